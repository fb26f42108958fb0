"""The five benchmark configurations at full size, in the launch configuration bench.py times
(one plan over all rows, TRIL): sampled output rows against the CPU oracle, plus properties that
hold at any size (closed-form counts, diagonal = squared row norms, the sum identity, mirror and
Jaccard invariants)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_09713_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = {np.dtype(np.float64): 1e-12, np.dtype(np.float32): 1e-5}


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available()
    from paper_2608_09713_b200 import binding
    return binding


def sample_rows(m, deg, k, seed):
    rng = np.random.default_rng(seed)
    rows = set(rng.integers(0, m, size=k).tolist()) | {0, 1, m // 2, m - 2, m - 1}
    heavy = np.argsort(deg)[-3:]                       # the heaviest rows of A as well
    return sorted(rows | set(int(x) for x in heavy))


def check_rows_against_oracle(a, cols, mode, rows, rp, ci, cv):
    for r in rows:
        ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode, r, r + 1, cols=cols)
        lo, hi = int(rp[r]), int(rp[r + 1])
        assert hi - lo == ref.nnz, f"row {r}: count"
        got_c = ci[lo:hi].cpu().numpy()
        got_v = cv[lo:hi].cpu().numpy()
        assert np.array_equal(got_c, ref.colidx), f"row {r}: structure"
        if np.issubdtype(a.vals.dtype, np.integer):
            assert np.array_equal(got_v, oracle.to_int32(ref.vals)), f"row {r}: values"
        else:
            err = np.abs(got_v.astype(np.float64) - ref.vals)
            assert np.all(err <= TOL[np.dtype(a.vals.dtype)] * ref.absvals), f"row {r}: values"


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_full_size_configuration(B, idx):
    a = W.config(idx)
    deg = np.diff(a.rowptr)
    d = (torch.from_numpy(a.rowptr).cuda(), torch.from_numpy(a.colidx).cuda(), torch.from_numpy(a.vals).cuda())
    rp, ci, cv, plan = B.tril_syrk(a.m, a.n, *d)
    torch.cuda.synchronize()
    rp_h = rp.cpu().numpy()
    nnz = int(rp_h[-1])

    # closed forms: multiply-add count of the half (Section III-C restricted to pairs j <= i)
    dk = np.bincount(a.colidx, minlength=a.n).astype(np.int64)
    work, classes = B.spsyrk_plan_stats(plan)
    assert work == int((dk * (dk + 1) // 2).sum())
    assert sum(classes) == a.m
    cnt = np.diff(rp_h)
    assert np.array_equal(cnt >= 1, deg > 0) and np.all(cnt <= np.arange(a.m) + 1)
    if idx == 2:
        assert dk.max() == a.m and nnz == a.m * (a.m + 1) // 2          # a column in every row: dense output

    # the diagonal is the last entry of every non-empty row and equals the squared row norm
    last = rp[1:][torch.from_numpy(deg > 0).cuda()] - 1
    rows_ne = torch.from_numpy(np.nonzero(deg > 0)[0]).cuda()
    assert torch.equal(ci[last].to(torch.int64), rows_ne)
    sq = torch.zeros(a.m, dtype=torch.float64, device="cuda")
    sq.index_add_(0, torch.repeat_interleave(torch.arange(a.m, device="cuda"), torch.from_numpy(deg).cuda()),
                  d[2].to(torch.float64) ** 2)
    diag = cv[last].to(torch.float64)
    tol = 1e-5 if a.vals.dtype == np.float32 else 1e-12
    assert torch.all((diag - sq[rows_ne]).abs() <= tol * sq[rows_ne])

    # sum identity: 2 sum(C_L) - trace = sum_k (sum_i a_ik)^2
    colsum = np.zeros(a.n)
    np.add.at(colsum, a.colidx, a.vals.astype(np.float64))
    abssum = np.zeros(a.n)
    np.add.at(abssum, a.colidx, np.abs(a.vals.astype(np.float64)))
    if a.vals.dtype == np.int32:
        lhs = 2 * int(cv.sum(dtype=torch.int64).item()) - int(diag.sum().item())
        assert lhs == int((colsum ** 2).sum())
    else:
        lhs = 2 * float(cv.to(torch.float64).sum().item()) - float(diag.sum().item())
        assert abs(lhs - (colsum ** 2).sum()) <= (1e-4 if a.vals.dtype == np.float32 else 1e-9) * (abssum ** 2).sum()

    # sampled rows against the oracle
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    rows = sample_rows(a.m, deg, 12 if idx == 2 else 40, idx)
    check_rows_against_oracle(a, cols, oracle.TRIL, rows, rp_h, ci, cv)

    # Jaccard on the binary configuration
    if a.vals.dtype == np.int32:
        jac = B.spsyrk_jaccard(a.m, 0, a.m, d[0], rp, ci, cv)
        assert torch.all(jac[last] == 1.0)
        for r in rows[:6]:
            lo, hi = int(rp_h[r]), int(rp_h[r + 1])
            exp = oracle.jaccard(r, 1, a.rowptr, np.array([0, hi - lo]), ci[lo:hi].cpu().numpy(), cv[lo:hi].cpu().numpy())
            assert np.array_equal(jac[lo:hi].cpu().numpy(), exp)
        del jac

    # mirror on the configurations that ask for it (4 and 5) and on the small ones
    if idx in (1, 3, 4, 5):
        f_rowptr, f_colidx, f_vals = B.spsyrk_mirror(a.m, rp, ci, cv)
        torch.cuda.synchronize()
        frp = f_rowptr.cpu().numpy()
        assert int(frp[-1]) == 2 * nnz - int((deg > 0).sum())
        # rows of F are rows of the full product: same structure, values within the tolerance
        check_rows_against_oracle(a, cols, oracle.FULL, rows[:20], frp, f_colidx, f_vals)
        # lower parts are bit copies of C_L
        for r in rows[:20]:
            lo, hi = int(rp_h[r]), int(rp_h[r + 1])
            assert torch.equal(f_colidx[int(frp[r]):int(frp[r]) + hi - lo], ci[lo:hi])
            assert torch.equal(f_vals[int(frp[r]):int(frp[r]) + hi - lo], cv[lo:hi])


def test_more_than_2_pow_22_rows_uses_wide_sort_keys(B):
    """Above 2^22 rows the warp-class sort keys no longer fit 32 bits; the 64-bit variant runs."""
    m = (1 << 22) + 12345
    a = W.erdos_renyi(m, 300_000, 3, 4242, np.float64, -1.0, 1.0)
    d = (torch.from_numpy(a.rowptr).cuda(), torch.from_numpy(a.colidx).cuda(), torch.from_numpy(a.vals).cuda())
    rp, ci, cv, plan = B.tril_syrk(a.m, a.n, *d)
    torch.cuda.synchronize()
    rp_h = rp.cpu().numpy()
    dk = np.bincount(a.colidx, minlength=a.n).astype(np.int64)
    assert B.spsyrk_plan_stats(plan)[0] == int((dk * (dk + 1) // 2).sum())
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    rows = sample_rows(a.m, np.diff(a.rowptr), 60, 9)
    check_rows_against_oracle(a, cols, oracle.TRIL, rows, rp_h, ci, cv)
    f_rowptr, f_colidx, f_vals = B.spsyrk_mirror(a.m, rp, ci, cv)
    check_rows_against_oracle(a, cols, oracle.FULL, rows[:30], f_rowptr.cpu().numpy(), f_colidx, f_vals)


def test_row_tiles_at_scale(B):
    """Configuration 5's recipe at 2^19 rows in five ragged row tiles equals the untiled result bit for bit."""
    a = W.erdos_renyi(1 << 19, 1 << 19, 16, W.SEED + 5, np.float64, -1.0, 1.0)
    d = (torch.from_numpy(a.rowptr).cuda(), torch.from_numpy(a.colidx).cuda(), torch.from_numpy(a.vals).cuda())
    rp, ci, cv, plan = B.tril_syrk(a.m, a.n, *d)
    cuts = [0, 100_001, 100_002, 262_144, 500_000, a.m]
    cols, vals, counts = [], [], []
    for r0, r1 in zip(cuts[:-1], cuts[1:]):
        B.spsyrk_plan_set_rows(plan, r0, r1)
        trp, tci, tcv, _ = B.tril_syrk(a.m, a.n, *d, row_begin=r0, row_end=r1, plan=plan)
        cols.append(tci); vals.append(tcv); counts.append(trp[1:] - trp[:-1])
    assert torch.equal(torch.cat(counts), rp[1:] - rp[:-1])
    assert torch.equal(torch.cat(cols), ci)
    assert torch.equal(torch.cat(vals), cv)


def test_panels_accumulate_to_the_whole_at_scale(B):
    """The accumulating form on the large Erdos-Renyi configuration: two column panels, their products
    summed; the structure must be that of the unsplit product bit for bit and the values agree to
    rounding (both sides are sums of the same partial products, grouped differently)."""
    a = W.config(5)
    d = (torch.from_numpy(a.rowptr).cuda(), torch.from_numpy(a.colidx).cuda(), torch.from_numpy(a.vals).cuda())
    rp, ci, cv, _ = B.tril_syrk(a.m, a.n, *d)
    prods = []
    for k0, k1 in ((0, a.n // 2), (a.n // 2, a.n)):
        p = B.spsyrk_column_panel(a.m, *d, k0, k1)
        prods.append(B.tril_syrk(a.m, a.n, *p)[:3])
        del p
    assert int(prods[0][1].numel()) + int(prods[1][1].numel()) >= int(ci.numel())
    zr, zc, zv = B.spsyrk_accumulate(a.m, *prods[0], *prods[1])
    del prods
    torch.cuda.synchronize()
    assert torch.equal(zr, rp) and torch.equal(zc, ci)
    # |difference| <= 1e-12 * (sum of |partial products|) <= 1e-12 * 16 since values lie in [-1, 1) and rows hold 16 entries
    assert float((zv - cv).abs().max()) <= 16e-12


def test_permutation_at_scale(B):
    """The symmetric permutation on the R-MAT configuration: sampled rows of the permuted matrix against
    the definition, and the product of the permuted matrix has the nnz and the diagonal of the original."""
    a = W.config(3)
    rng = np.random.default_rng(77)
    perm = rng.permutation(a.m).astype(np.int32)
    d = (torch.from_numpy(a.rowptr).cuda(), torch.from_numpy(a.colidx).cuda(), torch.from_numpy(a.vals).cuda())
    pt = torch.from_numpy(perm).cuda()
    br, bc, bv = B.spsyrk_permute(a.m, a.n, *d, pt, pt)
    brh = br.cpu().numpy()
    assert np.array_equal(np.diff(brh)[perm], np.diff(a.rowptr))          # row i went to row perm[i] with its length
    deg = np.diff(a.rowptr)
    for i in sample_rows(a.m, deg, 40, 5):
        src_c, src_v = a.colidx[a.rowptr[i]:a.rowptr[i + 1]], a.vals[a.rowptr[i]:a.rowptr[i + 1]]
        order = np.argsort(perm[src_c], kind="stable")
        lo, hi = int(brh[perm[i]]), int(brh[perm[i] + 1])
        assert np.array_equal(bc[lo:hi].cpu().numpy(), perm[src_c][order])
        assert np.array_equal(bv[lo:hi].cpu().numpy(), src_v[order])
    rp, ci, cv, _ = B.tril_syrk(a.m, a.n, *d)
    prp, pci, pcv, plan = B.tril_syrk(a.m, a.n, br, bc, bv)
    # (P A P^T)(P A P^T)^T = P (A A^T) P^T: the lower triangles differ, the full products are permutations of each
    # other, so nnz(tril) (every off-diagonal pair is stored once either way) and the diagonal values carry over
    assert int(pci.numel()) == int(ci.numel())
    diag = cv[(rp[1:] - 1).clamp(min=0)][torch.from_numpy(deg > 0).cuda()]
    pdeg = torch.from_numpy(np.diff(brh) > 0).cuda()
    pdiag = pcv[(prp[1:] - 1).clamp(min=0)][pdeg]
    inv = torch.from_numpy(np.argsort(perm)).cuda()        # row r of the permuted matrix is row inv[r] of the original
    full_diag = torch.zeros(a.m, dtype=cv.dtype, device="cuda")
    full_diag[torch.from_numpy(deg > 0).cuda()] = diag
    full_pdiag = torch.zeros(a.m, dtype=cv.dtype, device="cuda")
    full_pdiag[pdeg] = pdiag
    # a column permutation reorders the additions of each squared norm: equal to rounding
    assert float((full_pdiag - full_diag[inv]).abs().max()) <= 1e-5 * float(full_diag.abs().max())
    # equal-work row ranges of the plan tile the rows
    b = B.spsyrk_plan_partition(plan, 8)
    assert b[0] == 0 and b[-1] == a.m and all(x <= y for x, y in zip(b, b[1:]))
