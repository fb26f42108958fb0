"""Parity of the CUDA path against the CPU oracle, element by element, through the C ABI.

Bars: CSR structure and int32 values bit-exact; fp64 values within 1e-12 and fp32 values within
1e-5 of the oracle relative to the sum of absolute partial products of the entry (which equals
the relative error whenever the partial products share a sign); Jaccard within 1e-5.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_09713_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = {np.dtype(np.float64): 1e-12, np.dtype(np.float32): 1e-5}


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2608_09713_b200 import binding
    return binding


def dev(a: W.CSR):
    return (torch.from_numpy(a.rowptr).cuda(), torch.from_numpy(a.colidx).cuda(), torch.from_numpy(a.vals).cuda())


def check_values(gpu_vals, ref, dtype):
    """gpu_vals: numpy array of the matrix dtype; ref: oracle SyrkResult-like (vals, absvals float64)."""
    if np.issubdtype(dtype, np.integer):
        assert np.array_equal(gpu_vals, oracle.to_int32(ref.vals))
        return 0.0
    err = np.abs(gpu_vals.astype(np.float64) - ref.vals)
    bound = TOL[np.dtype(dtype)] * ref.absvals
    assert np.all(err <= bound), f"max scaled error {np.max(err / np.maximum(ref.absvals, 1e-300)):.3e}"
    return float(np.max(err / np.maximum(ref.absvals, 1e-300))) if err.size else 0.0


def run_and_compare(B, a: W.CSR, mode, r0=0, r1=None, cols=None, plan=None):
    """Both ways of computing the light rows (with the item map lent to the plan and without it)
    against the oracle; returns the result of the run with the map."""
    r1 = a.m if r1 is None else r1
    d = dev(a)
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode, r0, r1, cols=cols)
    for item_map in (False, True):
        c_rowptr, c_colidx, c_vals, plan = B.tril_syrk(a.m, a.n, *d, mode=mode, row_begin=r0, row_end=r1, plan=plan,
                                                       item_map=item_map)
        torch.cuda.synchronize()
        assert np.array_equal(c_rowptr.cpu().numpy(), ref.rowptr), f"item_map={item_map}"
        assert np.array_equal(c_colidx.cpu().numpy(), ref.colidx), f"item_map={item_map}"
        check_values(c_vals.cpu().numpy(), ref, a.vals.dtype)
    work, classes = B.spsyrk_plan_stats(plan)
    assert work == int(ref.work.sum())
    assert sum(classes) == r1 - r0
    return (c_rowptr, c_colidx, c_vals), ref, plan


# ------------------------------------------------------------------ the five workloads, reduced
@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("mode", [0, 1])
def test_small_configs(B, idx, mode):
    a = W.small(idx)
    run_and_compare(B, a, mode)


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_plan_internals(B, idx):
    """Step a1 (column lists ascending by row) and step a2 (per-row work) against the oracle."""
    a = W.small(idx)
    plan = B.spsyrk_plan(a.m, a.n, *dev(a))
    colptr, at_row, at_val, work = (t.cpu().numpy() for t in B.spsyrk_plan_buffers(plan))
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    assert np.array_equal(colptr, cols.colptr)
    assert np.array_equal(at_row, cols.rows)
    assert np.array_equal(at_val.astype(np.float64), cols.vals)
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, cols=cols, counts_only=True)
    assert np.array_equal(work, ref.work)
    d = np.diff(cols.colptr)
    total, classes = B.spsyrk_plan_stats(plan)
    assert total == int((d * (d + 1) // 2).sum())           # closed form of the multiply-add count
    fplan = B.spsyrk_plan(a.m, a.n, *dev(a), mode=B.FULL)
    assert B.spsyrk_plan_stats(fplan)[0] == int((d * d).sum())


def test_rmat_unpermuted_and_row_classes(B):
    """Hubs at low indices; every row class must be populated somewhere in these cases."""
    seen = np.zeros(8, dtype=np.int64)
    for a in (W.rmat(13, 16, 21, permute=False), W.small(3), W.small(2), W.small(5)):
        _, _, plan = run_and_compare(B, a, 0)
        seen += np.array(B.spsyrk_plan_stats(plan)[1])
    assert (seen > 0).all(), f"row classes not all exercised: {seen}"


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("mode", [0, 1])
def test_numeric_by_row_blocks(B, idx, mode):
    """spsyrk_numeric_rows over a partition of the rows fills the same arrays as one spsyrk_numeric."""
    a = W.small(idx)
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode, 0, a.m)
    cuts = [0, 1, a.m // 5, a.m // 5, a.m // 2 + 3, a.m - 1, a.m]          # an empty block among them
    for item_map in (False, True):
        plan = B.spsyrk_plan(a.m, a.n, *dev(a), mode=mode)
        B.spsyrk_plan_lend_map(plan, B._workspace(B.spsyrk_plan_map_bytes(plan), torch.device("cuda")) if item_map else None)
        c_rowptr = torch.empty(a.m + 1, dtype=torch.int64, device="cuda")
        nnz = B.spsyrk_symbolic(plan, c_rowptr)
        c_colidx = torch.full((nnz,), -7, dtype=torch.int32, device="cuda")
        c_vals = torch.zeros(nnz, dtype=torch.from_numpy(a.vals).dtype, device="cuda")
        rp = c_rowptr.cpu().numpy()
        for r0, r1 in zip(cuts[:-1], cuts[1:]):
            B.spsyrk_numeric_rows(plan, r0, r1, c_rowptr, c_colidx, c_vals)
            torch.cuda.synchronize()
            got = c_colidx.cpu().numpy()
            assert np.array_equal(got[:rp[r1]], ref.colidx[:rp[r1]]) and np.all(got[rp[r1]:] == -7)   # nothing beyond the block
        check_values(c_vals.cpu().numpy(), ref, a.vals.dtype)
        with pytest.raises(B.SpsyrkError):
            B.spsyrk_numeric_rows(plan, 0, a.m + 1, c_rowptr, c_colidx, c_vals)
        B.spsyrk_destroy(plan)


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_one_pass_mode(B, idx):
    """Slots from the work estimate, rows computed into them with their counts found on the way, then compacted:
    the same C_L as symbolic + numeric; also for a row range and a block of columns."""
    a = W.small(idx)
    d = dev(a)
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, 0, 0, a.m)
    plan = B.spsyrk_plan(a.m, a.n, *d)
    rp, ci, cv = B.onepass_syrk(plan)
    torch.cuda.synchronize()
    assert np.array_equal(rp.cpu().numpy(), ref.rowptr) and np.array_equal(ci.cpu().numpy(), ref.colidx)
    check_values(cv.cpu().numpy(), ref, a.vals.dtype)
    # the four-array form the slot buffers hold before the compaction: the same rows, each in its slot
    rb, rp4, sc, sv_ = B.onepass_syrk(plan, compact=False)
    assert torch.equal(rp4, rp)
    lens = rp[1:] - rp[:-1]
    assert bool((rb[:-1] + lens <= rb[1:]).all())
    idx = torch.repeat_interleave(rb[:-1] - rp[:-1], lens) + torch.arange(ci.numel(), device="cuda")
    assert torch.equal(sc[idx], ci) and torch.equal(sv_[idx], cv)
    r0, r1 = a.m // 3, a.m - 5
    B.spsyrk_plan_set_rows(plan, r0, r1)
    rp, ci, cv = B.onepass_syrk(plan)
    part = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, 0, r0, r1)
    assert np.array_equal(rp.cpu().numpy(), part.rowptr) and np.array_equal(ci.cpu().numpy(), part.colidx)
    check_values(cv.cpu().numpy(), part, a.vals.dtype)
    h = a.m // 2
    B.spsyrk_plan_set_block(plan, h, a.m, 0, h)            # an off-diagonal block: no diagonal handled apart
    rp, ci, cv = B.onepass_syrk(plan)
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    blk = oracle_block(a, oracle.TRIL, h, a.m, 0, h, cols)
    assert np.array_equal(rp.cpu().numpy(), blk.rowptr) and np.array_equal(ci.cpu().numpy(), blk.colidx)
    check_values(cv.cpu().numpy(), blk, a.vals.dtype)
    fplan = B.spsyrk_plan(a.m, a.n, *d, mode=B.FULL)
    with pytest.raises(B.SpsyrkError):
        B.onepass_syrk(fplan)                              # the two-part full-output mode keeps the two-pass route


@pytest.mark.parametrize("idx", [1, 3])
def test_numeric_replays_from_a_cuda_graph(B, idx):
    """The numeric pass makes no host round trip, so a caller can capture it into a CUDA graph and replay it."""
    a = W.small(idx)
    rp, ci, v = dev(a)
    plan = B.spsyrk_plan(a.m, a.n, rp, ci, v)
    B.spsyrk_plan_lend_map(plan, B._workspace(B.spsyrk_plan_map_bytes(plan), torch.device("cuda")))
    c_rowptr = torch.empty(a.m + 1, dtype=torch.int64, device="cuda")
    nnz = B.spsyrk_symbolic(plan, c_rowptr)
    c_colidx = torch.empty(nnz, dtype=torch.int32, device="cuda")
    c_vals = torch.empty(nnz, dtype=v.dtype, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        B.spsyrk_numeric(plan, c_rowptr, c_colidx, c_vals)          # warm-up outside the capture (function attributes)
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        B.spsyrk_numeric(plan, c_rowptr, c_colidx, c_vals)
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, 0, 0, a.m)
    for _ in range(2):
        c_vals.zero_()
        c_colidx.fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(c_colidx.cpu().numpy(), ref.colidx)
        check_values(c_vals.cpu().numpy(), ref, a.vals.dtype)
    B.spsyrk_destroy(plan)


@pytest.mark.parametrize("idx", [2, 3, 5])
def test_row_tiles_concatenate(B, idx):
    a = W.small(idx)
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    full, ref, _ = run_and_compare(B, a, 0, cols=cols)
    cuts = [0, a.m // 7, a.m // 7 + 1, a.m // 2, a.m - 3, a.m]
    plan = None
    parts_col, parts_val, counts = [], [], []
    for r0, r1 in zip(cuts[:-1], cuts[1:]):
        if plan is not None:
            B.spsyrk_plan_set_rows(plan, r0, r1)        # re-target without repeating the transpose
        (rp, ci, cv), _, plan = run_and_compare(B, a, 0, r0, r1, cols=cols, plan=plan)
        parts_col.append(ci); parts_val.append(cv); counts.append(rp[1:] - rp[:-1])
    assert torch.equal(torch.cat(counts), full[0][1:] - full[0][:-1])
    assert torch.equal(torch.cat(parts_col), full[1])
    assert torch.equal(torch.cat(parts_val), full[2])   # deterministic row classes give identical bits


def test_warp_rows_are_bit_reproducible_and_match_oracle_order(B):
    """Light rows sum partial products in ascending k like the oracle: fp64 results are identical bits."""
    a = W.small(5)
    (_, _, v1), ref, _ = run_and_compare(B, a, 0)
    (_, _, v2), _, _ = run_and_compare(B, a, 0)
    assert torch.equal(v1, v2)
    assert np.array_equal(v1.cpu().numpy(), ref.vals)


# ------------------------------------------------------------------------------ edge cases
def _csr(dense):
    dense = np.asarray(dense, dtype=np.float64)
    m, n = dense.shape
    s = dense != 0
    rowptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(s.sum(axis=1), out=rowptr[1:])
    rr, cc = np.nonzero(s)
    return W.CSR(m, n, rowptr, cc.astype(np.int32), dense[rr, cc].copy())


@pytest.mark.parametrize("mode", [0, 1])
def test_edge_cases(B, mode):
    rng = np.random.default_rng(4)
    cases = []
    cases.append(_csr(np.zeros((5, 4))))                                          # nnz = 0
    cases.append(_csr(np.array([[2.0, 0.0, 3.0]])))                               # m = 1
    cases.append(_csr(np.array([[2.0], [0.0], [5.0], [1.0]])))                    # n = 1
    d = (rng.random((40, 30)) < 0.2) * rng.random((40, 30)); d[3] = 0; d[17] = 0; d[:, 5] = 0
    cases.append(_csr(d))                                                         # empty rows and column
    d = (rng.random((70, 50)) < 0.1) * rng.random((70, 50)); d[9] = rng.random(50) + 0.1
    cases.append(_csr(d))                                                         # a full row (more than 32 nonzeros)
    d = (rng.random((300, 40)) < 0.05) * rng.random((300, 40)); d[:, 7] = rng.random(300) + 0.1
    cases.append(_csr(d))                                                         # a full column: dense output
    d = (rng.random((64, 64)) < 0.3) * rng.random((64, 64)); d[40] = d[2]; d[63] = d[2]
    cases.append(_csr(d))                                                         # identical rows
    cases.append(_csr(rng.random((90, 70)) + 0.1))                                # fully dense A
    for a in cases:
        run_and_compare(B, a, mode)


def test_zero_rows(B):
    a = W.CSR(0, 5, np.zeros(1, dtype=np.int64), np.zeros(0, dtype=np.int32), np.zeros(0, dtype=np.float64))
    rp, ci, cv, plan = B.tril_syrk(0, 5, *dev(a))
    assert rp.cpu().tolist() == [0] and ci.numel() == 0


def test_cancellation_keeps_structural_entries(B):
    d = np.array([[1.0, 1.0, 0.0], [1.0, -1.0, 0.0], [0.0, 0.0, 2.0]])
    rp, ci, cv, _ = B.tril_syrk(3, 3, *dev(_csr(d)))
    assert rp.cpu().tolist() == [0, 1, 3, 4] and ci.cpu().tolist() == [0, 0, 1, 2]
    assert cv.cpu().tolist() == [2.0, 0.0, 2.0, 4.0]


def test_bad_csr_is_rejected(B):
    a = W.small(1)
    rowptr, colidx, vals = dev(a)
    bad = colidx.clone(); bad[3], bad[4] = colidx[4].item(), colidx[3].item()       # unsorted row
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_plan(a.m, a.n, rowptr, bad, vals)
    assert e.value.status == 2
    bad = colidx.clone(); bad[10] = a.n                                               # out of range
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_plan(a.m, a.n, rowptr, bad, vals)
    assert e.value.status == 2
    bad = colidx.clone(); bad[1] = bad[0]                                             # duplicate
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_plan(a.m, a.n, rowptr, bad, vals)
    assert e.value.status == 2
    badp = rowptr.clone(); badp[5] = badp[6] + 1                                      # non-monotone
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_plan(a.m, a.n, badp, colidx, vals)
    assert e.value.status == 2
    plan = B.spsyrk_plan(a.m, a.n, rowptr, colidx, vals)
    with pytest.raises(B.SpsyrkError) as e:                                           # numeric before symbolic
        B.spsyrk_numeric(plan, torch.zeros(a.m + 1, dtype=torch.int64, device="cuda"),
                         torch.zeros(1, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.float64, device="cuda"))
    assert e.value.status == 5


# ----------------------------------------------------------------------------------- mirror
@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_mirror(B, idx):
    a = W.small(idx)
    (rp, ci, cv), ref, _ = run_and_compare(B, a, 0)
    f_rowptr, f_colidx, f_vals = B.spsyrk_mirror(a.m, rp, ci, cv)
    torch.cuda.synchronize()
    lv = cv.cpu().numpy()
    o_rowptr, o_colidx, o_vals = oracle.mirror(a.m, rp.cpu().numpy(), ci.cpu().numpy(), lv.astype(np.float64))
    assert np.array_equal(f_rowptr.cpu().numpy(), o_rowptr)
    assert np.array_equal(f_colidx.cpu().numpy(), o_colidx)
    assert np.array_equal(f_vals.cpu().numpy().astype(np.float64), o_vals)      # values are bit copies
    # same structure as the full-output variant of the same kernels
    (frp, fci, _), _, _ = run_and_compare(B, a, 1)
    assert torch.equal(frp, f_rowptr) and torch.equal(fci, f_colidx)


def test_mirror_rejects_upper_entries(B):
    rp = torch.tensor([0, 1, 2], dtype=torch.int64, device="cuda")
    ci = torch.tensor([1, 1], dtype=torch.int32, device="cuda")
    cv = torch.tensor([1.0, 1.0], dtype=torch.float64, device="cuda")
    with pytest.raises(B.SpsyrkError) as e:
        B.spsyrk_mirror(2, rp, ci, cv)
    assert e.value.status == 2


@pytest.mark.parametrize("m,density,diag", [(7, 0.5, "some"), (200, 0.1, "some"), (200, 0.1, "none"), (3000, 0.004, "all"),
                                            (70000, 0.0001, "some"), (2 ** 24 + 77, 2e-8, "some")])
def test_mirror_general_lower_triangles(B, m, density, diag):
    """Lower triangles that are not products: rows without a diagonal entry, empty rows, one pass
    (m < 256) up to four radix passes (m > 2^24); with every diagonal stored the record buffer that
    lives in F's value array is at its shortest."""
    rng = np.random.default_rng(m)
    nnz_target = int(density * m * m / 2) + m
    r = rng.integers(0, m, size=nnz_target)
    c = (rng.random(nnz_target) * (r + 1)).astype(np.int64)     # c <= r
    keep = c < r
    r, c = r[keep], c[keep]
    if diag != "none":
        d = np.arange(m) if diag == "all" else rng.choice(m, size=m // 2, replace=False)
        r, c = np.concatenate([r, d]), np.concatenate([c, d])
    key = np.unique(r * m + c)
    r, c = key // m, key % m
    rp = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(np.bincount(r, minlength=m), out=rp[1:])
    for dtype in (np.float64, np.float32):      # 16-byte records / separate arrays: both keep scratch in F's arrays
        vals = rng.standard_normal(c.size).astype(dtype)
        got = B.spsyrk_mirror(m, torch.from_numpy(rp).cuda(), torch.from_numpy(c.astype(np.int32)).cuda(), torch.from_numpy(vals).cuda())
        exp = oracle.mirror(m, rp, c.astype(np.int32), vals.astype(np.float64))
        assert np.array_equal(got[0].cpu().numpy(), exp[0]) and np.array_equal(got[1].cpu().numpy(), exp[1])
        assert np.array_equal(got[2].cpu().numpy().astype(np.float64), exp[2])


def test_mirror_few_entries_many_rows(B):
    """Three radix passes over five entries: the digit bytes do not fit F's column array and stay in the workspace."""
    m = 100000
    r = np.array([5, 70000, 70000, 99999, 99999]); c = np.array([5, 5, 69999, 0, 99999], dtype=np.int32)
    rp = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(np.bincount(r, minlength=m), out=rp[1:])
    vals = np.arange(1.0, 6.0)
    got = B.spsyrk_mirror(m, torch.from_numpy(rp).cuda(), torch.from_numpy(c).cuda(), torch.from_numpy(vals).cuda())
    exp = oracle.mirror(m, rp, c, vals)
    for g, e in zip(got, exp):
        assert np.array_equal(g.cpu().numpy(), e)


def test_mirror_of_nothing(B):
    z = (torch.zeros(1, dtype=torch.int64, device="cuda"), torch.zeros(0, dtype=torch.int32, device="cuda"),
         torch.zeros(0, dtype=torch.float64, device="cuda"))
    assert B.spsyrk_mirror(0, *z)[0].cpu().tolist() == [0]
    z5 = (torch.zeros(6, dtype=torch.int64, device="cuda"), z[1], z[2])
    f = B.spsyrk_mirror(5, *z5)
    assert f[0].cpu().tolist() == [0] * 6 and f[1].numel() == 0


# ---------------------------------------------------------------------------------- jaccard
def test_jaccard(B):
    a = W.small(2)
    (rp, ci, cv), ref, plan = run_and_compare(B, a, 0)
    rowptr_a = torch.from_numpy(a.rowptr).cuda()
    jac = B.spsyrk_jaccard(a.m, 0, a.m, rowptr_a, rp, ci, cv).cpu().numpy()
    exp = oracle.jaccard(0, a.m, a.rowptr, ref.rowptr, ref.colidx, oracle.to_int32(ref.vals))
    assert np.all(np.abs(jac - exp) <= 1e-5 * np.abs(exp))
    # fused into the numeric pass: the same numbers, bit for bit, with and without the item map
    for item_map in (False, True):
        plan = B.spsyrk_plan(a.m, a.n, *dev(a))
        B.spsyrk_plan_lend_map(plan, torch.empty(max(B.spsyrk_plan_map_bytes(plan), 256), dtype=torch.uint8, device="cuda") if item_map else None)
        rp2 = torch.empty(a.m + 1, dtype=torch.int64, device="cuda")
        nnz = B.spsyrk_symbolic(plan, rp2)
        ci2 = torch.empty(nnz, dtype=torch.int32, device="cuda")
        cv2 = torch.empty(nnz, dtype=torch.int32, device="cuda")
        fused = torch.full((nnz,), -1.0, dtype=torch.float32, device="cuda")
        B.spsyrk_plan_set_jaccard(plan, fused)
        B.spsyrk_numeric(plan, rp2, ci2, cv2)
        assert torch.equal(ci2, ci) and torch.equal(cv2, cv)
        assert np.array_equal(fused.cpu().numpy(), jac)
    assert np.array_equal(jac, exp)                          # one correctly rounded division on both sides
    rows = np.repeat(np.arange(a.m), np.diff(ref.rowptr))
    assert np.all(jac[rows == ref.colidx] == 1.0)
    # a row tile
    r0, r1 = 1000, 1777
    B.spsyrk_plan_set_rows(plan, r0, r1)
    trp, tci, tcv, _ = B.tril_syrk(a.m, a.n, *dev(a), row_begin=r0, row_end=r1, plan=plan)
    tj = B.spsyrk_jaccard(a.m, r0, r1 - r0, rowptr_a, trp, tci, tcv).cpu().numpy()
    assert np.array_equal(tj, exp[ref.rowptr[r0]:ref.rowptr[r1]])
    # arrays that do not start on 16 bytes take the scalar path; short rows straddle the 4-entry steps
    def shifted(t):
        buf = torch.empty(t.numel() + 1, dtype=t.dtype, device=t.device)
        buf[1:].copy_(t)
        return buf[1:]
    out = shifted(torch.zeros(ci.numel(), dtype=torch.float32, device="cuda"))
    uj = B.spsyrk_jaccard(a.m, 0, a.m, rowptr_a, rp, shifted(ci), shifted(cv), out=out).cpu().numpy()
    assert np.array_equal(uj, exp)
    b = W.small(4)                                            # binary values, about 50 entries per output row
    (rp4, ci4, cv4), ref4, _ = run_and_compare(B, W.CSR(b.m, b.n, b.rowptr, b.colidx, np.ones(b.nnz, dtype=np.int32)), 0)
    j4 = B.spsyrk_jaccard(b.m, 0, b.m, torch.from_numpy(b.rowptr).cuda(), rp4, ci4, cv4).cpu().numpy()
    assert np.array_equal(j4, oracle.jaccard(0, b.m, b.rowptr, ref4.rowptr, ref4.colidx, oracle.to_int32(ref4.vals)))


# --------------------------------------------------------------------- host-buffer entry point
def test_host_entry_point(B):
    a = W.small(4)
    rp, ci, cv = B.spsyrk_host_tril(a.m, a.n, torch.from_numpy(a.rowptr), torch.from_numpy(a.colidx),
                                    torch.from_numpy(a.vals), pinned=False)
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    assert np.array_equal(rp.numpy(), ref.rowptr) and np.array_equal(ci.numpy(), ref.colidx)
    check_values(cv.numpy(), ref, a.vals.dtype)


def test_host_entry_point_reuses_its_device_blocks(B):
    """Calls of different sizes in a row (the cached blocks grow, then serve a smaller problem), a
    release in between, and a mode change: results stay those of the oracle."""
    for idx, mode in [(1, 0), (5, 0), (1, 1), (3, 0)]:
        if idx == 3:
            B.spsyrk_host_release_cache()
        a = W.small(idx)
        rp, ci, cv = B.spsyrk_host_tril(a.m, a.n, torch.from_numpy(a.rowptr), torch.from_numpy(a.colidx),
                                        torch.from_numpy(a.vals), mode=mode)
        ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode)
        assert np.array_equal(rp.numpy(), ref.rowptr) and np.array_equal(ci.numpy(), ref.colidx)
        check_values(cv.numpy(), ref, a.vals.dtype)
    B.spsyrk_host_release_cache()


# ------------------------------------------------------------------ further dtypes and error paths
def test_int32_general_values_and_fp32_light_rows(B):
    rng = np.random.default_rng(11)
    a = W.erdos_renyi(3000, 2500, 9, 123, np.float64, 0.0, 1.0)
    ai = W.CSR(a.m, a.n, a.rowptr, a.colidx, rng.integers(-50, 51, size=a.nnz).astype(np.int32))
    run_and_compare(B, ai, 0)
    run_and_compare(B, ai, 1)
    af = W.CSR(a.m, a.n, a.rowptr, a.colidx, (rng.random(a.nnz) * 2 - 1).astype(np.float32))
    run_and_compare(B, af, 0)
    hf = W.hypergraph(20_000, 5_000, 77)
    run_and_compare(B, W.CSR(hf.m, hf.n, hf.rowptr, hf.colidx, hf.vals.astype(np.float32)), 0)


def test_workspace_and_alignment_errors(B):
    import ctypes
    a = W.small(1)
    rowptr, colidx, vals = dev(a)
    need = B.spsyrk_plan_workspace_bytes(a.m, a.n, a.nnz, torch.float64)
    small_ws = torch.empty(need // 2, dtype=torch.uint8, device="cuda")
    with pytest.raises(AssertionError):
        B.spsyrk_plan(a.m, a.n, rowptr, colidx, vals, workspace=small_ws)
    sz = ctypes.c_size_t(small_ws.numel())
    h = ctypes.c_void_p()
    st = B._lib.spsyrk_plan(ctypes.byref(h), a.m, a.n, a.nnz, B._p(rowptr), B._p(colidx), B._p(vals), 0, 0, 0, a.m,
                            B._p(small_ws), ctypes.byref(sz), None)
    assert st == 3                                                      # workspace too small
    ws = torch.empty(need + 64, dtype=torch.uint8, device="cuda")
    sz = ctypes.c_size_t(need)
    st = B._lib.spsyrk_plan(ctypes.byref(h), a.m, a.n, a.nnz, B._p(rowptr), B._p(colidx), B._p(vals), 0, 0, 0, a.m,
                            ctypes.c_void_p(ws.data_ptr() + 8), ctypes.byref(sz), None)
    assert st == 1                                                      # misaligned workspace
    # inputs need no particular alignment: column ids and values that start 4 / 8 bytes into an allocation
    sc = torch.empty(a.nnz + 1, dtype=torch.int32, device="cuda")
    sc[1:] = colidx
    sv_ = torch.empty(a.nnz + 1, dtype=vals.dtype, device="cuda")
    sv_[1:] = vals
    rp2, ci2, cv2, _ = B.tril_syrk(a.m, a.n, rowptr, sc[1:], sv_[1:])
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    assert np.array_equal(rp2.cpu().numpy(), ref.rowptr) and np.array_equal(ci2.cpu().numpy(), ref.colidx)
    check_values(cv2.cpu().numpy(), ref, a.vals.dtype)
    sl = torch.empty(ci2.numel() + 1, dtype=torch.int32, device="cuda")
    sl[1:] = ci2
    f = B.spsyrk_mirror(a.m, rp2, sl[1:], cv2)
    g = B.spsyrk_mirror(a.m, rp2, ci2, cv2)
    assert all(torch.equal(x, y) for x, y in zip(f, g))


# ---------------------------------------------------------------- blocks C[R, S] (Algorithm 2, lines 4 and 6)
def oracle_block(a, mode, r0, r1, s0, s1, cols):
    """Rows [r0, r1) of the product restricted to columns [s0, s1): the definition, then a column filter."""
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode, r0, r1, cols=cols)
    keep = (ref.colidx >= s0) & (ref.colidx < s1)
    rows = np.repeat(np.arange(r1 - r0), np.diff(ref.rowptr))
    rowptr = np.zeros(r1 - r0 + 1, dtype=np.int64)
    np.cumsum(np.bincount(rows[keep], minlength=r1 - r0), out=rowptr[1:])

    class R:  # same fields as the oracle's result
        pass
    out = R()
    out.rowptr, out.colidx, out.vals, out.absvals = rowptr, ref.colidx[keep], ref.vals[keep], ref.absvals[keep]
    return out


@pytest.mark.parametrize("idx", [2, 3, 4, 5])
def test_blocks(B, idx):
    a = W.small(idx)
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    d = dev(a)
    plan = B.spsyrk_plan(a.m, a.n, *d, mode=B.FULL)
    h = a.m // 2
    blocks = [(0, h // 2, h, a.m),            # row top half of a lower block x the other operand
              (h, a.m, h + (a.m - h) // 2, a.m),   # all rows x right half of the columns
              (h, a.m, 0, h),                 # an off-diagonal block
              (10, 50, 0, 1),                 # one output column
              (h, h + 7, 3, 3)]               # empty column range
    for r0, r1, s0, s1 in blocks:
        B.spsyrk_plan_set_block(plan, r0, r1, s0, s1)
        rp, ci, cv, _ = B.tril_syrk(a.m, a.n, *d, plan=plan)
        ref = oracle_block(a, oracle.FULL, r0, r1, s0, s1, cols)
        assert np.array_equal(rp.cpu().numpy(), ref.rowptr), (r0, r1, s0, s1)
        assert np.array_equal(ci.cpu().numpy(), ref.colidx)
        check_values(cv.cpu().numpy(), ref, a.vals.dtype)
    # TRIL mode with S = R is the lower triangle of a diagonal block
    tplan = B.spsyrk_plan(a.m, a.n, *d, mode=B.TRIL)
    B.spsyrk_plan_set_block(tplan, h, a.m, h, a.m)
    rp, ci, cv, _ = B.tril_syrk(a.m, a.n, *d, plan=tplan)
    ref = oracle_block(a, oracle.TRIL, h, a.m, h, a.m, cols)
    assert np.array_equal(rp.cpu().numpy(), ref.rowptr) and np.array_equal(ci.cpu().numpy(), ref.colidx)
    check_values(cv.cpu().numpy(), ref, a.vals.dtype)
    # four blocks tile the full product: entry counts add up
    B.spsyrk_plan_set_rows(plan, 0, a.m)
    total = B.tril_syrk(a.m, a.n, *d, plan=plan)[1].numel()
    parts = 0
    for r0, r1 in ((0, h), (h, a.m)):
        for s0, s1 in ((0, h), (h, a.m)):
            B.spsyrk_plan_set_block(plan, r0, r1, s0, s1)
            parts += B.tril_syrk(a.m, a.n, *d, plan=plan)[1].numel()
    assert parts == total


# ------------------------------------------------------------------ consuming the triangle (Section V-F)
@pytest.mark.parametrize("idx", [1, 3, 4, 5])
def test_symv(B, idx):
    a = W.small(idx)
    (rp, ci, cv), ref, _ = run_and_compare(B, a, 0)
    rng = np.random.default_rng(2)
    x = rng.standard_normal(a.m).astype(a.vals.dtype)
    y = B.spsyrk_symv(a.m, rp, ci, cv, torch.from_numpy(x).cuda()).cpu().numpy()
    exp, scale = oracle.symv(a.m, rp.cpu().numpy(), ci.cpu().numpy(), cv.cpu().numpy().astype(np.float64), x.astype(np.float64))
    tol = 1e-12 if a.vals.dtype == np.float64 else 2e-5
    assert np.all(np.abs(y.astype(np.float64) - exp) <= tol * (scale + 1e-300))


@pytest.mark.parametrize("idx", [1, 3, 4, 5])
@pytest.mark.parametrize("p", [1, 8, 33])
def test_symm(B, idx, p):
    """Y = C_L X + (X^T C_L)^T - D X (Section V-F, second equation) against the oracle, element by element."""
    a = W.small(idx)
    (rp, ci, cv), ref, _ = run_and_compare(B, a, 0)
    rng = np.random.default_rng(20 + p)
    x = rng.standard_normal((a.m, p)).astype(a.vals.dtype)
    y = B.spsyrk_symm(a.m, rp, ci, cv, torch.from_numpy(x).cuda()).cpu().numpy()
    exp, scale = oracle.symm(a.m, rp.cpu().numpy(), ci.cpu().numpy(), cv.cpu().numpy().astype(np.float64), x.astype(np.float64))
    tol = 1e-12 if a.vals.dtype == np.float64 else 2e-5
    assert y.shape == exp.shape
    assert np.all(np.abs(y.astype(np.float64) - exp) <= tol * (scale + 1e-300))
    if p == 1:                                             # one column is the vector form
        yv = B.spsyrk_symv(a.m, rp, ci, cv, torch.from_numpy(x[:, 0].copy()).cuda()).cpu().numpy()
        assert np.all(np.abs(yv.astype(np.float64) - exp[:, 0]) <= tol * (scale[:, 0] + 1e-300))


def test_symm_degenerate(B):
    z = (torch.zeros(1, dtype=torch.int64, device="cuda"), torch.zeros(0, dtype=torch.int32, device="cuda"),
         torch.zeros(0, dtype=torch.float64, device="cuda"))
    assert B.spsyrk_symm(0, *z, torch.zeros((0, 3), dtype=torch.float64, device="cuda")).shape == (0, 3)
    rp = torch.tensor([0, 1, 2], dtype=torch.int64, device="cuda")
    ci = torch.tensor([0, 1], dtype=torch.int32, device="cuda")
    cv = torch.tensor([2.0, 3.0], dtype=torch.float64, device="cuda")
    x = torch.tensor([[1.0, -1.0], [4.0, 0.5]], dtype=torch.float64, device="cuda")
    assert B.spsyrk_symm(2, rp, ci, cv, x).cpu().tolist() == [[2.0, -2.0], [12.0, 1.5]]    # the diagonal counts once


# ------------------------------------------- accumulating form over column panels (Section III-A, Algorithm 2)
def _np(*ts):
    return [t.cpu().numpy() for t in ts]


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_column_panel(B, idx):
    a = W.small(idx)
    d = dev(a)
    for k0, k1 in [(0, a.n), (0, a.n // 3), (a.n // 3, a.n // 3), (a.n // 3, a.n - 1), (a.n - 1, a.n), (a.n, a.n + 7)]:
        pr, pc, pv = _np(*B.spsyrk_column_panel(a.m, *d, k0, k1))
        er, ec, ev = oracle.column_panel(a.m, a.rowptr, a.colidx, a.vals, k0, k1)
        assert np.array_equal(pr, er) and np.array_equal(pc, ec)
        assert np.array_equal(pv.astype(np.float64), ev)       # values are copied bit for bit


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("npanels", [2, 5])
def test_accumulate_panels(B, idx, npanels):
    """C_L = sum over panels of tril(A_s A_s^T): every step against the oracle's sum of the same operands
    (bit-exact, one rounded addition per shared entry), the end against the unsplit product."""
    a = W.small(idx)
    d = dev(a)
    edges = np.linspace(0, a.n, npanels + 1).astype(np.int64)
    acc = None
    for s in range(npanels):
        p = B.spsyrk_column_panel(a.m, *d, int(edges[s]), int(edges[s + 1]))
        t_rowptr, t_colidx, t_vals, _ = B.tril_syrk(a.m, a.n, *p)
        if acc is None:
            acc = (t_rowptr, t_colidx, t_vals)
            continue
        z = B.spsyrk_accumulate(a.m, *acc, t_rowptr, t_colidx, t_vals)
        xr, xc, xv, yr, yc, yv = _np(*acc, t_rowptr, t_colidx, t_vals)
        er, ec, ev = oracle.add(a.m, xr, xc, xv.astype(np.float64), yr, yc, yv.astype(np.float64))
        zr, zc, zv = _np(*z)
        assert np.array_equal(zr, er) and np.array_equal(zc, ec)
        if a.vals.dtype == np.float32:
            assert np.array_equal(zv, ev.astype(np.float32))   # the double sum of two floats rounds to the float sum
        else:
            assert np.array_equal(zv.astype(np.float64), ev)
        acc = z
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    zr, zc, zv = _np(*acc)
    assert np.array_equal(zr, ref.rowptr) and np.array_equal(zc, ref.colidx)   # union of panel structures = structure of the whole
    check_values(zv, ref, a.vals.dtype)


def test_accumulate_edge_cases(B):
    dev0 = torch.device("cuda")
    def csr(m, rows):
        rp = np.zeros(m + 1, dtype=np.int64)
        ci, va = [], []
        for i, r in enumerate(rows):
            rp[i + 1] = rp[i] + len(r)
            ci += [c for c, _ in r]
            va += [v for _, v in r]
        return (torch.from_numpy(rp).to(dev0), torch.tensor(ci, dtype=torch.int32, device=dev0),
                torch.tensor(va, dtype=torch.float64, device=dev0))
    # empty + empty, empty + something, cancellation keeps the entry, disjoint and identical rows
    x = csr(5, [[], [(0, 1.0), (3, 2.0)], [(1, 1.5)], [(0, 1.0), (1, 1.0), (2, 1.0)], []])
    y = csr(5, [[], [], [(1, -1.5)], [(0, 2.0), (1, 3.0), (2, 4.0)], [(4, 9.0)]])
    zr, zc, zv = _np(*B.spsyrk_accumulate(5, *x, *y))
    assert zr.tolist() == [0, 0, 2, 3, 6, 7]
    assert zc.tolist() == [0, 3, 1, 0, 1, 2, 4]
    assert zv.tolist() == [1.0, 2.0, 0.0, 3.0, 4.0, 5.0, 9.0]
    e = csr(5, [[], [], [], [], []])
    zr, zc, zv = _np(*B.spsyrk_accumulate(5, *e, *e))
    assert zr.tolist() == [0] * 6 and zc.size == 0
    # m = 0
    z0 = csr(0, [])
    assert B.spsyrk_accumulate(0, *z0, *z0)[0].cpu().tolist() == [0]
    # a row that is not ascending is refused
    bad = csr(2, [[(3, 1.0), (1, 1.0)], []])
    ok = csr(2, [[(1, 1.0)], []])
    for args in ((bad, ok), (ok, bad)):
        with pytest.raises(B.SpsyrkError) as ei:
            B.spsyrk_accumulate(2, *args[0], *args[1])
        assert ei.value.status == 2


def test_accumulate_long_rows(B):
    """Rows much longer than a group of lanes, with many shared entries (the running match count
    crosses many 32-entry steps), int32 values."""
    rng = np.random.default_rng(11)
    m, n = 37, 20000
    def rand_csr(density):
        mask = rng.random((m, n)) < density
        mask[5] = False
        rp = np.zeros(m + 1, dtype=np.int64)
        np.cumsum(mask.sum(axis=1), out=rp[1:])
        rr, cc = np.nonzero(mask)
        return rp, cc.astype(np.int32), rng.integers(-5, 6, size=cc.size).astype(np.int32)
    x, y = rand_csr(0.3), rand_csr(0.4)
    z = B.spsyrk_accumulate(m, *[torch.from_numpy(t).cuda() for t in x], *[torch.from_numpy(t).cuda() for t in y])
    er, ec, ev = oracle.add(m, x[0], x[1], x[2].astype(np.float64), y[0], y[1], y[2].astype(np.float64))
    zr, zc, zv = _np(*z)
    assert np.array_equal(zr, er) and np.array_equal(zc, ec) and np.array_equal(zv, oracle.to_int32(ev))


# ------------------------------ symmetric permutation and equal-work row ranges (Section III-A, load balance)
@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_permute(B, idx):
    a = W.small(idx)
    d = dev(a)
    rng = np.random.default_rng(40 + idx)
    rp, cp = rng.permutation(a.m).astype(np.int32), rng.permutation(a.n).astype(np.int32)
    for cperm in (cp, None):
        got = _np(*B.spsyrk_permute(a.m, a.n, *d, torch.from_numpy(rp).cuda(), None if cperm is None else torch.from_numpy(cperm).cuda()))
        er, ec, ev = oracle.permute(a.m, a.n, a.rowptr, a.colidx, a.vals, rp, cperm)
        assert np.array_equal(got[0], er) and np.array_equal(got[1], ec)
        assert np.array_equal(got[2].astype(np.float64), ev)   # values are moved bit for bit


def test_permute_then_product(B):
    """The product of the symmetrically permuted matrix against the oracle on the same permuted input."""
    a = W.small(3)
    rng = np.random.default_rng(5)
    perm = rng.permutation(a.m).astype(np.int32)
    pt = torch.from_numpy(perm).cuda()
    b = B.spsyrk_permute(a.m, a.n, *dev(a), pt, pt)
    br, bc, bv = _np(*b)
    pa = W.CSR(a.m, a.n, br, bc, bv)
    run_and_compare(B, pa, 0)


def test_permute_edge_cases(B):
    a = W.small(1)
    d = dev(a)
    ident = torch.arange(a.m, dtype=torch.int32, device="cuda")
    got = _np(*B.spsyrk_permute(a.m, a.n, *d, ident, torch.arange(a.n, dtype=torch.int32, device="cuda")))
    assert np.array_equal(got[0], a.rowptr) and np.array_equal(got[1], a.colidx) and np.array_equal(got[2], a.vals)
    bad = ident.clone()
    bad[3] = bad[4]
    with pytest.raises(B.SpsyrkError) as ei:
        B.spsyrk_permute(a.m, a.n, *d, bad)
    assert ei.value.status == 1
    bad = ident.clone()
    bad[0] = a.m
    with pytest.raises(B.SpsyrkError):
        B.spsyrk_permute(a.m, a.n, *d, bad)
    # row pointers that leave [0, nnz] or do not end at nnz are rejected before any entry is moved by them
    for where, value in ((a.m, a.nnz + 5), (a.m, a.nnz - 1), (0, 1), (7, a.nnz + 1000)):
        badp = d[0].clone()
        badp[where] = value
        with pytest.raises(B.SpsyrkError) as ei:
            B.spsyrk_permute(a.m, a.n, badp, d[1], d[2], ident)
        assert ei.value.status == 2
    # no rows, no entries
    e = (torch.zeros(1, dtype=torch.int64, device="cuda"), torch.zeros(0, dtype=torch.int32, device="cuda"),
         torch.zeros(0, dtype=torch.float64, device="cuda"))
    assert B.spsyrk_permute(0, 5, *e, torch.zeros(0, dtype=torch.int32, device="cuda"))[0].cpu().tolist() == [0]
    z = (torch.zeros(4, dtype=torch.int64, device="cuda"), torch.zeros(0, dtype=torch.int32, device="cuda"),
         torch.zeros(0, dtype=torch.float64, device="cuda"))
    assert B.spsyrk_permute(3, 5, *z, torch.tensor([2, 0, 1], dtype=torch.int32, device="cuda"))[0].cpu().tolist() == [0, 0, 0, 0]


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_plan_partition(B, idx):
    a = W.small(idx)
    plan = B.spsyrk_plan(a.m, a.n, *dev(a))
    ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, counts_only=True)
    for parts in (1, 2, 3, 8, 64):
        assert B.spsyrk_plan_partition(plan, parts) == oracle.partition(ref.work, parts).tolist()
    # a row range: bounds are absolute row ids inside it
    r0, r1 = a.m // 4, a.m - a.m // 3
    B.spsyrk_plan_set_rows(plan, r0, r1)
    got = B.spsyrk_plan_partition(plan, 5)
    assert got == (oracle.partition(ref.work[r0:r1], 5) + r0).tolist()
    # the ranges tile the product: concatenating the parts gives the whole
    whole = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, r0, r1)
    pieces = []
    for p in range(5):
        if got[p + 1] > got[p]:
            B.spsyrk_plan_set_rows(plan, got[p], got[p + 1])
            rp = torch.empty(got[p + 1] - got[p] + 1, dtype=torch.int64, device="cuda")
            nnz = B.spsyrk_symbolic(plan, rp)
            ci = torch.empty(max(nnz, 1), dtype=torch.int32, device="cuda")
            cv = torch.empty(max(nnz, 1), dtype=torch.from_numpy(a.vals).dtype, device="cuda")
            B.spsyrk_numeric(plan, rp, ci, cv)
            pieces.append(ci[:nnz].cpu().numpy())
    assert np.array_equal(np.concatenate(pieces), whole.colidx)
    with pytest.raises(B.SpsyrkError):
        B.spsyrk_plan_partition(plan, 0)


# ------------------------------------------------------------------ rows exactly at the class boundaries
def test_rows_at_every_class_boundary(B):
    """One column shared by all rows: row i has exactly i + 1 partial products and i + 1 output entries,
    so consecutive rows walk through every class boundary (32|33, 64|65, ..., 512|513, 32768|32769).
    Structure by closed form for every row, values (single products, exact) for every entry, and rows
    around the boundaries against the oracle."""
    m = 33000
    rng = np.random.default_rng(3)
    vals = rng.standard_normal(m)
    a = W.CSR(m, 1, np.arange(m + 1, dtype=np.int64), np.zeros(m, dtype=np.int32), vals)
    for item_map in (False, True):
        rp, ci, cv, plan = B.tril_syrk(a.m, a.n, *dev(a), item_map=item_map)
        i = np.arange(m + 1, dtype=np.int64)
        assert np.array_equal(rp.cpu().numpy(), i * (i + 1) // 2)
        work, classes = B.spsyrk_plan_stats(plan)
        assert work == m * (m + 1) // 2
        # a light row is classed by its products without the diagonal one (row i has i of them here)
        assert classes == [0, 33, 32, 64, 128, 256, 32768 - 513, m - 32768]
        v = torch.from_numpy(vals).cuda()
        for r0 in range(0, m, 6000):                          # row blocks: the whole triangle at once would take tens of GB
            r1 = min(r0 + 6000, m)
            lo, hi = int(rp[r0]), int(rp[r1])
            rows = torch.repeat_interleave(torch.arange(r0, r1, device="cuda"), torch.arange(r0 + 1, r1 + 1, device="cuda"))
            cols = torch.arange(lo, hi, device="cuda") - rp[:-1][rows]
            assert torch.equal(ci[lo:hi].long(), cols)
            assert torch.equal(cv[lo:hi], v[rows] * v[cols])  # one product per entry: no rounding to differ in
            del rows, cols
        for r in (0, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257, 511, 512, 513, 8191, 8192, 32766, 32767, 32768, m - 1):
            ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, r, r + 1)
            lo, hi = int(rp[r]), int(rp[r + 1])
            assert np.array_equal(ci[lo:hi].cpu().numpy(), ref.colidx)
            assert np.array_equal(cv[lo:hi].cpu().numpy(), ref.vals)


def test_rows_with_33_nonzeros_leave_the_warp_classes(B):
    """At most 32 nonzeros fit the one-warp kernels: a row with 33 goes to the CTA kernels whatever its work."""
    m, n = 40, 33
    rng = np.random.default_rng(4)
    dense = rng.standard_normal((m, n))
    dense[::2, 32] = 0.0                                     # every other row has 32 nonzeros, the rest 33
    rr, cc = np.nonzero(dense)
    rowptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(np.bincount(rr, minlength=m), out=rowptr[1:])
    a = W.CSR(m, n, rowptr, cc.astype(np.int32), dense[rr, cc].copy())
    _, _, plan = run_and_compare(B, a, 0)
    _, classes = B.spsyrk_plan_stats(plan)
    assert sum(classes[6:]) >= m // 2
    run_and_compare(B, a, 1)


# ------------------------------------------------ binary matrices: heavy columns through bit masks
@pytest.mark.parametrize("dtype", [np.int32, np.float64])
@pytest.mark.parametrize("mode", [0, 1])
def test_binary_matrix_with_heavy_columns(B, dtype, mode):
    """All values one, a column in every row (every output row is dense), more than 64 columns with 256 or more
    entries (so only the heaviest go through the bit masks) and rows of every class."""
    rng = np.random.default_rng(31)
    m, n = 3000, 5000
    mask = rng.random((m, n)) < 0.004
    mask[:, 17] = True
    for k, dens in zip(rng.choice(n, size=90, replace=False), np.linspace(0.09, 0.9, 90)):
        mask[:, k] |= rng.random(m) < dens
    for r in (5, 1500, 2990):                                # rows of more than 255 nonzeros: their counts need full words,
        mask[r, rng.choice(n, size=400, replace=False)] = True   # the other rows pack four 8-bit counters per word
    rr, cc = np.nonzero(mask)
    rowptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(np.bincount(rr, minlength=m), out=rowptr[1:])
    assert np.diff(rowptr).max() > 255 and np.median(np.diff(rowptr)) < 255
    a = W.CSR(m, n, rowptr, cc.astype(np.int32), np.ones(cc.size, dtype=dtype))
    (rp, ci, cv), ref, plan = run_and_compare(B, a, mode)
    if dtype == np.int32 and mode == 0:
        jac = torch.empty(ci.numel(), dtype=torch.float32, device="cuda")
        B.spsyrk_plan_set_jaccard(plan, jac)
        B.spsyrk_numeric(plan, rp, ci, cv)
        exp = oracle.jaccard(0, a.m, a.rowptr, ref.rowptr, ref.colidx, oracle.to_int32(ref.vals))
        assert np.array_equal(jac.cpu().numpy(), exp)
    # the same structure with one value that is not one: the plain path must give the plain answer
    vals = np.ones(cc.size, dtype=dtype)
    vals[cc.size // 2] = 3
    run_and_compare(B, W.CSR(m, n, rowptr, cc.astype(np.int32), vals), mode)


# ------------------------------------------------ heavy rows beyond one bitmap chunk (more than 2^20 rows)
def _hub_matrix(dtype):
    """Three uniform columns per row, one column stored in 36000 scattered rows and three rows of 40
    nonzeros near the end, with more than 2^20 rows: the heavy rows sit at high row indices, so their
    output range spans several bitmap chunks of the one-CTA-per-row kernels in both passes."""
    m = n = (1 << 20) + 1000
    rng = np.random.default_rng(77)
    cols = rng.integers(0, n, size=(m, 3))
    hub_rows = np.sort(rng.choice(m, size=36000, replace=False))
    wide_rows = np.array([m - 700, m - 350, m - 2])
    lists = {}
    for r in hub_rows:
        lists[int(r)] = np.union1d(cols[r], [7])
    for r in wide_rows:
        base = lists.get(int(r), np.unique(cols[r]))
        lists[int(r)] = np.union1d(base, rng.choice(n, size=40, replace=False))
    rowptr = np.zeros(m + 1, dtype=np.int64)
    srt = np.sort(cols, axis=1)
    dup = (srt[:, 1:] == srt[:, :-1])
    base_deg = 3 - dup.sum(axis=1)
    degs = base_deg.copy()
    for r, l in lists.items():
        degs[r] = l.size
    np.cumsum(degs, out=rowptr[1:])
    colidx = np.empty(rowptr[-1], dtype=np.int32)
    keep = np.ones((m, 3), dtype=bool)
    keep[:, 1:] &= ~dup
    plain = np.ones(m, dtype=bool)
    plain[list(lists.keys())] = False
    # rows without additions: their distinct sorted columns, written in one go
    sel = keep & plain[:, None]
    pos = (rowptr[:-1][:, None] + np.cumsum(keep, axis=1) - 1)
    colidx[pos[sel]] = srt[sel]
    for r, l in lists.items():
        colidx[rowptr[r]:rowptr[r + 1]] = l
    if np.issubdtype(dtype, np.integer):
        vals = rng.integers(1, 4, size=colidx.size).astype(dtype)
    else:
        vals = rng.standard_normal(colidx.size).astype(dtype)
    return W.CSR(m, n, rowptr, colidx, vals), hub_rows, wide_rows


@pytest.mark.parametrize("dtype", [np.float64, np.int32])
@pytest.mark.parametrize("mode", [0, 1])
def test_heavy_rows_beyond_one_chunk(B, dtype, mode):
    a, hub_rows, wide_rows = _hub_matrix(dtype)
    assert np.all(np.diff(a.rowptr) >= 1)
    d = dev(a)
    rp, ci, cv, plan = B.tril_syrk(a.m, a.n, *d, mode=mode)
    _, classes = B.spsyrk_plan_stats(plan)
    assert classes[6] > 0 and classes[7] > 0, classes      # both one-CTA-per-row classes are exercised
    rp_h = rp.cpu().numpy()
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    # rows of every kind: hub rows early (short prefix), in the middle of the block class (one and several
    # accumulator tiles), in the large class, the rows with more than 32 nonzeros, and a few light neighbours
    picks = [hub_rows[10], hub_rows[600], hub_rows[3000], hub_rows[5000], hub_rows[8500], hub_rows[20000], hub_rows[33500], hub_rows[-1],
             *wide_rows, hub_rows[-1] - 1 if hub_rows[-1] - 1 not in hub_rows else hub_rows[-1] + 1, a.m - 1]
    for r in picks:
        r = int(r)
        ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode, r, r + 1, cols=cols)
        lo, hi = int(rp_h[r]), int(rp_h[r + 1])
        assert hi - lo == ref.nnz, (r, hi - lo, ref.nnz)
        assert np.array_equal(ci[lo:hi].cpu().numpy(), ref.colidx), r
        check_values(cv[lo:hi].cpu().numpy(), ref, a.vals.dtype)
    # every row's count against the closed form where there is one: a hub row's lower part holds the hub
    # rows before it (through column 7), itself, and what its other columns add
    if mode == 0:
        cnt = np.diff(rp_h)
        rank = np.arange(1, hub_rows.size + 1)
        assert np.all(cnt[hub_rows] >= rank)
