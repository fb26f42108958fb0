"""Seeded random matrices of every dtype, mode and row range, some with very heavy rows and columns,
through every entry point and against the CPU oracle.  Catches what the structured workloads do not
exercise (odd shapes, near-empty and near-dense inputs, ranges that start and end anywhere)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_09713_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    assert torch.cuda.is_available()
    from paper_2608_09713_b200 import binding
    return binding


def random_csr(rng, m, n, density, dtype, heavy):
    mask = rng.random((m, n)) < density
    if heavy:
        for _ in range(int(rng.integers(1, 4))):
            mask[rng.integers(0, m)] = rng.random(n) < 0.9
            mask[:, rng.integers(0, n)] = rng.random(m) < 0.9
    rr, cc = np.nonzero(mask)
    rowptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(np.bincount(rr, minlength=m), out=rowptr[1:])
    if dtype == np.int32:
        vals = rng.integers(-4, 5, size=cc.size).astype(np.int32)
    else:
        vals = rng.standard_normal(cc.size).astype(dtype)
    return W.CSR(m, n, rowptr, cc.astype(np.int32), vals)


def check_values(vals, ref, dtype):
    if np.issubdtype(dtype, np.integer):
        assert np.array_equal(vals, oracle.to_int32(ref.vals))
    else:
        tol = 1e-12 if dtype == np.float64 else 1e-5
        assert np.all(np.abs(vals.astype(np.float64) - ref.vals) <= tol * ref.absvals + 1e-300)


@pytest.mark.parametrize("seed", range(6))
def test_random_matrices_through_every_entry_point(B, seed):
    rng = np.random.default_rng(1000 + seed)
    for case in range(12):
        m, n = int(rng.integers(1, 700)), int(rng.integers(1, 700))
        dtype = [np.float64, np.float32, np.int32][int(rng.integers(0, 3))]
        a = random_csr(rng, m, n, float(rng.choice([0.002, 0.01, 0.05, 0.2, 0.6])), dtype, rng.random() < 0.4)
        mode = int(rng.integers(0, 2))
        r0 = int(rng.integers(0, m))
        r1 = int(rng.integers(r0, m + 1))
        if rng.random() < 0.5:
            r0, r1 = 0, m
        d = [torch.from_numpy(x).cuda() for x in (a.rowptr, a.colidx, a.vals)]
        rp, ci, cv, plan = B.tril_syrk(a.m, a.n, *d, mode=mode, row_begin=r0, row_end=r1)
        ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode, r0, r1)
        assert np.array_equal(rp.cpu().numpy(), ref.rowptr)
        assert np.array_equal(ci.cpu().numpy(), ref.colidx)
        check_values(cv.cpu().numpy(), ref, dtype)
        if r1 > r0:                                           # the same rows again, block by block
            cuts = sorted({r0, r1, *(int(x) for x in rng.integers(r0, r1 + 1, size=3))})
            crp = torch.empty(r1 - r0 + 1, dtype=torch.int64, device="cuda")
            nn = B.spsyrk_symbolic(plan, crp)
            cci = torch.full((max(nn, 1),), -3, dtype=torch.int32, device="cuda")
            ccv = torch.zeros(max(nn, 1), dtype=cv.dtype, device="cuda")
            for x0, x1 in zip(cuts[:-1], cuts[1:]):
                B.spsyrk_numeric_rows(plan, x0, x1, crp, cci, ccv)
            assert torch.equal(cci[:nn], ci)
            check_values(ccv[:nn].cpu().numpy(), ref, dtype)
        if rng.random() < 0.5:                                # a block of the product anywhere
            b0 = int(rng.integers(0, m)); b1 = int(rng.integers(b0, m + 1))
            s0 = int(rng.integers(0, m)); s1 = int(rng.integers(s0, m + 1))
            bmode = int(rng.integers(0, 2))
            bplan = B.spsyrk_plan(a.m, a.n, *d, mode=bmode)
            B.spsyrk_plan_set_block(bplan, b0, b1, s0, s1)
            brp, bci, bcv, _ = B.tril_syrk(a.m, a.n, *d, plan=bplan)
            bref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, bmode, b0, b1)
            keep = (bref.colidx >= s0) & (bref.colidx < s1)
            rows = np.repeat(np.arange(b1 - b0), np.diff(bref.rowptr))
            erp = np.zeros(b1 - b0 + 1, dtype=np.int64)
            np.cumsum(np.bincount(rows[keep], minlength=b1 - b0), out=erp[1:])
            assert np.array_equal(brp.cpu().numpy(), erp) and np.array_equal(bci.cpu().numpy(), bref.colidx[keep])

            class Kept:
                vals, absvals = bref.vals[keep], bref.absvals[keep]
            check_values(bcv.cpu().numpy(), Kept, dtype)
            B.spsyrk_destroy(bplan)
        if mode != 0 or (r0, r1) != (0, m):
            continue
        f = B.spsyrk_mirror(m, rp, ci, cv)
        e = oracle.mirror(m, ref.rowptr, ref.colidx, cv.cpu().numpy().astype(np.float64))
        assert np.array_equal(f[0].cpu().numpy(), e[0]) and np.array_equal(f[1].cpu().numpy(), e[1])
        assert np.array_equal(f[2].cpu().numpy().astype(np.float64), e[2])
        k = int(rng.integers(0, n + 1))                       # two column panels, summed
        acc = None
        for k0, k1 in ((0, k), (k, n)):
            t = B.tril_syrk(m, n, *B.spsyrk_column_panel(m, *d, k0, k1))[:3]
            acc = t if acc is None else B.spsyrk_accumulate(m, *acc, *t)
        assert torch.equal(acc[0], rp) and torch.equal(acc[1], ci)
        check_values(acc[2].cpu().numpy(), ref, dtype)
        perm, cperm = rng.permutation(m).astype(np.int32), rng.permutation(n).astype(np.int32)
        b = B.spsyrk_permute(m, n, *d, torch.from_numpy(perm).cuda(), torch.from_numpy(cperm).cuda())
        eb = oracle.permute(m, n, a.rowptr, a.colidx, a.vals, perm, cperm)
        assert np.array_equal(b[0].cpu().numpy(), eb[0]) and np.array_equal(b[1].cpu().numpy(), eb[1])
        assert np.array_equal(b[2].cpu().numpy().astype(np.float64), eb[2])
        parts = int(rng.integers(1, 9))
        assert B.spsyrk_plan_partition(plan, parts) == oracle.partition(ref.work, parts).tolist()
