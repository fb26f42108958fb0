"""Pins for the CPU oracle: it is checked against things other than itself.

Each test names what fixes the expected value: the definition of Section II-A evaluated by
brute force, closed forms of Section III-C, the identities of Section V-F, a third-party
routine in a special case, or an independent algorithm.
"""
import os

import numpy as np
import pytest
import scipy.sparse as sp

import oracle
from paper_2608_09713_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers
def csr_from_dense(d, structure=None):
    """Canonical CSR of a dense array; `structure` (bool array) marks stored entries so
    that explicit zeros can be stored."""
    d = np.asarray(d, dtype=np.float64)
    s = (d != 0) if structure is None else np.asarray(structure, dtype=bool)
    m, n = d.shape
    rowptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(s.sum(axis=1), out=rowptr[1:])
    rr, cc = np.nonzero(s)
    return W.CSR(m, n, rowptr, cc.astype(np.int32), d[rr, cc].copy())


def brute_force(a: W.CSR, mode):
    """Pure-Python statement of the definition: for every pair (i, j) the dot product over
    the shared stored columns in ascending k, stored iff a column is shared."""
    rows = []
    for i in range(a.m):
        cols_i = {int(a.colidx[p]): float(a.vals[p]) for p in range(a.rowptr[i], a.rowptr[i + 1])}
        out = []
        for j in range(a.m if mode == oracle.FULL else i + 1):
            acc, absacc, shared, nprod = 0.0, 0.0, False, 0
            for p in range(a.rowptr[j], a.rowptr[j + 1]):
                k = int(a.colidx[p])
                if k in cols_i:
                    shared = True
                    prod = cols_i[k] * float(a.vals[p])
                    acc = acc + prod
                    absacc = absacc + abs(prod)
                    nprod += 1
            if shared:
                out.append((j, acc, absacc, nprod))
        rows.append(out)
    return rows


def check_against_brute_force(a, mode):
    ref = brute_force(a, mode)
    res = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, mode)
    for i in range(a.m):
        lo, hi = res.rowptr[i], res.rowptr[i + 1]
        assert list(res.colidx[lo:hi]) == [t[0] for t in ref[i]], f"structure of row {i}"
        # same summation order (ascending k), separate multiply and add: bit-identical
        assert list(res.vals[lo:hi]) == [t[1] for t in ref[i]], f"values of row {i}"
        assert list(res.absvals[lo:hi]) == [t[2] for t in ref[i]]
        assert res.work[i] == sum(t[3] for t in ref[i])


def random_dense(rng, m, n, density, ints=False):
    d = rng.random((m, n))
    mask = rng.random((m, n)) < density
    if ints:
        d = rng.integers(-3, 4, size=(m, n)).astype(np.float64)
        d[d == 0] = 1
    return d * mask


def scipy_tril_product(a: W.CSR):
    s = sp.csr_matrix((np.ones(a.nnz), a.colidx, a.rowptr), shape=(a.m, a.n))
    v = sp.csr_matrix((a.vals.astype(np.float64), a.colidx, a.rowptr), shape=(a.m, a.n))
    pat = sp.tril(s @ s.T, format="csr")  # pattern: counts >= 1, never cancels
    val = sp.tril(v @ v.T, format="csr")
    pat.sort_indices()
    val.sort_indices()
    return pat, val


# ----------------------------------------------------------------------- golden fixture
def load_worked_example():
    lines = [l.strip() for l in open(os.path.join(GOLDEN, "worked_example.txt")) if l.strip() and not l.startswith("#")]
    it = iter(lines)
    hdr = next(it).split()
    m, n = int(hdr[1]), int(hdr[2])
    dense = np.array([[float(x) for x in next(it).split()] for _ in range(m)])
    hdr = next(it).split()
    trip = [next(it).split() for _ in range(int(hdr[1]))]
    work = [int(x) for x in next(it).split()[1:]]
    return dense, [(int(r), int(c), float(v)) for r, c, v in trip], work


def test_worked_example():
    dense, triples, work = load_worked_example()
    a = csr_from_dense(dense)
    res = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    got = [(i, int(res.colidx[p]), float(res.vals[p])) for i in range(a.m) for p in range(res.rowptr[i], res.rowptr[i + 1])]
    assert got == triples
    assert list(res.work) == work


# ------------------------------------------------------------------ definition, tiny inputs
@pytest.mark.parametrize("mode", [oracle.TRIL, oracle.FULL])
@pytest.mark.parametrize("seed", range(6))
def test_brute_force_random(seed, mode):
    rng = np.random.default_rng(seed)
    m, n = int(rng.integers(1, 40)), int(rng.integers(1, 40))
    a = csr_from_dense(random_dense(rng, m, n, rng.choice([0.05, 0.2, 0.6])) - 0.3 * (seed % 2))
    check_against_brute_force(a, mode)


@pytest.mark.parametrize("mode", [oracle.TRIL, oracle.FULL])
def test_brute_force_edge_cases(mode):
    rng = np.random.default_rng(99)
    cases = []
    d = random_dense(rng, 12, 9, 0.3); d[3, :] = 0; d[7, :] = 0; d[:, 2] = 0          # empty rows / column
    cases.append(csr_from_dense(d))
    d = random_dense(rng, 10, 8, 0.2); d[4, :] = rng.random(8) + 0.1                   # a full row
    cases.append(csr_from_dense(d))
    d = random_dense(rng, 10, 8, 0.2); d[:, 5] = rng.random(10) + 0.1                  # a full column
    cases.append(csr_from_dense(d))
    d = random_dense(rng, 9, 7, 0.4); d[6] = d[2]; d[8] = d[2]                          # identical rows
    cases.append(csr_from_dense(d))
    cases.append(csr_from_dense(np.array([[2.0, 0.0, 3.0]])))                          # m = 1
    cases.append(csr_from_dense(np.array([[2.0], [0.0], [5.0], [1.0]])))               # n = 1
    cases.append(csr_from_dense(np.zeros((5, 4))))                                     # nnz = 0
    cases.append(csr_from_dense(np.zeros((0, 4)).reshape(0, 4)))                       # m = 0
    for a in cases:
        check_against_brute_force(a, mode)


def test_structural_zeros_are_kept():
    """Products that cancel, and explicit zeros of A, still give stored entries."""
    d = np.array([[1.0, 1.0, 0.0], [1.0, -1.0, 0.0], [0.0, 0.0, 0.0]])
    s = np.array([[1, 1, 0], [1, 1, 0], [0, 0, 1]], dtype=bool)  # (2,2) is an explicit zero
    a = csr_from_dense(d, s)
    res = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    assert list(res.rowptr) == [0, 1, 3, 4]
    assert list(res.colidx) == [0, 0, 1, 2]
    assert list(res.vals) == [2.0, 0.0, 2.0, 0.0]
    check_against_brute_force(a, oracle.TRIL)


# --------------------------------------------------- small copies of the five workloads
@pytest.fixture(scope="module", params=[1, 2, 3, 4, 5])
def small_case(request):
    a = W.small(request.param)
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    tril = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, cols=cols)
    return request.param, a, cols, tril


def test_transpose_matches_scipy_csc(small_case):
    _, a, cols, _ = small_case
    csc = sp.csr_matrix((a.vals.astype(np.float64), a.colidx, a.rowptr), shape=(a.m, a.n)).tocsc()
    csc.sort_indices()
    assert np.array_equal(cols.colptr, csc.indptr)
    assert np.array_equal(cols.rows, csc.indices)
    assert np.array_equal(cols.vals, csc.data)


def test_matches_scipy_product(small_case):
    """Third-party routine: scipy's SpGEMM, then tril.  Structure from the pattern product
    (cannot cancel), values within rounding of the sum of absolute partial products."""
    _, a, _, tril = small_case
    pat, val = scipy_tril_product(a)
    assert np.array_equal(tril.rowptr, pat.indptr)
    assert np.array_equal(tril.colidx, pat.indices)
    dense_lookup = val.tocsr()
    rows = np.repeat(np.arange(a.m), np.diff(tril.rowptr))
    ref = np.asarray(dense_lookup[rows, tril.colidx]).ravel()
    assert np.all(np.abs(ref - tril.vals) <= 1e-13 * np.maximum(tril.absvals, 1e-300))


def test_independent_algorithm_expand_sort_compress(small_case):
    """Outer-product formulation: every column k contributes a_ik a_jk for all pairs of its
    rows; sort the triples by (i, j) and reduce.  Shares nothing with the row-wise oracle."""
    idx, a, cols, tril = small_case
    if idx == 2:
        pytest.skip("pair expansion of the Zipf case is too large for this check")
    d = np.diff(cols.colptr)
    ii, jj, vv = [], [], []
    for k in np.nonzero(d)[0]:
        r = cols.rows[cols.colptr[k]:cols.colptr[k + 1]].astype(np.int64)
        v = cols.vals[cols.colptr[k]:cols.colptr[k + 1]]
        i, j = np.meshgrid(r, r, indexing="ij")
        keep = j <= i
        ii.append(i[keep]); jj.append(j[keep]); vv.append(np.outer(v, v)[keep])
    ii, jj, vv = np.concatenate(ii), np.concatenate(jj), np.concatenate(vv)
    code = ii * a.m + jj
    order = np.argsort(code, kind="stable")
    code, vv = code[order], vv[order]
    uniq, start = np.unique(code, return_index=True)
    sums = np.add.reduceat(vv, start)
    rows = np.repeat(np.arange(a.m), np.diff(tril.rowptr))
    assert np.array_equal(uniq, rows * a.m + tril.colidx)
    assert np.all(np.abs(sums - tril.vals) <= 1e-13 * np.maximum(tril.absvals, 1e-300))
    assert ii.size == tril.work.sum()


def test_diagonal_is_squared_row_norm(small_case):
    _, a, _, tril = small_case
    deg = np.diff(a.rowptr)
    rows = np.repeat(np.arange(a.m), np.diff(tril.rowptr))
    on_diag = rows == tril.colidx
    assert np.array_equal(np.nonzero(deg > 0)[0], rows[on_diag])        # present iff row non-empty
    sq = np.zeros(a.m)
    np.add.at(sq, np.repeat(np.arange(a.m), deg), a.vals.astype(np.float64) ** 2)
    d = tril.vals[on_diag]
    assert np.allclose(d, sq[deg > 0], rtol=1e-14, atol=0)
    # the diagonal entry is the last of its row
    assert np.array_equal(np.nonzero(on_diag)[0], tril.rowptr[1:][deg > 0] - 1)


def test_work_closed_forms(small_case):
    """Multiply-add count: sum_k d_k^2 for A A^T (Section III-C); pairs j <= i inside a
    column number d_k (d_k + 1) / 2."""
    _, a, cols, tril = small_case
    d = np.diff(cols.colptr)
    assert tril.work.sum() == (d * (d + 1) // 2).sum()
    full = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.FULL, cols=cols, counts_only=True)
    assert full.work.sum() == (d * d).sum()
    # per row: sum over the row's columns of the column's length
    assert np.array_equal(full.work, np.add.reduceat(np.append(d[a.colidx], 0), a.rowptr[:-1]) * (np.diff(a.rowptr) > 0))


def test_spmv_identity(small_case):
    """Section V-F: C x = C_L x + (x^T C_L)^T - D x, and C x = A (A^T x)."""
    _, a, _, tril = small_case
    rng = np.random.default_rng(5)
    x = rng.standard_normal(a.m)
    A = sp.csr_matrix((a.vals.astype(np.float64), a.colidx, a.rowptr), shape=(a.m, a.n))
    L = sp.csr_matrix((tril.vals, tril.colidx, tril.rowptr), shape=(a.m, a.m))
    lhs = L @ x + L.T @ x - L.diagonal() * x
    rhs = A @ (A.T @ x)
    scale = sp.csr_matrix((tril.absvals, tril.colidx, tril.rowptr), shape=(a.m, a.m))
    bound = (scale + scale.T) @ np.abs(x) + 1e-300
    assert np.all(np.abs(lhs - rhs) <= 1e-12 * bound)


def test_sum_identity(small_case):
    """2 sum(C_L) - trace = sum_k (sum_i a_ik)^2."""
    _, a, cols, tril = small_case
    rows = np.repeat(np.arange(a.m), np.diff(tril.rowptr))
    tr = tril.vals[rows == tril.colidx].sum()
    colsum = np.zeros(a.n)
    np.add.at(colsum, a.colidx, a.vals.astype(np.float64))
    lhs, rhs = 2 * tril.vals.sum() - tr, (colsum ** 2).sum()
    assert abs(lhs - rhs) <= 1e-10 * tril.absvals.sum()


def test_tril_is_half_of_full(small_case):
    idx, a, cols, tril = small_case
    full = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.FULL, cols=cols)
    F = sp.csr_matrix((full.vals, full.colidx, full.rowptr), shape=(a.m, a.m))
    S = sp.csr_matrix((np.ones(full.nnz), full.colidx, full.rowptr), shape=(a.m, a.m))
    assert (S != S.T).nnz == 0                                          # symmetric structure
    assert abs(F - F.T).max() <= 1e-12 * max(full.absvals.max(), 1e-300)
    rows = np.repeat(np.arange(a.m), np.diff(full.rowptr))
    low = full.colidx <= rows
    assert np.array_equal(full.colidx[low], tril.colidx)
    assert np.array_equal(full.vals[low], tril.vals)                     # same order of sums
    assert full.nnz == 2 * tril.nnz - int((np.diff(a.rowptr) > 0).sum())
    # counts bound
    cnt = np.diff(tril.rowptr)
    assert np.all(cnt <= np.minimum(tril.work, np.arange(a.m) + 1))
    assert np.array_equal(cnt >= 1, np.diff(a.rowptr) > 0)


def test_row_tiles_concatenate(small_case):
    _, a, cols, tril = small_case
    cuts = [0, a.m // 5, a.m // 5 + 1, a.m // 2, a.m]
    colidx, vals, counts = [], [], []
    for r0, r1 in zip(cuts[:-1], cuts[1:]):
        t = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, r0, r1, cols=cols)
        assert t.rowptr[0] == 0
        colidx.append(t.colidx); vals.append(t.vals); counts.append(np.diff(t.rowptr))
    assert np.array_equal(np.concatenate(counts), np.diff(tril.rowptr))
    assert np.array_equal(np.concatenate(colidx), tril.colidx)
    assert np.array_equal(np.concatenate(vals), tril.vals)


# -------------------------------------------------------------------------- binary input
def test_binary_counts_are_set_intersections():
    a = W.small(2)
    tril = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    counts = oracle.to_int32(tril.vals)
    sets = [set(a.colidx[a.rowptr[i]:a.rowptr[i + 1]].tolist()) for i in range(a.m)]
    rng = np.random.default_rng(3)
    rows = np.repeat(np.arange(a.m), np.diff(tril.rowptr))
    for p in rng.integers(0, tril.nnz, size=4000):
        assert counts[p] == len(sets[rows[p]] & sets[int(tril.colidx[p])])
    assert np.all(counts[rows == tril.colidx] == 100)                    # c_ii = nnz(a_i)
    # pairs that are not stored share nothing
    stored = set(zip(rows.tolist(), tril.colidx.tolist()))
    for _ in range(2000):
        i = int(rng.integers(0, a.m)); j = int(rng.integers(0, i + 1))
        assert ((i, j) in stored) == (len(sets[i] & sets[j]) > 0)


def test_zipf_top_column_makes_output_dense():
    a = W.small(2)
    d = np.bincount(a.colidx, minlength=a.n)
    tril = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, counts_only=True)
    if d.max() == a.m:
        assert tril.nnz == a.m * (a.m + 1) // 2


# ------------------------------------------------------------------------------- mirror
def test_mirror_invariants(small_case):
    idx, a, cols, tril = small_case
    f_rowptr, f_colidx, f_vals = oracle.mirror(a.m, tril.rowptr, tril.colidx, tril.vals)
    full = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.FULL, cols=cols)
    assert np.array_equal(f_rowptr, full.rowptr)                         # same structure as A A^T
    assert np.array_equal(f_colidx, full.colidx)
    assert np.all(np.abs(f_vals - full.vals) <= 1e-12 * np.maximum(full.absvals, 1e-300))
    F = sp.csr_matrix((f_vals, f_colidx, f_rowptr), shape=(a.m, a.m))
    Ft = F.T.tocsr(); Ft.sort_indices()
    assert np.array_equal(Ft.indptr, f_rowptr) and np.array_equal(Ft.indices, f_colidx)
    assert np.array_equal(Ft.data, f_vals)                               # exactly symmetric
    rows = np.repeat(np.arange(a.m), np.diff(f_rowptr))
    low = f_colidx <= rows
    assert np.array_equal(f_colidx[low], tril.colidx) and np.array_equal(f_vals[low], tril.vals)
    ndiag = int((np.diff(a.rowptr) > 0).sum())
    assert f_rowptr[-1] == 2 * tril.nnz - ndiag


def test_mirror_tiny_by_hand():
    # C_L = [[5],[., 9],[14, ., 42]]  ->  F row 0 = (0:5, 2:14), row 1 = (1:9), row 2 = (0:14, 2:42)
    f_rowptr, f_colidx, f_vals = oracle.mirror(3, [0, 1, 2, 4], [0, 1, 0, 2], [5.0, 9.0, 14.0, 42.0])
    assert list(f_rowptr) == [0, 2, 3, 5]
    assert list(f_colidx) == [0, 2, 1, 0, 2]
    assert list(f_vals) == [5.0, 14.0, 9.0, 14.0, 42.0]


def test_mirror_rejects_upper_entries():
    with pytest.raises(AssertionError):
        oracle.mirror(2, [0, 1, 2], [1, 1], [1.0, 1.0])


# ------------------------------------------------------------------------------ jaccard
def test_jaccard_set_formula():
    a = W.zipf_binary(257, 4096, 20, 1.1, 77)
    tril = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    counts = oracle.to_int32(tril.vals)
    jac = oracle.jaccard(0, a.m, a.rowptr, tril.rowptr, tril.colidx, counts)
    sets = [set(a.colidx[a.rowptr[i]:a.rowptr[i + 1]].tolist()) for i in range(a.m)]
    rows = np.repeat(np.arange(a.m), np.diff(tril.rowptr))
    for p in range(tril.nnz):
        si, sj = sets[rows[p]], sets[int(tril.colidx[p])]
        assert jac[p] == np.float32(len(si & sj)) / np.float32(len(si | sj))
    assert np.all(jac[rows == tril.colidx] == 1.0)
    assert np.all((jac > 0) & (jac <= 1))
    # a tile gives the same numbers
    r0, r1 = 100, 180
    t = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, r0, r1)
    jt = oracle.jaccard(r0, r1 - r0, a.rowptr, t.rowptr, t.colidx, oracle.to_int32(t.vals))
    assert np.array_equal(jt, jac[tril.rowptr[r0]:tril.rowptr[r1]])


def test_jaccard_identical_rows_give_one():
    d = np.zeros((4, 6)); d[0, [1, 3]] = 1; d[1, [1, 3]] = 1; d[2, [1, 2]] = 1; d[3, [5]] = 1
    a = csr_from_dense(d)
    tril = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL)
    jac = oracle.jaccard(0, a.m, a.rowptr, tril.rowptr, tril.colidx, oracle.to_int32(tril.vals))
    rows = np.repeat(np.arange(a.m), np.diff(tril.rowptr))
    lookup = {(int(r), int(c)): float(j) for r, c, j in zip(rows, tril.colidx, jac)}
    assert lookup[(1, 0)] == 1.0
    assert lookup[(2, 0)] == np.float32(1) / np.float32(3)
    assert (3, 0) not in lookup


# -------------------------------------------------------------------- triangular SpMV
def test_symv_equals_a_at_x(small_case):
    """Section V-F: C x from the lower triangle equals A (A^T x), and equals scipy's product with the
    mirrored matrix."""
    _, a, _, tril = small_case
    rng = np.random.default_rng(8)
    x = rng.standard_normal(a.m)
    y, ay = oracle.symv(a.m, tril.rowptr, tril.colidx, tril.vals, x)
    A = sp.csr_matrix((a.vals.astype(np.float64), a.colidx, a.rowptr), shape=(a.m, a.n))
    ref = A @ (A.T @ x)
    absA = abs(A)
    bound = absA @ (absA.T @ np.abs(x)) + 1e-300
    assert np.all(np.abs(y - ref) <= 1e-12 * bound)
    f_rowptr, f_colidx, f_vals = oracle.mirror(a.m, tril.rowptr, tril.colidx, tril.vals)
    F = sp.csr_matrix((f_vals, f_colidx, f_rowptr), shape=(a.m, a.m))
    assert np.all(np.abs(y - F @ x) <= 1e-13 * (ay + 1e-300))


def test_symv_tiny_by_hand():
    # C_L = [[5], [., 9], [14, ., 42]], x = (1, 2, 3): C x = (5 + 42, 18, 14 + 126)
    y, _ = oracle.symv(3, [0, 1, 2, 4], [0, 1, 0, 2], [5.0, 9.0, 14.0, 42.0], [1.0, 2.0, 3.0])
    assert list(y) == [47.0, 18.0, 140.0]


@pytest.mark.parametrize("p", [1, 3, 8])
def test_symm_equals_a_at_x(small_case, p):
    """Section V-F, second equation: C X from the lower triangle equals A (A^T X) (the paper's own
    alternative evaluation) and scipy's product of the mirrored matrix with X; one column is the
    vector form."""
    _, a, _, tril = small_case
    rng = np.random.default_rng(80 + p)
    x = rng.standard_normal((a.m, p))
    y, ay = oracle.symm(a.m, tril.rowptr, tril.colidx, tril.vals, x)
    A = sp.csr_matrix((a.vals.astype(np.float64), a.colidx, a.rowptr), shape=(a.m, a.n))
    ref = A @ (A.T @ x)
    absA = abs(A)
    bound = absA @ (absA.T @ np.abs(x)) + 1e-300
    assert np.all(np.abs(y - ref) <= 1e-12 * bound)
    f_rowptr, f_colidx, f_vals = oracle.mirror(a.m, tril.rowptr, tril.colidx, tril.vals)
    F = sp.csr_matrix((f_vals, f_colidx, f_rowptr), shape=(a.m, a.m))
    assert np.all(np.abs(y - F @ x) <= 1e-13 * (ay + 1e-300))
    for c in range(p):                                   # every column on its own is the vector identity
        yc, _ = oracle.symv(a.m, tril.rowptr, tril.colidx, tril.vals, x[:, c])
        assert np.array_equal(yc, y[:, c])


def test_symm_tiny_by_hand():
    # C_L = [[5], [., 9], [14, ., 42]], so C = [[5, 0, 14], [0, 9, 0], [14, 0, 42]];
    # X = [[1, 0], [2, 1], [3, -1]]: C X = [[5 + 42, -14], [18, 9], [14 + 126, -42]]
    y, ay = oracle.symm(3, [0, 1, 2, 4], [0, 1, 0, 2], [5.0, 9.0, 14.0, 42.0], [[1.0, 0.0], [2.0, 1.0], [3.0, -1.0]])
    assert y.tolist() == [[47.0, -14.0], [18.0, 9.0], [140.0, -42.0]]
    # a wrong sign on the diagonal term or a missing reflected term changes these; a transposed X cannot be passed
    assert ay.tolist() == [[5.0 + 42.0 + 5.0 + 5.0, 14.0], [18.0 * 3, 9.0 * 3], [14.0 + 126.0 + 126.0 + 126.0, 42.0 * 3]]


def test_symm_degenerate_shapes():
    y, _ = oracle.symm(0, [0], [], [], np.zeros((0, 4)))
    assert y.shape == (0, 4)
    y, _ = oracle.symm(2, [0, 0, 0], [], [], np.ones((2, 3)))       # an empty triangle gives zeros
    assert np.array_equal(y, np.zeros((2, 3)))
    y, _ = oracle.symm(2, [0, 1, 2], [0, 1], [2.0, 3.0], np.array([[1.0], [4.0]]))   # diagonal only: counted once
    assert y.tolist() == [[2.0], [12.0]]


# ------------------------------------------------- accumulating form over column panels
def dense_add_reference(x, sx, y, sy):
    """Dense statement of Z = X + Y with explicit structure masks: stored iff stored in either."""
    rows = []
    for i in range(x.shape[0]):
        out = []
        for j in range(x.shape[1]):
            if sx[i, j] and sy[i, j]:
                out.append((j, x[i, j] + y[i, j]))
            elif sx[i, j]:
                out.append((j, x[i, j]))
            elif sy[i, j]:
                out.append((j, y[i, j]))
        rows.append(out)
    return rows


@pytest.mark.parametrize("seed", range(4))
def test_add_dense_brute_force(seed):
    """Pin: the definition of a sparse sum evaluated entry by entry on dense arrays, with stored
    zeros on both sides and values that cancel (the entry stays stored)."""
    rng = np.random.default_rng(100 + seed)
    m, n = 13, 17
    x = rng.integers(-2, 3, size=(m, n)).astype(np.float64)
    y = rng.integers(-2, 3, size=(m, n)).astype(np.float64)
    sx, sy = rng.random((m, n)) < 0.3, rng.random((m, n)) < 0.3
    sx[3], sy[5], sx[7], sy[7] = False, False, False, False  # empty rows on either side and on both
    cx, cy = csr_from_dense(x, sx), csr_from_dense(y, sy)
    zr, zc, zv = oracle.add(m, cx.rowptr, cx.colidx, cx.vals, cy.rowptr, cy.colidx, cy.vals)
    ref = dense_add_reference(x, sx, y, sy)
    for i in range(m):
        assert list(zip(zc[zr[i]:zr[i + 1]], zv[zr[i]:zr[i + 1]])) == ref[i]
    assert zr[m] == (sx | sy).sum()


def test_add_matches_scipy_on_positive_values():
    """Pin: scipy's CSR addition (third party); positive values, so it prunes nothing."""
    rng = np.random.default_rng(7)
    x = sp.random(200, 300, density=0.05, random_state=rng, format="csr", data_rvs=lambda k: rng.random(k) + 0.5)
    y = sp.random(200, 300, density=0.08, random_state=rng, format="csr", data_rvs=lambda k: rng.random(k) + 0.5)
    x.sort_indices(); y.sort_indices()
    zr, zc, zv = oracle.add(200, x.indptr, x.indices, x.data, y.indptr, y.indices, y.data)
    z = (x + y).tocsr()
    z.sort_indices()
    assert np.array_equal(zr, z.indptr) and np.array_equal(zc, z.indices)
    assert np.array_equal(zv, z.data)  # one addition per shared entry on both sides


def test_add_rejects_unsorted_rows():
    rowptr = np.array([0, 2], dtype=np.int64)
    bad = np.array([3, 1], dtype=np.int32)
    ok = np.array([1, 3], dtype=np.int32)
    v = np.ones(2)
    with pytest.raises(AssertionError):
        oracle.add(1, rowptr, bad, v, rowptr, ok, v)


def test_column_panel_matches_scipy_slice(small_case):
    """Pin: scipy column slicing (third party) for the panel's structure and values."""
    _, a, _, _ = small_case
    s = sp.csr_matrix((a.vals.astype(np.float64), a.colidx, a.rowptr), shape=(a.m, a.n))
    for k0, k1 in [(0, a.n), (0, a.n // 3), (a.n // 3, a.n // 3), (a.n // 3, a.n - 1), (a.n - 1, a.n)]:
        pr, pc, pv = oracle.column_panel(a.m, a.rowptr, a.colidx, a.vals, k0, k1)
        ref = s[:, k0:k1].tocsr()
        ref.sort_indices()
        assert np.array_equal(pr, ref.indptr)
        assert np.array_equal(pc, ref.indices + k0)
        assert np.array_equal(pv, ref.data)


@pytest.mark.parametrize("npanels", [1, 2, 5])
def test_panel_products_sum_to_the_whole(small_case, npanels):
    """Pin: Section III-A, C_ii = sum_s SYRK(A_is).  The union of the panel structures is the
    structure of tril(A A^T) exactly; the values agree to rounding (exactly for integer-valued
    inputs, where every partial sum is exact)."""
    cfg, a, _, tril = small_case
    edges = np.linspace(0, a.n, npanels + 1).astype(np.int64)
    acc = (np.zeros(a.m + 1, dtype=np.int64), np.zeros(0, dtype=np.int32), np.zeros(0))
    for s in range(npanels):
        pr, pc, pv = oracle.column_panel(a.m, a.rowptr, a.colidx, a.vals, int(edges[s]), int(edges[s + 1]))
        t = oracle.syrk(a.m, a.n, pr, pc, pv, oracle.TRIL)
        acc = oracle.add(a.m, *acc, t.rowptr, t.colidx, t.vals)
    zr, zc, zv = acc
    assert np.array_equal(zr, tril.rowptr) and np.array_equal(zc, tril.colidx)
    if cfg in (2, 4):  # integer-valued inputs
        assert np.array_equal(zv, tril.vals)
    else:
        assert np.all(np.abs(zv - tril.vals) <= 1e-13 * tril.absvals)


# ------------------------------------- symmetric permutation and row ranges of equal work
@pytest.mark.parametrize("seed", range(3))
def test_permute_dense_definition(seed):
    """Pin: B[rperm[i], cperm[k]] = A[i, k] evaluated on dense arrays, stored zeros kept."""
    rng = np.random.default_rng(300 + seed)
    m, n = 11, 14
    d = rng.integers(-3, 4, size=(m, n)).astype(np.float64)
    st = rng.random((m, n)) < 0.35
    st[4] = False
    a = csr_from_dense(d, st)
    rp, cp = rng.permutation(m).astype(np.int32), rng.permutation(n).astype(np.int32)
    for cperm in (cp, None):
        br, bc, bv = oracle.permute(m, n, a.rowptr, a.colidx, a.vals, rp, cperm)
        eb, es = np.zeros((m, n)), np.zeros((m, n), dtype=bool)
        cmap = np.arange(n) if cperm is None else cperm
        for i in range(m):
            for k in range(n):
                if st[i, k]:
                    eb[rp[i], cmap[k]] = d[i, k]
                    es[rp[i], cmap[k]] = True
        e = csr_from_dense(eb, es)
        assert np.array_equal(br, e.rowptr) and np.array_equal(bc, e.colidx) and np.array_equal(bv, e.vals)


def test_permute_matches_scipy_indexing(small_case):
    """Pin: scipy fancy indexing (third party): B = A[inv_r][:, inv_c]."""
    cfg, a, _, _ = small_case
    rng = np.random.default_rng(cfg)
    rp, cp = rng.permutation(a.m).astype(np.int32), rng.permutation(a.n).astype(np.int32)
    s = sp.csr_matrix((a.vals.astype(np.float64), a.colidx, a.rowptr), shape=(a.m, a.n))
    inv_r, inv_c = np.argsort(rp), np.argsort(cp)
    ref = s[inv_r][:, inv_c].tocsr()
    ref.sort_indices()
    br, bc, bv = oracle.permute(a.m, a.n, a.rowptr, a.colidx, a.vals, rp, cp)
    assert np.array_equal(br, ref.indptr) and np.array_equal(bc, ref.indices) and np.array_equal(bv, ref.data)


def test_permuted_product_is_permuted_product():
    """Pin: (P A)(P A)^T = P (A A^T) P^T, so the full product of the permuted matrix is the
    symmetric permutation of the full product; a column permutation changes nothing but the order
    of the additions (integer values: exact)."""
    a = W.small(4)
    rng = np.random.default_rng(9)
    rp, cp = rng.permutation(a.m).astype(np.int32), rng.permutation(a.n).astype(np.int32)
    full = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.FULL)
    b = oracle.permute(a.m, a.n, a.rowptr, a.colidx, a.vals, rp, cp)
    fb = oracle.syrk(a.m, a.n, *b, oracle.FULL)
    pr, pc, pv = oracle.permute(a.m, a.m, full.rowptr, full.colidx, full.vals, rp, rp)
    assert np.array_equal(fb.rowptr, pr) and np.array_equal(fb.colidx, pc) and np.array_equal(fb.vals, pv)


def test_permute_rejects_non_permutations():
    a = W.small(1)
    bad = np.zeros(a.m, dtype=np.int32)
    with pytest.raises(AssertionError):
        oracle.permute(a.m, a.n, a.rowptr, a.colidx, a.vals, bad)


def test_partition_definition_and_invariants(small_case):
    """Pin: the definition by brute force (exact integer arithmetic in Python), plus what any such
    split must satisfy: monotone bounds covering all rows, and no part heavier than its share by
    more than one row's work."""
    _, a, _, tril = small_case
    work = tril.work
    total = int(work.sum())
    prefix = np.concatenate([[0], np.cumsum(work)])
    for parts in (1, 2, 3, 8, 64):
        b = oracle.partition(work, parts)
        assert b[0] == 0 and b[parts] == a.m and np.all(np.diff(b) >= 0)
        for p in range(1, parts):
            r = next(r for r in range(a.m + 1) if int(prefix[r]) * parts >= p * total)
            assert b[p] == r
        share = [int(prefix[b[p + 1]] - prefix[b[p]]) for p in range(parts)]
        assert sum(share) == total
        assert max(share) <= total / parts + int(work.max()) + 1


def test_partition_degenerate():
    assert oracle.partition(np.zeros(5, dtype=np.int64), 3).tolist() == [0, 0, 0, 5]
    assert oracle.partition(np.zeros(0, dtype=np.int64), 2).tolist() == [0, 0, 0]
    assert oracle.partition(np.array([7], dtype=np.int64), 4).tolist() == [0, 1, 1, 1, 1]
