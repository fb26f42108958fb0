"""The seeded generators: canonical CSR, stated shapes and degrees, reproducible."""
import numpy as np
import pytest

from paper_2608_09713_b200 import workloads as W


def is_canonical(a):
    assert a.rowptr.dtype == np.int64 and a.colidx.dtype == np.int32
    assert a.rowptr[0] == 0 and a.rowptr[-1] == a.colidx.size == a.vals.size
    deg = np.diff(a.rowptr)
    assert (deg >= 0).all()
    if a.nnz:
        assert a.colidx.min() >= 0 and a.colidx.max() < a.n
        rows = np.repeat(np.arange(a.m), deg)
        same = rows[1:] == rows[:-1]
        assert np.all((a.colidx[1:] > a.colidx[:-1]) | ~same)
    return deg


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_small_configs_canonical_and_reproducible(idx):
    a, b = W.small(idx), W.small(idx)
    is_canonical(a)
    assert np.array_equal(a.rowptr, b.rowptr) and np.array_equal(a.colidx, b.colidx)
    assert np.array_equal(a.vals, b.vals)


def test_config1_shape_and_values():
    a = W.config(1)
    deg = is_canonical(a)
    assert (a.m, a.n, a.nnz) == (4096, 4096, 32768) and (deg == 8).all()
    assert a.vals.dtype == np.float64 and a.vals.min() >= 0 and a.vals.max() < 1


def test_zipf_degrees_and_skew():
    a = W.zipf_binary(2000, 1 << 16, 100, 1.1, 5)
    deg = is_canonical(a)
    assert (deg == 100).all() and a.vals.dtype == np.int32 and (a.vals == 1).all()
    d = np.sort(np.bincount(a.colidx, minlength=a.n))[::-1]
    assert d[0] >= 0.99 * a.m and d[100] < 0.3 * a.m          # a few columns in nearly every row


def test_rmat_properties():
    a = W.rmat(12, 16, 9)
    deg = is_canonical(a)
    rows = np.repeat(np.arange(a.m), deg)
    assert (rows != a.colidx).all()                            # no self-loops
    assert a.vals.dtype == np.float32 and a.vals.min() >= 0.5 and a.vals.max() < 1.5
    assert deg.max() > 20 * deg.mean() and (deg == 0).sum() > 0.2 * a.m   # power law, many empty rows
    b = W.rmat(12, 16, 9, permute=False)
    assert b.nnz == a.nnz


def test_hypergraph_band():
    a = W.hypergraph(40_000, 10_000, 3, band=512)
    deg = is_canonical(a)
    assert deg.min() >= 2 and deg.max() <= 8 and set(np.unique(deg)) == set(range(2, 9))
    rows = np.repeat(np.arange(a.m), deg)
    centre = rows * a.n // a.m
    far = np.abs(a.colidx - centre) > 512
    assert 0.05 < far.mean() < 0.15                            # about 10 % outliers
    assert (a.vals == 1.0).all()


def test_row_range_view():
    a = W.small(1)
    t = a.row_range(10, 20)
    assert t.m == 10 and t.rowptr[0] == 0 and t.nnz == 80
    assert np.array_equal(t.colidx, a.colidx[80:160])
