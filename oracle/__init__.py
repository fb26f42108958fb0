"""CPU oracle for tril(A * A^T), the mirror step and the Jaccard normalisation.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline leg, never by the product path.  It wraps ``spsyrk_oracle.c`` (plain,
single-threaded C compiled with gcc) through ctypes; it neither imports nor links anything
of the CUDA path.

All functions take and return numpy arrays.  Values of any input type (float64, float32,
int32) are promoted to float64, which represents them exactly; see the C file's header for
the definition that is followed and the readings taken where the paper is silent.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spsyrk_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

TRIL = 0
FULL = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-std=c99",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_transpose.argtypes = [i64, i64, p, p, p, p, p, p]
        lib.oracle_syrk_rows.argtypes = [i64, i64, p, p, p, p, p, p, ctypes.c_int, i64, i64,
                                         p, p, p, p, p, p]
        lib.oracle_mirror.argtypes = [i64, p, p, p, p, p, p]
        lib.oracle_jaccard.argtypes = [i64, i64, p, p, p, p, p]
        lib.oracle_symv.argtypes = [i64, p, p, p, p, p, p]
        lib.oracle_column_panel.argtypes = [i64, p, p, p, i64, i64, p, p, p]
        lib.oracle_add.argtypes = [i64, p, p, p, p, p, p, p, p, p]
        lib.oracle_permute.argtypes = [i64, i64, p, p, p, p, p, p, p, p]
        lib.oracle_partition.argtypes = [i64, p, i64, p]
        lib.oracle_symv.restype = ctypes.c_int
        lib.oracle_symm.argtypes = [i64, i64, p, p, p, p, p, p]
        lib.oracle_symm.restype = ctypes.c_int
        for f in (lib.oracle_transpose, lib.oracle_syrk_rows, lib.oracle_mirror, lib.oracle_jaccard):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


class ColumnLists:
    """Column lists of A: colptr (int64, n+1), rows (int32), vals (float64)."""

    def __init__(self, colptr, rows, vals):
        self.colptr, self.rows, self.vals = colptr, rows, vals


def transpose(m, n, rowptr, colidx, vals) -> ColumnLists:
    """Column lists of A, each ascending by row (counting sort over the rows in order)."""
    lib = _load()
    rowptr, colidx, vals = _c(rowptr, np.int64), _c(colidx, np.int32), _c(vals, np.float64)
    nnz = int(rowptr[m])
    colptr = np.empty(n + 1, dtype=np.int64)
    at_row = np.empty(max(nnz, 1), dtype=np.int32)
    at_val = np.empty(max(nnz, 1), dtype=np.float64)
    rc = lib.oracle_transpose(m, n, _ptr(rowptr), _ptr(colidx), _ptr(vals), _ptr(colptr),
                              _ptr(at_row), _ptr(at_val))
    assert rc == 0
    return ColumnLists(colptr, at_row[:nnz], at_val[:nnz])


class SyrkResult:
    """Rows [r0, r1) of C_L (or of the full C): tile-local rowptr, global column ids,
    float64 values, float64 sums of absolute partial products, per-row product counts."""

    def __init__(self, r0, r1, rowptr, colidx, vals, absvals, work):
        self.r0, self.r1 = r0, r1
        self.rowptr, self.colidx, self.vals, self.absvals, self.work = rowptr, colidx, vals, absvals, work

    @property
    def nnz(self):
        return int(self.rowptr[-1])


def syrk(m, n, rowptr, colidx, vals, mode=TRIL, r0=0, r1=None, cols: ColumnLists | None = None,
         counts_only=False) -> SyrkResult:
    """tril(A A^T) (mode TRIL) or A A^T (mode FULL), output rows [r0, r1)."""
    lib = _load()
    r1 = m if r1 is None else r1
    rowptr, colidx, vals = _c(rowptr, np.int64), _c(colidx, np.int32), _c(vals, np.float64)
    if cols is None:
        cols = transpose(m, n, rowptr, colidx, vals)
    rows = r1 - r0
    cnt = np.zeros(max(rows, 1), dtype=np.int64)
    work = np.zeros(max(rows, 1), dtype=np.int64)
    args = (m, n, _ptr(rowptr), _ptr(colidx), _ptr(vals), _ptr(cols.colptr), _ptr(cols.rows),
            _ptr(cols.vals), mode, r0, r1)
    rc = lib.oracle_syrk_rows(*args, _ptr(cnt), _ptr(work), None, None, None, None)
    assert rc == 0
    c_rowptr = np.zeros(rows + 1, dtype=np.int64)
    np.cumsum(cnt[:rows], out=c_rowptr[1:])
    if counts_only:
        return SyrkResult(r0, r1, c_rowptr, None, None, None, work[:rows])
    nnz = int(c_rowptr[-1])
    c_colidx = np.empty(max(nnz, 1), dtype=np.int32)
    c_vals = np.empty(max(nnz, 1), dtype=np.float64)
    c_abs = np.empty(max(nnz, 1), dtype=np.float64)
    rc = lib.oracle_syrk_rows(*args, None, None, _ptr(c_rowptr), _ptr(c_colidx), _ptr(c_vals), _ptr(c_abs))
    assert rc == 0
    return SyrkResult(r0, r1, c_rowptr, c_colidx[:nnz], c_vals[:nnz], c_abs[:nnz], work[:rows])


def to_int32(vals: np.ndarray) -> np.ndarray:
    """Integer results computed in double: check exactness and int32 range, convert."""
    r = np.rint(vals)
    assert np.array_equal(r, vals), "integer product left the exact range of double"
    assert (np.abs(r) < 2 ** 31).all(), "integer product does not fit int32"
    return r.astype(np.int32)


def mirror(m, l_rowptr, l_colidx, l_vals):
    """F = C_L + C_L^T - D as full CSR (rowptr int64, colidx int32, vals float64)."""
    lib = _load()
    l_rowptr, l_colidx, l_vals = _c(l_rowptr, np.int64), _c(l_colidx, np.int32), _c(l_vals, np.float64)
    f_rowptr = np.empty(m + 1, dtype=np.int64)
    rc = lib.oracle_mirror(m, _ptr(l_rowptr), _ptr(l_colidx), _ptr(l_vals), _ptr(f_rowptr), None, None)
    assert rc == 0, "input is not lower triangular"
    nnz = int(f_rowptr[m])
    f_colidx = np.empty(max(nnz, 1), dtype=np.int32)
    f_vals = np.empty(max(nnz, 1), dtype=np.float64)
    rc = lib.oracle_mirror(m, _ptr(l_rowptr), _ptr(l_colidx), _ptr(l_vals), _ptr(f_rowptr),
                           _ptr(f_colidx), _ptr(f_vals))
    assert rc == 0
    return f_rowptr, f_colidx[:nnz], f_vals[:nnz]


def jaccard(row_begin, rows, a_rowptr, c_rowptr, c_colidx, c_counts) -> np.ndarray:
    """float32 J = c / (|a_i| + |a_j| - c) for rows [row_begin, row_begin + rows) of C_L."""
    lib = _load()
    a_rowptr, c_rowptr = _c(a_rowptr, np.int64), _c(c_rowptr, np.int64)
    c_colidx, c_counts = _c(c_colidx, np.int32), _c(c_counts, np.int32)
    nnz = int(c_rowptr[rows])
    jac = np.empty(max(nnz, 1), dtype=np.float32)
    rc = lib.oracle_jaccard(row_begin, rows, _ptr(a_rowptr), _ptr(c_rowptr), _ptr(c_colidx),
                            _ptr(c_counts), _ptr(jac))
    assert rc == 0
    return jac[:nnz]


def symv(m, l_rowptr, l_colidx, l_vals, x):
    """(y, abs_y): y = C x = C_L x + C_L^T x - D x from the lower triangle; abs_y is the sum of the
    absolute contributions per row (the scale for rounding comparisons)."""
    lib = _load()
    l_rowptr, l_colidx, l_vals, x = _c(l_rowptr, np.int64), _c(l_colidx, np.int32), _c(l_vals, np.float64), _c(x, np.float64)
    y = np.empty(max(m, 1), dtype=np.float64)
    ay = np.empty(max(m, 1), dtype=np.float64)
    rc = lib.oracle_symv(m, _ptr(l_rowptr), _ptr(l_colidx), _ptr(l_vals), _ptr(x), _ptr(y), _ptr(ay))
    assert rc == 0
    return y[:m], ay[:m]


def symm(m, l_rowptr, l_colidx, l_vals, x):
    """(Y, abs_Y): Y = C X = C_L X + (X^T C_L)^T - D X for a dense X of shape (m, p) from the lower
    triangle (Section V-F, second equation); abs_Y holds the sums of the absolute contributions."""
    lib = _load()
    l_rowptr, l_colidx, l_vals = _c(l_rowptr, np.int64), _c(l_colidx, np.int32), _c(l_vals, np.float64)
    x = _c(x, np.float64)
    assert x.ndim == 2 and x.shape[0] == m
    p = x.shape[1]
    y = np.empty((max(m, 1), max(p, 1)), dtype=np.float64)
    ay = np.empty_like(y)
    rc = lib.oracle_symm(m, p, _ptr(l_rowptr), _ptr(l_colidx), _ptr(l_vals), _ptr(x), _ptr(y), _ptr(ay))
    assert rc == 0
    return y[:m, :p].copy(), ay[:m, :p].copy()


def column_panel(m, rowptr, colidx, vals, k0, k1):
    """A(:, [k0, k1)) as CSR with unchanged column ids (rowptr int64, colidx int32, vals float64)."""
    lib = _load()
    rowptr, colidx, vals = _c(rowptr, np.int64), _c(colidx, np.int32), _c(vals, np.float64)
    out_rowptr = np.empty(m + 1, dtype=np.int64)
    rc = lib.oracle_column_panel(m, _ptr(rowptr), _ptr(colidx), _ptr(vals), k0, k1, _ptr(out_rowptr), None, None)
    assert rc == 0
    nnz = int(out_rowptr[m])
    out_colidx = np.empty(max(nnz, 1), dtype=np.int32)
    out_vals = np.empty(max(nnz, 1), dtype=np.float64)
    rc = lib.oracle_column_panel(m, _ptr(rowptr), _ptr(colidx), _ptr(vals), k0, k1, _ptr(out_rowptr),
                                 _ptr(out_colidx), _ptr(out_vals))
    assert rc == 0
    return out_rowptr, out_colidx[:nnz], out_vals[:nnz]


def add(m, x_rowptr, x_colidx, x_vals, y_rowptr, y_colidx, y_vals):
    """Z = X + Y on sorted CSR rows: union structure, x + y where both store the entry."""
    lib = _load()
    x_rowptr, x_colidx, x_vals = _c(x_rowptr, np.int64), _c(x_colidx, np.int32), _c(x_vals, np.float64)
    y_rowptr, y_colidx, y_vals = _c(y_rowptr, np.int64), _c(y_colidx, np.int32), _c(y_vals, np.float64)
    z_rowptr = np.empty(m + 1, dtype=np.int64)
    args = (m, _ptr(x_rowptr), _ptr(x_colidx), _ptr(x_vals), _ptr(y_rowptr), _ptr(y_colidx), _ptr(y_vals))
    rc = lib.oracle_add(*args, _ptr(z_rowptr), None, None)
    assert rc == 0, "rows must be strictly ascending in column"
    nnz = int(z_rowptr[m])
    z_colidx = np.empty(max(nnz, 1), dtype=np.int32)
    z_vals = np.empty(max(nnz, 1), dtype=np.float64)
    rc = lib.oracle_add(*args, _ptr(z_rowptr), _ptr(z_colidx), _ptr(z_vals))
    assert rc == 0
    return z_rowptr, z_colidx[:nnz], z_vals[:nnz]


def permute(m, n, rowptr, colidx, vals, rperm, cperm=None):
    """B with row i of A at row rperm[i] and column k at column cperm[k] (None: columns stay);
    rows of B ascending in column.  Returns (rowptr, colidx, vals float64)."""
    lib = _load()
    rowptr, colidx, vals = _c(rowptr, np.int64), _c(colidx, np.int32), _c(vals, np.float64)
    rperm = _c(rperm, np.int32)
    cperm = None if cperm is None else _c(cperm, np.int32)
    nnz = int(rowptr[m])
    b_rowptr = np.empty(m + 1, dtype=np.int64)
    b_colidx = np.empty(max(nnz, 1), dtype=np.int32)
    b_vals = np.empty(max(nnz, 1), dtype=np.float64)
    rc = lib.oracle_permute(m, n, _ptr(rowptr), _ptr(colidx), _ptr(vals), _ptr(rperm), _ptr(cperm),
                            _ptr(b_rowptr), _ptr(b_colidx), _ptr(b_vals))
    assert rc == 0, "not a permutation"
    return b_rowptr, b_colidx[:nnz], b_vals[:nnz]


def partition(work, parts) -> np.ndarray:
    """Row bounds (parts + 1 int64) of contiguous ranges with near-equal sums of `work`."""
    lib = _load()
    work = _c(work, np.int64)
    bounds = np.empty(parts + 1, dtype=np.int64)
    rc = lib.oracle_partition(work.size, _ptr(work), parts, _ptr(bounds))
    assert rc == 0
    return bounds
