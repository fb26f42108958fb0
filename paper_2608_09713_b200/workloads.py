"""Seeded synthetic CSR inputs shaped like the paper's workload classes.

The paper evaluates on random matrices of varying density (Section V-C), a Kronecker
power-law graph, rectangular incidence-like matrices (Table I) and names Jaccard
similarity on genomics data as the motivating application (Section I).  Those matrices
are not redistributed here; the five generators below are seeded stand-ins with the same
shape, degree structure and value types.

This module holds no arithmetic of the method itself (no products, no transposes): it only
draws matrices.  It is the one module that the CUDA path's tests, the benchmark and the CPU
oracle's tests all share.  Everything is a pure function of its arguments: randomness comes
from a counter-based 64-bit mixer keyed by (seed, row, slot, attempt), so the output does
not depend on numpy's generator or on any library version.

Canonical CSR is produced throughout: int64 row pointers, int32 column ids strictly
ascending inside a row, no duplicates, no explicit zeros on purpose.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_K0 = np.uint64(0x9E3779B97F4A7C15)
_K1 = np.uint64(0xBF58476D1CE4E5B9)
_K2 = np.uint64(0x94D049BB133111EB)
_KA = np.uint64(0xD6E8FEB86659FD93)
_KB = np.uint64(0xA0761D6478BD642F)
_KC = np.uint64(0xE7037ED1A0B428DB)


@dataclass
class CSR:
    """A host CSR matrix (numpy arrays)."""

    m: int
    n: int
    rowptr: np.ndarray  # int64, m+1
    colidx: np.ndarray  # int32, nnz
    vals: np.ndarray  # float64 | float32 | int32, nnz
    name: str = ""

    @property
    def nnz(self) -> int:
        return int(self.rowptr[-1])

    def row_range(self, r0: int, r1: int) -> "CSR":
        """Rows [r0, r1) as a CSR of their own (column ids unchanged)."""
        p0, p1 = int(self.rowptr[r0]), int(self.rowptr[r1])
        return CSR(r1 - r0, self.n, (self.rowptr[r0:r1 + 1] - p0).copy(),
                   self.colidx[p0:p1].copy(), self.vals[p0:p1].copy(), self.name)


def _mix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        x = x + _K0
        x ^= x >> np.uint64(30)
        x *= _K1
        x ^= x >> np.uint64(27)
        x *= _K2
        x ^= x >> np.uint64(31)
    return x


def _key(seed: int, a, b=None, c=None) -> np.ndarray:
    """64-bit hash of (seed, a[, b[, c]]); a, b, c are integer arrays that broadcast."""
    with np.errstate(over="ignore"):
        h = _mix64(np.uint64(seed) ^ (np.asarray(a).astype(np.uint64) * _KA))
        if b is not None:
            h = _mix64(h ^ (np.asarray(b).astype(np.uint64) * _KB))
        if c is not None:
            h = _mix64(h ^ (np.asarray(c).astype(np.uint64) * _KC))
    return h


def _u01(h: np.ndarray) -> np.ndarray:
    """Uniform double in [0, 1) from the top 53 bits of a hash."""
    return (h >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def _distinct_columns(m: int, dmax: int, deg: np.ndarray, n: int, draw) -> np.ndarray:
    """Draw `deg[i]` distinct columns for every row; a duplicate slot is redrawn.

    draw(rows, slots, attempts) -> int64 column ids.  Returns an (m, dmax) int64 array
    sorted inside each row, unused slots holding sentinels >= n at the end.
    """
    rows = np.arange(m, dtype=np.int64)[:, None]
    slots = np.arange(dmax, dtype=np.int64)[None, :]
    cols = draw(np.broadcast_to(rows, (m, dmax)), np.broadcast_to(slots, (m, dmax)),
                np.zeros((m, dmax), dtype=np.int64)).astype(np.int64)
    unused = slots >= deg[:, None]
    cols[unused] = (n + np.broadcast_to(slots, (m, dmax)))[unused]  # distinct sentinels
    srt = np.sort(cols, axis=1)
    bad_rows = np.nonzero((srt[:, 1:] == srt[:, :-1]).any(axis=1))[0]
    if bad_rows.size:
        sub = cols[bad_rows]
        att = np.zeros(sub.shape, dtype=np.int64)
        active = np.arange(bad_rows.size)
        while active.size:
            cur = sub[active]
            order = np.argsort(cur, axis=1, kind="stable")
            s = np.take_along_axis(cur, order, axis=1)
            dup = s[:, 1:] == s[:, :-1]
            has = dup.any(axis=1)
            if not has.any():
                break
            rr, pp = np.nonzero(dup)
            slot_idx = order[rr, pp + 1]
            g = active[rr]
            att[g, slot_idx] += 1
            sub[g, slot_idx] = draw(bad_rows[g], slot_idx, att[g, slot_idx])
            active = active[has]
        cols[bad_rows] = sub
        srt[bad_rows] = np.sort(sub, axis=1)
    return srt


def _finish(m: int, n: int, srt: np.ndarray, deg: np.ndarray, name: str) -> tuple:
    rowptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(deg, out=rowptr[1:])
    dmax = srt.shape[1]
    if (deg == dmax).all():
        colidx = srt.reshape(-1).astype(np.int32)
    else:
        keep = np.arange(dmax)[None, :] < deg[:, None]
        colidx = srt[keep].astype(np.int32)
    return rowptr, colidx


def _values(seed: int, nnz: int, dtype, lo: float, hi: float) -> np.ndarray:
    u = _u01(_key(seed ^ 0x5A17, np.arange(nnz, dtype=np.int64)))
    return (lo + (hi - lo) * u).astype(dtype)


def erdos_renyi(m: int, n: int, d: int, seed: int, dtype=np.float64,
                lo: float = 0.0, hi: float = 1.0) -> CSR:
    """Exactly `d` distinct uniform columns per row, values uniform in [lo, hi)."""
    assert d <= n

    def draw(rows, slots, attempts):
        return np.minimum((_u01(_key(seed, rows, slots, attempts)) * n).astype(np.int64), n - 1)

    deg = np.full(m, d, dtype=np.int64)
    srt = _distinct_columns(m, d, deg, n, draw)
    rowptr, colidx = _finish(m, n, srt, deg, "er")
    return CSR(m, n, rowptr, colidx, _values(seed, m * d, dtype, lo, hi), f"er_{m}x{n}_d{d}")


def zipf_binary(m: int, n: int, d: int, s: float, seed: int) -> CSR:
    """`d` distinct columns per row with ranks from a bounded Zipf(s) law, values int32 1.

    rank r in 1..n has probability proportional to r**-s (inverse-CDF sampling on a
    double-precision cumulative table); the column is perm[r-1] for a seeded permutation.
    """
    assert d <= n
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    perm = np.argsort(_key(seed ^ 0x7E57, np.arange(n, dtype=np.int64)), kind="stable")

    def draw(rows, slots, attempts):
        u = _u01(_key(seed, rows, slots, attempts))
        r = np.minimum(np.searchsorted(cdf, u, side="right"), n - 1)
        return perm[r]

    deg = np.full(m, d, dtype=np.int64)
    srt = _distinct_columns(m, d, deg, n, draw)
    rowptr, colidx = _finish(m, n, srt, deg, "zipf")
    return CSR(m, n, rowptr, colidx, np.ones(m * d, dtype=np.int32), f"zipf_{m}x{n}_d{d}")


def rmat(scale: int, edge_factor: int, seed: int, abcd=(0.57, 0.19, 0.19, 0.05),
         permute: bool = True, dtype=np.float32, lo: float = 0.5, hi: float = 1.5) -> CSR:
    """Directed R-MAT adjacency, duplicates and self-loops removed, optional relabelling."""
    nv = 1 << scale
    ne = edge_factor * nv
    a, b, c, _ = abcd
    e = np.arange(ne, dtype=np.int64)
    rows = np.zeros(ne, dtype=np.int64)
    cols = np.zeros(ne, dtype=np.int64)
    for level in range(scale):
        u = _u01(_key(seed, e, level))
        q = (u >= a).astype(np.int64) + (u >= a + b) + (u >= a + b + c)
        rows = (rows << 1) | (q >> 1)
        cols = (cols << 1) | (q & 1)
    keep = rows != cols
    rows, cols = rows[keep], cols[keep]
    if permute:
        perm = np.argsort(_key(seed ^ 0x9E11, np.arange(nv, dtype=np.int64)), kind="stable")
        rows, cols = perm[rows], perm[cols]
    code = np.unique((rows << 32) | cols)
    rows, cols = code >> 32, code & 0xFFFFFFFF
    rowptr = np.zeros(nv + 1, dtype=np.int64)
    np.cumsum(np.bincount(rows, minlength=nv), out=rowptr[1:])
    nnz = code.size
    return CSR(nv, nv, rowptr, cols.astype(np.int32), _values(seed, nnz, dtype, lo, hi),
               f"rmat_s{scale}_ef{edge_factor}{'' if permute else '_noperm'}")


def hypergraph(m: int, n: int, seed: int, band: int = 4096, outlier: float = 0.1,
               dmin: int = 2, dmax: int = 8) -> CSR:
    """Tall incidence matrix: row degree uniform in [dmin, dmax]; columns in a band of
    width `band` around row*n/m (clipped at the edges), a fraction `outlier` uniform."""
    band = min(band, n)
    span = dmax - dmin + 1
    rws = np.arange(m, dtype=np.int64)
    deg = dmin + np.minimum((_u01(_key(seed ^ 0xDE6, rws)) * span).astype(np.int64), span - 1)
    deg = np.minimum(deg, n)

    def draw(rows, slots, attempts):
        h = _key(seed, rows, slots, attempts)
        is_out = _u01(h) < outlier
        u2 = _u01(_mix64(h ^ _KC))
        centre = (np.asarray(rows, dtype=np.int64) * n) // m
        lo_ = np.clip(centre - band // 2, 0, n - band)
        inband = lo_ + np.minimum((u2 * band).astype(np.int64), band - 1)
        anywhere = np.minimum((u2 * n).astype(np.int64), n - 1)
        return np.where(is_out, anywhere, inband)

    srt = _distinct_columns(m, dmax, deg, n, draw)
    rowptr, colidx = _finish(m, n, srt, deg, "hyper")
    return CSR(m, n, rowptr, colidx, np.ones(int(rowptr[-1]), dtype=np.float64),
               f"hyper_{m}x{n}")


# --------------------------------------------------------------------------------------
# The five benchmark configurations and reduced copies of each for fast parity tests.
# --------------------------------------------------------------------------------------
SEED = 0x5EED0000

CONFIG_NAMES = {
    1: "er_4096_d8_f64",
    2: "zipf_binary_100000x4194304_d100_i32",
    3: "rmat_s18_ef16_f32",
    4: "hypergraph_2000000x500000_f64",
    5: "er_4194304_d16_f64",
}


def config(idx: int) -> CSR:
    """Full-size benchmark configuration `idx` (1..5)."""
    if idx == 1:
        a = erdos_renyi(4096, 4096, 8, SEED + 1, np.float64, 0.0, 1.0)
    elif idx == 2:
        a = zipf_binary(100_000, 1 << 22, 100, 1.1, SEED + 2)
    elif idx == 3:
        a = rmat(18, 16, SEED + 3)
    elif idx == 4:
        a = hypergraph(2_000_000, 500_000, SEED + 4)
    elif idx == 5:
        a = erdos_renyi(1 << 22, 1 << 22, 16, SEED + 5, np.float64, -1.0, 1.0)
    else:
        raise ValueError("config index must be 1..5")
    a.name = CONFIG_NAMES[idx]
    return a


def small(idx: int) -> CSR:
    """A reduced copy of configuration `idx` with the same structure, sized so that the
    CPU oracle finishes in seconds while the GPU path still spans several tiles, every
    row class and a ragged tail."""
    if idx == 1:
        return erdos_renyi(1000, 1111, 8, SEED + 11, np.float64, 0.0, 1.0)
    if idx == 2:
        return zipf_binary(3001, 1 << 17, 100, 1.1, SEED + 12)
    if idx == 3:
        return rmat(13, 16, SEED + 13)
    if idx == 4:
        return hypergraph(50_003, 12_500, SEED + 14)
    if idx == 5:
        return erdos_renyi(60_001, 60_001, 16, SEED + 15, np.float64, -1.0, 1.0)
    raise ValueError("config index must be 1..5")
