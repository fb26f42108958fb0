// The accumulating form of the local product (Section III-A: C_ii = sum over s of SYRK(A_is);
// Algorithm 2 line 2: C_local += SYRK(A_recv)).
//
//   spsyrk_column_panel : A_s = A(:, [k0, k1)), the operand of one term of the sum;
//   spsyrk_accumulate   : Z = X + Y on sorted CSR rows, the "+=" itself.
//
// The sum works row by row: G lanes per row when rows are short, one warp walking both rows in
// windows when they are longer (add_merge_kernel).  Both input rows are ascending, so an entry's
// place in the merged row is
//     its own index + the number of entries of the other row below it - the matches below it,
// where a match is a column stored in both rows (it is emitted once, from X's side, with x + y).
// The other row's count is a binary search; the matches below come from a running count over the
// row, advanced G entries at a time with a vote inside the group.
#include <algorithm>

#include "common.cuh"

using namespace spsyrk;

namespace {

constexpr size_t ALIGN = 256;

int group_width(int64_t nnz, int64_t m) {
    const double avg = m > 0 ? (double)nnz / (double)m : 0.0;
    return avg <= 4 ? 4 : avg <= 8 ? 8 : avg <= 16 ? 16 : 32;
}

struct RowWs {
    uint32_t* cnt;  // m
    int64_t* partials;
    uint32_t* err;
};

size_t carve(RowWs* w, void* ws, int64_t m) {
    char* base = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) -> void* {
        off = (off + ALIGN - 1) / ALIGN * ALIGN;
        void* p = base ? base + off : nullptr;
        off += bytes;
        return p;
    };
    const int64_t items = std::max<int64_t>(m, 1);
    RowWs t;
    t.cnt = (uint32_t*)take(items * 4);
    t.partials = (int64_t*)take(scan_partials_count(items + 1) * 8);
    t.err = (uint32_t*)take(4);
    if (w) *w = t;
    return (off + ALIGN - 1) / ALIGN * ALIGN;
}

// lanes of the G-wide group this lane belongs to
template <int G>
__device__ __forceinline__ unsigned group_mask() {
    return (uint32_t)((1ull << G) - 1ull) << (lane_id() & ~(G - 1));
}

// ------------------------------------------------------------------------------ column panel
__global__ void __launch_bounds__(256) panel_count_kernel(int64_t m, const int64_t* __restrict__ rowptr,
                                                          const int32_t* __restrict__ colidx, int32_t k0, int32_t k1,
                                                          uint32_t* __restrict__ cnt) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= m) return;
    const int64_t p0 = rowptr[r];
    const uint32_t len = (uint32_t)(rowptr[r + 1] - p0);
    const uint32_t a = lower_bound_i32(colidx + p0, len, k0);
    const uint32_t b = a + lower_bound_i32(colidx + p0 + a, len - a, k1);
    cnt[r] = b - a;
}

template <typename V, int G>
__global__ void __launch_bounds__(256) panel_fill_kernel(int64_t m, const int64_t* __restrict__ rowptr,
                                                         const int32_t* __restrict__ colidx, const V* __restrict__ vals, int32_t k0,
                                                         const int64_t* __restrict__ p_rowptr, int32_t* __restrict__ p_colidx,
                                                         V* __restrict__ p_vals) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= m) return;
    const int64_t o0 = p_rowptr[r];
    const uint32_t n = (uint32_t)(p_rowptr[r + 1] - o0);
    if (n == 0) return;
    const int64_t p0 = rowptr[r];
    const int64_t src = p0 + lower_bound_i32(colidx + p0, (uint32_t)(rowptr[r + 1] - p0), k0);
    for (uint32_t t = gl; t < n; t += G) {
        p_colidx[o0 + t] = colidx[src + t];
        p_vals[o0 + t] = vals[src + t];
    }
}

// ------------------------------------------------------------------------------- sparse sum
// Walk row `self` G entries at a time; for each entry report (index, lower bound in `other`, match,
// matches before it) to `visit`.  Returns the number of matches of the row.  Loop bounds are
// uniform inside the group, so the votes see all of its lanes.
template <int G, typename Visit>
__device__ __forceinline__ uint32_t walk_row(const int32_t* __restrict__ self, uint32_t ls, const int32_t* __restrict__ other,
                                             uint32_t lo_len, uint32_t* err, Visit visit) {
    const unsigned gmask = group_mask<G>();
    const int gl = lane_id() & (G - 1);
    const int gshift = lane_id() & ~(G - 1);
    uint32_t matched = 0;
    for (uint32_t t0 = 0; t0 < ls; t0 += G) {
        const uint32_t t = t0 + gl;
        bool match = false;
        uint32_t lb = 0;
        int32_t col = 0;
        if (t < ls) {
            col = self[t];
            if (t > 0 && self[t - 1] >= col) atomicOr(err, ERRW_UNSORTED);
            lb = lower_bound_i32(other, lo_len, col);
            match = lb < lo_len && other[lb] == col;
        }
        const unsigned votes = (__ballot_sync(gmask, match) >> gshift) & (uint32_t)((1ull << G) - 1ull);
        if (t < ls) visit(t, lb, match, matched + __popc(votes & ((1u << gl) - 1u)), col);
        matched += __popc(votes);
    }
    return matched;
}

// One warp per row for rows of more than a few entries: the two rows are walked in windows of
// MERGE_WIN column ids each.  Everything up to the smaller of the two windows' last ids is known
// completely, so those entries are merged at once: an entry's place is the output position reached
// so far + its index in its own window + the entries of the other window below it (a search over the
// window in shared memory) - the matches below it (votes).  All global accesses are coalesced and a
// step brings in up to 2 x MERGE_WIN ids with one round of loads.
constexpr int MERGE_WARPS = 8;
constexpr int MERGE_PER_LANE = 1;  // ids per lane and window; 4 was measured: no faster on long rows, slower on short ones
constexpr int MERGE_WIN = 32 * MERGE_PER_LANE;

template <typename V, bool FILL>
__global__ void __launch_bounds__(MERGE_WARPS * 32) add_merge_kernel(int64_t m, const int64_t* __restrict__ x_rowptr,
                                                                     const int32_t* __restrict__ x_colidx, const V* __restrict__ x_vals,
                                                                     const int64_t* __restrict__ y_rowptr,
                                                                     const int32_t* __restrict__ y_colidx, const V* __restrict__ y_vals,
                                                                     uint32_t* __restrict__ cnt, const int64_t* __restrict__ z_rowptr,
                                                                     int32_t* __restrict__ z_colidx, V* __restrict__ z_vals, uint32_t* err) {
    constexpr int32_t INF = 0x7fffffff;  // above every column id
    constexpr int U = MERGE_PER_LANE;
    constexpr uint32_t WIN = MERGE_WIN;
    __shared__ int32_t s_x[MERGE_WARPS][MERGE_WIN];
    __shared__ int32_t s_y[MERGE_WARPS][MERGE_WIN];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t r = (int64_t)blockIdx.x * MERGE_WARPS + warp;
    if (r >= m) return;
    const int64_t x0 = x_rowptr[r], y0 = y_rowptr[r];
    const int64_t lx64 = x_rowptr[r + 1] - x0, ly64 = y_rowptr[r + 1] - y0;
    if (lx64 < 0 || ly64 < 0 || lx64 + ly64 > 0x7fffffffLL) {
        if (lane == 0) {
            atomicOr(err, ERRW_BAD_ROWPTR);
            if (!FILL) cnt[r] = 0;
        }
        return;
    }
    const uint32_t lx = (uint32_t)lx64, ly = (uint32_t)ly64;
    const int64_t z0 = FILL ? z_rowptr[r] : 0;
    const uint32_t lz = FILL ? (uint32_t)(z_rowptr[r + 1] - z0) : 0u;
    const unsigned lt = (1u << lane) - 1u;
    int32_t* wx = s_x[warp];
    int32_t* wy = s_y[warp];
    // number of ids below key among the first n (ascending) ids of a window
    auto below = [&](const int32_t* win, uint32_t n, int32_t key) -> uint32_t {
        uint32_t pos = 0;
#pragma unroll
        for (uint32_t step = WIN / 2; step > 0; step >>= 1)
            if (pos + step <= n && win[pos + step - 1] < key) pos += step;
        if (pos < n && win[pos] < key) ++pos;  // a full window with every probed id below: the last one
        return pos;
    };
    uint32_t ix = 0, iy = 0, out = 0, matches = 0;
    int32_t lastx = -1, lasty = -1;
    while (ix < lx || iy < ly) {  // warp-uniform
        const uint32_t nx = min(WIN, lx - ix), ny = min(WIN, ly - iy);
        int32_t xa[U], ya[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t e = u * 32 + lane;
            xa[u] = e < nx ? x_colidx[x0 + ix + e] : INF;
            ya[u] = e < ny ? y_colidx[y0 + iy + e] : INF;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            wx[u * 32 + lane] = xa[u];
            wy[u * 32 + lane] = ya[u];
        }
        __syncwarp();
        const int32_t bx = ix + WIN < lx ? wx[WIN - 1] : INF, by = iy + WIN < ly ? wy[WIN - 1] : INF;
        const int32_t bound = min(bx, by);
        uint32_t cx = 0, cy = 0, cmx = 0, cmy = 0;  // taken from x, from y, matches seen from either side so far
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t e = u * 32 + lane;
            // rows must be strictly ascending (also across windows)
            const int32_t px = e == 0 ? lastx : wx[e - 1], py = e == 0 ? lasty : wy[e - 1];
            if ((e < nx && px >= xa[u]) || (e < ny && py >= ya[u])) atomicOr(err, ERRW_UNSORTED);
            const bool takex = e < nx && xa[u] <= bound, takey = e < ny && ya[u] <= bound;
            const uint32_t ry = takex ? below(wy, ny, xa[u]) : 0u;
            const bool mx = takex && ry < ny && wy[ry] == xa[u];
            const uint32_t rx = takey ? below(wx, nx, ya[u]) : 0u;
            const bool my = takey && rx < nx && wx[rx] == ya[u];
            const unsigned vx = __ballot_sync(FULL_MASK, takex), vy = __ballot_sync(FULL_MASK, takey);
            const unsigned vmx = __ballot_sync(FULL_MASK, mx), vmy = __ballot_sync(FULL_MASK, my);
            if (FILL) {
                if (takex) {
                    const uint32_t pos = out + e + ry - (cmx + __popc(vmx & lt));
                    if (pos < lz) {
                        z_colidx[z0 + pos] = xa[u];
                        const V xv = x_vals[x0 + ix + e];
                        z_vals[z0 + pos] = mx ? (V)(xv + y_vals[y0 + iy + ry]) : xv;
                    }
                }
                if (takey && !my) {
                    const uint32_t pos = out + e + rx - (cmy + __popc(vmy & lt));
                    if (pos < lz) {
                        z_colidx[z0 + pos] = ya[u];
                        z_vals[z0 + pos] = y_vals[y0 + iy + e];
                    }
                }
            }
            cx += __popc(vx);
            cy += __popc(vy);
            cmx += __popc(vmx);
            cmy += __popc(vmy);
        }
        if (cx > 0) lastx = wx[cx - 1];
        if (cy > 0) lasty = wy[cy - 1];
        out += cx + cy - cmx;
        matches += cmx;
        ix += cx;
        iy += cy;
        __syncwarp();  // the windows are rewritten
    }
    if (!FILL && lane == 0) cnt[r] = lx + ly - matches;
}

template <int G>
__global__ void __launch_bounds__(256) add_count_kernel(int64_t m, const int64_t* __restrict__ x_rowptr,
                                                        const int32_t* __restrict__ x_colidx, const int64_t* __restrict__ y_rowptr,
                                                        const int32_t* __restrict__ y_colidx, uint32_t* __restrict__ cnt,
                                                        uint32_t* err) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= m) return;  // whole groups leave together
    const int64_t x0 = x_rowptr[r], y0 = y_rowptr[r];
    const int64_t lx64 = x_rowptr[r + 1] - x0, ly64 = y_rowptr[r + 1] - y0;
    if (lx64 < 0 || ly64 < 0 || lx64 + ly64 > 0x7fffffffLL) {
        if (gl == 0) { atomicOr(err, ERRW_BAD_ROWPTR); cnt[r] = 0; }
        return;
    }
    const uint32_t lx = (uint32_t)lx64, ly = (uint32_t)ly64;
    // the sortedness of X is checked here, that of Y inside the walk
    for (uint32_t t = 1 + gl; t < lx; t += G)
        if (x_colidx[x0 + t - 1] >= x_colidx[x0 + t]) atomicOr(err, ERRW_UNSORTED);
    const uint32_t matched =
        walk_row<G>(y_colidx + y0, ly, x_colidx + x0, lx, err, [](uint32_t, uint32_t, bool, uint32_t, int32_t) {});
    if (gl == 0) cnt[r] = lx + ly - matched;
}

template <typename V, int G>
__global__ void __launch_bounds__(256) add_fill_kernel(int64_t m, const int64_t* __restrict__ x_rowptr,
                                                       const int32_t* __restrict__ x_colidx, const V* __restrict__ x_vals,
                                                       const int64_t* __restrict__ y_rowptr, const int32_t* __restrict__ y_colidx,
                                                       const V* __restrict__ y_vals, const int64_t* __restrict__ z_rowptr,
                                                       int32_t* __restrict__ z_colidx, V* __restrict__ z_vals, uint32_t* err) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    if (r >= m) return;
    const int64_t x0 = x_rowptr[r], y0 = y_rowptr[r], z0 = z_rowptr[r];
    const uint32_t lx = (uint32_t)(x_rowptr[r + 1] - x0), ly = (uint32_t)(y_rowptr[r + 1] - y0);
    const uint32_t lz = (uint32_t)(z_rowptr[r + 1] - z0);
    // entries of X: all are emitted, matched ones with the sum
    walk_row<G>(x_colidx + x0, lx, y_colidx + y0, ly, err, [&](uint32_t t, uint32_t lb, bool match, uint32_t before, int32_t col) {
        const uint32_t pos = t + lb - before;
        if (pos < lz) {  // always true for the row pointer of the size step; keeps a stale one from writing outside
            z_colidx[z0 + pos] = col;
            const V xv = x_vals[x0 + t];
            z_vals[z0 + pos] = match ? (V)(xv + y_vals[y0 + lb]) : xv;
        }
    });
    // entries of Y: only the ones X does not store
    walk_row<G>(y_colidx + y0, ly, x_colidx + x0, lx, err, [&](uint32_t t, uint32_t lb, bool match, uint32_t before, int32_t col) {
        const uint32_t pos = t + lb - before;
        if (!match && pos < lz) {
            z_colidx[z0 + pos] = col;
            z_vals[z0 + pos] = y_vals[y0 + t];
        }
    });
}

spsyrk_status_t read_err_and_total(const RowWs& w, const int64_t* d_rowptr_out, int64_t m, int64_t* total, cudaStream_t st) {
    int64_t nnz = 0;
    uint32_t e = 0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&nnz, d_rowptr_out + m, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, w.err, 4, cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    if (e) return SPSYRK_ERR_BAD_CSR;
    *total = nnz;
    return SPSYRK_OK;
}

template <typename V>
void launch_panel_fill(int g, int64_t m, const int64_t* rowptr, const int32_t* colidx, const void* vals, int32_t k0,
                       const int64_t* p_rowptr, int32_t* p_colidx, void* p_vals, cudaStream_t st) {
#define FILL(G)                                                                                                            \
    panel_fill_kernel<V, G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(m, rowptr, colidx, static_cast<const V*>(vals), k0, \
                                                                             p_rowptr, p_colidx, static_cast<V*>(p_vals))
    switch (g) {
        case 4: FILL(4); break;
        case 8: FILL(8); break;
        case 16: FILL(16); break;
        default: FILL(32); break;
    }
#undef FILL
    note_launches(1);
}

template <typename V>
void launch_add_fill(int g, int64_t m, const int64_t* xr, const int32_t* xc, const void* xv, const int64_t* yr, const int32_t* yc,
                     const void* yv, const int64_t* zr, int32_t* zc, void* zv, uint32_t* err, cudaStream_t st) {
#define FILL(G)                                                                                                             \
    add_fill_kernel<V, G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(m, xr, xc, static_cast<const V*>(xv), yr, yc,          \
                                                                           static_cast<const V*>(yv), zr, zc, static_cast<V*>(zv), \
                                                                           err)
    switch (g) {
        case 4: FILL(4); break;
        case 8: FILL(8); break;
        case 16: FILL(16); break;
        default:
            add_merge_kernel<V, true><<<(unsigned)((m + MERGE_WARPS - 1) / MERGE_WARPS), MERGE_WARPS * 32, 0, st>>>(
                m, xr, xc, static_cast<const V*>(xv), yr, yc, static_cast<const V*>(yv), nullptr, zr, zc, static_cast<V*>(zv), err);
            break;
    }
#undef FILL
    note_launches(1);
}

bool dtype_ok(spsyrk_dtype_t t) { return t == SPSYRK_F64 || t == SPSYRK_F32 || t == SPSYRK_I32; }

}  // namespace

extern "C" spsyrk_status_t spsyrk_column_panel(int64_t m, int64_t nnz, spsyrk_dtype_t dtype, const int64_t* d_rowptr,
                                               const int32_t* d_colidx, const void* d_vals, int64_t k0, int64_t k1,
                                               int64_t* d_p_rowptr, int32_t* d_p_colidx, void* d_p_vals, int64_t* nnz_out,
                                               void* d_workspace, size_t* workspace_bytes, void* cuda_stream) {
    if (!workspace_bytes || m < 0 || nnz < 0 || !dtype_ok(dtype)) return SPSYRK_ERR_INVALID_ARG;
    if (k0 < 0 || k1 < k0) return SPSYRK_ERR_INVALID_ARG;
    const size_t need = carve(nullptr, nullptr, m);
    if (!d_workspace) {
        *workspace_bytes = need;
        return SPSYRK_OK;
    }
    if (*workspace_bytes < need) return SPSYRK_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_workspace) % ALIGN) return SPSYRK_ERR_INVALID_ARG;
    if (!d_rowptr || !d_p_rowptr || (nnz > 0 && !d_colidx)) return SPSYRK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    RowWs w;
    carve(&w, d_workspace, m);
    // column ids are below 2^31, so larger bounds mean "to the end"
    const int32_t c0 = (int32_t)std::min<int64_t>(k0, 0x7fffffffLL), c1 = (int32_t)std::min<int64_t>(k1, 0x7fffffffLL);
    if (!d_p_colidx) {  // step 2: sizes
        if (!nnz_out) return SPSYRK_ERR_INVALID_ARG;
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, st));
        if (m > 0) {
            panel_count_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(m, d_rowptr, d_colidx, c0, c1, w.cnt);
            note_launches(1);
        }
        SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.cnt, m, d_p_rowptr, w.partials, st));
        return read_err_and_total(w, d_p_rowptr, m, nnz_out, st);
    }
    if (!d_p_vals || (nnz > 0 && !d_vals)) return SPSYRK_ERR_INVALID_ARG;
    if (m == 0) return SPSYRK_OK;
    const int g = group_width(nnz, m);
    if (dtype == SPSYRK_F64) launch_panel_fill<uint64_t>(g, m, d_rowptr, d_colidx, d_vals, c0, d_p_rowptr, d_p_colidx, d_p_vals, st);
    else launch_panel_fill<uint32_t>(g, m, d_rowptr, d_colidx, d_vals, c0, d_p_rowptr, d_p_colidx, d_p_vals, st);
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}

extern "C" spsyrk_status_t spsyrk_accumulate(int64_t m, spsyrk_dtype_t dtype, int64_t nnz_x, const int64_t* d_x_rowptr,
                                             const int32_t* d_x_colidx, const void* d_x_vals, int64_t nnz_y,
                                             const int64_t* d_y_rowptr, const int32_t* d_y_colidx, const void* d_y_vals,
                                             int64_t* d_z_rowptr, int32_t* d_z_colidx, void* d_z_vals, int64_t* nnz_out,
                                             void* d_workspace, size_t* workspace_bytes, void* cuda_stream) {
    if (!workspace_bytes || m < 0 || nnz_x < 0 || nnz_y < 0 || !dtype_ok(dtype)) return SPSYRK_ERR_INVALID_ARG;
    const size_t need = carve(nullptr, nullptr, m);
    if (!d_workspace) {
        *workspace_bytes = need;
        return SPSYRK_OK;
    }
    if (*workspace_bytes < need) return SPSYRK_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_workspace) % ALIGN) return SPSYRK_ERR_INVALID_ARG;
    if (!d_x_rowptr || !d_y_rowptr || !d_z_rowptr || (nnz_x > 0 && !d_x_colidx) || (nnz_y > 0 && !d_y_colidx))
        return SPSYRK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    RowWs w;
    carve(&w, d_workspace, m);
    const int g = group_width(nnz_x + nnz_y, m);
    if (!d_z_colidx) {  // step 2: sizes
        if (!nnz_out) return SPSYRK_ERR_INVALID_ARG;
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, st));
        if (m > 0) {
#define COUNT(G) \
    add_count_kernel<G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(m, d_x_rowptr, d_x_colidx, d_y_rowptr, d_y_colidx, w.cnt, w.err)
            switch (g) {
                case 4: COUNT(4); break;
                case 8: COUNT(8); break;
                case 16: COUNT(16); break;
                default:
                    add_merge_kernel<uint32_t, false><<<(unsigned)((m + MERGE_WARPS - 1) / MERGE_WARPS), MERGE_WARPS * 32, 0, st>>>(
                        m, d_x_rowptr, d_x_colidx, nullptr, d_y_rowptr, d_y_colidx, nullptr, w.cnt, nullptr, nullptr, nullptr, w.err);
                    break;
            }
#undef COUNT
            note_launches(1);
        }
        SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.cnt, m, d_z_rowptr, w.partials, st));
        return read_err_and_total(w, d_z_rowptr, m, nnz_out, st);
    }
    if (!d_z_vals || (nnz_x > 0 && !d_x_vals) || (nnz_y > 0 && !d_y_vals)) return SPSYRK_ERR_INVALID_ARG;
    if (m == 0) return SPSYRK_OK;
    switch (dtype) {
        case SPSYRK_F64:
            launch_add_fill<double>(g, m, d_x_rowptr, d_x_colidx, d_x_vals, d_y_rowptr, d_y_colidx, d_y_vals, d_z_rowptr, d_z_colidx,
                                    d_z_vals, w.err, st);
            break;
        case SPSYRK_F32:
            launch_add_fill<float>(g, m, d_x_rowptr, d_x_colidx, d_x_vals, d_y_rowptr, d_y_colidx, d_y_vals, d_z_rowptr, d_z_colidx,
                                   d_z_vals, w.err, st);
            break;
        default:
            // unsigned addition wraps modulo 2^32, which is also what two's-complement int32 addition means
            launch_add_fill<uint32_t>(g, m, d_x_rowptr, d_x_colidx, d_x_vals, d_y_rowptr, d_y_colidx, d_y_vals, d_z_rowptr,
                                      d_z_colidx, d_z_vals, w.err, st);
            break;
    }
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}
