// Steps a4 / a6 for light rows (at most 32 nonzeros, at most N <= 512 partial products):
// one warp per output row.
//
// The partial products of row i are the entries of the column prefixes named by the row's
// descriptors, flattened to items t = 0 .. w-1 in (ascending column k, ascending row j) order.
//   symbolic : insert every j into a per-warp shared-memory hash set, count the distinct ones.
//   numeric  : key = (j << log2 N) | t, value a_ik * a_jk stored at slot t; a register bitonic
//              sort orders the keys by j (ties by t, i.e. by ascending k); the first key of each
//              run of equal j sums its run left to right and the row is written out coalesced.
//              The summation order per entry is therefore ascending k, the same for every run
//              of the program, and fused multiply-add is not used.
#pragma once
#include "transpose.cuh"

namespace spsyrk {

constexpr int ROW_WARPS = 8;  // warps (rows) per CTA in the symbolic warp-class kernel
// warps per CTA of the numeric warp-class kernel: keeps static shared memory under 48 KB
__host__ __device__ constexpr int numeric_warps(int n) { return n >= 512 ? 2 : n >= 256 ? 4 : 8; }

template <int N>
__global__ void __launch_bounds__(ROW_WARPS * 32) symbolic_warp_kernel(PlanDev P, const int32_t* __restrict__ rows, int64_t nrows,
                                                                       int32_t* __restrict__ cnt) {
    constexpr int T = 2 * N;  // hash slots per warp
    constexpr int RND = N / 32;
    constexpr int SHIFT = 32 - ilog2_ce(T);
    __shared__ uint32_t s_tab[ROW_WARPS][T];
    __shared__ uint32_t s_off[ROW_WARPS][32];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t widx = (int64_t)blockIdx.x * ROW_WARPS + warp;
    if (widx >= nrows) return;
    const int32_t rloc = rows[widx];
    const int64_t i = (int64_t)P.r0 + rloc;
    const int64_t p0 = P.rowptr[i];
    const int deg = (int)(P.rowptr[i + 1] - p0);
    uint2 d = lane < deg ? P.desc[p0 + lane] : make_uint2(0u, 0u);
    const uint32_t incl = warp_inclusive_scan(d.y);
    const uint32_t w = __shfl_sync(FULL_MASK, incl, 31);
    s_off[warp][lane] = lane < deg ? incl - d.y : 0xffffffffu;
#pragma unroll
    for (int s = lane; s < T; s += 32) s_tab[warp][s] = 0xffffffffu;
    __syncwarp();
    int local = 0;
#pragma unroll
    for (int r = 0; r < RND; ++r) {
        if ((uint32_t)(r * 32) < w) {  // warp-uniform
            const uint32_t t = r * 32 + lane;
            int s = 0;
#pragma unroll
            for (int st = 16; st > 0; st >>= 1)
                if (s_off[warp][s + st] <= t) s += st;
            const uint32_t start = __shfl_sync(FULL_MASK, d.x, s);
            if (t < w) {
                const uint32_t j = (uint32_t)P.at_row[start + (t - s_off[warp][s])];
                uint32_t h = (j * 2654435761u) >> SHIFT;
                for (int probe = 0; probe < T; ++probe) {  // bounded: the table is at most half full
                    uint32_t old = atomicCAS(&s_tab[warp][h], 0xffffffffu, j);
                    if (old == 0xffffffffu) { ++local; break; }
                    if (old == j) break;
                    h = (h + 1) & (T - 1);
                }
            }
        }
    }
    local = warp_reduce_sum(local);
    if (lane == 0) cnt[rloc] = local;
}

template <typename V, int N, typename Key>
__global__ void __launch_bounds__(numeric_warps(N) * 32) numeric_warp_kernel(PlanDev P, const int32_t* __restrict__ rows, int64_t nrows,
                                                                      const int64_t* __restrict__ c_rowptr,
                                                                      int32_t* __restrict__ c_colidx, V* __restrict__ c_vals) {
    using Acc = typename AccOf<V>::type;
    constexpr int NW = numeric_warps(N);
    constexpr int R = N / 32;
    constexpr int IDXB = ilog2_ce(N);
    constexpr Key PAD = ~Key(0);
    __shared__ Acc s_val[NW][N];   // products by item index t
    __shared__ Key s_key[NW][N];   // sorted keys
    __shared__ Acc s_oval[NW][N];  // compacted output staging
    __shared__ int32_t s_oj[NW][N];
    __shared__ uint32_t s_off[NW][32];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t widx = (int64_t)blockIdx.x * NW + warp;
    if (widx >= nrows) return;
    const int32_t rloc = rows[widx];
    const int64_t i = (int64_t)P.r0 + rloc;
    const int64_t p0 = P.rowptr[i];
    const int deg = (int)(P.rowptr[i + 1] - p0);
    uint2 d = lane < deg ? P.desc[p0 + lane] : make_uint2(0u, 0u);
    const Acc a = lane < deg ? (Acc) static_cast<const V*>(P.vals)[p0 + lane] : Acc(0);
    const uint32_t incl = warp_inclusive_scan(d.y);
    const uint32_t w = __shfl_sync(FULL_MASK, incl, 31);
    s_off[warp][lane] = lane < deg ? incl - d.y : 0xffffffffu;
    __syncwarp();

    Key key[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        key[r] = PAD;
        if ((uint32_t)(r * 32) < w) {  // warp-uniform
            const uint32_t t = r * 32 + lane;
            int s = 0;
#pragma unroll
            for (int st = 16; st > 0; st >>= 1)
                if (s_off[warp][s + st] <= t) s += st;
            const uint32_t start = __shfl_sync(FULL_MASK, d.x, s);
            const Acc av = __shfl_sync(FULL_MASK, a, s);
            if (t < w) {
                const uint32_t q = start + (t - s_off[warp][s]);
                const uint32_t j = (uint32_t)P.at_row[q];
                const Acc v = (Acc) static_cast<const V*>(P.at_val)[q];
                s_val[warp][t] = acc_mul(av, v);
                key[r] = ((Key)j << IDXB) | (Key)t;
            }
        }
    }
    group_bitonic_sort<Key, R, 32>(key);
#pragma unroll
    for (int r = 0; r < R; ++r) s_key[warp][lane * R + r] = key[r];
    __syncwarp();

    // heads of runs of equal j
    Key prev_last = __shfl_up_sync(FULL_MASK, key[R - 1], 1);
    int nheads = 0;
    bool head[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const Key pk = r == 0 ? prev_last : key[r - 1];
        const bool first = (r == 0 && lane == 0);
        head[r] = key[r] != PAD && (first || (pk >> IDXB) != (key[r] >> IDXB));
        nheads += head[r];
    }
    const int hincl = warp_inclusive_scan(nheads);
    const int total = __shfl_sync(FULL_MASK, hincl, 31);
    int pos = hincl - nheads;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (head[r]) {
            const Key jk = key[r] >> IDXB;
            Acc sum = s_val[warp][(uint32_t)(key[r] & (Key)(N - 1))];
            for (uint32_t e = lane * R + r + 1; e < w; ++e) {
                const Key nk = s_key[warp][e];
                if ((nk >> IDXB) != jk) break;
                sum = acc_add(sum, s_val[warp][(uint32_t)(nk & (Key)(N - 1))]);
            }
            s_oj[warp][pos] = (int32_t)jk;
            s_oval[warp][pos] = sum;
            ++pos;
        }
    }
    __syncwarp();
    const int64_t ob = c_rowptr[rloc];
    for (int o = lane; o < total; o += 32) {
        c_colidx[ob + o] = s_oj[warp][o];
        c_vals[ob + o] = (V)s_oval[warp][o];
    }
}

}  // namespace spsyrk
