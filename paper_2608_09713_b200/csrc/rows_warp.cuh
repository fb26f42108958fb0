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
__host__ __device__ constexpr int numeric_warps(int n) { return n >= 512 ? 4 : 8; }

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
    __shared__ Acc s_val[NW][N];      // products by item index t; later the compacted output values
    __shared__ int32_t s_oj[NW][N];   // compacted output column ids
    __shared__ Acc s_a[NW][32];       // a_ik per list
    __shared__ uint32_t s_smo[NW][32];  // list start minus list offset: item t of list s is entry t + smo[s]
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t widx = (int64_t)blockIdx.x * NW + warp;
    if (widx >= nrows) return;
    const int32_t rloc = rows[widx];
    const int64_t i = (int64_t)P.r0 + rloc;
    const int64_t p0 = P.rowptr[i];
    const int deg = (int)(P.rowptr[i + 1] - p0);
    const bool live = lane < deg;
    uint2 d = live ? P.desc[p0 + lane] : make_uint2(0u, 0u);
    const uint32_t incl = warp_inclusive_scan(d.y);
    const uint32_t w = __shfl_sync(FULL_MASK, incl, 31);
    const uint32_t off = live ? incl - d.y : 0xffffffffu;  // first item of this lane's list
    s_smo[warp][lane] = d.x - off;
    s_a[warp][lane] = live ? (Acc) static_cast<const V*>(P.vals)[p0 + lane] : Acc(0);
    __syncwarp();

    Key key[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        key[r] = PAD;
        if ((uint32_t)(r * 32) < w) {  // warp-uniform
            // owner list of item t = 32 r + lane: the list active at item 32 r, plus the lists that
            // start inside (32 r, t]; starts are distinct because every list has at least one item
            const uint32_t rel = off - (uint32_t)(r * 32);  // in 1..31 iff the list starts inside this round
            const uint32_t before = __popc(__ballot_sync(FULL_MASK, off <= (uint32_t)(r * 32)));
            const uint32_t startbits = __reduce_or_sync(FULL_MASK, (rel - 1u < 31u) ? (1u << rel) : 0u);
            const uint32_t s = before - 1u + __popc(startbits & (0xfffffffeu >> (31 - lane)));
            const uint32_t t = r * 32 + lane;
            if (t < w) {
                const uint32_t q = t + s_smo[warp][s];
                const uint32_t j = (uint32_t)P.at_row[q];
                const Acc v = (Acc) static_cast<const V*>(P.at_val)[q];
                s_val[warp][t] = acc_mul(s_a[warp][s], v);
                key[r] = ((Key)j << IDXB) | (Key)t;
            }
        }
    }
    group_bitonic_sort<Key, R, 32>(key);
    __syncwarp();

    // products in sorted order with an ordered segmented sum inside the lane: after it the last
    // element of a run of equal j holds the run's sum as far as this lane can see
    Acc sum[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const Acc v = key[r] != PAD ? s_val[warp][(uint32_t)(key[r] & (Key)(N - 1))] : Acc(0);
        sum[r] = (r > 0 && (key[r] >> IDXB) == (key[r > 0 ? r - 1 : 0] >> IDXB)) ? acc_add(sum[r > 0 ? r - 1 : 0], v) : v;
    }
    // runs that continue from the previous lane: restart the leading run from the carried sum, in
    // order; repeat while a lane that is one single run passes a changed sum on (almost never)
    const Key firstj = key[0] >> IDXB;
    const Key prevj = __shfl_up_sync(FULL_MASK, key[R - 1] >> IDXB, 1);
    const bool joins = lane > 0 && key[0] != PAD && prevj == firstj;
    for (int iter = 0; iter < 32; ++iter) {
        const Acc carry = __shfl_up_sync(FULL_MASK, sum[R - 1], 1);
        const Acc old_tail = sum[R - 1];
        if (joins) {
            Acc acc = carry;
            bool in_run = true;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                in_run = in_run && ((key[r] >> IDXB) == firstj) && key[r] != PAD;
                if (in_run) { acc = acc_add(acc, s_val[warp][(uint32_t)(key[r] & (Key)(N - 1))]); sum[r] = acc; }
            }
        }
        if (!__any_sync(FULL_MASK, joins && !(sum[R - 1] == old_tail))) break;
    }
    __syncwarp();  // every lane has read its products: s_val is free for the output

    // the last element of each run is emitted
    const Key nextj = __shfl_down_sync(FULL_MASK, firstj, 1);
    const bool next_valid = __shfl_down_sync(FULL_MASK, key[0] != PAD ? 1 : 0, 1) != 0 && lane < 31;
    int ntails = 0;
    bool tail[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const bool same_next = (r + 1 < R) ? (key[r + 1] != PAD && (key[r + 1] >> IDXB) == (key[r] >> IDXB))
                                           : (next_valid && nextj == (key[r] >> IDXB));
        tail[r] = key[r] != PAD && !same_next;
        ntails += tail[r];
    }
    const int tincl = warp_inclusive_scan(ntails);
    const int total = __shfl_sync(FULL_MASK, tincl, 31);
    int pos = tincl - ntails;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        if (tail[r]) {
            s_oj[warp][pos] = (int32_t)(key[r] >> IDXB);
            s_val[warp][pos] = sum[r];
            ++pos;
        }
    }
    __syncwarp();
    const int64_t ob = c_rowptr[rloc];
    for (int o = lane; o < total; o += 32) {
        c_colidx[ob + o] = s_oj[warp][o];
        c_vals[ob + o] = (V)s_val[warp][o];
    }
}

}  // namespace spsyrk
