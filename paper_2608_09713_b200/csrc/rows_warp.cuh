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

// warps per CTA of the symbolic warp-class kernel (static shared memory stays under 48 KB)
__host__ __device__ constexpr int symbolic_warps(int n) { return n >= 512 ? 4 : 8; }
// warps per CTA of the numeric warp-class kernel: keeps static shared memory under 48 KB
__host__ __device__ constexpr int numeric_warps(int n) { return n >= 512 ? 2 : n >= 256 ? 4 : 8; }
// register budget: at least this many CTAs of the numeric kernel must fit on an SM
__host__ __device__ constexpr int numeric_min_ctas(int n) { return n == 256 ? 6 : n == 128 ? 4 : n == 64 ? 5 : 1; }

// lane holding the s-th (0-based) set bit of mask
__device__ __forceinline__ uint32_t nth_set_lane(unsigned mask, uint32_t s) {
    for (uint32_t k = 0; k < s; ++k) mask &= mask - 1;
    return (uint32_t)(__ffs(mask) - 1);
}

// Asynchronous global -> shared copies of 4 or 8 bytes (no register staging), grouped per thread.
template <int BYTES>
__device__ __forceinline__ void cp_async(void* smem_dst, const void* gmem_src) {
    static_assert(BYTES == 4 || BYTES == 8, "cp.async size");
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2;\n" ::"r"(dst), "l"(gmem_src), "n"(BYTES) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int KEEP>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(KEEP) : "memory"); }

// Per-row header in class order, written by the plan: the row's index inside the plan's range, the
// position of its first nonzero in A and its number of nonzeros.
__global__ void __launch_bounds__(256) row_header_kernel(PlanDev P, const int32_t* __restrict__ perm, int64_t rows,
                                                         uint4* __restrict__ hdr) {
    const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= rows) return;
    const int32_t rloc = perm[n];
    const int64_t i = (int64_t)P.r0 + rloc;
    const int64_t p0 = P.rowptr[i], p1 = P.rowptr[i + 1];
    hdr[n] = make_uint4((uint32_t)rloc, (uint32_t)p0, (uint32_t)(p1 - p0), 0u);
}

// Numeric pass for light rows, one warp per row, software-pipelined over the rows a warp owns:
// while row n is sorted and written, the column-list entries of row n+1 stream into shared memory
// through cp.async, the descriptors of row n+2 and the header of row n+3 are in flight in
// registers.  Memory latency is hidden inside the warp instead of by occupancy.
// GAPS: descriptors may have zero length (plan restricted to a column range)
template <typename V, int N, typename Key, bool GAPS>
__global__ void __launch_bounds__(numeric_warps(N) * 32, numeric_min_ctas(N)) numeric_warp_kernel(PlanDev P, const uint4* __restrict__ hdr, int64_t nrows,
                                                                      const int64_t* __restrict__ c_rowptr,
                                                                      int32_t* __restrict__ c_colidx, V* __restrict__ c_vals) {
    using Acc = typename AccOf<V>::type;
    constexpr int NW = numeric_warps(N);
    constexpr int R = N / 32;
    constexpr int IDXB = ilog2_ce(N);
    constexpr Key PAD = ~Key(0);
    // double-buffered landing zones of the gathers; buffer b is reused for row n's products and
    // then for its compacted output
    // the output staging indexes these arrays through pad(): one spare slot per eight keeps the
    // stride-R writes of the compaction off a single bank
    constexpr int NP = N + N / 8;
    __shared__ uint32_t s_j[NW][2][NP];
    __shared__ Acc s_v[NW][2][NP];
    __shared__ uint8_t s_own[NW][2][N];
    __shared__ Acc s_a[NW][2][32];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t stride = (int64_t)gridDim.x * NW;
    int64_t n = (int64_t)blockIdx.x * NW + warp;
    if (n >= nrows) return;

    const uint4 none = make_uint4(0u, 0u, 0u, 0u);
    auto load_hdr = [&](int64_t idx) { return idx < nrows ? hdr[idx] : none; };
    auto load_desc = [&](const uint4& h) { return (uint32_t)lane < h.z ? P.desc[(int64_t)h.y + lane] : make_uint2(0u, 0u); };
    auto load_a = [&](const uint4& h) { return (uint32_t)lane < h.z ? (Acc) static_cast<const V*>(P.vals)[(int64_t)h.y + lane] : Acc(0); };
    // issue the gathers of one row into buffer b; returns its item count
    auto issue = [&](const uint4& h, const uint2& d, Acc a, int b) -> uint32_t {
        const uint32_t incl = warp_inclusive_scan(d.y);
        const uint32_t w = __shfl_sync(FULL_MASK, incl, 31);
        // a list without items (possible when the plan is restricted to a column range) takes no part
        const unsigned nzmask = GAPS ? __ballot_sync(FULL_MASK, d.y > 0) : 0u;
        const bool gaps = GAPS && (nzmask & (nzmask + 1u)) != 0;  // the non-empty lists are not lanes 0..k-1
        const uint32_t off = d.y > 0 ? incl - d.y : 0xffffffffu;  // first item of this lane's list
        const uint32_t smo = d.x - off;                           // item t of this list is entry t + smo
        s_a[warp][b][lane] = a;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if ((uint32_t)(r * 32) < w) {  // warp-uniform
                // owner list of item t = 32 r + lane: the list active at item 32 r plus the lists that
                // start inside (32 r, t]; starts are distinct because every list has at least one item
                const uint32_t rel = off - (uint32_t)(r * 32);
                const uint32_t before = __popc(__ballot_sync(FULL_MASK, off <= (uint32_t)(r * 32)));
                const uint32_t startbits = __reduce_or_sync(FULL_MASK, (rel - 1u < 31u) ? (1u << rel) : 0u);
                uint32_t s = before - 1u + __popc(startbits & (0xfffffffeu >> (31 - lane)));
                if (gaps) s = nth_set_lane(nzmask, s & 31);  // s counted non-empty lists: back to a lane
                const uint32_t q = r * 32 + lane + __shfl_sync(FULL_MASK, smo, s & 31);
                const uint32_t t = r * 32 + lane;
                if (t < w) {
                    cp_async<4>(&s_j[warp][b][t], P.at_row + q);
                    cp_async<sizeof(V)>(&s_v[warp][b][t], static_cast<const V*>(P.at_val) + q);
                    s_own[warp][b][t] = (uint8_t)s;
                }
            }
        }
        cp_async_commit();
        return w;
    };

    // prologue
    uint4 h0 = load_hdr(n), hB = load_hdr(n + stride), hA = load_hdr(n + 2 * stride);
    uint2 d0 = load_desc(h0);
    Acc a0 = load_a(h0);
    uint2 dB = load_desc(hB);
    Acc aB = load_a(hB);
    uint32_t rloc_n = h0.x;
    int64_t ob_n = c_rowptr[rloc_n];
    uint32_t w_n = issue(h0, d0, a0, 0);
    int b = 0;

    for (; n < nrows; n += stride, b ^= 1) {
        // stage A: header of row n+3; stage B: descriptors of row n+2; stage C: gathers of row n+1
        const uint4 hNew = load_hdr(n + 3 * stride);
        const uint2 dNew = load_desc(hA);
        const Acc aNew = load_a(hA);
        const int64_t ob_next = hB.z ? c_rowptr[hB.x] : 0;
        const uint32_t w_next = issue(hB, dB, aB, b ^ 1);

        // stage D: row n.  Its gathers were committed one group ago.
        cp_async_wait<1>();
        __syncwarp();
        Key key[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            key[r] = PAD;
            const uint32_t t = r * 32 + lane;
            if (t < w_n) {
                const uint32_t j = s_j[warp][b][t];
                const Acc v = (Acc) * reinterpret_cast<const V*>(&s_v[warp][b][t]);
                s_v[warp][b][t] = acc_mul(s_a[warp][b][s_own[warp][b][t]], v);
                key[r] = ((Key)j << IDXB) | (Key)t;
            }
        }
        group_bitonic_sort<Key, R, 32>(key);
        __syncwarp();

        // same[r]: element r continues the run of equal j of element r-1 (same[0]: of the previous
        // lane's last element).  Padding keys sort to the end and never equal a real j.
        constexpr Key JUNIT = Key(1) << IDXB;
        const Key prev_last = __shfl_up_sync(FULL_MASK, key[R - 1], 1);
        bool same[R + 1];
        same[0] = lane > 0 && ((key[0] ^ prev_last) < JUNIT);
#pragma unroll
        for (int r = 1; r < R; ++r) same[r] = (key[r] ^ key[r - 1]) < JUNIT;
        same[R] = __shfl_down_sync(FULL_MASK, same[0] ? 1 : 0, 1) != 0 && lane < 31;
        // products in sorted order with an ordered segmented sum inside the lane: after it the last
        // element of a run holds the run's sum as far as this lane can see
        Acc sum[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const Acc v = s_v[warp][b][(uint32_t)(key[r] & (Key)(N - 1))];
            sum[r] = (r > 0 && same[r]) ? acc_add(sum[r > 0 ? r - 1 : 0], v) : v;
        }
        // runs that continue from the previous lane: restart the leading run from the carried sum, in
        // order; repeat while a lane that is one single run passes a changed sum on (almost never)
        const bool joins = same[0] && key[0] != PAD;
        if (__any_sync(FULL_MASK, joins)) {
            // a leading run of three or more (or, with one or two keys per lane, possibly the whole lane)
            const bool deep = joins && (R >= 3 ? (same[1] && same[R >= 3 ? 2 : 0]) : true);
            if (!__any_sync(FULL_MASK, deep)) {
                // common case: the run reaches at most two elements into the lane, so no lane's last
                // sum changes and one step settles everything
                const Acc carry = __shfl_up_sync(FULL_MASK, sum[R - 1], 1);
                if (joins) {
                    const Acc a0 = acc_add(carry, s_v[warp][b][(uint32_t)(key[0] & (Key)(N - 1))]);
                    sum[0] = a0;
                    if (R >= 2 && same[R >= 2 ? 1 : 0]) sum[R >= 2 ? 1 : 0] = acc_add(a0, s_v[warp][b][(uint32_t)(key[R >= 2 ? 1 : 0] & (Key)(N - 1))]);
                }
            } else {
                for (int iter = 0; iter < 32; ++iter) {
                    const Acc carry = __shfl_up_sync(FULL_MASK, sum[R - 1], 1);
                    const Acc old_tail = sum[R - 1];
                    if (joins) {
                        Acc acc = carry;
                        bool in_run = true;
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            in_run = in_run && (r == 0 || same[r]);
                            if (in_run) { acc = acc_add(acc, s_v[warp][b][(uint32_t)(key[r] & (Key)(N - 1))]); sum[r] = acc; }
                        }
                    }
                    if (!__any_sync(FULL_MASK, joins && !(sum[R - 1] == old_tail))) break;
                }
            }
        }
        __syncwarp();  // every lane has read its products: the buffer is free for the output

        // the last element of each run is emitted; element e = lane * R + r is real iff e < w
        const int nreal = (int)w_n - lane * R;
        int ntails = 0;
        bool tail[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            tail[r] = r < nreal && !(same[r + 1] && r + 1 < nreal);
            ntails += tail[r];
        }
        const int tincl = warp_inclusive_scan(ntails);
        const int total = __shfl_sync(FULL_MASK, tincl, 31);
        int pos = tincl - ntails;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (tail[r]) {
                s_j[warp][b][pos + (pos >> 3)] = (uint32_t)(key[r] >> IDXB);
                s_v[warp][b][pos + (pos >> 3)] = sum[r];
                ++pos;
            }
        }
        __syncwarp();
        for (int o = lane; o < total; o += 32) {
            c_colidx[ob_n + o] = (int32_t)s_j[warp][b][o + (o >> 3)];
            c_vals[ob_n + o] = (V)s_v[warp][b][o + (o >> 3)];
        }
        __syncwarp();  // buffer b is handed to the gathers of row n+2 in the next iteration

        rloc_n = hB.x; w_n = w_next; ob_n = ob_next;
        hB = hA; dB = dNew; aB = aNew; hA = hNew;
    }
    cp_async_wait<0>();
    (void)rloc_n;
}

// Symbolic pass for light rows: the same persistent, software-pipelined walk as the numeric kernel
// (header, descriptors and column-list row ids of later rows in flight while a row is counted), but
// only the row ids are gathered and they go into a per-warp hash set; the count is the number of
// successful inserts.
template <int N, bool GAPS>
__global__ void __launch_bounds__(symbolic_warps(N) * 32) symbolic_warp_kernel(PlanDev P, const uint4* __restrict__ hdr, int64_t nrows,
                                                                       int32_t* __restrict__ cnt) {
    constexpr int SW = symbolic_warps(N);
    constexpr int T = 2 * N;  // hash slots per warp
    constexpr int R = N / 32;
    constexpr int SHIFT = 32 - ilog2_ce(T);
    __shared__ uint32_t s_tab[SW][T];
    __shared__ uint32_t s_j[SW][2][N];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t stride = (int64_t)gridDim.x * SW;
    int64_t n = (int64_t)blockIdx.x * SW + warp;
    if (n >= nrows) return;

    const uint4 none = make_uint4(0u, 0u, 0u, 0u);
    auto load_hdr = [&](int64_t idx) { return idx < nrows ? hdr[idx] : none; };
    auto load_desc = [&](const uint4& h) { return (uint32_t)lane < h.z ? P.desc[(int64_t)h.y + lane] : make_uint2(0u, 0u); };
    auto issue = [&](const uint4& h, const uint2& d, int b) -> uint32_t {
        const uint32_t incl = warp_inclusive_scan(d.y);
        const uint32_t w = __shfl_sync(FULL_MASK, incl, 31);
        const unsigned nzmask = GAPS ? __ballot_sync(FULL_MASK, d.y > 0) : 0u;
        const bool gaps = GAPS && (nzmask & (nzmask + 1u)) != 0;
        const uint32_t off = d.y > 0 ? incl - d.y : 0xffffffffu;
        const uint32_t smo = d.x - off;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if ((uint32_t)(r * 32) < w) {  // warp-uniform
                const uint32_t rel = off - (uint32_t)(r * 32);
                const uint32_t before = __popc(__ballot_sync(FULL_MASK, off <= (uint32_t)(r * 32)));
                const uint32_t startbits = __reduce_or_sync(FULL_MASK, (rel - 1u < 31u) ? (1u << rel) : 0u);
                uint32_t s = before - 1u + __popc(startbits & (0xfffffffeu >> (31 - lane)));
                if (gaps) s = nth_set_lane(nzmask, s & 31);
                const uint32_t q = r * 32 + lane + __shfl_sync(FULL_MASK, smo, s & 31);
                if ((uint32_t)(r * 32 + lane) < w) cp_async<4>(&s_j[warp][b][r * 32 + lane], P.at_row + q);
            }
        }
        cp_async_commit();
        return w;
    };

    uint4 h0 = load_hdr(n), hB = load_hdr(n + stride), hA = load_hdr(n + 2 * stride);
    uint2 d0 = load_desc(h0);
    uint2 dB = load_desc(hB);
    uint32_t rloc_n = h0.x;
    uint32_t w_n = issue(h0, d0, 0);
    int b = 0;
    for (; n < nrows; n += stride, b ^= 1) {
        const uint4 hNew = load_hdr(n + 3 * stride);
        const uint2 dNew = load_desc(hA);
        const uint32_t w_next = issue(hB, dB, b ^ 1);
#pragma unroll
        for (int s = lane; s < T; s += 32) s_tab[warp][s] = 0xffffffffu;
        cp_async_wait<1>();
        __syncwarp();
        int local = 0;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const uint32_t t = r * 32 + lane;
            if (t < w_n) {
                const uint32_t j = s_j[warp][b][t];
                uint32_t h = (j * 2654435761u) >> SHIFT;
                for (int probe = 0; probe < T; ++probe) {  // bounded: the table is at most half full
                    const uint32_t old = atomicCAS(&s_tab[warp][h], 0xffffffffu, j);
                    if (old == 0xffffffffu) { ++local; break; }
                    if (old == j) break;
                    h = (h + 1) & (T - 1);
                }
            }
        }
        local = warp_reduce_sum(local);
        if (lane == 0) cnt[rloc_n] = local;
        __syncwarp();  // the table and buffer b are reused by the next rows
        rloc_n = hB.x; w_n = w_next;
        hB = hA; dB = dNew; hA = hNew;
    }
    cp_async_wait<0>();
}

}  // namespace spsyrk
