// Steps a4 / a6 for light rows (at most 32 nonzeros, at most N <= 512 partial products):
// a group of G lanes (8, 16 or 32) per output row, 32 / G rows per warp.
//
// The partial products of row i are the entries of the column prefixes named by the row's
// descriptors, flattened to items t = 0 .. w-1 in (ascending column k, ascending row j) order.
//   symbolic : insert every j into a per-group shared-memory hash set, count the distinct ones.
//   numeric  : key = (j << log2 N) | t, value a_ik * a_jk stored at slot t; a register bitonic
//              sort orders the keys by j (ties by t, i.e. by ascending k); the first key of each
//              run of equal j sums its run left to right and the row is written out coalesced.
//              The summation order per entry is therefore ascending k, the same for every run
//              of the program, and fused multiply-add is not used.
//
// DIAG (lower-triangle mode over the whole column range): every column prefix of row i ends
// with the entry (i, a_ik) itself.  Those entries are left out of the gather; the diagonal
// c_ii = sum_k a_ik^2 is folded left to right from the row's own values and appended as the last
// entry of the row, and the symbolic count is the distinct j < i plus one.
//
// Gathers.  Column-list entries are fetched in pieces of up to four entries per lane and round:
// the pieces of all lists of a row are numbered consecutively (a prefix sum of the pieces per
// list), a lane finds the list of its piece by a five-step search in a 32-entry table in shared
// memory (lists without entries drop out of that search by themselves), and issues the
// asynchronous copies.  The numeric pass reads the interleaved (row id, value) records, whose
// alignment unit is the record, so the items land densely in item order; the symbolic pass reads
// aligned 16-byte pieces of the plain row-id array and masks the entries outside the prefix.
#pragma once
#include "transpose.cuh"

namespace spsyrk {

// lanes per row for the class with N item slots
__host__ __device__ constexpr int warp_class_group(int n) { return n <= 32 ? 8 : n <= 128 ? 16 : 32; }
// warps per CTA
__host__ __device__ constexpr int numeric_warps(int n) { return n >= 512 ? 2 : 4; }
__host__ __device__ constexpr int symbolic_warps(int n) { return n >= 512 ? 4 : 8; }
// register budget: at least this many CTAs must fit on an SM
__host__ __device__ constexpr int numeric_min_ctas(int n) { return n == 256 ? 5 : n == 512 ? 4 : 4; }

// Asynchronous global -> shared copies (no register staging), grouped per thread.
template <int BYTES>
__device__ __forceinline__ void cp_async(void* smem_dst, const void* gmem_src) {
    static_assert(BYTES == 4 || BYTES == 8 || BYTES == 16, "cp.async size");
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    if constexpr (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gmem_src) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], %2;\n" ::"r"(dst), "l"(gmem_src), "n"(BYTES) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int KEEP>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(KEEP) : "memory"); }

template <int G>
__device__ __forceinline__ uint32_t group_inclusive_scan(uint32_t v, int gl) {
#pragma unroll
    for (int o = 1; o < G; o <<= 1) {
        const uint32_t t = __shfl_up_sync(FULL_MASK, v, o, G);
        if (gl >= o) v += t;
    }
    return v;
}

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

// last s in [0, 32) with tab[s] <= c; tab is non-decreasing and tab[0] = 0
__device__ __forceinline__ uint32_t last_not_above(const uint32_t* tab, uint32_t c) {
    uint32_t s = 0;
#pragma unroll
    for (uint32_t step = 16; step > 0; step >>= 1)
        if (tab[s + step] <= c) s += step;
    return s;
}

// ---------------------------------------------------------------------------------------------
// numeric
// ---------------------------------------------------------------------------------------------
template <typename V, int N>
struct NumericWarpSmem {
    using Acc = typename AccOf<V>::type;
    using Rec = ColRec<V>;
    static constexpr int NP = N + N / 8 + 2;  // output staging: one spare slot per eight, room for the diagonal
    static constexpr int BUF = (int)(((sizeof(Rec) * N > (4 + sizeof(V)) * NP ? sizeof(Rec) * N : (4 + sizeof(V)) * NP) + 15) / 16 * 16);
    // per group: two landing buffers, two owner arrays, two copies of the row's own values, the tables
    static constexpr int GROUP = 2 * BUF + 2 * N + 2 * 32 * (int)sizeof(Acc) + 32 * 16 + 32 * 4;
};

// Numeric pass for light rows, software-pipelined over the rows a group owns: while row n is sorted
// and written, the column-list records of row n+1 stream into shared memory through cp.async, the
// descriptors of row n+2 and the header of row n+3 are in flight in registers.  Memory latency is
// hidden inside the warp instead of by occupancy.
template <typename V, int N, int G, typename Key, bool DIAG>
__global__ void __launch_bounds__(numeric_warps(N) * 32, numeric_min_ctas(N))
numeric_warp_kernel(PlanDev P, const uint4* __restrict__ hdr, int64_t nrows, const int64_t* __restrict__ c_rowptr,
                    const int64_t* __restrict__ c_rowend, int32_t* __restrict__ c_colidx, V* __restrict__ c_vals,
                    int32_t* __restrict__ cnt_out = nullptr) {
    // c_rowptr[r] / c_rowend[r]: where row r's part of the output starts and ends (c_rowend = c_rowptr + 1 unless the
    // rows are written in two parts, see the full-output mode of the plan).  cnt_out: the kernel counts the entries of
    // a row itself while it merges equal column ids, so it can also serve rows whose slots were sized by an upper
    // bound (the one-pass mode); it then reports the counts here.
    using Acc = typename AccOf<V>::type;
    using Rec = ColRec<V>;
    using SM = NumericWarpSmem<V, N>;
    constexpr int NW = numeric_warps(N);
    constexpr int W = 32 / G;   // rows per warp
    constexpr int LD = 32 / G;  // lists per lane: a light row has at most 32
    constexpr int R = N / G;
    constexpr int IDXB = ilog2_ce(N);
    constexpr Key PAD = ~Key(0);
    constexpr int NP = SM::NP;
    static_assert(R >= 1 && (R & (R - 1)) == 0, "keys per lane");
    extern __shared__ __align__(16) unsigned char nw_smem[];

    const int lane = lane_id(), gl = lane & (G - 1);
    const int gq = threadIdx.x / G;  // group inside the CTA
    unsigned char* gs = nw_smem + (size_t)gq * SM::GROUP;
    unsigned char* s_buf = gs;                                            // [2][BUF]
    uint8_t* s_own = gs + 2 * SM::BUF;                                    // [2][N]
    Acc* s_a = reinterpret_cast<Acc*>(gs + 2 * SM::BUF + 2 * N);          // [2][32]
    uint4* s_tab = reinterpret_cast<uint4*>(s_a + 64);                    // [32] (start, first item, items, first piece)
    uint32_t* s_first = reinterpret_cast<uint32_t*>(s_tab + 32);          // [32] first piece per list

    const int64_t stride = (int64_t)gridDim.x * NW * W;
    int64_t n = (int64_t)blockIdx.x * NW * W + gq;
    int64_t n_warp = n - (gq & (W - 1));  // row of the warp's first group: the loop bound is warp-uniform
    if (n_warp >= nrows) return;

    const uint4 none = make_uint4(0u, 0u, 0u, 0u);
    const Rec* __restrict__ recs = static_cast<const Rec*>(P.at_rec);
    auto load_hdr = [&](int64_t idx) { return idx < nrows ? hdr[idx] : none; };
    struct Lists {
        uint2 d[LD];
        Acc a[LD];
    };
    auto load_lists = [&](const uint4& h) {
        Lists L;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const uint32_t s = (uint32_t)(gl * LD + u);
            const bool on = s < h.z;
            L.d[u] = on ? P.desc[(int64_t)h.y + s] : make_uint2(0u, 0u);
            L.a[u] = on ? (Acc) static_cast<const V*>(P.vals)[(int64_t)h.y + s] : Acc(0);
        }
        return L;
    };
    // issue the gathers of one row into buffer b; returns its item count
    auto issue = [&](const uint4& h, const Lists& L, int b) -> uint32_t {
        uint32_t pk[LD], mine = 0;
        __syncwarp();  // the tables may still be searched for the previous row
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            uint32_t len = L.d[u].y;
            if (DIAG && len > 0) --len;  // the entry (i, a_ik) closes the prefix
            pk[u] = (((len + 3u) >> 2) << 16) | len;  // pieces of four in the high half, items in the low half
            mine += pk[u];
        }
        const uint32_t incl = group_inclusive_scan<G>(mine, gl);
        const uint32_t tot = __shfl_sync(FULL_MASK, incl, G - 1, G);
        uint32_t run = incl - mine;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const int s = gl * LD + u;
            s_tab[s] = make_uint4(L.d[u].x, run & 0xffffu, pk[u] & 0xffffu, run >> 16);
            s_first[s] = run >> 16;
            s_a[b * 32 + s] = L.a[u];
            run += pk[u];
        }
        __syncwarp();
        const uint32_t npieces = tot >> 16;
        Rec* buf = reinterpret_cast<Rec*>(s_buf + b * SM::BUF);
        uint8_t* own = s_own + b * N;
        for (uint32_t c = gl; c < npieces; c += G) {
            const uint32_t s = last_not_above(s_first, c);
            const uint4 t = s_tab[s];
            const uint32_t e0 = (c - t.w) * 4u;
            const uint32_t left = t.z - e0;
            const Rec* src = recs + t.x + e0;
            const uint32_t slot = t.y + e0;
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) {
                if (e < left && SPSYRK_IN_RANGE(slot + e < (uint32_t)N, P.err)) {
                    cp_async<sizeof(Rec)>(buf + slot + e, src + e);
                    own[slot + e] = (uint8_t)s;
                }
            }
        }
        cp_async_commit();
        (void)h;
        return tot & 0xffffu;
    };

    // prologue
    uint4 h0 = load_hdr(n), hB = load_hdr(n + stride), hA = load_hdr(n + 2 * stride);
    Lists l0 = load_lists(h0);
    Lists lB = load_lists(hB);
    uint4 h_n = h0;
    int64_t ob_n = h0.z ? c_rowptr[h0.x] : 0;
    uint32_t w_n = issue(h0, l0, 0);
    int b = 0;

    for (; n_warp < nrows; n_warp += stride, n += stride, b ^= 1) {
        // stage A: header of row n+3; stage B: descriptors of row n+2; stage C: gathers of row n+1
        const uint4 hNew = load_hdr(n + 3 * stride);
        const Lists lNew = load_lists(hA);
        const int64_t ob_next = hB.z ? c_rowptr[hB.x] : 0;
        const uint32_t w_next = issue(hB, lB, b ^ 1);

        // stage D: row n.  Its gathers were committed one group ago.
        cp_async_wait<1>();
        __syncwarp();
        unsigned char* bufb = s_buf + b * SM::BUF;
        Rec* buf = reinterpret_cast<Rec*>(bufb);
        const uint8_t* own = s_own + b * N;
        // product of slot t: written over the record it came from
        auto prod_at = [&](uint32_t t) -> Acc* {
            if constexpr (sizeof(Acc) == sizeof(Rec)) return reinterpret_cast<Acc*>(buf + t);
            else return reinterpret_cast<Acc*>(&buf[t].v);
        };
        Key key[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            key[r] = PAD;
            const uint32_t t = r * G + gl;
            if (t < w_n) {
                const Rec rc = buf[t];
                const Acc a = s_a[b * 32 + own[t]];
                *prod_at(t) = acc_mul(a, (Acc)rc.v);
                key[r] = ((Key)(uint32_t)rc.j << IDXB) | (Key)t;
            }
        }
        Acc diag = Acc(0);
        if (DIAG) {
            // c_ii: the squares of the row's own values, folded left to right (ascending k)
            uint32_t dmax = h_n.z;
            if (G < 32) dmax = __reduce_max_sync(FULL_MASK, dmax);
            for (uint32_t s = 0; s < dmax; ++s) {
                const Acc a = s_a[b * 32 + (s & 31)];
                if (s < h_n.z) diag = acc_add(diag, acc_mul(a, a));
            }
        }
        group_bitonic_sort<Key, R, G>(key);
        __syncwarp();

        // same[r]: element r continues the run of equal j of element r-1 (same[0]: of the previous
        // lane's last element).  Padding keys sort to the end and never equal a real j.
        constexpr Key JUNIT = Key(1) << IDXB;
        const Key prev_last = __shfl_up_sync(FULL_MASK, key[R - 1], 1, G);
        bool same[R + 1];
        same[0] = gl > 0 && ((key[0] ^ prev_last) < JUNIT);
#pragma unroll
        for (int r = 1; r < R; ++r) same[r] = (key[r] ^ key[r - 1]) < JUNIT;
        same[R] = __shfl_down_sync(FULL_MASK, same[0] ? 1 : 0, 1, G) != 0 && gl < G - 1;
        // products in sorted order with an ordered segmented sum inside the lane: after it the last
        // element of a run holds the run's sum as far as this lane can see
        Acc sum[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const Acc v = *prod_at((uint32_t)(key[r] & (Key)(N - 1)));
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
                const Acc carry = __shfl_up_sync(FULL_MASK, sum[R - 1], 1, G);
                if (joins) {
                    const Acc a0 = acc_add(carry, *prod_at((uint32_t)(key[0] & (Key)(N - 1))));
                    sum[0] = a0;
                    if (R >= 2 && same[R >= 2 ? 1 : 0]) sum[R >= 2 ? 1 : 0] = acc_add(a0, *prod_at((uint32_t)(key[R >= 2 ? 1 : 0] & (Key)(N - 1))));
                }
            } else {
                for (int iter = 0; iter < 32; ++iter) {
                    const Acc carry = __shfl_up_sync(FULL_MASK, sum[R - 1], 1, G);
                    const Acc old_tail = sum[R - 1];
                    if (joins) {
                        Acc acc = carry;
                        bool in_run = true;
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            in_run = in_run && (r == 0 || same[r]);
                            if (in_run) { acc = acc_add(acc, *prod_at((uint32_t)(key[r] & (Key)(N - 1)))); sum[r] = acc; }
                        }
                    }
                    if (!__any_sync(FULL_MASK, joins && !(sum[R - 1] == old_tail))) break;
                }
            }
        }
        __syncwarp();  // every lane has read its products: the buffer is free for the output

        // the last element of each run is emitted; element e = gl * R + r is real iff e < w
        const int nreal = (int)w_n - gl * R;
        int ntails = 0;
        bool tail[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            tail[r] = r < nreal && !(same[r + 1] && r + 1 < nreal);
            ntails += tail[r];
        }
        const int tincl = (int)group_inclusive_scan<G>((uint32_t)ntails, gl);
        int total = __shfl_sync(FULL_MASK, tincl, G - 1, G);
        int pos = tincl - ntails;
        uint32_t* o_j = reinterpret_cast<uint32_t*>(bufb);        // [NP]
        V* o_v = reinterpret_cast<V*>(bufb + 4 * NP);             // [NP]
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (tail[r]) {
                o_j[pos + (pos >> 3)] = (uint32_t)(key[r] >> IDXB);
                o_v[pos + (pos >> 3)] = (V)sum[r];
                ++pos;
            }
        }
        if (DIAG && h_n.z > 0) {
            if (gl == 0) {
                o_j[total + (total >> 3)] = (uint32_t)P.r0 + h_n.x;
                o_v[total + (total >> 3)] = (V)diag;
            }
            ++total;
        }
        __syncwarp();
#ifdef SPSYRK_CHECKED
        {
            const int64_t room = h_n.z ? c_rowend[h_n.x] - ob_n : 0;  // the row's entries counted by the symbolic pass
            if (!SPSYRK_IN_RANGE((int64_t)total <= room && total <= NP - 1, P.err)) total = 0;
        }
#endif
        if (cnt_out && gl == 0 && h_n.z > 0) cnt_out[h_n.x] = total;
        for (int o = gl; o < total; o += G) {
            const int32_t j = (int32_t)o_j[o + (o >> 3)];
            const V cv = o_v[o + (o >> 3)];
            c_colidx[ob_n + o] = j;
            c_vals[ob_n + o] = cv;
            if constexpr (std::is_same<V, int32_t>::value) {
                if (P.jaccard) {
                    const int64_t na_j = P.adeg[j];
                    P.jaccard[ob_n + o] = __fdiv_rn((float)cv, (float)((int64_t)h_n.z + na_j - (int64_t)cv));
                }
            }
        }
        __syncwarp();  // buffer b is handed to the gathers of row n+2 in the next iteration

        h_n = hB; w_n = w_next; ob_n = ob_next;
        hB = hA; lB = lNew; hA = hNew;
    }
    cp_async_wait<0>();
    (void)c_rowend;
}

// ---------------------------------------------------------------------------------------------
// symbolic
// ---------------------------------------------------------------------------------------------
template <int N>
struct SymbolicWarpSmem {
    static constexpr int T = 2 * N;       // hash slots per group
    static constexpr int NS = N + 8 * 32;  // landing slots: aligned pieces carry up to 3 + 3 foreign entries per list
    // per group: hash table, two landing buffers, two mask arrays (one byte per piece), the tables
    static constexpr int GROUP = T * 4 + 2 * NS * 4 + 2 * (NS / 4) + 32 * 16 + 32 * 4;
};

// Symbolic pass for light rows: the same persistent, software-pipelined walk as the numeric kernel
// (header, descriptors and column-list row ids of later rows in flight while a row is counted), but
// only the row ids are gathered, in aligned 16-byte pieces, and they go into a per-group hash set;
// the count is the number of successful inserts.
template <int N, int G, bool DIAG>
__global__ void __launch_bounds__(symbolic_warps(N) * 32) symbolic_warp_kernel(PlanDev P, const uint4* __restrict__ hdr, int64_t nrows,
                                                                       int32_t* __restrict__ cnt) {
    using SM = SymbolicWarpSmem<N>;
    constexpr int SW = symbolic_warps(N);
    constexpr int W = 32 / G;
    constexpr int LD = 32 / G;
    constexpr int T = SM::T;
    constexpr int NS = SM::NS;
    constexpr int SHIFT = 32 - ilog2_ce(T);
    extern __shared__ __align__(16) unsigned char sw_smem[];

    const int lane = lane_id(), gl = lane & (G - 1);
    const int gq = threadIdx.x / G;
    unsigned char* gs = sw_smem + (size_t)gq * SM::GROUP;
    uint32_t* s_tabh = reinterpret_cast<uint32_t*>(gs);                  // [T]
    uint32_t* s_j = s_tabh + T;                                          // [2][NS]
    uint8_t* s_mask = reinterpret_cast<uint8_t*>(s_j + 2 * NS);          // [2][NS / 4]
    uint4* s_tab = reinterpret_cast<uint4*>(s_mask + 2 * (NS / 4));      // [32] (aligned start, lead, lead + items, first piece)
    uint32_t* s_first = reinterpret_cast<uint32_t*>(s_tab + 32);         // [32]

    const int64_t stride = (int64_t)gridDim.x * SW * W;
    int64_t n = (int64_t)blockIdx.x * SW * W + gq;
    int64_t n_warp = n - (gq & (W - 1));
    if (n_warp >= nrows) return;

    const uint4 none = make_uint4(0u, 0u, 0u, 0u);
    auto load_hdr = [&](int64_t idx) { return idx < nrows ? hdr[idx] : none; };
    struct Lists {
        uint2 d[LD];
    };
    auto load_lists = [&](const uint4& h) {
        Lists L;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const uint32_t s = (uint32_t)(gl * LD + u);
            L.d[u] = s < h.z ? P.desc[(int64_t)h.y + s] : make_uint2(0u, 0u);
        }
        return L;
    };
    // issue the gathers of one row into buffer b; returns its number of pieces
    auto issue = [&](const Lists& L, int b) -> uint32_t {
        uint32_t np[LD], mine = 0;
        __syncwarp();  // the tables may still be searched for the previous row
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            uint32_t len = L.d[u].y;
            if (DIAG && len > 0) --len;
            np[u] = len ? (((L.d[u].x & 3u) + len + 3u) >> 2) : 0u;  // aligned pieces that cover the prefix
            mine += np[u];
        }
        const uint32_t incl = group_inclusive_scan<G>(mine, gl);
        const uint32_t tot = __shfl_sync(FULL_MASK, incl, G - 1, G);
        uint32_t run = incl - mine;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const int s = gl * LD + u;
            uint32_t len = L.d[u].y;
            if (DIAG && len > 0) --len;
            const uint32_t lead = L.d[u].x & 3u;
            s_tab[s] = make_uint4(L.d[u].x - lead, lead, lead + len, run);
            s_first[s] = run;
            run += np[u];
        }
        __syncwarp();
        uint32_t* buf = s_j + b * NS;
        uint8_t* mask = s_mask + b * (NS / 4);
        for (uint32_t c = gl; c < tot; c += G) {
            const uint32_t s = last_not_above(s_first, c);
            const uint4 t = s_tab[s];
            const uint32_t e0 = (c - t.w) * 4u;
            if (!SPSYRK_IN_RANGE(4 * c + 3 < (uint32_t)NS, P.err)) continue;
            cp_async<16>(buf + 4 * c, P.at_row + t.x + e0);
            // entries e0 .. e0 + 3 of the aligned run; the prefix is [lead, lead + items)
            uint32_t mk = 0;
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) mk |= (e0 + e >= t.y && e0 + e < t.z) ? (1u << e) : 0u;
            mask[c] = (uint8_t)mk;
        }
        cp_async_commit();
        return tot;
    };

    uint4 h0 = load_hdr(n), hB = load_hdr(n + stride), hA = load_hdr(n + 2 * stride);
    Lists l0 = load_lists(h0);
    Lists lB = load_lists(hB);
    uint4 h_n = h0;
    uint32_t np_n = issue(l0, 0);
    int b = 0;
    for (; n_warp < nrows; n_warp += stride, n += stride, b ^= 1) {
        const uint4 hNew = load_hdr(n + 3 * stride);
        const Lists lNew = load_lists(hA);
        const uint32_t np_next = issue(lB, b ^ 1);
        {
            uint4* t4 = reinterpret_cast<uint4*>(s_tabh);
#pragma unroll
            for (int s = gl; s < T / 4; s += G) t4[s] = make_uint4(0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu);
        }
        cp_async_wait<1>();
        __syncwarp();
        const uint4* buf4 = reinterpret_cast<const uint4*>(s_j + b * NS);
        const uint8_t* mask = s_mask + b * (NS / 4);
        int local = 0;
        for (uint32_t c = gl; c < np_n; c += G) {
            const uint4 q = buf4[c];
            const uint32_t mk = mask[c];
            const uint32_t jj[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (mk & (1u << e)) {
                    const uint32_t j = jj[e];
                    uint32_t h = (j * 2654435761u) >> SHIFT;
                    bool placed = false;
                    for (int probe = 0; probe < T; ++probe) {  // bounded: the table is at most half full
                        const uint32_t old = atomicCAS(&s_tabh[h], 0xffffffffu, j);
                        if (old == 0xffffffffu) { ++local; placed = true; break; }
                        if (old == j) { placed = true; break; }
                        h = (h + 1) & (T - 1);
                    }
                    if (!placed) atomicOr(P.err, ERRW_INTERNAL);
                }
            }
        }
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) local += __shfl_xor_sync(FULL_MASK, local, o);
        if (gl == 0 && h_n.z > 0) cnt[h_n.x] = local + (DIAG ? 1 : 0);
        __syncwarp();  // the table and buffer b are reused by the next rows
        h_n = hB; np_n = np_next;
        hB = hA; lB = lNew; hA = hNew;
    }
    cp_async_wait<0>();
}

// =============================================================================================
// Light rows with an item map.
//
// When the caller lends a map buffer (two bytes per partial product of the light rows), the
// ordering work is done once: the symbolic pass sorts the items of a row by output column and
// records, for item t (in ascending-k, ascending-j order), the output slot it adds into and its
// place q among the items of that slot (0 for the first, in ascending k).  The numeric pass then
// gathers, multiplies and adds: items with q = 0 store their product into their slot, the items
// with q = 1, 2, ... are added round by round, which is the ascending-k summation order again,
// and the row leaves shared memory already sorted.  No sort and no hash table in the numeric pass.
//   map word = slot | q << 9        (slot < 512 items per row, q < 32 lists per row)
// The items of a row occupy a multiple of eight words in the map (16-byte pieces).
// =============================================================================================
constexpr int MAP_SLOT_BITS = 9;

// items of the light rows in class order, rounded up to eight: the scan of these is where a row's map words start
static __global__ void __launch_bounds__(256) row_items_kernel(PlanDev P, const uint4* __restrict__ hdr, const uint8_t* __restrict__ cls,
                                                               int64_t rows, bool diag, uint32_t* __restrict__ items8) {
    const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= rows) return;
    const uint4 h = hdr[n];
    const uint8_t c = cls[h.x];
    uint32_t it = 0;
    if (c >= 1 && c <= 5) it = (uint32_t)(P.work[h.x] - (diag ? (int64_t)h.z : 0));
    items8[n] = (it + 7u) & ~7u;
}

template <int N>
struct SymbolicSortSmem {
    static constexpr int NS = N + 8 * 32;  // landing slots: aligned pieces carry up to 3 + 3 foreign entries per list
    // per group: two landing buffers, two piece-meta arrays (16 bits per piece), the dense row ids, the map words, the tables
    static constexpr int GROUP = 2 * NS * 4 + 2 * (NS / 4) * 2 + N * 4 + N * 2 + 32 * 16 + 32 * 4;
};

__host__ __device__ constexpr int symbolic_sort_warps(int n) { return n >= 512 ? 2 : 4; }
__host__ __device__ constexpr int symbolic_sort_min_ctas(int n) { return n >= 512 ? 4 : 5; }

template <int N, int G, typename Key, bool DIAG>
__global__ void __launch_bounds__(symbolic_sort_warps(N) * 32, symbolic_sort_min_ctas(N))
symbolic_sort_warp_kernel(PlanDev P, const uint4* __restrict__ hdr, const int64_t* __restrict__ itemoff, int64_t nrows,
                          int32_t* __restrict__ cnt, uint16_t* __restrict__ map) {
    using SM = SymbolicSortSmem<N>;
    constexpr int SW = symbolic_sort_warps(N);
    constexpr int W = 32 / G;
    constexpr int LD = 32 / G;
    constexpr int R = N / G;
    constexpr int NS = SM::NS;
    constexpr int IDXB = ilog2_ce(N);
    constexpr Key PAD = ~Key(0);
    extern __shared__ __align__(16) unsigned char ss_smem[];

    const int lane = lane_id(), gl = lane & (G - 1);
    const int gq = threadIdx.x / G;
    unsigned char* gs = ss_smem + (size_t)gq * SM::GROUP;
    uint32_t* s_j = reinterpret_cast<uint32_t*>(gs);                          // [2][NS]
    uint16_t* s_meta = reinterpret_cast<uint16_t*>(s_j + 2 * NS);             // [2][NS / 4]
    uint32_t* s_jd = reinterpret_cast<uint32_t*>(s_meta + 2 * (NS / 4));      // [N] row ids in item order
    uint16_t* s_map = reinterpret_cast<uint16_t*>(s_jd + N);                  // [N]
    uint4* s_tab = reinterpret_cast<uint4*>(s_map + N);                       // [32]
    uint32_t* s_first = reinterpret_cast<uint32_t*>(s_tab + 32);              // [32]

    const int64_t stride = (int64_t)gridDim.x * SW * W;
    int64_t n = (int64_t)blockIdx.x * SW * W + gq;
    int64_t n_warp = n - (gq & (W - 1));
    if (n_warp >= nrows) return;

    const uint4 none = make_uint4(0u, 0u, 0u, 0u);
    auto load_hdr = [&](int64_t idx) { return idx < nrows ? hdr[idx] : none; };
    struct Lists {
        uint2 d[LD];
    };
    auto load_lists = [&](const uint4& h) {
        Lists L;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const uint32_t s = (uint32_t)(gl * LD + u);
            L.d[u] = s < h.z ? P.desc[(int64_t)h.y + s] : make_uint2(0u, 0u);
        }
        return L;
    };
    // issue the gathers of one row into buffer b; returns pieces << 16 | items
    auto issue = [&](const Lists& L, int b) -> uint32_t {
        uint32_t pk[LD], mine = 0;
        __syncwarp();  // the tables may still be searched for the previous row
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            uint32_t len = L.d[u].y;
            if (DIAG && len > 0) --len;
            const uint32_t np = len ? (((L.d[u].x & 3u) + len + 3u) >> 2) : 0u;  // aligned pieces that cover the prefix
            pk[u] = (np << 16) | len;
            mine += pk[u];
        }
        const uint32_t incl = group_inclusive_scan<G>(mine, gl);
        const uint32_t tot = __shfl_sync(FULL_MASK, incl, G - 1, G);
        uint32_t run = incl - mine;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const int s = gl * LD + u;
            const uint32_t lead = L.d[u].x & 3u;
            s_tab[s] = make_uint4(L.d[u].x - lead, lead | ((run & 0xffffu) << 8), lead + (pk[u] & 0xffffu), run >> 16);
            s_first[s] = run >> 16;
            run += pk[u];
        }
        __syncwarp();
        uint32_t* buf = s_j + b * NS;
        uint16_t* meta = s_meta + b * (NS / 4);
        const uint32_t npieces = tot >> 16;
        for (uint32_t c = gl; c < npieces; c += G) {
            const uint32_t s = last_not_above(s_first, c);
            const uint4 t = s_tab[s];
            const uint32_t e0 = (c - t.w) * 4u;
            const uint32_t lead = t.y & 0xffu, off = t.y >> 8;
            if (!SPSYRK_IN_RANGE(4 * c + 3 < (uint32_t)NS && off + e0 + 3u - lead < (uint32_t)N + 3u, P.err)) {
                meta[c] = 0;
                continue;
            }
            cp_async<16>(buf + 4 * c, P.at_row + t.x + e0);
            uint32_t mk = 0;
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) mk |= (e0 + e >= lead && e0 + e < t.z) ? (1u << e) : 0u;
            // item index of the piece's entry 0, plus 3 (the first piece of a list can start before its prefix)
            meta[c] = (uint16_t)(mk | ((off + e0 + 3u - lead) << 4));
        }
        cp_async_commit();
        return tot;
    };

    uint4 h0 = load_hdr(n), hB = load_hdr(n + stride), hA = load_hdr(n + 2 * stride);
    Lists l0 = load_lists(h0);
    Lists lB = load_lists(hB);
    uint4 h_n = h0;
    int64_t io_n = n < nrows ? itemoff[n] : 0;
    uint32_t pw_n = issue(l0, 0);
    int b = 0;
    for (; n_warp < nrows; n_warp += stride, n += stride, b ^= 1) {
        const uint4 hNew = load_hdr(n + 3 * stride);
        const Lists lNew = load_lists(hA);
        const int64_t io_next = n + stride < nrows ? itemoff[n + stride] : 0;
        const uint32_t pw_next = issue(lB, b ^ 1);
        cp_async_wait<1>();
        __syncwarp();
        const uint32_t w_n = pw_n & 0xffffu, np_n = pw_n >> 16;
        {
            // the valid entries of the pieces, in item order
            const uint4* buf4 = reinterpret_cast<const uint4*>(s_j + b * NS);
            const uint16_t* meta = s_meta + b * (NS / 4);
            for (uint32_t c = gl; c < np_n; c += G) {
                const uint4 q = buf4[c];
                const uint32_t mt = meta[c];
                const int tb = (int)(mt >> 4) - 3;
                if (!SPSYRK_IN_RANGE(tb + 3 >= 0 && tb < N, P.err)) continue;
                if ((mt & 1u) && SPSYRK_IN_RANGE(tb >= 0, P.err)) s_jd[tb] = q.x;
                if ((mt & 2u) && SPSYRK_IN_RANGE(tb + 1 >= 0 && tb + 1 < N, P.err)) s_jd[tb + 1] = q.y;
                if ((mt & 4u) && SPSYRK_IN_RANGE(tb + 2 >= 0 && tb + 2 < N, P.err)) s_jd[tb + 2] = q.z;
                if ((mt & 8u) && SPSYRK_IN_RANGE(tb + 3 < N, P.err)) s_jd[tb + 3] = q.w;
            }
        }
        __syncwarp();
        Key key[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const uint32_t t = r * G + gl;
            key[r] = t < w_n ? (((Key)s_jd[t] << IDXB) | (Key)t) : PAD;
        }
        group_bitonic_sort<Key, R, G>(key);

        // same[r]: element r continues the run of equal j of element r-1
        constexpr Key JUNIT = Key(1) << IDXB;
        const Key prev_last = __shfl_up_sync(FULL_MASK, key[R - 1], 1, G);
        const int e0 = gl * R;  // sorted position of this lane's first element
        int nheads = 0, last_head = -1;
        bool head[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool same = r == 0 ? (gl > 0 && ((key[0] ^ prev_last) < JUNIT)) : ((key[r] ^ key[r - 1]) < JUNIT);
            head[r] = (uint32_t)(e0 + r) < w_n && !same;
            nheads += head[r];
            if (head[r]) last_head = e0 + r;
        }
        // slot = heads up to and including the element, minus one; q = distance to the head of the run
        const int hincl = (int)group_inclusive_scan<G>((uint32_t)nheads, gl);
        const int total = __shfl_sync(FULL_MASK, hincl, G - 1, G);
        int hp = last_head;  // inclusive max-scan of the last head position over the lanes
#pragma unroll
        for (int o = 1; o < G; o <<= 1) {
            const int t = __shfl_up_sync(FULL_MASK, hp, o, G);
            if (gl >= o) hp = max(hp, t);
        }
        int cur = __shfl_up_sync(FULL_MASK, hp, 1, G);  // last head before this lane
        if (gl == 0) cur = -1;
        int hc = hincl - nheads;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if ((uint32_t)(e0 + r) < w_n) {
                if (head[r]) { cur = e0 + r; ++hc; }
                const uint32_t t = (uint32_t)(key[r] & (Key)(N - 1));
                s_map[t] = (uint16_t)((uint32_t)(hc - 1) | ((uint32_t)(e0 + r - cur) << MAP_SLOT_BITS));
            }
        }
        if (gl == 0 && h_n.z > 0) cnt[h_n.x] = total + (DIAG ? 1 : 0);
        __syncwarp();
        {
            const uint4* src = reinterpret_cast<const uint4*>(s_map);
            uint4* dst = reinterpret_cast<uint4*>(map + io_n);
            const uint32_t nch = (w_n + 7u) >> 3;
            for (uint32_t c = gl; c < nch; c += G) dst[c] = src[c];
        }
        __syncwarp();  // the dense arrays and buffer b are reused by the next rows
        h_n = hB; pw_n = pw_next; io_n = io_next;
        hB = hA; lB = lNew; hA = hNew;
    }
    cp_async_wait<0>();
}

template <typename V, int N>
struct NumericMapSmem {
    using Acc = typename AccOf<V>::type;
    using Rec = ColRec<V>;
    // per group: two record buffers, two owner arrays, two map buffers, two copies of the row's own values,
    // the output row (column ids, sums), the tables
    static constexpr int GROUP = 2 * (int)sizeof(Rec) * N + 2 * N + 2 * 2 * N + 2 * 32 * (int)sizeof(Acc) + 4 * (N + 4) +
                                 (int)sizeof(Acc) * (N + 4) + 32 * 16 + 32 * 4;
};

__host__ __device__ constexpr int numeric_map_warps(int n) { return n >= 512 ? 2 : 4; }

template <typename V, int N, int G, bool DIAG>
__global__ void __launch_bounds__(numeric_map_warps(N) * 32)
numeric_map_warp_kernel(PlanDev P, const uint4* __restrict__ hdr, const int64_t* __restrict__ itemoff, int64_t nrows,
                        const uint16_t* __restrict__ map, const int64_t* __restrict__ c_rowptr, const int64_t* __restrict__ c_rowend,
                        int32_t* __restrict__ c_colidx, V* __restrict__ c_vals) {
    using Acc = typename AccOf<V>::type;
    using Rec = ColRec<V>;
    using SM = NumericMapSmem<V, N>;
    constexpr int NW = numeric_map_warps(N);
    constexpr int W = 32 / G;
    constexpr int LD = 32 / G;
    constexpr int R = N / G;
    extern __shared__ __align__(16) unsigned char nm_smem[];

    const int lane = lane_id(), gl = lane & (G - 1);
    const int gq = threadIdx.x / G;
    unsigned char* gs = nm_smem + (size_t)gq * SM::GROUP;
    Rec* s_rec = reinterpret_cast<Rec*>(gs);                                   // [2][N]
    uint8_t* s_own = reinterpret_cast<uint8_t*>(s_rec + 2 * N);                // [2][N]
    uint16_t* s_mapw = reinterpret_cast<uint16_t*>(s_own + 2 * N);             // [2][N]
    Acc* s_a = reinterpret_cast<Acc*>(s_mapw + 2 * N);                         // [2][32]
    Acc* o_v = s_a + 64;                                                       // [N + 4]
    uint32_t* o_j = reinterpret_cast<uint32_t*>(o_v + N + 4);                  // [N + 4]
    uint4* s_tab = reinterpret_cast<uint4*>(o_j + N + 4);                      // [32]
    uint32_t* s_first = reinterpret_cast<uint32_t*>(s_tab + 32);               // [32]

    const int64_t stride = (int64_t)gridDim.x * NW * W;
    int64_t n = (int64_t)blockIdx.x * NW * W + gq;
    int64_t n_warp = n - (gq & (W - 1));
    if (n_warp >= nrows) return;

    const uint4 none = make_uint4(0u, 0u, 0u, 0u);
    const Rec* __restrict__ recs = static_cast<const Rec*>(P.at_rec);
    auto load_hdr = [&](int64_t idx) { return idx < nrows ? hdr[idx] : none; };
    struct Lists {
        uint2 d[LD];
        Acc a[LD];
    };
    auto load_lists = [&](const uint4& h) {
        Lists L;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const uint32_t s = (uint32_t)(gl * LD + u);
            const bool on = s < h.z;
            L.d[u] = on ? P.desc[(int64_t)h.y + s] : make_uint2(0u, 0u);
            L.a[u] = on ? (Acc) static_cast<const V*>(P.vals)[(int64_t)h.y + s] : Acc(0);
        }
        return L;
    };
    auto issue = [&](const Lists& L, int64_t io, int b) -> uint32_t {
        uint32_t pk[LD], mine = 0;
        __syncwarp();
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            uint32_t len = L.d[u].y;
            if (DIAG && len > 0) --len;
            pk[u] = (((len + 3u) >> 2) << 16) | len;
            mine += pk[u];
        }
        const uint32_t incl = group_inclusive_scan<G>(mine, gl);
        const uint32_t tot = __shfl_sync(FULL_MASK, incl, G - 1, G);
        uint32_t run = incl - mine;
#pragma unroll
        for (int u = 0; u < LD; ++u) {
            const int s = gl * LD + u;
            s_tab[s] = make_uint4(L.d[u].x, run & 0xffffu, pk[u] & 0xffffu, run >> 16);
            s_first[s] = run >> 16;
            s_a[b * 32 + s] = L.a[u];
            run += pk[u];
        }
        __syncwarp();
        const uint32_t npieces = tot >> 16, w = tot & 0xffffu;
        Rec* buf = s_rec + b * N;
        uint8_t* own = s_own + b * N;
        for (uint32_t c = gl; c < npieces; c += G) {
            const uint32_t s = last_not_above(s_first, c);
            const uint4 t = s_tab[s];
            const uint32_t e0 = (c - t.w) * 4u;
            const uint32_t left = t.z - e0;
            const Rec* src = recs + t.x + e0;
            const uint32_t slot = t.y + e0;
#pragma unroll
            for (uint32_t e = 0; e < 4; ++e) {
                if (e < left && SPSYRK_IN_RANGE(slot + e < (uint32_t)N, P.err)) {
                    cp_async<sizeof(Rec)>(buf + slot + e, src + e);
                    own[slot + e] = (uint8_t)s;
                }
            }
        }
        {
            const uint4* src = reinterpret_cast<const uint4*>(map + io);
            uint4* dst = reinterpret_cast<uint4*>(s_mapw + b * N);
            const uint32_t nch = (w + 7u) >> 3;
            for (uint32_t c = gl; c < nch; c += G) cp_async<16>(dst + c, src + c);
        }
        cp_async_commit();
        return w;
    };

    uint4 h0 = load_hdr(n), hB = load_hdr(n + stride), hA = load_hdr(n + 2 * stride);
    Lists l0 = load_lists(h0);
    Lists lB = load_lists(hB);
    int64_t ioB = n + stride < nrows ? itemoff[n + stride] : 0;
    uint4 h_n = h0;
    int64_t ob_n = h0.z ? c_rowptr[h0.x] : 0, oe_n = h0.z ? c_rowend[h0.x] : 0;
    uint32_t w_n = issue(l0, n < nrows ? itemoff[n] : 0, 0);
    int b = 0;

    for (; n_warp < nrows; n_warp += stride, n += stride, b ^= 1) {
        const uint4 hNew = load_hdr(n + 3 * stride);
        const Lists lNew = load_lists(hA);
        const int64_t ioNew = n + 2 * stride < nrows ? itemoff[n + 2 * stride] : 0;
        const int64_t ob_next = hB.z ? c_rowptr[hB.x] : 0, oe_next = hB.z ? c_rowend[hB.x] : 0;
        const uint32_t w_next = issue(lB, ioB, b ^ 1);

        cp_async_wait<1>();
        __syncwarp();
        const Rec* buf = s_rec + b * N;
        const uint8_t* own = s_own + b * N;
        const uint16_t* mw = s_mapw + b * N;
        Acc prod[R];
        uint32_t word[R];
        uint32_t qmax = 0;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const uint32_t t = r * G + gl;
            word[r] = 0xffffffffu;
            prod[r] = Acc(0);
            if (t < w_n) {
                const Rec rc = buf[t];
                const Acc a = s_a[b * 32 + own[t]];
                prod[r] = acc_mul(a, (Acc)rc.v);
                word[r] = mw[t];
                const uint32_t slot = word[r] & ((1u << MAP_SLOT_BITS) - 1u);
                if (!SPSYRK_IN_RANGE(slot < (uint32_t)N, P.err)) {
                    word[r] = 0xffffffffu;
                } else if ((word[r] >> MAP_SLOT_BITS) == 0) {
                    o_j[slot] = (uint32_t)rc.j;
                    o_v[slot] = prod[r];
                } else {
                    qmax = max(qmax, word[r] >> MAP_SLOT_BITS);
                }
            }
        }
        Acc diag = Acc(0);
        if (DIAG) {
            uint32_t dmax = h_n.z;
            if (G < 32) dmax = __reduce_max_sync(FULL_MASK, dmax);
            for (uint32_t s = 0; s < dmax; ++s) {
                const Acc a = s_a[b * 32 + (s & 31)];
                if (s < h_n.z) diag = acc_add(diag, acc_mul(a, a));
            }
        }
        qmax = __reduce_max_sync(FULL_MASK, qmax);
        // later items of a slot, one place at a time: ascending k inside every entry
        for (uint32_t q = 1; q <= qmax; ++q) {
            __syncwarp();
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (word[r] != 0xffffffffu && (word[r] >> MAP_SLOT_BITS) == q) {
                    const uint32_t slot = word[r] & ((1u << MAP_SLOT_BITS) - 1u);
                    o_v[slot] = acc_add(o_v[slot], prod[r]);
                }
            }
        }
        int total = (int)(oe_n - ob_n);
        if (!SPSYRK_IN_RANGE(total >= 0 && total <= N + (DIAG ? 1 : 0), P.err)) total = 0;
        if (DIAG && h_n.z > 0 && total > 0 && gl == 0) {
            o_j[total - 1] = (uint32_t)P.r0 + h_n.x;
            o_v[total - 1] = diag;
        }
        __syncwarp();
        for (int o = gl; o < total; o += G) {
            const int32_t j = (int32_t)o_j[o];
            const V cv = (V)o_v[o];
            c_colidx[ob_n + o] = j;
            c_vals[ob_n + o] = cv;
            if constexpr (std::is_same<V, int32_t>::value) {
                if (P.jaccard) {
                    const int64_t na_j = P.adeg[j];
                    P.jaccard[ob_n + o] = __fdiv_rn((float)cv, (float)((int64_t)h_n.z + na_j - (int64_t)cv));
                }
            }
        }
        __syncwarp();  // the output row and buffer b are reused

        h_n = hB; w_n = w_next; ob_n = ob_next; oe_n = oe_next;
        hB = hA; lB = lNew; hA = hNew; ioB = ioNew;
    }
    cp_async_wait<0>();
}

}  // namespace spsyrk
