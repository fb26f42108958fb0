// Steps a4 / a6 for heavy rows: one CTA per output row.
//
// The output columns j of row i lie in [0, U), U = i + 1 (TRIL) or m (FULL).  The range is cut
// into chunks of `chunk_bits` columns.  For each chunk a shared-memory bitmap records which j
// occur; a prefix population count over its words turns the bitmap into an order-preserving map
// j -> output slot (number of set bits below j), so rows come out sorted with no sort at all:
//   symbolic : the row count is the number of set bits over all chunks;
//   numeric  : partial products are added into shared-memory accumulators indexed by slot
//              (tiles of `acc_slots` slots; a tile is a contiguous range of j, found per column
//              list by binary search, the lists being ascending in j), then tiles are written out
//              contiguously; column ids are regenerated from the bitmap.
// Work is spread over the CTA by flattening the (list, position) pairs of up to THREADS lists at
// a time through a prefix sum of their lengths, so that one very long list is shared by all lanes.
#pragma once
#include "transpose.cuh"

namespace spsyrk {

enum : int { CTA_SETBITS = 0, CTA_ACCUM = 1 };

// CTAs per SM the launches are sized for (shared memory allows no more): stated so that the register allocation
// does not trade spills for an occupancy the kernel cannot reach
// (the counting pass holds little state: it keeps the 32 registers that let 2048 threads share an SM)
__host__ __device__ constexpr int cta_min_blocks(int threads, bool numeric) {
    return !numeric ? 2048 / threads : threads >= 1024 ? 1 : threads >= 512 ? 2 : 3;
}

template <typename V, int THREADS, bool NUMERIC>
struct CtaRowSmem {
    using Acc = typename AccOf<V>::type;
    static size_t bytes(uint32_t chunk_bits, uint32_t acc_slots) {
        size_t words = (size_t)(chunk_bits >> 5) * (NUMERIC ? 2 : 1) + 5 * THREADS + 1;
        words = (words + 3) & ~size_t(3);
        size_t b = words * 4;
        if (NUMERIC) b += (size_t)THREADS * sizeof(Acc) + (size_t)acc_slots * sizeof(Acc);
        return b;
    }
};

// GLOBAL_ACC: the variant for rows whose output does not fit the shared-memory accumulator tile.
// Instead of walking the lists once per tile, it accumulates the whole row in one pass into a
// global-memory slice owned by the CTA (global atomics, served by L2).  It runs as a persistent grid:
// CTAs fetch rows from a counter, so that the slice indexed by blockIdx.x is never shared.  The
// two variants are launched over the same row list and each skips the rows of the other.
template <typename V, int THREADS, bool NUMERIC, bool GLOBAL_ACC = false>
__global__ void __launch_bounds__(THREADS, cta_min_blocks(THREADS, NUMERIC)) rows_cta_kernel(PlanDev P, const int32_t* __restrict__ rows,
                                                           uint32_t chunk_bits, uint32_t acc_slots,
                                                           int32_t* __restrict__ cnt,
                                                           const int64_t* __restrict__ c_rowptr, const int64_t* __restrict__ c_rowend,
                                                           int32_t* __restrict__ c_colidx, V* __restrict__ c_vals,
                                                           uint32_t nrows = 0, uint32_t* row_counter = nullptr,
                                                           typename AccOf<V>::type* gscratch = nullptr, uint32_t gslots = 0) {
    using Acc = typename AccOf<V>::type;
    __shared__ uint32_t s_row;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t s_sel[2];
    __shared__ uint32_t s_nlong;
    const uint32_t cw = chunk_bits >> 5;
    uint32_t* bits = reinterpret_cast<uint32_t*>(smem_raw);
    uint32_t* rank = bits + cw;  // numeric only
    uint32_t* loff = bits + (size_t)cw * (NUMERIC ? 2 : 1);
    uint32_t* lstart = loff + THREADS + 1;
    uint32_t* llen = lstart + THREADS;      // lengths of the batch's lists
    uint32_t* long_idx = llen + THREADS;    // batch indices of the long lists
    uint32_t* lprev = long_idx + THREADS;   // where the previous slot tile ended inside each list
    size_t words = (size_t)cw * (NUMERIC ? 2 : 1) + 5 * THREADS + 1;
    words = (words + 3) & ~size_t(3);
    Acc* la = reinterpret_cast<Acc*>(smem_raw + words * 4);
    Acc* acc = GLOBAL_ACC ? gscratch + (size_t)blockIdx.x * gslots : la + THREADS;
    const uint32_t tile_slots = GLOBAL_ACC ? gslots : acc_slots;  // slots accumulated per pass over the lists

    const int tid = threadIdx.x;
    auto do_row = [&](const int32_t rloc) {
    const int64_t i = (int64_t)P.r0 + rloc;
    const uint32_t U = P.mode == SPSYRK_TRIL ? (uint32_t)i + 1u : (uint32_t)P.m;
    if (NUMERIC) {
        // rows that overflow the shared-memory tile (and are not full) belong to the global variant
        const int64_t row_cnt = c_rowend[rloc] - c_rowptr[rloc];
        const bool wants_global = gslots > 0 && row_cnt > (int64_t)acc_slots && U <= chunk_bits && row_cnt < (int64_t)U &&
                                  row_cnt <= (int64_t)gslots;
        if (wants_global != GLOBAL_ACC) return;
    }
    const int64_t p0 = P.rowptr[i];
    const uint32_t deg = (uint32_t)(P.rowptr[i + 1] - p0);
    const int64_t out_base = NUMERIC ? c_rowptr[rloc] : 0;
    const int64_t out_end = NUMERIC ? c_rowend[rloc] : 0;  // bounds-checked build: no write at or past it
    (void)out_end;
    uint32_t total_cnt = 0;

    // A row whose range fits one chunk and that holds a column present in every candidate row
    // (a list as long as the range) is dense: every j occurs, slot = j, no bitmap is needed.
    bool dense = false;
    if (U <= chunk_bits) {
        int hit = 0;
        for (uint32_t b0 = tid; b0 < deg; b0 += THREADS) hit |= (P.desc[p0 + b0].y == U);
        dense = __syncthreads_or(hit) != 0;
    }
    if (dense && !NUMERIC) {
        if (tid == 0) cnt[rloc] = (int32_t)U;
        return;
    }
    // Binary input: a partial product is 1.  In a dense row the heavy columns' share of every count comes
    // from the per-row bit masks (one population count per entry), and their lists are not walked.
    const bool binary = P.binary != 0;
    const bool use_masks = NUMERIC && dense && binary && P.nheavy > 0;
    const unsigned long long mask_i = use_masks ? P.heavy_mask[i] : 0ull;
    // Binary input, dense row of at most 255 nonzeros: every count is at most the row's own length, so four
    // 8-bit counters share a 32-bit word of the accumulator tile and a tile holds four times the columns
    // (a row of 1e5 columns is one tile: its lists are cut into column ranges once, not once per tile).
    const bool packed = NUMERIC && !GLOBAL_ACC && std::is_same<V, int32_t>::value && dense && binary && deg <= 255u;
    const uint32_t row_tile_slots = packed ? tile_slots * 4u : tile_slots;

    // One partial product: set its bit, or add it into its slot.
    auto apply = [&](auto what, auto dense_tag, uint32_t rel, Acc a, Acc v, uint32_t s0) {
        constexpr int WHAT = decltype(what)::value;
        constexpr bool DENSE = decltype(dense_tag)::value;
        if (WHAT == CTA_SETBITS) {
            if (SPSYRK_IN_RANGE((rel >> 5) < cw, P.err)) atomicOr(&bits[rel >> 5], 1u << (rel & 31));
        } else {
            if (!SPSYRK_IN_RANGE(DENSE || (rel >> 5) < cw, P.err)) return;
            const uint32_t slot = (DENSE ? rel : rank[rel >> 5] + __popc(bits[rel >> 5] & ((1u << (rel & 31)) - 1u))) - s0;
            if (!SPSYRK_IN_RANGE(slot < row_tile_slots, P.err)) return;
            if (DENSE && packed) atomicAdd(reinterpret_cast<uint32_t*>(acc) + (slot >> 2), 1u << ((slot & 3u) * 8u));  // a product of a binary matrix is 1
            else atomicAdd(&acc[slot], acc_mul(a, v));
        }
    };

    // Visit every partial product whose j lies in [lo, hi); `whole` skips the per-list search.
    // Lists of at least LONG_LIST entries are walked one after the other by the whole CTA (a lean
    // loop: two loads and one shared-memory atomic per product); the shorter ones are flattened
    // through a prefix sum of their lengths so that no lane idles on a short list.
    constexpr uint32_t LONG_LIST = THREADS / 2;
    constexpr int UNR = 4;
    // `resume`: the range starts where the previous call's range ended (consecutive slot tiles of a row
    // with at most THREADS lists), so each list's lower end is remembered instead of searched again.
    // ones_tag: the partial products are ones (binary input, or the bit-setting pass): only row ids are read
    auto for_each_product = [&](auto what, auto dense_tag, auto ones_tag, uint32_t lo, uint32_t hi, bool whole, uint32_t c0, uint32_t s0,
                                bool resume) {
        constexpr int WHAT = decltype(what)::value;
        constexpr bool ONES = decltype(ones_tag)::value || WHAT != CTA_ACCUM;
        for (uint32_t b0 = 0; b0 < deg; b0 += THREADS) {
            uint32_t sublen = 0, substart = 0;
            Acc a = Acc(0);
            if (tid == 0) s_nlong = 0;
            if (b0 + tid < deg) {
                uint2 d = P.desc[p0 + b0 + tid];
                if (WHAT == CTA_ACCUM && use_masks && P.heavy_id[P.colidx[p0 + b0 + tid]] != 0xff) d.y = 0;  // counted through the masks
                if (whole) {
                    substart = d.x;
                    sublen = d.y;
                } else {
                    const int32_t* lst = P.at_row + d.x;
                    const uint32_t a0 = lo == 0 ? 0u : resume ? lprev[tid] : lower_bound_i32(lst, d.y, (int32_t)lo);
                    const uint32_t a1 = a0 + lower_bound_i32(lst + a0, d.y - a0, (int32_t)hi);
                    if (deg <= THREADS) lprev[tid] = a1;
                    substart = d.x + a0;
                    sublen = a1 - a0;
                }
                if (WHAT == CTA_ACCUM) a = binary ? Acc(1) : (Acc) static_cast<const V*>(P.vals)[p0 + b0 + tid];
            }
            const bool is_long = sublen >= LONG_LIST;
            uint32_t T;
            const uint32_t ex = block_exclusive_scan<uint32_t, THREADS>(is_long ? 0u : sublen, scratch, &T);
            loff[tid] = ex;
            lstart[tid] = substart;
            llen[tid] = sublen;
            if (WHAT == CTA_ACCUM) la[tid] = a;
            if (tid == 0) loff[THREADS] = T;
            if (is_long) long_idx[atomicAdd(&s_nlong, 1u)] = tid;
            __syncthreads();
            // short lists, flattened: every warp takes a contiguous run of items and its lanes interleave
            // inside it, so that a warp's loads are coalesced and UNR different lines are in flight; a lane
            // steps from list to list as its items advance (no search per item)
            {
                constexpr uint32_t NW = THREADS / 32;
                const uint32_t per_warp = ((T + NW - 1) / NW + 31u) & ~31u;
                const uint32_t wfirst = min((uint32_t)(tid >> 5) * per_warp, T), last = min(wfirst + per_warp, T);
                const uint32_t first = wfirst + (tid & 31);
                if (first < last) {
                    uint32_t lo_l = 0, hi_l = THREADS;  // last list whose offset is <= first
                    while (hi_l - lo_l > 1) {
                        const uint32_t mid = (lo_l + hi_l) >> 1;
                        if (loff[mid] <= first) lo_l = mid; else hi_l = mid;
                    }
                    uint32_t cur = lo_l, cur_off = loff[cur], next_off = loff[cur + 1], cur_start = lstart[cur];
                    Acc cur_a = WHAT == CTA_ACCUM ? la[cur] : Acc(0);
                    for (uint32_t item0 = first; item0 < last; item0 += UNR * 32) {
                        uint32_t q[UNR];
                        Acc av[UNR];
#pragma unroll
                        for (int u = 0; u < UNR; ++u) {
                            const uint32_t item = item0 + u * 32;
                            q[u] = 0xffffffffu;
                            av[u] = Acc(0);
                            if (item < last) {
                                if (item >= next_off) {
                                    do { ++cur; } while (item >= loff[cur + 1]);
                                    cur_off = loff[cur];
                                    next_off = loff[cur + 1];
                                    cur_start = lstart[cur];
                                    if (WHAT == CTA_ACCUM) cur_a = la[cur];
                                }
                                q[u] = cur_start + (item - cur_off);
                                av[u] = cur_a;
                            }
                        }
                        uint32_t rel[UNR];
                        Acc val[UNR];
#pragma unroll
                        for (int u = 0; u < UNR; ++u) {
                            rel[u] = 0;
                            val[u] = Acc(0);
                            if (q[u] != 0xffffffffu) {
                                if constexpr (!ONES) {
                                    // one load brings the row id and the value (the records the light rows gather)
                                    const ColRec<V> rec = static_cast<const ColRec<V>*>(P.at_rec)[q[u]];
                                    rel[u] = (uint32_t)rec.j - c0;
                                    val[u] = (Acc)rec.v;
                                } else {
                                    rel[u] = (uint32_t)P.at_row[q[u]] - c0;
                                    val[u] = Acc(1);
                                }
                            }
                        }
#pragma unroll
                        for (int u = 0; u < UNR; ++u)
                            if (q[u] != 0xffffffffu) apply(what, dense_tag, rel[u], av[u], val[u], s0);
                    }
                }
            }
            // long lists, one after the other
            const uint32_t nlong = s_nlong;
            for (uint32_t li = 0; li < nlong; ++li) {
                const uint32_t t = long_idx[li];
                const uint32_t len = llen[t];
                const int32_t* __restrict__ rowp = P.at_row + lstart[t];
                const ColRec<V>* __restrict__ recp = static_cast<const ColRec<V>*>(P.at_rec) + lstart[t];
                const Acc fa = WHAT == CTA_ACCUM ? la[t] : Acc(0);
                uint32_t e = tid;
                for (; e + (UNR - 1) * THREADS < len; e += UNR * THREADS) {
                    uint32_t rel[UNR];
                    Acc val[UNR];
#pragma unroll
                    for (int u = 0; u < UNR; ++u) {
                        if constexpr (!ONES) {
                            const ColRec<V> rec = recp[e + u * THREADS];
                            rel[u] = (uint32_t)rec.j - c0;
                            val[u] = (Acc)rec.v;
                        } else {
                            rel[u] = (uint32_t)rowp[e + u * THREADS] - c0;
                            val[u] = Acc(1);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < UNR; ++u) apply(what, dense_tag, rel[u], fa, val[u], s0);
                }
                for (; e < len; e += THREADS) {
                    if constexpr (!ONES) {
                        const ColRec<V> rec = recp[e];
                        apply(what, dense_tag, (uint32_t)rec.j - c0, fa, (Acc)rec.v, s0);
                    } else {
                        apply(what, dense_tag, (uint32_t)rowp[e] - c0, fa, Acc(1), s0);
                    }
                }
            }
            __syncthreads();
        }
    };
    const std::integral_constant<int, CTA_SETBITS> SET{};
    const std::integral_constant<int, CTA_ACCUM> ACC{};
    const std::true_type IS_DENSE{};
    const std::false_type NOT_DENSE{};

    for (uint32_t c0 = 0; c0 < U; c0 += chunk_bits) {
        const uint32_t c1 = min(c0 + chunk_bits, U);
        const bool single_chunk = (c0 == 0 && c1 == U);
        const uint32_t cwa = (c1 - c0 + 31) >> 5;  // words of the bitmap this chunk uses
        const uint32_t per = (cwa + THREADS - 1) / THREADS;
        const uint32_t w0 = tid * per;
        uint32_t tot = c1 - c0;
        if (!dense) {
            for (uint32_t w = tid; w < cwa; w += THREADS) bits[w] = 0;
            __syncthreads();
            for_each_product(SET, NOT_DENSE, IS_DENSE, c0, c1, single_chunk, c0, 0u, false);
            uint32_t s = 0;
            for (uint32_t w = w0; w < w0 + per && w < cwa; ++w) s += __popc(bits[w]);
            uint32_t ex = block_exclusive_scan<uint32_t, THREADS>(s, scratch, &tot);
            if (NUMERIC) {
                for (uint32_t w = w0; w < w0 + per && w < cwa; ++w) { rank[w] = ex; ex += __popc(bits[w]); }
                __syncthreads();
            }
        }
        if (NUMERIC) {
            const int64_t ob = out_base + total_cnt;
            if (!dense) {  // (a dense row writes its column ids, c0 + slot, with its values below)
                // column ids straight from the bitmap
                for (uint32_t w = tid; w < cwa; w += THREADS) {
                    uint32_t b = bits[w], r = rank[w];
                    while (b) {
                        const int bit = __ffs(b) - 1;
                        if (SPSYRK_IN_RANGE(ob + r < out_end, P.err)) c_colidx[ob + r] = (int32_t)(c0 + (w << 5) + bit);
                        ++r;
                        b &= b - 1;
                    }
                }
            }
            for (uint32_t s0 = 0; s0 < tot; s0 += row_tile_slots) {
                const uint32_t s1 = min(s0 + row_tile_slots, tot);
                const bool single_tile = (s0 == 0 && s1 == tot);
                uint32_t jlo = c0, jhi = c1;
                if (!single_tile && dense) {
                    jlo = c0 + s0;
                    jhi = c0 + s1;
                } else if (!single_tile) {
                    if (tid < 2) {
                        const uint32_t sl = tid == 0 ? s0 : s1;
                        uint32_t res;
                        if (tid == 0 && s0 == 0) res = c0;
                        else if (tid == 1 && s1 == tot) res = c1;
                        else {
                            // last word whose rank is <= sl holds slot sl
                            uint32_t lo_w = 0, hi_w = cwa;
                            while (hi_w - lo_w > 1) {
                                uint32_t mid = (lo_w + hi_w) >> 1;
                                if (rank[mid] <= sl) lo_w = mid; else hi_w = mid;
                            }
                            uint32_t b = bits[lo_w];
                            for (uint32_t n = sl - rank[lo_w]; n > 0; --n) b &= b - 1;
                            res = c0 + (lo_w << 5) + (uint32_t)(__ffs(b) - 1);
                        }
                        s_sel[tid] = res;
                    }
                    __syncthreads();
                    jlo = s_sel[0];
                    jhi = s_sel[1];
                }
                if (packed) {
                    // slot t of a dense row is column c0 + s0 + t; word w holds slots 4 w .. 4 w + 3
                    const uint64_t* mk = P.heavy_mask + c0 + s0;
                    uint32_t* acc32 = reinterpret_cast<uint32_t*>(acc);
                    for (uint32_t w = tid; w < (s1 - s0 + 3u) / 4u; w += THREADS) {
                        uint32_t word = 0;
                        if (use_masks) {
#pragma unroll
                            for (uint32_t q = 0; q < 4; ++q)
                                if (4u * w + q < s1 - s0) word |= (uint32_t)__popcll((unsigned long long)mk[4u * w + q] & mask_i) << (8u * q);
                        }
                        acc32[w] = word;
                    }
                } else if (use_masks) {
                    // slot t of a dense row is column c0 + s0 + t
                    const uint64_t* mk = P.heavy_mask + c0 + s0;
                    for (uint32_t t = tid; t < s1 - s0; t += THREADS) acc[t] = Acc(__popcll((unsigned long long)mk[t] & mask_i));
                } else {
                    for (uint32_t t = tid; t < s1 - s0; t += THREADS) acc[t] = Acc(0);
                }
                __syncthreads();
                const bool resume = s0 > 0 && deg <= THREADS;
                const bool whole_row = single_chunk && single_tile;
                if (binary) {  // (the tags are std::true_type / std::false_type: here "the products are ones")
                    if (dense) for_each_product(ACC, IS_DENSE, IS_DENSE, jlo, jhi, whole_row, c0, s0, resume);
                    else for_each_product(ACC, NOT_DENSE, IS_DENSE, jlo, jhi, whole_row, c0, s0, resume);
                } else {
                    if (dense) for_each_product(ACC, IS_DENSE, NOT_DENSE, jlo, jhi, whole_row, c0, s0, resume);
                    else for_each_product(ACC, NOT_DENSE, NOT_DENSE, jlo, jhi, whole_row, c0, s0, resume);
                }
                for (uint32_t t = tid; t < s1 - s0; t += THREADS) {
                    if (!SPSYRK_IN_RANGE(ob + s0 + t < out_end, P.err)) continue;
                    const V cv = packed ? (V)((reinterpret_cast<const uint32_t*>(acc)[t >> 2] >> ((t & 3u) * 8u)) & 0xffu)
                                        : (V)(GLOBAL_ACC ? __ldcg(acc + t) : acc[t]);
                    c_vals[ob + s0 + t] = cv;
                    if (dense) c_colidx[ob + s0 + t] = (int32_t)(c0 + s0 + t);
                    if constexpr (std::is_same<V, int32_t>::value) {
                        if (P.jaccard) {
                            // J = c / (|a_i| + |a_j| - c); the column id was written above (dense rows: it is the slot's column)
                            const int64_t j = dense ? (int64_t)(c0 + s0 + t) : (int64_t)c_colidx[ob + s0 + t];
                            const int64_t na_j = P.adeg[j];
                            P.jaccard[ob + s0 + t] = __fdiv_rn((float)cv, (float)((int64_t)deg + na_j - (int64_t)cv));
                        }
                    }
                }
                __syncthreads();
            }
        }
        total_cnt += tot;
        __syncthreads();
    }
    if (!NUMERIC && tid == 0) cnt[rloc] = (int32_t)total_cnt;
    };  // do_row

    if (GLOBAL_ACC) {
        for (;;) {
            if (tid == 0) s_row = atomicAdd(row_counter, 1u);
            __syncthreads();
            const uint32_t r = s_row;
            __syncthreads();
            if (r >= nrows) break;
            do_row(rows[nrows - 1 - r]);
            __syncthreads();
        }
    } else {
        // later rows carry longer column prefixes: hand them out first so that the tail of the launch is light
        do_row(rows[gridDim.x - 1 - blockIdx.x]);
    }
}

}  // namespace spsyrk
