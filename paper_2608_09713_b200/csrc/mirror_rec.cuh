// Radix passes of the mirror for 8-byte values, on 16-byte records.
//
// The reflected part of F is a stable sort of C_L's entries by column id.  Here an entry travels
// as one aligned record (column, row, value): one 16-byte load, one 16-byte slot in the sorted tile
// in shared memory, one 16-byte store per pass, where separate arrays cost three of each.  The
// first pass reads C_L itself: the row of every entry of a tile comes from the tile's slice of the
// row pointers (row starts marked in shared memory, then a running maximum), so no (key, row)
// expansion is written and read back.  Every pass also writes the digit the next pass sorts on as
// one byte per element, so that the next pass's per-tile histogram reads bytes, not records.
//
// Keys are the column ids of all entries, the diagonal ones included: entry s of the sorted order,
// of column j and row r > j, lands at s + l_rowptr[j + 1] - (number of diagonal entries of the rows
// 0..j), because the sorted order up to it holds every strictly lower entry of the columns before
// j, the diagonals of rows 0..j, and the strictly lower entries of column j above it.
#pragma once
#include "radix.cuh"

namespace spsyrk {

// tile of the record passes: with 16-byte records a run of 8 elements per digit is already a full
// 128-byte line, so tiles can be half the size of the separate-array passes and four CTAs share an SM
constexpr int MR_THREADS = 256;
constexpr int MR_WARPS = MR_THREADS / 32;
constexpr int MR_ITEMS = 8;
constexpr int MR_TILE = MR_THREADS * MR_ITEMS;
constexpr int MR_CHUNK = MR_TILE / MR_WARPS;
constexpr int MR_MIN_CTAS = 4;
inline int64_t mirror_tiles(int64_t n) { return n > 0 ? (n + MR_TILE - 1) / MR_TILE : 0; }
// A CTA sorts MR_SUB consecutive tiles one after the other and carries its per-digit offsets from one to the
// next, so the histograms, their scan and the offsets a CTA fetches are per group of tiles: half of the
// per-tile figures in bytes and in scan time (measured: two tiles per CTA 19.4 ms for the whole mirror, one 20.9, four 20.4, eight 20.4, sixteen 21.5).
constexpr int MR_SUB = 2;
constexpr int MR_GROUP = MR_TILE * MR_SUB;
inline int64_t mirror_groups(int64_t n) { return n > 0 ? (n + MR_GROUP - 1) / MR_GROUP : 0; }

struct alignas(16) MirrorRec {
    uint32_t key;
    uint32_t row;
    uint64_t val;
};

// Per-group histograms for the record passes.  A CTA of MR_THREADS threads covers HIST_TILES groups: each
// warp owns whole groups (its private counters need no clearing race with other warps) and reads them
// 16 bytes per lane.
constexpr int MR_HIST_TILES = MR_THREADS / 32;  // one group per warp

// digit bytes written by the previous pass
template <int BITS>
__global__ void __launch_bounds__(MR_THREADS) radix_hist_u8_kernel(const uint8_t* __restrict__ digits, int64_t n,
                                                                   uint32_t* __restrict__ hist, int64_t ntiles) {
    constexpr int NB = 1 << BITS;
    static_assert(NB == 256, "one byte per digit");
    __shared__ uint32_t h[MR_HIST_TILES][NB];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t tile = (int64_t)blockIdx.x * MR_HIST_TILES + warp;
    for (int d = lane; d < NB; d += 32) h[warp][d] = 0;
    __syncwarp();
    if (tile < ntiles) {
        const int64_t base = tile * MR_GROUP;
        // MR_GROUP bytes = MR_GROUP / 16 pieces of 16 bytes (the array is 16-byte aligned and groups are multiples of 16)
        for (int c = lane; c < MR_GROUP / 16; c += 32) {
            const int64_t e = base + (int64_t)c * 16;
            if (e + 16 <= n) {
                const uint4 v = *reinterpret_cast<const uint4*>(digits + e);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    atomicAdd(&h[warp][w[q] & 0xffu], 1u);
                    atomicAdd(&h[warp][(w[q] >> 8) & 0xffu], 1u);
                    atomicAdd(&h[warp][(w[q] >> 16) & 0xffu], 1u);
                    atomicAdd(&h[warp][w[q] >> 24], 1u);
                }
            } else {
                for (int64_t x = e; x < n && x < e + 16; ++x) atomicAdd(&h[warp][digits[x]], 1u);
            }
        }
    }
    __syncwarp();
    if (tile < ntiles)
        for (int d = lane; d < NB; d += 32) hist[(int64_t)d * ntiles + tile] = h[warp][d];
}

// one digit of 32-bit keys (the first pass: column ids of C_L, any alignment)
template <int BITS>
__global__ void __launch_bounds__(MR_THREADS) mirror_hist_key_kernel(const uint32_t* __restrict__ keys, int64_t n, int shift,
                                                                    uint32_t* __restrict__ hist, int64_t ntiles) {
    constexpr int NB = 1 << BITS;
    __shared__ uint32_t h[MR_HIST_TILES][NB];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t tile = (int64_t)blockIdx.x * MR_HIST_TILES + warp;
    for (int d = lane; d < NB; d += 32) h[warp][d] = 0;
    __syncwarp();
    if (tile < ntiles) {
        const int64_t base = tile * MR_GROUP;
        constexpr int UNR = 8;
        for (int c0 = 0; c0 < MR_GROUP; c0 += 32 * UNR) {
            uint32_t k[UNR];
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                const int64_t e = base + c0 + u * 32 + lane;
                k[u] = e < n ? keys[e] : 0u;
            }
#pragma unroll
            for (int u = 0; u < UNR; ++u) {
                const int64_t e = base + c0 + u * 32 + lane;
                if (e < n) atomicAdd(&h[warp][(k[u] >> shift) & (NB - 1)], 1u);
            }
        }
    }
    __syncwarp();
    if (tile < ntiles)
        for (int d = lane; d < NB; d += 32) hist[(int64_t)d * ntiles + tile] = h[warp][d];
}

// row of the first and of the last entry of every tile: the last r with l_rowptr[r] <= position
static __global__ void mirror_tile_rows_kernel(const int64_t* __restrict__ l_rowptr, int64_t m, int64_t n, int64_t ntiles,
                                               int32_t* __restrict__ tile_rows) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= 2 * ntiles) return;
    const int64_t tile = t >> 1;
    const int64_t pos = (t & 1) ? min(tile * MR_TILE + MR_TILE, n) - 1 : tile * MR_TILE;
    int64_t lo = 0, hi = m;  // l_rowptr[0] = 0 <= pos < n = l_rowptr[m]
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (l_rowptr[mid] <= pos) lo = mid; else hi = mid;
    }
    tile_rows[t] = (int32_t)lo;
}

struct MirrorPassArgs {
    // source: C_L (first pass) or records
    const int64_t* l_rowptr;
    const int32_t* l_colidx;
    const uint64_t* l_vals;
    int64_t m;
    const int32_t* tile_rows;  // [2 * tiles]: row of each tile's first and last entry
    // A record buffer comes in two pieces: records [0, split) at `src` / `dst`, the rest at the tail pointer.
    // (The buffer that lives in F's value array while F is not yet written is a few records short; see mirror.cu.)
    const MirrorRec* src;
    const MirrorRec* src_tail;
    int64_t src_split;
    // destination: records and the next digit, or F (last pass)
    MirrorRec* dst;
    MirrorRec* dst_tail;
    int64_t dst_split;
    uint8_t* next_digit;
    const int64_t* fbase;  // l_rowptr[j + 1] - diagonals of rows 0..j
    int32_t* f_colidx;
    uint64_t* f_vals;
    unsigned long long* seg_start;
    unsigned long long* seg_end;
    const int64_t* dtotal;  // number of diagonal entries: F holds 2 n - *dtotal entries
    uint32_t* err;
};

template <int BITS>
struct MirrorPassSmem {
    static constexpr int NB = 1 << BITS;
    static size_t bytes() { return (size_t)NB * 16 + (size_t)MR_TILE * sizeof(MirrorRec) + (size_t)MR_WARPS * NB * 4 + (size_t)NB * 4; }
};

template <int BITS, bool FROM_CSR, bool FINAL>
__global__ void __launch_bounds__(MR_THREADS, MR_MIN_CTAS) mirror_pass_kernel(MirrorPassArgs A, int64_t n, int shift,
                                                                    const int64_t* __restrict__ goff_all, int64_t ntiles) {
    constexpr int NB = 1 << BITS;
    static_assert(MR_WARPS * NB * 4 >= MR_TILE * 4, "the row marks share the warp counters' space");
    extern __shared__ __align__(16) unsigned char mp_smem[];
    __shared__ uint32_t scratch[33];
    int64_t* goff = reinterpret_cast<int64_t*>(mp_smem);                     // [NB] offset of the tile's bin minus its start in the tile
    int64_t* gbase = goff + NB;                                              // [NB] where the current tile's bins start in the output
    MirrorRec* s_rec = reinterpret_cast<MirrorRec*>(gbase + NB);             // [TILE] sorted order
    uint32_t* wcount = reinterpret_cast<uint32_t*>(s_rec + MR_TILE);         // [WARPS][NB]; first: row marks [TILE]
    uint32_t* bin_start = wcount + MR_WARPS * NB;                            // [NB]

    const int tid = threadIdx.x, lane = lane_id(), warp = tid >> 5;
    for (int d = tid; d < NB; d += MR_THREADS) gbase[d] = goff_all[(int64_t)d * ntiles + blockIdx.x];
    for (int sub = 0; sub < MR_SUB; ++sub) {
    const int64_t tile = (int64_t)blockIdx.x * MR_SUB + sub;
    const int64_t tile_base = tile * MR_TILE;
    if (tile_base >= n) break;  // the same for every thread
    const int tile_n = (int)min((int64_t)MR_TILE, n - tile_base);
    uint32_t k[MR_ITEMS], a[MR_ITEMS];
    uint64_t b[MR_ITEMS];

    if (FROM_CSR) {
        // rows of the tile's entries: the last row that starts at or before an entry owns it
        uint32_t* mark = wcount;
        for (int t = tid; t < MR_TILE; t += MR_THREADS) mark[t] = 0;
        const int64_t r_lo = A.tile_rows[2 * tile], r_hi = A.tile_rows[2 * tile + 1];
        __syncthreads();
        for (int64_t r = r_lo + 1 + tid; r <= r_hi; r += MR_THREADS) {
            const int64_t p = A.l_rowptr[r] - tile_base;  // in (0, tile_n) by the choice of r_lo, r_hi
            if (p >= 0 && p < tile_n) atomicMax(&mark[p], (uint32_t)(r - r_lo));
        }
        __syncthreads();
        {
            // running maximum over the tile: thread t owns positions [t * ITEMS, t * ITEMS + ITEMS)
            uint32_t v[MR_ITEMS], run = 0;
#pragma unroll
            for (int i = 0; i < MR_ITEMS; ++i) {
                run = max(run, mark[tid * MR_ITEMS + i]);
                v[i] = run;
            }
            // exclusive maximum over the threads before this one
            uint32_t incl = run;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(FULL_MASK, incl, o);
                if (lane >= o) incl = max(incl, t);
            }
            if (lane == 31) scratch[warp] = incl;
            __syncthreads();
            uint32_t before = 0;
            for (int w = 0; w < warp; ++w) before = max(before, scratch[w]);
            const uint32_t prev = __shfl_up_sync(FULL_MASK, incl, 1);
            if (lane > 0) before = max(before, prev);
#pragma unroll
            for (int i = 0; i < MR_ITEMS; ++i) mark[tid * MR_ITEMS + i] = max(v[i], before);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < MR_ITEMS; ++i) {
            const int t = warp * MR_CHUNK + i * 32 + lane;
            const bool on = t < tile_n;
            k[i] = on ? (uint32_t)A.l_colidx[tile_base + t] : 0u;
            a[i] = on ? (uint32_t)(r_lo + mark[t]) : 0u;
            b[i] = on ? A.l_vals[tile_base + t] : 0ull;
        }
        __syncthreads();  // the marks are read: their space becomes the warp counters
    } else {
#pragma unroll
        for (int i = 0; i < MR_ITEMS; ++i) {
            const int t = warp * MR_CHUNK + i * 32 + lane;
            uint4 r = make_uint4(0u, 0u, 0u, 0u);
            if (t < tile_n) {  // one 16-byte load
                const int64_t e = tile_base + t;
                r = e < A.src_split ? reinterpret_cast<const uint4*>(A.src)[e] : reinterpret_cast<const uint4*>(A.src_tail)[e - A.src_split];
            }
            k[i] = r.x; a[i] = r.y; b[i] = (uint64_t)r.z | ((uint64_t)r.w << 32);
        }
    }
    for (int d = tid; d < MR_WARPS * NB; d += MR_THREADS) wcount[d] = 0;
    __syncthreads();

    uint32_t rk[MR_ITEMS];
    uint32_t* mycount = wcount + warp * NB;
#pragma unroll
    for (int i = 0; i < MR_ITEMS; ++i) {
        const int t = warp * MR_CHUNK + i * 32 + lane;
        const bool valid = t < tile_n;
        const uint32_t d = valid ? ((k[i] >> shift) & (NB - 1)) : 0u;
        unsigned peers = __ballot_sync(FULL_MASK, valid);
#pragma unroll
        for (int bit = 0; bit < BITS; ++bit) {
            const bool set = (d >> bit) & 1u;
            const unsigned bal = __ballot_sync(FULL_MASK, set);
            peers &= set ? bal : ~bal;
        }
        const int leader = __ffs(peers) - 1;
        uint32_t prev = 0;
        if (valid && lane == leader) {
            prev = mycount[d];
            mycount[d] = prev + __popc(peers);
        }
        prev = __shfl_sync(FULL_MASK, prev, leader);
        rk[i] = (prev + __popc(peers & ((1u << lane) - 1u))) | (d << 16);
        __syncwarp();
    }
    __syncthreads();
    for (int d = tid; d < NB; d += MR_THREADS) {
        uint32_t run = 0;
#pragma unroll
        for (int w = 0; w < MR_WARPS; ++w) {
            const uint32_t c = wcount[w * NB + d];
            wcount[w * NB + d] = run;
            run += c;
        }
        bin_start[d] = run;  // the bin's count for now
        goff[d] = gbase[d];
        gbase[d] += (int64_t)run;  // the next tile of the group continues behind this one's entries
    }
    __syncthreads();
    {
        constexpr int PER = (NB + MR_THREADS - 1) / MR_THREADS;
        uint32_t s = 0;
#pragma unroll
        for (int q = 0; q < PER; ++q)
            if (tid * PER + q < NB) s += bin_start[tid * PER + q];
        uint32_t tot;
        uint32_t ex = block_exclusive_scan<uint32_t, MR_THREADS>(s, scratch, &tot);
#pragma unroll
        for (int q = 0; q < PER; ++q) {
            if (tid * PER + q < NB) {
                const uint32_t t = bin_start[tid * PER + q];
                bin_start[tid * PER + q] = ex;
                ex += t;
            }
        }
    }
    __syncthreads();
    for (int e = tid; e < MR_WARPS * NB; e += MR_THREADS) wcount[e] += bin_start[e & (NB - 1)];
    for (int d = tid; d < NB; d += MR_THREADS) goff[d] -= (int64_t)bin_start[d];
    __syncthreads();
#pragma unroll
    for (int i = 0; i < MR_ITEMS; ++i) {
        const int t = warp * MR_CHUNK + i * 32 + lane;
        if (t < tile_n) {
            const uint32_t q = mycount[rk[i] >> 16] + (rk[i] & 0xffffu);
            if (SPSYRK_IN_RANGE(q < (uint32_t)MR_TILE, A.err))
                reinterpret_cast<uint4*>(s_rec)[q] = make_uint4(k[i], a[i], (uint32_t)b[i], (uint32_t)(b[i] >> 32));
        }
    }
    __syncthreads();
    for (int q = tid; q < tile_n; q += MR_THREADS) {
        const uint4 r4 = reinterpret_cast<const uint4*>(s_rec)[q];
        MirrorRec r;
        r.key = r4.x; r.row = r4.y; r.val = (uint64_t)r4.z | ((uint64_t)r4.w << 32);
        const int64_t dest = goff[(r.key >> shift) & (NB - 1)] + q;
        if (!SPSYRK_IN_RANGE(dest >= 0 && dest < n, A.err)) continue;
        if (!FINAL) {
            if (dest < A.dst_split) reinterpret_cast<uint4*>(A.dst)[dest] = r4;
            else reinterpret_cast<uint4*>(A.dst_tail)[dest - A.dst_split] = r4;
            A.next_digit[dest] = (uint8_t)((r.key >> (shift + BITS)) & (NB - 1));
        } else if (r.key < (uint32_t)A.m) {
            // ends of a run of one key inside the tile; a segment that spans tiles settles through min / max
            const uint32_t prev = q > 0 ? s_rec[q - 1].key : NO_KEY, next = q + 1 < tile_n ? s_rec[q + 1].key : NO_KEY;
            if (prev != r.key) atomicMin(&A.seg_start[r.key], (unsigned long long)dest);
            if (next != r.key) atomicMax(&A.seg_end[r.key], (unsigned long long)dest + 1ull);
            if (r.row > r.key) {
                const int64_t pos = dest + A.fbase[r.key];
                if (pos >= 0 && pos < 2 * n - *A.dtotal) {
                    A.f_colidx[pos] = (int32_t)r.row;
                    A.f_vals[pos] = r.val;
                } else {
                    atomicOr(A.err, ERRW_UPPER);  // only an input with entries above the diagonal gets here
                }
            } else if (r.row < r.key) {
                atomicOr(A.err, ERRW_UPPER);
            }
        } else {
            atomicOr(A.err, ERRW_UPPER);  // a column id outside [0, m)
        }
    }
    __syncthreads();  // the tile in shared memory and the offsets are rewritten by the next tile of the group
    }  // tiles of the group
}

}  // namespace spsyrk
