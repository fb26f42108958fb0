// Stable least-significant-digit radix partition passes over (key, payload a, payload b) records
// held as separate arrays.  A sparse transpose is a stable sort by column id: entries that arrive
// in ascending row order leave every column's segment in ascending row order, with no atomics and
// no per-segment sort, and every pass reads and writes memory in long runs.
//
// One pass = three launches: per-tile digit histogram, device-wide scan of the digit-major
// histogram, scatter.  In the scatter a warp owns a contiguous slice of the tile, keeps its elements
// in registers and ranks them 32 at a time (elements with equal digits find each other through one
// warp vote per digit bit, the lowest lane bumps the warp's counter), an exclusive prefix over the
// warps makes the ranks tile-wide and stable, every element is dropped into its slot of the
// digit-major tile in shared memory and the tile is written out in runs.  There is no waiting
// between CTAs.
#pragma once
#include <type_traits>

#include "common.cuh"

namespace spsyrk {

constexpr int RX_THREADS = 512;
constexpr int RX_WARPS = RX_THREADS / 32;
constexpr int RX_ITEMS = 8;
constexpr int RX_TILE = RX_THREADS * RX_ITEMS;  // elements per CTA
constexpr int RX_CHUNK = RX_TILE / RX_WARPS;    // contiguous elements per warp

inline int64_t radix_tiles(int64_t n) { return n > 0 ? (n + RX_TILE - 1) / RX_TILE : 0; }

template <int BITS>
__global__ void __launch_bounds__(RX_THREADS) radix_hist_kernel(const uint32_t* __restrict__ keys, int64_t n, int shift,
                                                                uint32_t* __restrict__ hist, int64_t ntiles) {
    constexpr int NB = 1 << BITS;
    __shared__ uint32_t h[RX_WARPS][NB];  // one histogram per warp keeps the atomics apart
    for (int d = threadIdx.x; d < RX_WARPS * NB; d += RX_THREADS) (&h[0][0])[d] = 0;
    __syncthreads();
    const int warp = threadIdx.x >> 5;
    const int64_t base = (int64_t)blockIdx.x * RX_TILE;
    uint32_t k[RX_ITEMS];
#pragma unroll
    for (int it = 0; it < RX_ITEMS; ++it) {
        const int64_t e = base + it * RX_THREADS + threadIdx.x;
        k[it] = e < n ? keys[e] : 0u;
    }
#pragma unroll
    for (int it = 0; it < RX_ITEMS; ++it) {
        const int64_t e = base + it * RX_THREADS + threadIdx.x;
        if (e < n) atomicAdd(&h[warp][(k[it] >> shift) & (NB - 1)], 1u);
    }
    __syncthreads();
    for (int d = threadIdx.x; d < NB; d += RX_THREADS) {
        uint32_t t = 0;
#pragma unroll
        for (int w = 0; w < RX_WARPS; ++w) t += h[w][d];
        hist[(int64_t)d * ntiles + blockIdx.x] = t;
    }
}

// A functor that declares `static constexpr bool NEIGHBOURS = true` is also handed the keys next to the
// element in the tile's sorted order.
constexpr uint32_t NO_KEY = 0xffffffffu;
template <typename E, typename = void>
struct emit_wants_neighbours : std::false_type {};
template <typename E>
struct emit_wants_neighbours<E, std::void_t<decltype(E::NEIGHBOURS)>> : std::bool_constant<E::NEIGHBOURS> {};

template <int BITS, typename PB, bool HAS_PC = false>
struct RadixSmem {
    static constexpr int NB = 1 << BITS;
    static size_t bytes() {
        return (size_t)NB * 8 + (size_t)RX_TILE * sizeof(PB) + (size_t)RX_TILE * (4 + 4 + (HAS_PC ? 4 : 0)) + (size_t)RX_WARPS * NB * 4 +
               (size_t)NB * 4;
    }
};

// `err` is the device error word of the caller (used by the bounds-checked build only).
// Emit(dest, key, pa, pb) is called once per element with its position `dest` in the order sorted
// by the digits seen so far.  pa == nullptr (pb == nullptr) means "this payload is the element's own
// index".
//
// A thread keeps its RX_ITEMS elements in registers (coalesced loads straight from global memory,
// the payloads still in flight while the keys are ranked), learns each element's slot in the tile's
// digit-major order, drops key and payloads into that slot of shared memory, and the tile is then
// read back slot by slot and written out in runs.
// HAS_PC: a third payload pc (32 bits; nullptr = the element's own index) travels along and the functor is
// called as emit(dest, key, pa, pb, pc).
template <int BITS, typename PB, typename Emit, bool HAS_PC = false>
__global__ void __launch_bounds__(RX_THREADS, 2) radix_scatter_kernel(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ pa,
                                                                      const PB* __restrict__ pb, const uint32_t* __restrict__ pc,
                                                                      int64_t n, int shift, const int64_t* __restrict__ goff_all,
                                                                      int64_t ntiles, Emit emit, uint32_t* err) {
    constexpr int NB = 1 << BITS;
    static_assert(BITS <= 12, "digit width");
    extern __shared__ __align__(16) unsigned char rx_smem[];
    __shared__ uint32_t scratch[33];
    int64_t* goff = reinterpret_cast<int64_t*>(rx_smem);               // [NB]
    PB* s_pb = reinterpret_cast<PB*>(goff + NB);                       // [TILE] sorted order
    uint32_t* s_key = reinterpret_cast<uint32_t*>(s_pb + RX_TILE);     // [TILE] sorted order
    uint32_t* s_pa = s_key + RX_TILE;                                  // [TILE] sorted order
    uint32_t* s_pc = s_pa + RX_TILE;                                   // [TILE] sorted order (HAS_PC only)
    uint32_t* wcount = s_pc + (HAS_PC ? RX_TILE : 0);                  // [WARPS][NB]
    uint32_t* bin_start = wcount + RX_WARPS * NB;                      // [NB]

    const int tid = threadIdx.x, lane = lane_id(), warp = tid >> 5;
    const int64_t tile_base = (int64_t)blockIdx.x * RX_TILE;
    const int tile_n = (int)min((int64_t)RX_TILE, n - tile_base);
    uint32_t k[RX_ITEMS], a[RX_ITEMS];
    PB b[RX_ITEMS];
#pragma unroll
    for (int i = 0; i < RX_ITEMS; ++i) {
        const int t = warp * RX_CHUNK + i * 32 + lane;
        k[i] = t < tile_n ? keys[tile_base + t] : 0u;
    }
#pragma unroll
    for (int i = 0; i < RX_ITEMS; ++i) {
        const int t = warp * RX_CHUNK + i * 32 + lane;
        a[i] = (pa && t < tile_n) ? pa[tile_base + t] : (uint32_t)(tile_base + t);
        b[i] = (pb && t < tile_n) ? pb[tile_base + t] : (PB)(tile_base + t);
    }
    for (int d = tid; d < RX_WARPS * NB; d += RX_THREADS) wcount[d] = 0;
    __syncthreads();

    uint32_t rk[RX_ITEMS];
    uint32_t* mycount = wcount + warp * NB;
#pragma unroll
    for (int i = 0; i < RX_ITEMS; ++i) {
        const int t = warp * RX_CHUNK + i * 32 + lane;
        const bool valid = t < tile_n;
        const uint32_t d = valid ? ((k[i] >> shift) & (NB - 1)) : 0u;
        // lanes with the same digit, found one bit at a time with warp votes (cheaper here than the
        // match instruction, whose unit saturates long before memory does)
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
    // exclusive prefix over the warps per digit; digit totals; this tile's global offsets
    for (int d = tid; d < NB; d += RX_THREADS) {
        uint32_t run = 0;
#pragma unroll
        for (int w = 0; w < RX_WARPS; ++w) {
            const uint32_t c = wcount[w * NB + d];
            wcount[w * NB + d] = run;
            run += c;
        }
        bin_start[d] = run;
        goff[d] = goff_all[(int64_t)d * ntiles + blockIdx.x];
    }
    __syncthreads();
    {
        // exclusive scan of the digit totals: thread t owns digits [t * PER, t * PER + PER)
        constexpr int PER = (NB + RX_THREADS - 1) / RX_THREADS;
        uint32_t s = 0;
#pragma unroll
        for (int q = 0; q < PER; ++q)
            if (tid * PER + q < NB) s += bin_start[tid * PER + q];
        uint32_t tot;
        uint32_t ex = block_exclusive_scan<uint32_t, RX_THREADS>(s, scratch, &tot);
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
    // a warp's first slot of digit d = start of the digit + the elements of the warps before it; slot q of
    // digit d goes to goff[d] + (q - bin_start[d]): fold the tables
    for (int e = tid; e < RX_WARPS * NB; e += RX_THREADS) wcount[e] += bin_start[e & (NB - 1)];
    for (int d = tid; d < NB; d += RX_THREADS) goff[d] -= (int64_t)bin_start[d];
    __syncthreads();
    // elements into their slots
#pragma unroll
    for (int i = 0; i < RX_ITEMS; ++i) {
        const int t = warp * RX_CHUNK + i * 32 + lane;
        if (t < tile_n) {
            const uint32_t q = mycount[rk[i] >> 16] + (rk[i] & 0xffffu);
            if (!SPSYRK_IN_RANGE(q < (uint32_t)RX_TILE, err)) continue;
            s_key[q] = k[i];
            s_pa[q] = a[i];
            s_pb[q] = b[i];
            // the third payload is loaded only now: it would not fit the registers next to the others
            if constexpr (HAS_PC) s_pc[q] = pc ? pc[tile_base + t] : (uint32_t)(tile_base + t);
        }
    }
    __syncthreads();
    for (int q = tid; q < tile_n; q += RX_THREADS) {
        const uint32_t key = s_key[q];
        const int64_t dest = goff[(key >> shift) & (NB - 1)] + q;
        if (!SPSYRK_IN_RANGE(dest >= 0 && dest < n, err)) continue;
        if constexpr (HAS_PC) {
            emit(dest, key, s_pa[q], s_pb[q], s_pc[q]);
        } else if constexpr (emit_wants_neighbours<Emit>::value) {
            // the keys of the slots before and after (NO_KEY at the ends of the tile): in the last pass of a
            // sort equal keys are adjacent, so a functor can tell where a run of one key starts and ends
            emit(dest, key, s_pa[q], s_pb[q], q > 0 ? s_key[q - 1] : NO_KEY, q + 1 < tile_n ? s_key[q + 1] : NO_KEY);
        } else {
            emit(dest, key, s_pa[q], s_pb[q]);
        }
    }
}

template <typename PB>
struct EmitArrays {
    uint32_t* keys;
    uint32_t* pa;
    PB* pb;
    __device__ __forceinline__ void operator()(int64_t dest, uint32_t k, uint32_t a, PB b) const {
        keys[dest] = k;
        pa[dest] = a;
        pb[dest] = b;
    }
};

template <typename PB>
struct EmitArrays3 {
    uint32_t* keys;
    uint32_t* pa;
    PB* pb;
    uint32_t* pc;
    __device__ __forceinline__ void operator()(int64_t dest, uint32_t k, uint32_t a, PB b, uint32_t c) const {
        keys[dest] = k;
        pa[dest] = a;
        pb[dest] = b;
        pc[dest] = c;
    }
};

// hist: NB * ntiles uint32; offsets: NB * ntiles + 1 int64; partials: scan_partials_count(NB * ntiles) int64
template <int BITS, typename PB, bool HAS_PC, typename Emit>
inline cudaError_t radix_pass_impl(const uint32_t* keys, const uint32_t* pa, const PB* pb, const uint32_t* pc, int64_t n, int shift,
                                   uint32_t* hist, int64_t* offsets, int64_t* partials, Emit emit, uint32_t* err, cudaStream_t st) {
    constexpr int NB = 1 << BITS;
    const int64_t nt = radix_tiles(n);
    if (nt == 0) return cudaSuccess;
    radix_hist_kernel<BITS><<<(unsigned)nt, RX_THREADS, 0, st>>>(keys, n, shift, hist, nt);
    cudaError_t e = exclusive_scan_i64<uint32_t>(hist, (int64_t)NB * nt, offsets, partials, st);
    if (e != cudaSuccess) return e;
    auto kern = radix_scatter_kernel<BITS, PB, Emit, HAS_PC>;
    const size_t smem = RadixSmem<BITS, PB, HAS_PC>::bytes();
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)nt, RX_THREADS, smem, st>>>(keys, pa, pb, pc, n, shift, offsets, nt, emit, err);
    note_launches(2);
    return cudaGetLastError();
}

template <int BITS, typename PB, typename Emit>
inline cudaError_t radix_pass(const uint32_t* keys, const uint32_t* pa, const PB* pb, int64_t n, int shift, uint32_t* hist,
                              int64_t* offsets, int64_t* partials, Emit emit, uint32_t* err, cudaStream_t st) {
    return radix_pass_impl<BITS, PB, false>(keys, pa, pb, nullptr, n, shift, hist, offsets, partials, emit, err, st);
}

// the same with a third 32-bit payload (pc == nullptr: the element's own index)
template <int BITS, typename PB, typename Emit>
inline cudaError_t radix_pass3(const uint32_t* keys, const uint32_t* pa, const PB* pb, const uint32_t* pc, int64_t n, int shift,
                               uint32_t* hist, int64_t* offsets, int64_t* partials, Emit emit, uint32_t* err, cudaStream_t st) {
    return radix_pass_impl<BITS, PB, true>(keys, pa, pb, pc, n, shift, hist, offsets, partials, emit, err, st);
}

inline int bits_for(uint64_t max_value) {
    int b = 1;
    while (b < 64 && (max_value >> b)) ++b;
    return b;
}

}  // namespace spsyrk
