// Stable least-significant-digit radix partition passes over (key, payload a, payload b) records
// held as separate arrays.  A sparse transpose is a stable sort by column id: entries that arrive
// in ascending row order leave every column's segment in ascending row order, with no atomics and
// no per-segment sort, and every pass reads and writes memory in long runs.
//
// One pass = three launches: per-tile digit histogram, device-wide scan of the digit-major
// histogram, scatter.  In the scatter a warp owns a contiguous slice of the tile and ranks its
// elements 32 at a time (elements with equal digits find each other through one warp vote per digit
// bit, the lowest lane bumps the warp's counter), an exclusive prefix over the warps makes the ranks
// tile-wide and stable, the tile is reordered digit-major in shared memory and written out in
// runs.  There is no waiting between CTAs.
#pragma once
#include "common.cuh"

namespace spsyrk {

constexpr int RX_THREADS = 512;
constexpr int RX_WARPS = RX_THREADS / 32;
constexpr int RX_ITEMS = 8;
constexpr int RX_TILE = RX_THREADS * RX_ITEMS;  // elements per CTA
constexpr int RX_CHUNK = RX_TILE / RX_WARPS;    // contiguous elements per warp

inline int64_t radix_tiles(int64_t n) { return n > 0 ? (n + RX_TILE - 1) / RX_TILE : 0; }

// 16-byte asynchronous global -> shared copy; both addresses 16-byte aligned
__device__ __forceinline__ void rx_cp_async16(void* smem_dst, const void* gmem_src) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void rx_cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int KEEP>
__device__ __forceinline__ void rx_cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(KEEP) : "memory"); }

// Copy `count` elements of T from src (element `first` of a 16-byte aligned array, `first` a multiple
// of 16 / sizeof(T)) to shared memory: whole 16-byte pieces asynchronously, a ragged tail by plain loads.
template <typename T>
__device__ __forceinline__ void rx_tile_load(T* s_dst, const T* __restrict__ src, int64_t first, int count) {
    constexpr int PER = 16 / sizeof(T);
    const int whole = count / PER;
    for (int c = threadIdx.x; c < whole; c += RX_THREADS) rx_cp_async16(s_dst + c * PER, src + first + (int64_t)c * PER);
    for (int t = whole * PER + threadIdx.x; t < count; t += RX_THREADS) s_dst[t] = src[first + t];
}

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

template <int BITS, typename PB>
struct RadixSmem {
    static constexpr int NB = 1 << BITS;
    static size_t bytes() {
        return (size_t)NB * 8 + (size_t)RX_TILE * sizeof(PB) + (size_t)RX_WARPS * NB * 4 + (size_t)NB * 4 +
               (size_t)RX_TILE * (4 + 4 + 2 + 2);
    }
};

// Emit(dest, key, pa, pb) is called once per element with its position `dest` in the order sorted
// by the digits seen so far.  pa == nullptr (pb == nullptr) means "this payload is the element's own
// index".
// All input arrays must be 16-byte aligned.
template <int BITS, typename PB, typename Emit>
__global__ void __launch_bounds__(RX_THREADS) radix_scatter_kernel(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ pa,
                                                                   const PB* __restrict__ pb, int64_t n, int shift,
                                                                   const int64_t* __restrict__ goff_all, int64_t ntiles, Emit emit) {
    constexpr int NB = 1 << BITS;
    static_assert(BITS <= 12, "digit width");
    extern __shared__ __align__(16) unsigned char rx_smem[];
    __shared__ uint32_t scratch[33];
    int64_t* goff = reinterpret_cast<int64_t*>(rx_smem);               // [NB]
    PB* s_pb = reinterpret_cast<PB*>(goff + NB);                       // [TILE] source order
    uint32_t* s_key = reinterpret_cast<uint32_t*>(s_pb + RX_TILE);     // [TILE] source order
    uint32_t* s_pa = s_key + RX_TILE;                                  // [TILE] source order
    uint32_t* wcount = s_pa + RX_TILE;                                 // [WARPS][NB]
    uint32_t* bin_start = wcount + RX_WARPS * NB;                      // [NB]
    uint32_t* s_perm = bin_start + NB;                                 // [TILE] (digit << 16) | source index of sorted slot q

    const int tid = threadIdx.x, lane = lane_id(), warp = tid >> 5;
    const int64_t tile_base = (int64_t)blockIdx.x * RX_TILE;
    const int tile_n = (int)min((int64_t)RX_TILE, n - tile_base);
    // the whole tile streams into shared memory while the ranking runs: keys first, payloads behind
    rx_tile_load(s_key, keys, tile_base, tile_n);
    rx_cp_async_commit();
    if (pa) rx_tile_load(s_pa, pa, tile_base, tile_n);
    if (pb) rx_tile_load(s_pb, pb, tile_base, tile_n);
    rx_cp_async_commit();
    for (int d = tid; d < RX_WARPS * NB; d += RX_THREADS) wcount[d] = 0;
    rx_cp_async_wait<1>();
    __syncthreads();

    uint32_t rk[RX_ITEMS];
    uint32_t* mycount = wcount + warp * NB;
#pragma unroll
    for (int i = 0; i < RX_ITEMS; ++i) {
        const int t = warp * RX_CHUNK + i * 32 + lane;
        const bool valid = t < tile_n;
        const uint32_t d = valid ? ((s_key[t] >> shift) & (NB - 1)) : 0u;
        // lanes with the same digit, found one bit at a time with warp votes (cheaper here than the
        // match instruction, whose unit saturates long before memory does)
        unsigned peers = __ballot_sync(FULL_MASK, valid);
#pragma unroll
        for (int b = 0; b < BITS; ++b) {
            const bool bit = (d >> b) & 1u;
            const unsigned bal = __ballot_sync(FULL_MASK, bit);
            peers &= bit ? bal : ~bal;
        }
        const int leader = __ffs(peers) - 1;
        uint32_t prev = 0;
        if (valid && lane == leader) {
            prev = mycount[d];
            mycount[d] = prev + __popc(peers);
        }
        prev = __shfl_sync(FULL_MASK, prev, leader);
        rk[i] = (prev + __popc(peers & ((1u << lane) - 1u))) | (d << 12) | (valid ? 0u : 0x80000000u);
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
        for (int k = 0; k < PER; ++k)
            if (tid * PER + k < NB) s += bin_start[tid * PER + k];
        uint32_t tot;
        uint32_t ex = block_exclusive_scan<uint32_t, RX_THREADS>(s, scratch, &tot);
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            if (tid * PER + k < NB) {
                const uint32_t t = bin_start[tid * PER + k];
                bin_start[tid * PER + k] = ex;
                ex += t;
            }
        }
    }
    __syncthreads();
    // sorted slot -> source index
#pragma unroll
    for (int i = 0; i < RX_ITEMS; ++i) {
        if (!(rk[i] & 0x80000000u)) {
            const uint32_t d = (rk[i] >> 12) & 0xfffu;
            const uint32_t q = bin_start[d] + mycount[d] + (rk[i] & 0xfffu);
            s_perm[q] = (d << 16) | (uint32_t)(warp * RX_CHUNK + i * 32 + lane);
        }
    }
    rx_cp_async_wait<0>();
    __syncthreads();
    // slot q of digit d goes to goff[d] + (q - bin_start[d]): fold the two tables into one
    for (int d = tid; d < NB; d += RX_THREADS) goff[d] -= (int64_t)bin_start[d];
    __syncthreads();
    for (int q = tid; q < tile_n; q += RX_THREADS) {
        const uint32_t pd = s_perm[q];
        const uint32_t src = pd & 0xffffu;
        emit(goff[pd >> 16] + q, s_key[src], pa ? s_pa[src] : (uint32_t)(tile_base + src), pb ? s_pb[src] : (PB)(tile_base + src));
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

// hist: NB * ntiles uint32; offsets: NB * ntiles + 1 int64; partials: scan_partials_count(NB * ntiles) int64
template <int BITS, typename PB, typename Emit>
inline cudaError_t radix_pass(const uint32_t* keys, const uint32_t* pa, const PB* pb, int64_t n, int shift, uint32_t* hist,
                              int64_t* offsets, int64_t* partials, Emit emit, cudaStream_t st) {
    constexpr int NB = 1 << BITS;
    const int64_t nt = radix_tiles(n);
    if (nt == 0) return cudaSuccess;
    radix_hist_kernel<BITS><<<(unsigned)nt, RX_THREADS, 0, st>>>(keys, n, shift, hist, nt);
    cudaError_t e = exclusive_scan_i64<uint32_t>(hist, (int64_t)NB * nt, offsets, partials, st);
    if (e != cudaSuccess) return e;
    auto kern = radix_scatter_kernel<BITS, PB, Emit>;
    const size_t smem = RadixSmem<BITS, PB>::bytes();
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)nt, RX_THREADS, smem, st>>>(keys, pa, pb, n, shift, offsets, nt, emit);
    note_launches(2);
    return cudaGetLastError();
}

inline int bits_for(uint64_t max_value) {
    int b = 1;
    while (b < 64 && (max_value >> b)) ++b;
    return b;
}

}  // namespace spsyrk
