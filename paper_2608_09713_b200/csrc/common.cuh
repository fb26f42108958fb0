// Shared device utilities: warp/block scans, register bitonic sort, device-wide scan,
// stable class binning.  Header-only; included by every translation unit of libspsyrk.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <type_traits>

#include "../../include/spsyrk.h"

namespace spsyrk {

constexpr unsigned FULL_MASK = 0xffffffffu;

// bits of the device error word
enum : uint32_t {
    ERRW_BAD_ROWPTR = 1u,
    ERRW_BAD_COL = 2u,
    ERRW_UNSORTED = 4u,
    ERRW_INTERNAL = 8u,
    ERRW_UPPER = 16u,
};

// Bounds-checked build (-DSPSYRK_CHECKED, a second library next to the regular one): every index into a
// shared-memory accumulator, hash or landing slot and every output offset that the kernels compute is
// tested first; a violation sets ERRW_INTERNAL in the device error word and the access is skipped, so the
// caller gets SPSYRK_ERR_INTERNAL instead of a memory fault.  In the regular build the test is `true`.
#ifdef SPSYRK_CHECKED
#define SPSYRK_IN_RANGE(cond, errptr) ((cond) ? true : (atomicOr((errptr), ::spsyrk::ERRW_INTERNAL), false))
#else
#define SPSYRK_IN_RANGE(cond, errptr) true
#endif

constexpr int NCLASS = 8;  // row / column classes produced by the binning pass

// kernel-launch bookkeeping behind spsyrk_launch_count (defined in api.cu)
void note_launches(int n);

#define SPSYRK_CUDA_TRY(expr)                                  \
    do {                                                       \
        cudaError_t _e = (expr);                               \
        if (_e != cudaSuccess) return SPSYRK_ERR_CUDA;         \
    } while (0)

__host__ __device__ constexpr int ilog2_ce(int v) { return v <= 1 ? 0 : 1 + ilog2_ce(v >> 1); }

__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

template <typename T>
__device__ __forceinline__ T warp_inclusive_scan(T v) {
    const int lane = lane_id();
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T t = __shfl_up_sync(FULL_MASK, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

template <typename T>
__device__ __forceinline__ T warp_reduce_sum(T v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL_MASK, v, o);
    return v;
}

// Exclusive scan over the threads of a CTA.  `scratch` holds 33 elements of T in shared memory.
// Returns the exclusive prefix of `v`; *total receives the CTA-wide sum.  Contains barriers.
template <typename T, int THREADS>
__device__ __forceinline__ T block_exclusive_scan(T v, T* scratch, T* total) {
    static_assert(THREADS % 32 == 0 && THREADS <= 1024, "bad CTA size");
    constexpr int NW = THREADS / 32;
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    T incl = warp_inclusive_scan(v);
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        T s = lane < NW ? scratch[lane] : T(0);
        T si = warp_inclusive_scan(s);
        scratch[lane] = si - s;
        if (lane == 31) scratch[32] = si;
    }
    __syncthreads();
    T res = scratch[warp] + incl - v;
    *total = scratch[32];
    __syncthreads();
    return res;
}

// ---------------------------------------------------------------------------------------
// Bitonic sort of G*R keys held in registers by groups of G lanes (G = 8, 16 or 32), R keys per
// lane, ascending.  Element e of a group lives in lane (e / R) of the group, register e % R, so
// that compare-exchanges at a distance below R stay inside a lane and the others are one
// shuffle per register.  After the call lane l of a group holds sorted elements [l*R, l*R+R).
//
// Every compare-exchange is a plain min/max: merge levels whose direction depends on the
// register index are resolved at compile time, and levels whose direction depends on the lane
// run on complemented keys in the descending lanes (x -> ~x reverses the order), so that the
// whole level is an ascending merge.
// ---------------------------------------------------------------------------------------
template <typename K>
__device__ __forceinline__ K kmin(K a, K b) { return a < b ? a : b; }
template <typename K>
__device__ __forceinline__ K kmax(K a, K b) { return a < b ? b : a; }
template <>
__device__ __forceinline__ uint32_t kmin<uint32_t>(uint32_t a, uint32_t b) { return min(a, b); }
template <>
__device__ __forceinline__ uint32_t kmax<uint32_t>(uint32_t a, uint32_t b) { return max(a, b); }

// x -> ~x for every key when `flip`, else unchanged.  ~x = -x - 1, written as x * c + d with
// (c, d) = (-1, -1) or (1, 0): an integer multiply-add, which issues on the FMA pipe and leaves the
// ALU pipe (busy with the min/max of the network) alone.
template <typename K, int R>
__device__ __forceinline__ void flip_keys(K (&x)[R], bool flip) {
    const K c = flip ? ~K(0) : K(1);
    const K d = flip ? ~K(0) : K(0);
#pragma unroll
    for (int r = 0; r < R; ++r) x[r] = x[r] * c + d;
}

template <typename K, int R, int G = 32>
__device__ __forceinline__ void group_bitonic_sort(K (&x)[R]) {
    static_assert((R & (R - 1)) == 0 && (G & (G - 1)) == 0 && G <= 32, "powers of two");
    const int gl = lane_id() & (G - 1);
    bool flipped = false;
#pragma unroll
    for (int k = 2; k <= G * R; k <<= 1) {
        if (k >= R && k < G * R) {
            // direction of this level is per lane: descending lanes work on complemented keys
            const bool want = (gl & (k / R)) != 0;
            flip_keys<K, R>(x, want != flipped);
            flipped = want;
        } else if (k == G * R && G * R > R) {
            flip_keys<K, R>(x, flipped);
            flipped = false;
        }
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j < R) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int pr = r ^ j;
                    if (pr > r) {
                        // for k < R the direction depends on r only (compile time); otherwise ascending
                        const bool up = (k < R) ? ((r & k) == 0) : true;
                        const K lo = kmin(x[r], x[pr]), hi = kmax(x[r], x[pr]);
                        x[r] = up ? lo : hi;
                        x[pr] = up ? hi : lo;
                    }
                }
            } else {
                const int lj = j / R;
                const bool lower = (gl & lj) == 0;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const K other = __shfl_xor_sync(FULL_MASK, x[r], lj);
                    x[r] = lower ? kmin(x[r], other) : kmax(x[r], other);
                }
            }
        }
    }
}

// first position in a[0, len) whose value is >= key (a ascending)
__device__ __forceinline__ uint32_t lower_bound_i32(const int32_t* __restrict__ a, uint32_t len, int32_t key) {
    uint32_t lo = 0, hi = len;
    while (lo < hi) {
        uint32_t mid = (lo + hi) >> 1;
        if (a[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// ---------------------------------------------------------------------------------------
// Device-wide exclusive scan, reduce-then-scan in three launches (no inter-CTA waiting):
//   out[i] = sum_{r<i} in[r] for i in [0, n], so out has n + 1 entries and out[n] is the total.
// `partials` needs scan_partials_count(n) int64 entries.
// ---------------------------------------------------------------------------------------
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

inline int64_t scan_partials_count(int64_t n) { return (n + SCAN_TILE - 1) / SCAN_TILE + 1; }

template <typename InT>
static __global__ void __launch_bounds__(SCAN_THREADS) scan_tile_sums_kernel(const InT* __restrict__ in, int64_t n,
                                                                       int64_t* __restrict__ partials) {
    __shared__ int64_t red[SCAN_THREADS / 32];
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE;
    int64_t s = 0;
#pragma unroll
    for (int it = 0; it < SCAN_ITEMS; ++it) {
        int64_t idx = base + it * SCAN_THREADS + threadIdx.x;
        if (idx < n) s += (int64_t)in[idx];
    }
    s = warp_reduce_sum(s);
    if (lane_id() == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t t = 0;
        for (int w = 0; w < SCAN_THREADS / 32; ++w) t += red[w];
        partials[blockIdx.x] = t;
    }
}

// one CTA: exclusive scan of partials[0, ntiles) in place
static __global__ void __launch_bounds__(1024) scan_partials_kernel(int64_t* __restrict__ partials, int64_t ntiles) {
    __shared__ int64_t scratch[33];
    int64_t carry = 0;
    for (int64_t b = 0; b < ntiles; b += 1024) {
        int64_t idx = b + threadIdx.x;
        int64_t v = idx < ntiles ? partials[idx] : 0, tot;
        int64_t ex = block_exclusive_scan<int64_t, 1024>(v, scratch, &tot);
        if (idx < ntiles) partials[idx] = carry + ex;
        carry += tot;
    }
}

template <typename InT>
static __global__ void __launch_bounds__(SCAN_THREADS) scan_tiles_kernel(const InT* __restrict__ in, int64_t n,
                                                                   const int64_t* __restrict__ partials,
                                                                   int64_t* __restrict__ out) {
    __shared__ int64_t scratch[33];
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int64_t v[SCAN_ITEMS], s = 0;
#pragma unroll
    for (int it = 0; it < SCAN_ITEMS; ++it) {
        int64_t idx = base + it;
        v[it] = idx < n ? (int64_t)in[idx] : 0;
        s += v[it];
    }
    int64_t tot;
    int64_t ex = block_exclusive_scan<int64_t, SCAN_THREADS>(s, scratch, &tot) + partials[blockIdx.x];
#pragma unroll
    for (int it = 0; it < SCAN_ITEMS; ++it) {
        int64_t idx = base + it;
        if (idx < n) out[idx] = ex;
        ex += v[it];
        if (idx == n - 1) out[n] = ex;
    }
}

template <typename InT>
inline cudaError_t exclusive_scan_i64(const InT* in, int64_t n, int64_t* out, int64_t* partials, cudaStream_t st) {
    if (n <= 0) return cudaMemsetAsync(out, 0, sizeof(int64_t), st);
    const int64_t ntiles = (n + SCAN_TILE - 1) / SCAN_TILE;
    scan_tile_sums_kernel<InT><<<(unsigned)ntiles, SCAN_THREADS, 0, st>>>(in, n, partials);
    scan_partials_kernel<<<1, 1024, 0, st>>>(partials, ntiles);
    scan_tiles_kernel<InT><<<(unsigned)ntiles, SCAN_THREADS, 0, st>>>(in, n, partials, out);
    note_launches(3);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------
// Stable binning of items 0..n-1 into NCLASS classes (a counting sort on the class id):
// perm lists the items of class 0, then class 1, ..., each in ascending item order;
// class_start[c] (c = 0..NCLASS) are the offsets.  cls[i] is a byte per item.
//   blockhist : NCLASS * nblocks int32      offsets : NCLASS * nblocks + 1 int64
// ---------------------------------------------------------------------------------------
constexpr int BIN_THREADS = 256;
constexpr int BIN_ROUNDS = 8;
constexpr int BIN_TILE = BIN_THREADS * BIN_ROUNDS;

inline int64_t bin_blocks(int64_t n) { return n > 0 ? (n + BIN_TILE - 1) / BIN_TILE : 1; }

static __global__ void __launch_bounds__(BIN_THREADS) bin_count_kernel(const uint8_t* __restrict__ cls, int64_t n,
                                                                 int32_t* __restrict__ blockhist, int64_t nblocks) {
    __shared__ int32_t hist[NCLASS];
    if (threadIdx.x < NCLASS) hist[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * BIN_TILE;
#pragma unroll
    for (int r = 0; r < BIN_ROUNDS; ++r) {
        int64_t idx = base + r * BIN_THREADS + threadIdx.x;
        if (idx < n) atomicAdd(&hist[cls[idx]], 1);
    }
    __syncthreads();
    if (threadIdx.x < NCLASS) blockhist[(int64_t)threadIdx.x * nblocks + blockIdx.x] = hist[threadIdx.x];
}

static __global__ void __launch_bounds__(BIN_THREADS) bin_scatter_kernel(const uint8_t* __restrict__ cls, int64_t n,
                                                                   const int64_t* __restrict__ offsets, int64_t nblocks,
                                                                   int32_t* __restrict__ perm) {
    constexpr int NW = BIN_THREADS / 32;
    __shared__ int64_t running[NCLASS];
    __shared__ int32_t wcount[NW][NCLASS];
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    if (threadIdx.x < NCLASS) running[threadIdx.x] = offsets[(int64_t)threadIdx.x * nblocks + blockIdx.x];
    const int64_t base = (int64_t)blockIdx.x * BIN_TILE;
    for (int r = 0; r < BIN_ROUNDS; ++r) {
        int64_t idx = base + r * BIN_THREADS + threadIdx.x;
        int c = idx < n ? (int)cls[idx] : -1;
        int myrank = 0;
#pragma unroll
        for (int k = 0; k < NCLASS; ++k) {
            unsigned b = __ballot_sync(FULL_MASK, c == k);
            if (c == k) myrank = __popc(b & ((1u << lane) - 1u));
            if (lane == 0) wcount[warp][k] = __popc(b);
        }
        __syncthreads();
        if (c >= 0) {
            int64_t pos = running[c] + myrank;
            for (int w = 0; w < warp; ++w) pos += wcount[w][c];
            perm[pos] = (int32_t)idx;
        }
        __syncthreads();
        if (threadIdx.x < NCLASS) {
            int t = 0;
            for (int w = 0; w < NW; ++w) t += wcount[w][threadIdx.x];
            running[threadIdx.x] += t;
        }
        __syncthreads();
    }
}

static __global__ void bin_class_starts_kernel(const int64_t* __restrict__ offsets, int64_t nblocks, int64_t* __restrict__ class_start) {
    int c = threadIdx.x;
    if (c < NCLASS) class_start[c] = offsets[(int64_t)c * nblocks];
    if (c == NCLASS) class_start[c] = offsets[(int64_t)NCLASS * nblocks];
}

// scratch sizes (in elements) for bin_items: blockhist int32, offsets int64, partials int64
inline cudaError_t bin_items(const uint8_t* cls, int64_t n, int32_t* perm, int64_t* class_start /*device, NCLASS+1*/,
                             int32_t* blockhist, int64_t* offsets, int64_t* partials, cudaStream_t st) {
    const int64_t nb = bin_blocks(n);
    bin_count_kernel<<<(unsigned)nb, BIN_THREADS, 0, st>>>(cls, n, blockhist, nb);
    cudaError_t e = exclusive_scan_i64<int32_t>(blockhist, NCLASS * nb, offsets, partials, st);
    if (e != cudaSuccess) return e;
    bin_scatter_kernel<<<(unsigned)nb, BIN_THREADS, 0, st>>>(cls, n, offsets, nb, perm);
    bin_class_starts_kernel<<<1, 32, 0, st>>>(offsets, nb, class_start);
    note_launches(3);
    return cudaGetLastError();
}

// value-type traits: accumulator type and exact conversions
template <typename V> struct AccOf { using type = double; };
template <> struct AccOf<int32_t> { using type = int32_t; };

__device__ __forceinline__ double acc_mul(double a, double b) { return __dmul_rn(a, b); }
__device__ __forceinline__ int32_t acc_mul(int32_t a, int32_t b) { return (int32_t)((uint32_t)a * (uint32_t)b); }
__device__ __forceinline__ double acc_add(double a, double b) { return __dadd_rn(a, b); }
__device__ __forceinline__ int32_t acc_add(int32_t a, int32_t b) { return (int32_t)((uint32_t)a + (uint32_t)b); }

}  // namespace spsyrk
