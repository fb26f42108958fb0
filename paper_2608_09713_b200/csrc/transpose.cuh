// Step a1: on-device CSR transpose of A into column lists whose entries are ascending by row,
// plus the per-nonzero descriptors the row kernels consume.
//
//   colptr[n+1]        column pointers (int64)
//   at_row[q], at_val[q]  entries of the column lists, q in [colptr[k], colptr[k+1]) ascending by row
//   desc[p] = (start, len) for nonzero p = (i, k) of A: start = colptr[k]; len = number of entries
//             of column k with row <= i (TRIL: the rank of i in the list, plus one) or the whole
//             column length (FULL).  "Rows j <= i of column k" is then at_row[start, start+len).
//
// Method: histogram of column ids (atomics), scan, scatter of (row, p) keys through per-column
// atomic cursors (arbitrary order inside a column), then a sort of every column segment by row:
// register bitonic sort for short columns, a bitmap-rank pass for long ones (row ids inside a
// column are distinct, so the rank of a row is the number of set bits below it).
#pragma once
#include "common.cuh"

namespace spsyrk {

struct PlanDev {
    int32_t m, n;
    int64_t nnz;
    int32_t r0, r1;
    int32_t mode;
    const int64_t* rowptr;
    const int32_t* colidx;
    const void* vals;
    int64_t* colptr;
    int32_t* at_row;
    void* at_val;
    uint2* desc;
    int64_t* work;  // per row of the range
    uint32_t* err;
};

static __global__ void validate_rowptr_kernel(const int64_t* __restrict__ rowptr, int64_t m, int64_t nnz, uint32_t* err) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) {
        int64_t a = rowptr[i], b = rowptr[i + 1];
        if (a > b || a < 0 || b > nnz) atomicOr(err, ERRW_BAD_ROWPTR);
    }
    if (i == 0 && (rowptr[0] != 0 || rowptr[m] != nnz)) atomicOr(err, ERRW_BAD_ROWPTR);
}

static __global__ void column_histogram_kernel(const int32_t* __restrict__ colidx, int64_t nnz, int32_t n,
                                        uint32_t* __restrict__ colcnt, uint32_t* err) {
    int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; p < nnz; p += stride) {
        int32_t k = colidx[p];
        if ((uint32_t)k >= (uint32_t)n) atomicOr(err, ERRW_BAD_COL);
        else atomicAdd(&colcnt[k], 1u);
    }
}

// G lanes per row: scatter (row, p) keys into the column segments; also checks that column ids are
// strictly ascending inside the row.
template <int G>
static __global__ void __launch_bounds__(256) column_fill_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ colidx,
                                                          int32_t m, int32_t n, const int64_t* __restrict__ colptr,
                                                          uint32_t* __restrict__ cursor, uint64_t* __restrict__ keys, uint32_t* err) {
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (gid >= m) return;
    const int64_t p0 = rowptr[gid], p1 = rowptr[gid + 1];
    for (int64_t p = p0 + gl; p < p1; p += G) {
        int32_t k = colidx[p];
        if ((uint32_t)k >= (uint32_t)n) continue;  // already reported by the histogram
        if (p > p0 && colidx[p - 1] >= k) atomicOr(err, ERRW_UNSORTED);
        uint32_t slot = atomicAdd(&cursor[k], 1u);
        keys[colptr[k] + slot] = ((uint64_t)(uint32_t)gid << 32) | (uint32_t)p;
    }
}

// column classes: 0 empty, 1: d<=8, 2: <=16, 3: <=32, 4: <=64, 5: <=128, 6: <=256, 7: larger
static __global__ void column_class_kernel(const int64_t* __restrict__ colptr, int32_t n, uint8_t* __restrict__ cls) {
    int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    int64_t d = colptr[k + 1] - colptr[k];
    uint8_t c = d == 0 ? 0 : d <= 8 ? 1 : d <= 16 ? 2 : d <= 32 ? 3 : d <= 64 ? 4 : d <= 128 ? 5 : d <= 256 ? 6 : 7;
    cls[k] = c;
}

template <typename V>
__device__ __forceinline__ void emit_column_entry(const PlanDev& P, int64_t cs, uint32_t q, uint32_t d, uint64_t key) {
    const uint32_t row = (uint32_t)(key >> 32), p = (uint32_t)key;
    P.at_row[cs + q] = (int32_t)row;
    static_cast<V*>(P.at_val)[cs + q] = static_cast<const V*>(P.vals)[p];
    P.desc[p] = make_uint2((uint32_t)cs, P.mode == SPSYRK_TRIL ? q + 1 : d);
}

// groups of G lanes sort one column of at most G*R entries
template <typename V, int R, int G>
static __global__ void __launch_bounds__(256) column_sort_group_kernel(PlanDev P, const int32_t* __restrict__ cols, int64_t ncols,
                                                                const uint64_t* __restrict__ keys) {
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    // all lanes of a warp take part in the shuffles; groups past the end sort padding
    const bool live = gid < ncols;
    int64_t cs = 0;
    uint32_t d = 0;
    if (live) {
        const int32_t k = cols[gid];
        cs = P.colptr[k];
        d = (uint32_t)(P.colptr[k + 1] - cs);
    }
    uint64_t x[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        uint32_t e = r * G + gl;  // any input order will do
        x[r] = e < d ? keys[cs + e] : ~0ull;
    }
    group_bitonic_sort<uint64_t, R, G>(x);
#pragma unroll
    for (int r = 0; r < R; ++r) {
        uint32_t q = gl * R + r;
        if (q < d) emit_column_entry<V>(P, cs, q, d, x[r]);
    }
}

// one CTA per long column: rank rows through a bitmap over row-id chunks of `chunk_bits` bits.
// dynamic shared memory: 2 * chunk_bits / 32 words.
template <typename V, int THREADS>
static __global__ void __launch_bounds__(THREADS) column_sort_cta_kernel(PlanDev P, const int32_t* __restrict__ cols,
                                                                  const uint64_t* __restrict__ keys, uint32_t chunk_bits) {
    extern __shared__ uint32_t smem_u32[];
    __shared__ uint32_t scratch[33];
    const uint32_t cw = chunk_bits >> 5;
    uint32_t* bits = smem_u32;
    uint32_t* rank = smem_u32 + cw;
    const int32_t k = cols[blockIdx.x];
    const int64_t cs = P.colptr[k];
    const uint32_t d = (uint32_t)(P.colptr[k + 1] - cs);
    const uint32_t per = (cw + THREADS - 1) / THREADS;
    uint32_t base = 0;
    for (uint32_t c0 = 0; c0 < (uint32_t)P.m; c0 += chunk_bits) {
        for (uint32_t w = threadIdx.x; w < cw; w += THREADS) bits[w] = 0;
        __syncthreads();
        for (uint32_t e = threadIdx.x; e < d; e += THREADS) {
            uint32_t row = (uint32_t)(keys[cs + e] >> 32) - c0;
            if (row < chunk_bits) atomicOr(&bits[row >> 5], 1u << (row & 31));
        }
        __syncthreads();
        uint32_t s = 0;
        const uint32_t w0 = threadIdx.x * per;
        for (uint32_t w = w0; w < w0 + per && w < cw; ++w) s += __popc(bits[w]);
        uint32_t tot;
        uint32_t ex = block_exclusive_scan<uint32_t, THREADS>(s, scratch, &tot);
        for (uint32_t w = w0; w < w0 + per && w < cw; ++w) { rank[w] = ex; ex += __popc(bits[w]); }
        __syncthreads();
        for (uint32_t e = threadIdx.x; e < d; e += THREADS) {
            uint64_t key = keys[cs + e];
            uint32_t row = (uint32_t)(key >> 32) - c0;
            if (row < chunk_bits) {
                uint32_t q = base + rank[row >> 5] + __popc(bits[row >> 5] & ((1u << (row & 31)) - 1u));
                emit_column_entry<V>(P, cs, q, d, key);
            }
        }
        base += tot;
        __syncthreads();
    }
}

// Step a2: per-row work w[i] = sum of the descriptor lengths of row i (G lanes per row), and the
// class of the row.  Rows of the range [r0, r1) only.
//   class 0: no work; 1..5: w <= 32, 64, 128, 256, 512 and at most 32 nonzeros (one warp, register sort)
//   6: w <= block_max (one 256-thread CTA, bitmap accumulator); 7: larger (one 1024-thread CTA)
template <int G>
static __global__ void __launch_bounds__(256) row_work_kernel(PlanDev P, uint8_t* __restrict__ cls, int64_t block_max,
                                                        unsigned long long* __restrict__ work_total) {
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    const int64_t rows = P.r1 - P.r0;
    int64_t w = 0, deg = 0;
    if (gid < rows) {
        const int64_t i = P.r0 + gid;
        const int64_t p0 = P.rowptr[i], p1 = P.rowptr[i + 1];
        deg = p1 - p0;
        for (int64_t p = p0 + gl; p < p1; p += G) w += P.desc[p].y;
    }
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) w += __shfl_xor_sync(FULL_MASK, w, o);
    const bool owner = gid < rows && gl == 0;
    if (owner) {
        P.work[gid] = w;
        uint8_t c;
        if (w == 0) c = 0;
        else if (deg <= 32 && w <= 512) c = w <= 32 ? 1 : w <= 64 ? 2 : w <= 128 ? 3 : w <= 256 ? 4 : 5;
        else c = w <= block_max ? 6 : 7;
        cls[gid] = c;
    }
    // one atomic per CTA for the total
    __shared__ unsigned long long cta_sum;
    if (threadIdx.x == 0) cta_sum = 0;
    __syncthreads();
    unsigned long long ws = warp_reduce_sum<unsigned long long>(owner ? (unsigned long long)w : 0ull);
    if (lane_id() == 0 && ws) atomicAdd(&cta_sum, ws);
    __syncthreads();
    if (threadIdx.x == 0 && cta_sum) atomicAdd(work_total, cta_sum);
}

}  // namespace spsyrk
