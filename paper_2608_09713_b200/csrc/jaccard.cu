// Step a8: Jaccard normalisation of intersection counts, J = c / (|a_i| + |a_j| - c).
// One CTA per chunk of stored entries: the chunk's first row is found by a binary search over
// the row pointers, then each thread locates its entry's row inside the chunk's row span.
#include "common.cuh"

using namespace spsyrk;

namespace {

constexpr int JAC_THREADS = 256;
constexpr int JAC_ITEMS = 8;
constexpr int64_t JAC_CHUNK = JAC_THREADS * JAC_ITEMS;

// last row t in [lo, hi] with c_rowptr[t] <= e
__device__ __forceinline__ int64_t row_of_entry(const int64_t* __restrict__ c_rowptr, int64_t lo, int64_t hi, int64_t e) {
    while (lo < hi) {
        const int64_t mid = (lo + hi + 1) >> 1;
        if (c_rowptr[mid] <= e) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__global__ void __launch_bounds__(JAC_THREADS) jaccard_kernel(int64_t row_begin, int64_t rows, int64_t nnz,
                                                              const int64_t* __restrict__ a_rowptr,
                                                              const int64_t* __restrict__ c_rowptr,
                                                              const int32_t* __restrict__ c_colidx,
                                                              const int32_t* __restrict__ c_counts, float* __restrict__ jac) {
    __shared__ int64_t span[2];
    const int64_t e0 = (int64_t)blockIdx.x * JAC_CHUNK;
    const int64_t e1 = min(e0 + JAC_CHUNK, nnz);
    if (threadIdx.x < 2) span[threadIdx.x] = row_of_entry(c_rowptr, 0, rows - 1, threadIdx.x == 0 ? e0 : e1 - 1);
    __syncthreads();
    const int64_t t_lo = span[0], t_hi = span[1];
#pragma unroll
    for (int it = 0; it < JAC_ITEMS; ++it) {
        const int64_t e = e0 + (int64_t)it * JAC_THREADS + threadIdx.x;
        if (e >= e1) continue;
        const int64_t t = t_lo == t_hi ? t_lo : row_of_entry(c_rowptr, t_lo, t_hi, e);
        const int64_t i = row_begin + t;
        const int64_t j = c_colidx[e];
        const int64_t na_i = a_rowptr[i + 1] - a_rowptr[i];
        const int64_t na_j = a_rowptr[j + 1] - a_rowptr[j];
        const int64_t c = c_counts[e];
        jac[e] = __fdiv_rn((float)c, (float)(na_i + na_j - c));
    }
}

}  // namespace

extern "C" spsyrk_status_t spsyrk_jaccard(int64_t m, int64_t row_begin, int64_t rows, const int64_t* d_a_rowptr,
                                          const int64_t* d_c_rowptr, const int32_t* d_c_colidx, const int32_t* d_c_counts,
                                          float* d_jaccard, void* cuda_stream) {
    if (m < 0 || row_begin < 0 || rows < 0 || row_begin + rows > m) return SPSYRK_ERR_INVALID_ARG;
    if (!d_a_rowptr || !d_c_rowptr) return SPSYRK_ERR_INVALID_ARG;
    if (rows == 0) return SPSYRK_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int64_t nnz = 0;  // the grid size depends on the entry count: one small read-back
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&nnz, d_c_rowptr + rows, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    if (nnz == 0) return SPSYRK_OK;
    if (!d_c_colidx || !d_c_counts || !d_jaccard) return SPSYRK_ERR_INVALID_ARG;
    const int64_t blocks = (nnz + JAC_CHUNK - 1) / JAC_CHUNK;
    if (blocks >= (int64_t(1) << 31)) return SPSYRK_ERR_OVERFLOW;
    jaccard_kernel<<<(unsigned)blocks, JAC_THREADS, 0, st>>>(row_begin, rows, nnz, d_a_rowptr, d_c_rowptr, d_c_colidx,
                                                             d_c_counts, d_jaccard);
    note_launches(1);
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}
