// Consuming the triangular output without materialising the full matrix (Section V-F, Eq. 1):
//     y = C x = C_L x + (x^T C_L)^T - D x,
// one pass over the stored lower triangle: entry (r, j, v) adds v * x[j] to y[r] and, when j != r,
// v * x[r] to y[j]; the diagonal is therefore counted once and C_L^T is never formed.
#include "common.cuh"

using namespace spsyrk;

namespace {

template <typename V, int G>
__global__ void __launch_bounds__(256) symv_kernel(int64_t m, const int64_t* __restrict__ l_rowptr, const int32_t* __restrict__ l_colidx,
                                                   const V* __restrict__ l_vals, const V* __restrict__ x, V* __restrict__ y) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    V acc = V(0);
    V xr = V(0);
    if (r < m) {
        xr = x[r];
        const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
        for (int64_t p = p0 + gl; p < p1; p += G) {
            const int32_t j = l_colidx[p];
            const V v = l_vals[p];
            acc += v * x[j];
            if (j != r) atomicAdd(&y[j], v * xr);
        }
    }
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(FULL_MASK, acc, o);
    if (r < m && gl == 0) atomicAdd(&y[r], acc);
}

int group_width(int64_t nnz, int64_t m) {
    const double avg = m > 0 ? (double)nnz / (double)m : 0.0;
    return avg <= 4 ? 4 : avg <= 8 ? 8 : avg <= 16 ? 16 : 32;
}

template <typename V>
spsyrk_status_t symv_typed(int64_t m, int64_t nnz_l, const int64_t* l_rowptr, const int32_t* l_colidx, const void* l_vals,
                           const void* x, void* y, cudaStream_t st) {
    SPSYRK_CUDA_TRY(cudaMemsetAsync(y, 0, (size_t)m * sizeof(V), st));
    const V* lv = static_cast<const V*>(l_vals);
    const V* xv = static_cast<const V*>(x);
    V* yv = static_cast<V*>(y);
#define SYMV(G) symv_kernel<V, G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(m, l_rowptr, l_colidx, lv, xv, yv)
    switch (group_width(nnz_l, m)) {
        case 4: SYMV(4); break;
        case 8: SYMV(8); break;
        case 16: SYMV(16); break;
        default: SYMV(32); break;
    }
#undef SYMV
    note_launches(1);
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}

}  // namespace

namespace {

// Y = C_L X + (X^T C_L)^T - D X for a dense row-major X (m x p), columns in chunks of PC = 8: one warp per row
// of C_L, lane = (entry slot e = lane / 8, column c = lane % 8), so a warp instruction handles four stored
// entries times eight columns.  For entry (r, j, v) lane (e, c) adds v * X[j, c0 + c] to its partial of
// Y[r, c0 + c] (registers) and, when j != r, v * X[r, c0 + c] to Y[j, c0 + c] with an atomic add: the eight
// adds of one entry fall into one 64-byte piece of Y (one or two sectors), which the memory system
// handles together, instead of eight separate requests.  The diagonal is counted once and C_L^T is never formed.
template <typename V, int PC>
__global__ void __launch_bounds__(256) symm_kernel(int64_t m, int64_t p, int64_t c0, const int64_t* __restrict__ l_rowptr,
                                                   const int32_t* __restrict__ l_colidx, const V* __restrict__ l_vals,
                                                   const V* __restrict__ x, V* __restrict__ y) {
    static_assert(PC == 8, "lane layout");
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = lane_id(), c = lane & 7, e = lane >> 3;
    if (r >= m) return;  // warp-uniform
    const bool col_on = c0 + c < p;
    const V xr = col_on ? x[r * p + c0 + c] : V(0);
    V acc = V(0);
    const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
    for (int64_t q = p0 + e; q < p1; q += 4) {
        const int64_t j = l_colidx[q];
        const V v = l_vals[q];
        if (col_on) {
            acc += v * x[j * p + c0 + c];
            if (j != r) atomicAdd(&y[j * p + c0 + c], v * xr);
        }
    }
    acc += __shfl_xor_sync(FULL_MASK, acc, 8);
    acc += __shfl_xor_sync(FULL_MASK, acc, 16);
    if (e == 0 && col_on) atomicAdd(&y[r * p + c0 + c], acc);
}

template <typename V>
spsyrk_status_t symm_typed(int64_t m, int64_t p, int64_t nnz_l, const int64_t* l_rowptr, const int32_t* l_colidx, const void* l_vals,
                           const void* x, void* y, cudaStream_t st) {
    SPSYRK_CUDA_TRY(cudaMemsetAsync(y, 0, (size_t)m * (size_t)p * sizeof(V), st));
    const V* lv = static_cast<const V*>(l_vals);
    const V* xv = static_cast<const V*>(x);
    V* yv = static_cast<V*>(y);
    constexpr int PC = 8;
    for (int64_t c0 = 0; c0 < p; c0 += PC) {
        symm_kernel<V, PC><<<(unsigned)((m * 32 + 255) / 256), 256, 0, st>>>(m, p, c0, l_rowptr, l_colidx, lv, xv, yv);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}

}  // namespace

extern "C" spsyrk_status_t spsyrk_symm(int64_t m, int64_t p, int64_t nnz_l, spsyrk_dtype_t dtype, const int64_t* d_l_rowptr,
                                       const int32_t* d_l_colidx, const void* d_l_vals, const void* d_x, void* d_y,
                                       void* cuda_stream) {
    if (m < 0 || p < 0 || nnz_l < 0 || !d_l_rowptr || (m > 0 && p > 0 && (!d_x || !d_y)) || (nnz_l > 0 && (!d_l_colidx || !d_l_vals)))
        return SPSYRK_ERR_INVALID_ARG;
    if (dtype != SPSYRK_F64 && dtype != SPSYRK_F32) return SPSYRK_ERR_INVALID_ARG;
    if (m == 0 || p == 0) return SPSYRK_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    return dtype == SPSYRK_F64 ? symm_typed<double>(m, p, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_x, d_y, st)
                               : symm_typed<float>(m, p, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_x, d_y, st);
}

extern "C" spsyrk_status_t spsyrk_symv(int64_t m, int64_t nnz_l, spsyrk_dtype_t dtype, const int64_t* d_l_rowptr,
                                       const int32_t* d_l_colidx, const void* d_l_vals, const void* d_x, void* d_y,
                                       void* cuda_stream) {
    if (m < 0 || nnz_l < 0 || !d_l_rowptr || (m > 0 && (!d_x || !d_y)) || (nnz_l > 0 && (!d_l_colidx || !d_l_vals)))
        return SPSYRK_ERR_INVALID_ARG;
    if (dtype != SPSYRK_F64 && dtype != SPSYRK_F32) return SPSYRK_ERR_INVALID_ARG;
    if (m == 0) return SPSYRK_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    return dtype == SPSYRK_F64 ? symv_typed<double>(m, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_x, d_y, st)
                               : symv_typed<float>(m, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_x, d_y, st);
}
