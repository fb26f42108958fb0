// spsyrk_host_tril: the whole path on host buffers.  Device memory is allocated here with
// cudaMalloc; the computation itself goes through the same entry points a device caller uses.
#include <new>

#include <cuda_runtime.h>

#include "../../include/spsyrk.h"

struct spsyrk_session_s {
    spsyrk_plan_t plan = nullptr;
    cudaStream_t stream = nullptr;
    int64_t m = 0, nnz_c = 0;
    size_t sv = 0;
    void *d_rowptr = nullptr, *d_colidx = nullptr, *d_vals = nullptr, *d_ws = nullptr;
    void *d_c_rowptr = nullptr, *d_c_colidx = nullptr, *d_c_vals = nullptr;
};

namespace {
void release(spsyrk_session_s* s) {
    if (!s) return;
    if (s->plan) spsyrk_destroy(s->plan);
    cudaFree(s->d_rowptr); cudaFree(s->d_colidx); cudaFree(s->d_vals); cudaFree(s->d_ws);
    cudaFree(s->d_c_rowptr); cudaFree(s->d_c_colidx); cudaFree(s->d_c_vals);
    if (s->stream) cudaStreamDestroy(s->stream);
    delete s;
}
}  // namespace

#define HOST_TRY(expr) do { if ((expr) != cudaSuccess) { release(s); return SPSYRK_ERR_CUDA; } } while (0)
#define HOST_ST(expr) do { spsyrk_status_t _st = (expr); if (_st != SPSYRK_OK) { release(s); return _st; } } while (0)

extern "C" spsyrk_status_t spsyrk_host_tril(spsyrk_session_t* session, int64_t m, int64_t n, int64_t nnz,
                                            const int64_t* h_rowptr, const int32_t* h_colidx, const void* h_vals,
                                            spsyrk_dtype_t dtype, spsyrk_mode_t mode, int64_t* h_c_rowptr, int64_t* nnz_out,
                                            int32_t* h_c_colidx, void* h_c_vals) {
    if (!session) return SPSYRK_ERR_INVALID_ARG;
    if (!h_c_colidx) {  // call 1: upload, plan, symbolic
        if (!h_rowptr || !h_c_rowptr || !nnz_out || m < 0 || nnz < 0 || (nnz > 0 && (!h_colidx || !h_vals)))
            return SPSYRK_ERR_INVALID_ARG;
        spsyrk_session_s* s = new (std::nothrow) spsyrk_session_s();
        if (!s) return SPSYRK_ERR_INTERNAL;
        s->m = m;
        s->sv = dtype == SPSYRK_F64 ? 8 : 4;
        size_t ws_bytes = 0;
        HOST_ST(spsyrk_plan(nullptr, m, n, nnz, nullptr, nullptr, nullptr, dtype, mode, 0, m, nullptr, &ws_bytes, nullptr));
        HOST_TRY(cudaStreamCreate(&s->stream));
        HOST_TRY(cudaMalloc(&s->d_rowptr, (size_t)(m + 1) * 8));
        HOST_TRY(cudaMalloc(&s->d_colidx, (size_t)(nnz > 0 ? nnz : 1) * 4));
        HOST_TRY(cudaMalloc(&s->d_vals, (size_t)(nnz > 0 ? nnz : 1) * s->sv));
        HOST_TRY(cudaMalloc(&s->d_ws, ws_bytes));
        HOST_TRY(cudaMalloc(&s->d_c_rowptr, (size_t)(m + 1) * 8));
        HOST_TRY(cudaMemcpyAsync(s->d_rowptr, h_rowptr, (size_t)(m + 1) * 8, cudaMemcpyHostToDevice, s->stream));
        if (nnz > 0) {
            HOST_TRY(cudaMemcpyAsync(s->d_colidx, h_colidx, (size_t)nnz * 4, cudaMemcpyHostToDevice, s->stream));
            HOST_TRY(cudaMemcpyAsync(s->d_vals, h_vals, (size_t)nnz * s->sv, cudaMemcpyHostToDevice, s->stream));
        }
        HOST_ST(spsyrk_plan(&s->plan, m, n, nnz, (const int64_t*)s->d_rowptr, (const int32_t*)s->d_colidx, s->d_vals, dtype, mode,
                            0, m, s->d_ws, &ws_bytes, s->stream));
        HOST_ST(spsyrk_symbolic(s->plan, (int64_t*)s->d_c_rowptr, &s->nnz_c, s->stream));
        HOST_TRY(cudaMemcpyAsync(h_c_rowptr, s->d_c_rowptr, (size_t)(m + 1) * 8, cudaMemcpyDeviceToHost, s->stream));
        HOST_TRY(cudaStreamSynchronize(s->stream));
        *nnz_out = s->nnz_c;
        *session = s;
        return SPSYRK_OK;
    }
    // call 2: numeric, download, release
    spsyrk_session_s* s = *session;
    if (!s || !h_c_vals) return SPSYRK_ERR_INVALID_ARG;
    *session = nullptr;
    const size_t cn = (size_t)(s->nnz_c > 0 ? s->nnz_c : 1);
    HOST_TRY(cudaMalloc(&s->d_c_colidx, cn * 4));
    HOST_TRY(cudaMalloc(&s->d_c_vals, cn * s->sv));
    HOST_ST(spsyrk_numeric(s->plan, (const int64_t*)s->d_c_rowptr, (int32_t*)s->d_c_colidx, s->d_c_vals, s->stream));
    if (s->nnz_c > 0) {
        HOST_TRY(cudaMemcpyAsync(h_c_colidx, s->d_c_colidx, (size_t)s->nnz_c * 4, cudaMemcpyDeviceToHost, s->stream));
        HOST_TRY(cudaMemcpyAsync(h_c_vals, s->d_c_vals, (size_t)s->nnz_c * s->sv, cudaMemcpyDeviceToHost, s->stream));
    }
    HOST_TRY(cudaStreamSynchronize(s->stream));
    release(s);
    return SPSYRK_OK;
}
