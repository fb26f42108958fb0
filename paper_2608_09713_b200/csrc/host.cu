// spsyrk_host_tril: the whole path on host buffers.  Device memory is allocated here with
// cudaMalloc; the computation itself goes through the same entry points a device caller uses.
#include <algorithm>
#include <mutex>
#include <new>

#include <cuda_runtime.h>

#include "../../include/spsyrk.h"

// Device memory of the host entry point comes from two grow-only arenas per device that outlive the
// call: allocating and freeing several GB per call costs more than the computation it serves.  A call
// that finds the arenas taken by a live session of another thread falls back to its own allocations.
namespace {
struct Arena {
    void* ptr = nullptr;
    size_t bytes = 0;
    bool busy = false;
};
constexpr int MAX_DEVICES = 64;
std::mutex g_arena_mutex;
Arena g_arena[MAX_DEVICES][2];  // [device][0: inputs, workspace, row pointers; 1: output entries]

constexpr size_t A256 = 256;
constexpr int HOST_MAX_BLOCKS = 8;
constexpr int64_t HOST_BLOCK_MIN_ENTRIES = int64_t(1) << 22;  // below this a block's launches cost more than its copy hides
size_t up256(size_t b) { return (b + A256 - 1) / A256 * A256; }
}  // namespace

struct spsyrk_session_s {
    spsyrk_plan_t plan = nullptr;
    cudaStream_t stream = nullptr;
    int64_t m = 0, nnz_c = 0;
    size_t sv = 0;
    int device = -1;
    void* block[2] = {nullptr, nullptr};  // the two device blocks of this session
    bool cached[2] = {false, false};      // block i belongs to the device's arena (else: owned, freed on release)
    void *d_rowptr = nullptr, *d_colidx = nullptr, *d_vals = nullptr, *d_ws = nullptr;
    void *d_c_rowptr = nullptr, *d_c_colidx = nullptr, *d_c_vals = nullptr;
    // call 2 computes and downloads C_L in row blocks of about equal numbers of entries: the copy of a block
    // runs while the next ones are computed
    cudaStream_t copy_stream = nullptr;
    int blocks = 0;
    int64_t block_row[HOST_MAX_BLOCKS + 1] = {};
    int64_t block_off[HOST_MAX_BLOCKS + 1] = {};
};

namespace {
// a block of `bytes` for slot `which` of session s: the device's arena when it is free, grown if needed
cudaError_t acquire(spsyrk_session_s* s, int which, size_t bytes) {
    if (s->device >= 0 && s->device < MAX_DEVICES) {
        std::lock_guard<std::mutex> lock(g_arena_mutex);
        Arena& a = g_arena[s->device][which];
        if (!a.busy) {
            if (a.bytes < bytes) {
                if (a.ptr) cudaFree(a.ptr);
                a.ptr = nullptr;
                a.bytes = 0;
                cudaError_t e = cudaMalloc(&a.ptr, bytes);
                if (e != cudaSuccess) return e;
                a.bytes = bytes;
            }
            a.busy = true;
            s->block[which] = a.ptr;
            s->cached[which] = true;
            return cudaSuccess;
        }
    }
    s->cached[which] = false;
    return cudaMalloc(&s->block[which], bytes);
}

void release(spsyrk_session_s* s) {
    if (!s) return;
    if (s->plan) spsyrk_destroy(s->plan);
    if (s->copy_stream) {
        cudaStreamSynchronize(s->copy_stream);
        cudaStreamDestroy(s->copy_stream);
    }
    if (s->stream) {
        cudaStreamSynchronize(s->stream);
        cudaStreamDestroy(s->stream);
    }
    for (int i = 0; i < 2; ++i) {
        if (!s->block[i]) continue;
        if (s->cached[i]) {
            std::lock_guard<std::mutex> lock(g_arena_mutex);
            g_arena[s->device][i].busy = false;
        } else {
            cudaFree(s->block[i]);
        }
    }
    delete s;
}
}  // namespace

extern "C" spsyrk_status_t spsyrk_host_release_cache(void) {
    std::lock_guard<std::mutex> lock(g_arena_mutex);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPSYRK_ERR_CUDA;
    if (dev < 0 || dev >= MAX_DEVICES) return SPSYRK_OK;
    for (int i = 0; i < 2; ++i) {
        Arena& a = g_arena[dev][i];
        if (a.busy) continue;  // a live session still uses it
        if (a.ptr) cudaFree(a.ptr);
        a.ptr = nullptr;
        a.bytes = 0;
    }
    return SPSYRK_OK;
}

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
        HOST_TRY(cudaGetDevice(&s->device));
        HOST_TRY(cudaStreamCreate(&s->stream));
        const size_t b_rowptr = up256((size_t)(m + 1) * 8), b_colidx = up256((size_t)(nnz > 0 ? nnz : 1) * 4);
        const size_t b_vals = up256((size_t)(nnz > 0 ? nnz : 1) * s->sv), b_ws = up256(ws_bytes);
        HOST_TRY(acquire(s, 0, 2 * b_rowptr + b_colidx + b_vals + b_ws));
        char* base = static_cast<char*>(s->block[0]);
        s->d_rowptr = base;
        s->d_c_rowptr = base + b_rowptr;
        s->d_colidx = base + 2 * b_rowptr;
        s->d_vals = base + 2 * b_rowptr + b_colidx;
        s->d_ws = base + 2 * b_rowptr + b_colidx + b_vals;
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
        // row blocks of call 2: boundaries where the output reaches k / blocks of its entries
        s->blocks = (int)std::max<int64_t>(1, std::min<int64_t>(HOST_MAX_BLOCKS, s->nnz_c / HOST_BLOCK_MIN_ENTRIES));
        for (int b = 0; b <= s->blocks; ++b) {
            const int64_t target = b == s->blocks ? s->nnz_c : s->nnz_c / s->blocks * b;
            const int64_t r = b == s->blocks ? m : b == 0 ? 0 : std::lower_bound(h_c_rowptr, h_c_rowptr + m + 1, target) - h_c_rowptr;
            s->block_row[b] = std::min<int64_t>(r, m);
            s->block_off[b] = h_c_rowptr[s->block_row[b]];
        }
        *nnz_out = s->nnz_c;
        *session = s;
        return SPSYRK_OK;
    }
    // call 2: numeric, download, release
    spsyrk_session_s* s = *session;
    if (!s || !h_c_vals) return SPSYRK_ERR_INVALID_ARG;
    *session = nullptr;
    const size_t cn = (size_t)(s->nnz_c > 0 ? s->nnz_c : 1);
    HOST_TRY(acquire(s, 1, up256(cn * 4) + up256(cn * s->sv)));
    s->d_c_colidx = s->block[1];
    s->d_c_vals = static_cast<char*>(s->block[1]) + up256(cn * 4);
    if (s->blocks <= 1) {
        HOST_ST(spsyrk_numeric(s->plan, (const int64_t*)s->d_c_rowptr, (int32_t*)s->d_c_colidx, s->d_c_vals, s->stream));
        if (s->nnz_c > 0) {
            HOST_TRY(cudaMemcpyAsync(h_c_colidx, s->d_c_colidx, (size_t)s->nnz_c * 4, cudaMemcpyDeviceToHost, s->stream));
            HOST_TRY(cudaMemcpyAsync(h_c_vals, s->d_c_vals, (size_t)s->nnz_c * s->sv, cudaMemcpyDeviceToHost, s->stream));
        }
        HOST_TRY(cudaStreamSynchronize(s->stream));
        release(s);
        return SPSYRK_OK;
    }
    HOST_TRY(cudaStreamCreate(&s->copy_stream));
    cudaEvent_t done[HOST_MAX_BLOCKS] = {};
    spsyrk_status_t st = SPSYRK_OK;
    for (int b = 0; b < s->blocks && st == SPSYRK_OK; ++b) {
        st = spsyrk_numeric_rows(s->plan, s->block_row[b], s->block_row[b + 1], (const int64_t*)s->d_c_rowptr, (int32_t*)s->d_c_colidx,
                                 s->d_c_vals, s->stream);
        if (st != SPSYRK_OK) break;
        const int64_t o0 = s->block_off[b], cnt = s->block_off[b + 1] - o0;
        if (cnt <= 0) continue;
        if (cudaEventCreateWithFlags(&done[b], cudaEventDisableTiming) != cudaSuccess || cudaEventRecord(done[b], s->stream) != cudaSuccess ||
            cudaStreamWaitEvent(s->copy_stream, done[b], 0) != cudaSuccess ||
            cudaMemcpyAsync(h_c_colidx + o0, (const int32_t*)s->d_c_colidx + o0, (size_t)cnt * 4, cudaMemcpyDeviceToHost, s->copy_stream) != cudaSuccess ||
            cudaMemcpyAsync((char*)h_c_vals + (size_t)o0 * s->sv, (const char*)s->d_c_vals + (size_t)o0 * s->sv, (size_t)cnt * s->sv,
                            cudaMemcpyDeviceToHost, s->copy_stream) != cudaSuccess)
            st = SPSYRK_ERR_CUDA;
    }
    if (cudaStreamSynchronize(s->stream) != cudaSuccess || cudaStreamSynchronize(s->copy_stream) != cudaSuccess) st = st == SPSYRK_OK ? SPSYRK_ERR_CUDA : st;
    for (int b = 0; b < HOST_MAX_BLOCKS; ++b)
        if (done[b]) cudaEventDestroy(done[b]);
    release(s);
    return st;
}
