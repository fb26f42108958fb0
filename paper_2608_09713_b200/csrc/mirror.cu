// Step a7: F = C_L + C_L^T - D, the full symmetric CSR from the stored lower triangle.
//
// Row j of F = row j of C_L (columns <= j) followed by the reflected entries (r, c_rj) of the
// later rows r > j that store column j, ascending in r.  That second part is a transpose of the
// strictly lower triangle:
//   count   : per column j the number of strictly lower entries (atomics), add the row's own
//             length, scan -> f_rowptr.
//   scatter : copy the lower parts in place; push every strictly lower entry (r, j, v) into the
//             staging segment of row j through an atomic cursor (arbitrary order inside a segment).
//   sort    : order every staging segment by r (rows are distinct inside a segment) and write it
//             behind the lower part: register bitonic sort for short segments, bitmap rank for
//             long ones.
#include <algorithm>
#include <mutex>

#include "common.cuh"

using namespace spsyrk;

namespace {

constexpr size_t ALIGN = 256;
constexpr uint32_t MIRROR_CHUNK_BITS_MAX = 1u << 19;

struct MirrorWs {
    uint32_t* ucnt;    // m: strictly-lower entries per column, later reused as cursor
    uint32_t* rowtot;  // m
    uint8_t* cls;      // m
    int32_t* perm;     // m
    int32_t* blockhist;
    int64_t* offsets;
    int64_t* partials;
    int64_t* class_start_dev;
    uint32_t* err;
    int32_t* stage_row;  // nnz_l
    void* stage_val;     // nnz_l * sv
};

size_t carve(MirrorWs* w, void* ws, int64_t m, int64_t nnz_l, size_t sv) {
    char* base = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) -> void* {
        off = (off + ALIGN - 1) / ALIGN * ALIGN;
        void* p = base ? base + off : nullptr;
        off += bytes;
        return p;
    };
    const int64_t items = std::max<int64_t>(m, 1);
    const int64_t nb = bin_blocks(items);
    MirrorWs t;
    t.ucnt = (uint32_t*)take(items * 4);
    t.rowtot = (uint32_t*)take(items * 4);
    t.cls = (uint8_t*)take(items);
    t.perm = (int32_t*)take(items * 4);
    t.blockhist = (int32_t*)take(NCLASS * nb * 4);
    t.offsets = (int64_t*)take((NCLASS * nb + 1) * 8);
    t.partials = (int64_t*)take(scan_partials_count(std::max<int64_t>(items + 1, NCLASS * nb)) * 8);
    t.class_start_dev = (int64_t*)take((NCLASS + 1) * 8);
    t.err = (uint32_t*)take(4);
    t.stage_row = (int32_t*)take(std::max<int64_t>(nnz_l, 1) * 4);
    t.stage_val = take(std::max<int64_t>(nnz_l, 1) * sv);
    if (w) *w = t;
    return (off + ALIGN - 1) / ALIGN * ALIGN;
}

template <int G>
__global__ void __launch_bounds__(256) mirror_count_kernel(const int64_t* __restrict__ l_rowptr, const int32_t* __restrict__ l_colidx,
                                                           int64_t m, uint32_t* __restrict__ ucnt, uint32_t* err) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= m) return;
    const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
    for (int64_t p = p0 + gl; p < p1; p += G) {
        const int64_t j = l_colidx[p];
        if (j > r || j < 0) atomicOr(err, ERRW_UPPER);
        else if (j < r) atomicAdd(&ucnt[j], 1u);
    }
}

__global__ void mirror_rowtot_kernel(const int64_t* __restrict__ l_rowptr, const uint32_t* __restrict__ ucnt, int64_t m,
                                     uint32_t* __restrict__ rowtot) {
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < m) rowtot[r] = (uint32_t)(l_rowptr[r + 1] - l_rowptr[r]) + ucnt[r];
}

// class of a row of F by the length u of its reflected part
__global__ void mirror_class_kernel(const int64_t* __restrict__ l_rowptr, const int64_t* __restrict__ f_rowptr, int64_t m,
                                    uint8_t* __restrict__ cls) {
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= m) return;
    const int64_t u = (f_rowptr[r + 1] - f_rowptr[r]) - (l_rowptr[r + 1] - l_rowptr[r]);
    cls[r] = u <= 0 ? 0 : u <= 32 ? 1 : u <= 64 ? 2 : u <= 128 ? 3 : u <= 256 ? 4 : u <= 512 ? 5 : 7;
}

template <typename V, int G>
__global__ void __launch_bounds__(256) mirror_scatter_kernel(const int64_t* __restrict__ l_rowptr, const int32_t* __restrict__ l_colidx,
                                                             const V* __restrict__ l_vals, int64_t m,
                                                             const int64_t* __restrict__ f_rowptr, int32_t* __restrict__ f_colidx,
                                                             V* __restrict__ f_vals, uint32_t* __restrict__ cursor,
                                                             int32_t* __restrict__ stage_row, V* __restrict__ stage_val) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= m) return;
    const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
    const int64_t fb = f_rowptr[r];
    for (int64_t p = p0 + gl; p < p1; p += G) {
        const int32_t j = l_colidx[p];
        const V v = l_vals[p];
        f_colidx[fb + (p - p0)] = j;
        f_vals[fb + (p - p0)] = v;
        if (j < r) {
            const uint32_t slot = atomicAdd(&cursor[j], 1u);
            const int64_t sp = (f_rowptr[j] - l_rowptr[j]) + slot;  // segment start = reflected entries of earlier rows
            stage_row[sp] = (int32_t)r;
            stage_val[sp] = v;
        }
    }
}

// one warp per row of F whose reflected part has at most 32*R entries
template <typename V, int R, typename Key>
__global__ void __launch_bounds__(256) mirror_sort_warp_kernel(const int32_t* __restrict__ rows, int64_t nrows,
                                                               const int64_t* __restrict__ l_rowptr, const int64_t* __restrict__ f_rowptr,
                                                               const int32_t* __restrict__ stage_row, const V* __restrict__ stage_val,
                                                               int32_t* __restrict__ f_colidx, V* __restrict__ f_vals) {
    constexpr int IDXB = ilog2_ce(32 * R);
    const int lane = lane_id();
    const int64_t widx = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (widx >= nrows) return;
    const int64_t j = rows[widx];
    const int64_t lcnt = l_rowptr[j + 1] - l_rowptr[j];
    const int64_t sb = f_rowptr[j] - l_rowptr[j];
    const int64_t fb = f_rowptr[j] + lcnt;
    const uint32_t u = (uint32_t)(f_rowptr[j + 1] - fb);
    Key x[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint32_t e = r * 32 + lane;
        x[r] = e < u ? (((Key)(uint32_t)stage_row[sb + e] << IDXB) | (Key)e) : ~Key(0);
    }
    group_bitonic_sort<Key, R, 32>(x);
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint32_t q = lane * R + r;
        if (q < u) {
            f_colidx[fb + q] = (int32_t)(x[r] >> IDXB);
            f_vals[fb + q] = stage_val[sb + (uint32_t)(x[r] & (Key)(32 * R - 1))];
        }
    }
}

// one CTA per row of F with a long reflected part: bitmap rank over chunks of the row-id range (j, m)
template <typename V, int THREADS>
__global__ void __launch_bounds__(THREADS) mirror_sort_cta_kernel(const int32_t* __restrict__ rows, int64_t m, uint32_t chunk_bits,
                                                                  const int64_t* __restrict__ l_rowptr, const int64_t* __restrict__ f_rowptr,
                                                                  const int32_t* __restrict__ stage_row, const V* __restrict__ stage_val,
                                                                  int32_t* __restrict__ f_colidx, V* __restrict__ f_vals) {
    extern __shared__ uint32_t smem_u32[];
    __shared__ uint32_t scratch[33];
    const uint32_t cw = chunk_bits >> 5;
    uint32_t* bits = smem_u32;
    uint32_t* rank = smem_u32 + cw;
    const int64_t j = rows[blockIdx.x];
    const int64_t lcnt = l_rowptr[j + 1] - l_rowptr[j];
    const int64_t sb = f_rowptr[j] - l_rowptr[j];
    const int64_t fb = f_rowptr[j] + lcnt;
    const uint32_t u = (uint32_t)(f_rowptr[j + 1] - fb);
    const uint32_t per = (cw + THREADS - 1) / THREADS;
    uint32_t base = 0;
    for (int64_t c0 = j + 1; c0 < m; c0 += chunk_bits) {
        for (uint32_t w = threadIdx.x; w < cw; w += THREADS) bits[w] = 0;
        __syncthreads();
        for (uint32_t e = threadIdx.x; e < u; e += THREADS) {
            const int64_t rel = (int64_t)stage_row[sb + e] - c0;
            if (rel >= 0 && rel < (int64_t)chunk_bits) atomicOr(&bits[rel >> 5], 1u << (rel & 31));
        }
        __syncthreads();
        uint32_t s = 0;
        const uint32_t w0 = threadIdx.x * per;
        for (uint32_t w = w0; w < w0 + per && w < cw; ++w) s += __popc(bits[w]);
        uint32_t tot;
        uint32_t ex = block_exclusive_scan<uint32_t, THREADS>(s, scratch, &tot);
        for (uint32_t w = w0; w < w0 + per && w < cw; ++w) { rank[w] = ex; ex += __popc(bits[w]); }
        __syncthreads();
        for (uint32_t e = threadIdx.x; e < u; e += THREADS) {
            const int32_t r = stage_row[sb + e];
            const int64_t rel = (int64_t)r - c0;
            if (rel >= 0 && rel < (int64_t)chunk_bits) {
                const uint32_t q = base + rank[rel >> 5] + __popc(bits[rel >> 5] & ((1u << (rel & 31)) - 1u));
                f_colidx[fb + q] = r;
                f_vals[fb + q] = stage_val[sb + e];
            }
        }
        base += tot;
        __syncthreads();
    }
}

int group_width(int64_t nnz, int64_t m) {
    const double avg = m > 0 ? (double)nnz / (double)m : 0.0;
    return avg <= 4 ? 4 : avg <= 8 ? 8 : avg <= 16 ? 16 : 32;
}

template <typename V, int R, typename Key>
void launch_sort_warp(const MirrorWs& w, const int64_t* cs, int c, const int64_t* l_rowptr, const int64_t* f_rowptr,
                      int32_t* f_colidx, void* f_vals, cudaStream_t st) {
    const int64_t count = cs[c + 1] - cs[c];
    if (count <= 0) return;
    mirror_sort_warp_kernel<V, R, Key><<<(unsigned)((count * 32 + 255) / 256), 256, 0, st>>>(
        w.perm + cs[c], count, l_rowptr, f_rowptr, w.stage_row, static_cast<const V*>(w.stage_val), f_colidx, static_cast<V*>(f_vals));
    note_launches(1);
}

template <typename V, typename Key>
void launch_sort_warp_all(const MirrorWs& w, const int64_t* cs, const int64_t* l_rowptr, const int64_t* f_rowptr,
                          int32_t* f_colidx, void* f_vals, cudaStream_t st) {
    launch_sort_warp<V, 1, Key>(w, cs, 1, l_rowptr, f_rowptr, f_colidx, f_vals, st);
    launch_sort_warp<V, 2, Key>(w, cs, 2, l_rowptr, f_rowptr, f_colidx, f_vals, st);
    launch_sort_warp<V, 4, Key>(w, cs, 3, l_rowptr, f_rowptr, f_colidx, f_vals, st);
    launch_sort_warp<V, 8, Key>(w, cs, 4, l_rowptr, f_rowptr, f_colidx, f_vals, st);
    launch_sort_warp<V, 16, Key>(w, cs, 5, l_rowptr, f_rowptr, f_colidx, f_vals, st);
}

template <typename V>
spsyrk_status_t mirror_fill(const MirrorWs& w, int64_t m, int64_t nnz_l, const int64_t* l_rowptr, const int32_t* l_colidx,
                            const void* l_vals, const int64_t* f_rowptr, int32_t* f_colidx, void* f_vals, cudaStream_t st) {
    SPSYRK_CUDA_TRY(cudaMemsetAsync(w.ucnt, 0, (size_t)m * 4, st));
    const V* lv = static_cast<const V*>(l_vals);
    V* fv = static_cast<V*>(f_vals);
    V* sv = static_cast<V*>(w.stage_val);
#define SCATTER(G)                                                                                                   \
    mirror_scatter_kernel<V, G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(l_rowptr, l_colidx, lv, m, f_rowptr, \
                                                                                 f_colidx, fv, w.ucnt, w.stage_row, sv)
    switch (group_width(nnz_l, m)) {
        case 4: SCATTER(4); break;
        case 8: SCATTER(8); break;
        case 16: SCATTER(16); break;
        default: SCATTER(32); break;
    }
#undef SCATTER
    mirror_class_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(l_rowptr, f_rowptr, m, w.cls);
    note_launches(2);  // scatter + class
    SPSYRK_CUDA_TRY(bin_items(w.cls, m, w.perm, w.class_start_dev, w.blockhist, w.offsets, w.partials, st));
    int64_t cs[NCLASS + 1];
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(cs, w.class_start_dev, sizeof(cs), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    if (m <= (int64_t(1) << 22)) launch_sort_warp_all<V, uint32_t>(w, cs, l_rowptr, f_rowptr, f_colidx, f_vals, st);
    else launch_sort_warp_all<V, uint64_t>(w, cs, l_rowptr, f_rowptr, f_colidx, f_vals, st);
    const int64_t big = cs[8] - cs[7];
    if (big > 0) {
        uint32_t cb = 1024;
        while (cb < MIRROR_CHUNK_BITS_MAX && cb < (uint64_t)m) cb <<= 1;
        const size_t smem = (size_t)(cb >> 5) * 2 * sizeof(uint32_t);
        auto kern = mirror_sort_cta_kernel<V, 512>;
        SPSYRK_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        kern<<<(unsigned)big, 512, smem, st>>>(w.perm + cs[7], m, cb, l_rowptr, f_rowptr, w.stage_row, sv, f_colidx, fv);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}

}  // namespace

extern "C" spsyrk_status_t spsyrk_mirror(int64_t m, int64_t nnz_l, spsyrk_dtype_t dtype, const int64_t* d_l_rowptr,
                                         const int32_t* d_l_colidx, const void* d_l_vals, int64_t* d_f_rowptr,
                                         int32_t* d_f_colidx, void* d_f_vals, int64_t* nnz_full_out, void* d_workspace,
                                         size_t* workspace_bytes, void* cuda_stream) {
    if (!workspace_bytes || m < 0 || nnz_l < 0) return SPSYRK_ERR_INVALID_ARG;
    if (dtype != SPSYRK_F64 && dtype != SPSYRK_F32 && dtype != SPSYRK_I32) return SPSYRK_ERR_INVALID_ARG;
    if (m >= (int64_t(1) << 31) - 1) return SPSYRK_ERR_OVERFLOW;
    const size_t sv = dtype == SPSYRK_F64 ? 8 : 4;
    const size_t need = carve(nullptr, nullptr, m, nnz_l, sv);
    if (!d_workspace) {
        *workspace_bytes = need;
        return SPSYRK_OK;
    }
    if (*workspace_bytes < need) return SPSYRK_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_workspace) % ALIGN) return SPSYRK_ERR_INVALID_ARG;
    if (!d_l_rowptr || !d_f_rowptr || (nnz_l > 0 && !d_l_colidx)) return SPSYRK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    MirrorWs w;
    carve(&w, d_workspace, m, nnz_l, sv);

    if (!d_f_colidx) {  // step 2: sizes
        if (!nnz_full_out) return SPSYRK_ERR_INVALID_ARG;
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, st));
        if (m > 0) {
            SPSYRK_CUDA_TRY(cudaMemsetAsync(w.ucnt, 0, (size_t)m * 4, st));
#define COUNT(G) mirror_count_kernel<G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(d_l_rowptr, d_l_colidx, m, w.ucnt, w.err)
            switch (group_width(nnz_l, m)) {
                case 4: COUNT(4); break;
                case 8: COUNT(8); break;
                case 16: COUNT(16); break;
                default: COUNT(32); break;
            }
#undef COUNT
            mirror_rowtot_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(d_l_rowptr, w.ucnt, m, w.rowtot);
            note_launches(2);  // count + row totals
        }
        SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.rowtot, m, d_f_rowptr, w.partials, st));
        int64_t nnz = 0;
        uint32_t e = 0;
        SPSYRK_CUDA_TRY(cudaMemcpyAsync(&nnz, d_f_rowptr + m, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
        SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, w.err, 4, cudaMemcpyDeviceToHost, st));
        SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
        if (e & ERRW_UPPER) return SPSYRK_ERR_BAD_CSR;
        *nnz_full_out = nnz;
        return SPSYRK_OK;
    }
    // step 3: fill
    if (!d_f_vals || (nnz_l > 0 && !d_l_vals)) return SPSYRK_ERR_INVALID_ARG;
    if (m == 0) return SPSYRK_OK;
    switch (dtype) {
        case SPSYRK_F64: return mirror_fill<uint64_t>(w, m, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_f_rowptr, d_f_colidx, d_f_vals, st);
        default: return mirror_fill<uint32_t>(w, m, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_f_rowptr, d_f_colidx, d_f_vals, st);
    }
}


// ------------------------------------------------------------------------------------------
// Allocation-free variant of the size step of spsyrk_mirror.
//
// Some callers have no device memory to lend and may not create any: a plug-in running inside a
// host application that has claimed the whole GPU for its own memory pool, or a service loop that
// cannot afford the device-wide synchronisation a cudaMalloc / cudaFree may bring.  For them the
// scratch of this one step lives in a fixed array that is part of the library image, so the call
// needs nothing but its inputs and outputs.  The price: the array occupies its bytes on every GPU
// that loads the library until the process exits, and the problem size is capped.
// ------------------------------------------------------------------------------------------
namespace {

constexpr int64_t NOALLOC_MAX_ROWS = SPSYRK_NOALLOC_MAX_ROWS;
// strictly-lower counts (4 B per row), row totals (4 B per row), scan partials, one error word
constexpr size_t NOALLOC_UCNT_OFF = 0;
constexpr size_t NOALLOC_ROWTOT_OFF = NOALLOC_UCNT_OFF + (size_t)NOALLOC_MAX_ROWS * 4;
constexpr size_t NOALLOC_PARTIALS_OFF = NOALLOC_ROWTOT_OFF + (size_t)NOALLOC_MAX_ROWS * 4;
constexpr size_t NOALLOC_PARTIALS_BYTES = ((size_t)(NOALLOC_MAX_ROWS / SCAN_TILE) + 2) * 8;
constexpr size_t NOALLOC_ERR_OFF = (NOALLOC_PARTIALS_OFF + NOALLOC_PARTIALS_BYTES + 255) / 256 * 256;
constexpr size_t NOALLOC_BYTES = NOALLOC_ERR_OFF + 256;

// In host code this name is only a handle for the runtime, not a device address: the address is
// looked up once per device with cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
unsigned char* g_noalloc_ptr[NOALLOC_MAX_DEVICES] = {};

// device address of the scratch array on the current device (set up on the first call per device)
cudaError_t noalloc_scratch(unsigned char** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" spsyrk_status_t spsyrk_mirror_rowptr_noalloc(int64_t m, const int64_t* d_l_rowptr, const int32_t* d_l_colidx,
                                                        int64_t* d_f_rowptr, int64_t* nnz_full_out, void* cuda_stream) {
    if (m < 0 || !d_l_rowptr || !d_f_rowptr || !nnz_full_out) return SPSYRK_ERR_INVALID_ARG;
    if (m > NOALLOC_MAX_ROWS) return SPSYRK_ERR_OVERFLOW;  // beyond the fixed scratch: use spsyrk_mirror
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned char* base = nullptr;
    SPSYRK_CUDA_TRY(noalloc_scratch(&base));
    uint32_t* ucnt = reinterpret_cast<uint32_t*>(base + NOALLOC_UCNT_OFF);
    uint32_t* rowtot = reinterpret_cast<uint32_t*>(base + NOALLOC_ROWTOT_OFF);
    int64_t* partials = reinterpret_cast<int64_t*>(base + NOALLOC_PARTIALS_OFF);
    uint32_t* err = reinterpret_cast<uint32_t*>(base + NOALLOC_ERR_OFF);
    // the array keeps whatever the previous call left: clear what is accumulated into
    SPSYRK_CUDA_TRY(cudaMemsetAsync(err, 0, 4, st));
    if (m > 0) {
        SPSYRK_CUDA_TRY(cudaMemsetAsync(ucnt, 0, (size_t)m * 4, st));
        // row lengths are not known on the host here, so the widest lane grouping is used
        mirror_count_kernel<32><<<(unsigned)((m * 32 + 255) / 256), 256, 0, st>>>(d_l_rowptr, d_l_colidx, m, ucnt, err);
        mirror_rowtot_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(d_l_rowptr, ucnt, m, rowtot);
        note_launches(2);
    }
    SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(rowtot, m, d_f_rowptr, partials, st));
    int64_t nnz = 0;
    uint32_t e = 0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&nnz, d_f_rowptr + m, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, err, 4, cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    if (e & ERRW_UPPER) return SPSYRK_ERR_BAD_CSR;
    *nnz_full_out = nnz;
    return SPSYRK_OK;
}
