// Row and column permutation of a CSR matrix: row i of A becomes row rperm[i] of B and column k
// becomes column cperm[k].  With a square A and cperm == rperm this is the symmetric random
// permutation used to balance the load (Section III-A; the load-balance study of Section V).
//
// B's entries are A's entries sorted by (new row, new column).  That is a stable
// least-significant-digit radix sort: first by the new column id, then by the new row id; the
// position of an entry in the final order is its position in B, so the last pass writes B's
// column ids and values in place.  Row pointers come from the permuted row lengths.  When the
// columns stay, rows keep their inner order and the column passes are skipped.
#include <algorithm>

#include "radix.cuh"

using namespace spsyrk;

namespace {

constexpr size_t ALIGN = 256;
constexpr int PERMUTE_RADIX_BITS = 8;

struct PermuteWs {
    uint32_t* len;   // m: lengths of B's rows
    uint32_t* seen;  // max(m, n): permutation check
    int64_t* partials;
    uint32_t* err;
    uint32_t *key_a, *pay_a, *key_b, *pay_b;  // nnz each
    void *val_a, *val_b;
    uint32_t* hist;
    int64_t* offsets;
};

size_t carve(PermuteWs* w, void* ws, int64_t m, int64_t n, int64_t nnz, size_t sv) {
    char* base = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) -> void* {
        off = (off + ALIGN - 1) / ALIGN * ALIGN;
        void* p = base ? base + off : nullptr;
        off += bytes;
        return p;
    };
    const int64_t items = std::max<int64_t>(std::max(m, n), 1);
    const int64_t ne = std::max<int64_t>(nnz, 1);
    const int64_t hist_n = (int64_t)(1 << PERMUTE_RADIX_BITS) * std::max<int64_t>(radix_tiles(nnz), 1);
    PermuteWs t;
    t.len = (uint32_t*)take(items * 4);
    t.seen = (uint32_t*)take(items * 4);
    t.partials = (int64_t*)take(scan_partials_count(std::max<int64_t>(items + 1, hist_n)) * 8);
    t.err = (uint32_t*)take(4);
    t.key_a = (uint32_t*)take(ne * 4);
    t.pay_a = (uint32_t*)take(ne * 4);
    t.key_b = (uint32_t*)take(ne * 4);
    t.pay_b = (uint32_t*)take(ne * 4);
    t.val_a = take(ne * sv);
    t.val_b = take(ne * sv);
    t.hist = (uint32_t*)take(hist_n * 4);
    t.offsets = (int64_t*)take((hist_n + 1) * 8);
    if (w) *w = t;
    return (off + ALIGN - 1) / ALIGN * ALIGN;
}

// every value of perm[0, count) must lie in [0, count) and occur once
__global__ void check_permutation_kernel(const int32_t* __restrict__ perm, int64_t count, uint32_t* __restrict__ seen, uint32_t* err) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const int64_t v = perm[i];
    if (v < 0 || v >= count) atomicOr(err, ERRW_BAD_COL);
    else if (atomicExch(&seen[v], 1u) != 0u) atomicOr(err, ERRW_BAD_COL);
}

// Also the row-pointer checks of the whole call: rowptr[0] = 0, rowptr[m] = nnz, non-decreasing, inside [0, nnz] -
// the expand kernel indexes arrays of nnz entries with these positions.
__global__ void permuted_lengths_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ rperm, int64_t m, int64_t nnz,
                                        uint32_t* __restrict__ len, uint32_t* err) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= m) return;
    const int64_t a = rowptr[i], b = rowptr[i + 1];
    const int64_t l = b - a;
    const int64_t r = rperm[i];
    if (i == 0 && (rowptr[0] != 0 || rowptr[m] != nnz)) atomicOr(err, ERRW_BAD_ROWPTR);
    if (l < 0 || a < 0 || b > nnz) atomicOr(err, ERRW_BAD_ROWPTR);
    else if (r >= 0 && r < m) len[r] = (uint32_t)l;
}

// G lanes per row: the (new column, new row) pair of every entry
template <int G>
__global__ void __launch_bounds__(256) permute_expand_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ colidx,
                                                             const int32_t* __restrict__ rperm, const int32_t* __restrict__ cperm,
                                                             int64_t m, int64_t n, uint32_t* __restrict__ newcol,
                                                             uint32_t* __restrict__ newrow, uint32_t* err) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= m) return;
    const uint32_t nr = (uint32_t)rperm[r];
    for (int64_t p = rowptr[r] + gl; p < rowptr[r + 1]; p += G) {
        const int64_t c = colidx[p];
        if (c < 0 || c >= n) {
            atomicOr(err, ERRW_BAD_COL);
            newcol[p] = 0;
        } else {
            newcol[p] = cperm ? (uint32_t)cperm[c] : (uint32_t)c;
        }
        newrow[p] = nr;
    }
}

// last pass: position in the sorted order == position in B
template <typename V>
struct EmitPermuted {
    int32_t* b_colidx;
    V* b_vals;
    __device__ __forceinline__ void operator()(int64_t dest, uint32_t /*new row*/, uint32_t newcol, V val) const {
        b_colidx[dest] = (int32_t)newcol;
        b_vals[dest] = val;
    }
};

int group_width(int64_t nnz, int64_t m) {
    const double avg = m > 0 ? (double)nnz / (double)m : 0.0;
    return avg <= 4 ? 4 : avg <= 8 ? 8 : avg <= 16 ? 16 : 32;
}

template <typename V>
spsyrk_status_t permute_sort(const PermuteWs& w, int64_t m, int64_t n, int64_t nnz, const void* vals, bool sort_columns,
                             int32_t* b_colidx, void* b_vals, cudaStream_t st) {
    constexpr int BITS = PERMUTE_RADIX_BITS;
    // after the expand: key_a = new column, pay_a = new row
    const uint32_t* key = w.key_a;
    const uint32_t* pay = w.pay_a;
    const V* val = static_cast<const V*>(vals);
    bool in_a = true;  // which buffer pair holds (key, pay)
    auto other_key = [&]() { return in_a ? w.key_b : w.key_a; };
    auto other_pay = [&]() { return in_a ? w.pay_b : w.pay_a; };
    auto other_val = [&]() { return static_cast<V*>(in_a ? w.val_b : w.val_a); };
    if (sort_columns) {
        const int npass = (bits_for((uint64_t)std::max<int64_t>(n - 1, 1)) + BITS - 1) / BITS;
        for (int p = 0; p < npass; ++p) {
            EmitArrays<V> emit{other_key(), other_pay(), other_val()};
            SPSYRK_CUDA_TRY((radix_pass<BITS, V>(key, pay, val, nnz, p * BITS, w.hist, w.offsets, w.partials, emit, w.err, st)));
            key = emit.keys; pay = emit.pa; val = emit.pb;
            in_a = !in_a;
        }
    }
    // now sort by the new row: the row array becomes the key, the column array the payload
    std::swap(key, pay);
    const int npass = (bits_for((uint64_t)std::max<int64_t>(m - 1, 1)) + BITS - 1) / BITS;
    for (int p = 0; p < npass; ++p) {
        if (p == npass - 1) {
            EmitPermuted<V> emit{b_colidx, static_cast<V*>(b_vals)};
            SPSYRK_CUDA_TRY((radix_pass<BITS, V>(key, pay, val, nnz, p * BITS, w.hist, w.offsets, w.partials, emit, w.err, st)));
        } else {
            // the roles of the two uint32 buffers of a pair are swapped with the arrays
            uint32_t* dk = in_a ? w.pay_b : w.pay_a;
            uint32_t* dp = in_a ? w.key_b : w.key_a;
            EmitArrays<V> emit{dk, dp, other_val()};
            SPSYRK_CUDA_TRY((radix_pass<BITS, V>(key, pay, val, nnz, p * BITS, w.hist, w.offsets, w.partials, emit, w.err, st)));
            key = dk; pay = dp; val = emit.pb;
            in_a = !in_a;
        }
    }
    return SPSYRK_OK;
}

}  // namespace

extern "C" spsyrk_status_t spsyrk_permute(int64_t m, int64_t n, int64_t nnz, spsyrk_dtype_t dtype, const int64_t* d_rowptr,
                                          const int32_t* d_colidx, const void* d_vals, const int32_t* d_rperm,
                                          const int32_t* d_cperm, int64_t* d_b_rowptr, int32_t* d_b_colidx, void* d_b_vals,
                                          void* d_workspace, size_t* workspace_bytes, void* cuda_stream) {
    if (!workspace_bytes || m < 0 || n < 0 || nnz < 0) return SPSYRK_ERR_INVALID_ARG;
    if (dtype != SPSYRK_F64 && dtype != SPSYRK_F32 && dtype != SPSYRK_I32) return SPSYRK_ERR_INVALID_ARG;
    if (m >= (int64_t(1) << 31) - 1 || n >= (int64_t(1) << 31) - 1) return SPSYRK_ERR_OVERFLOW;
    const size_t sv = dtype == SPSYRK_F64 ? 8 : 4;
    const size_t need = carve(nullptr, nullptr, m, n, nnz, sv);
    if (!d_workspace) {
        *workspace_bytes = need;
        return SPSYRK_OK;
    }
    if (*workspace_bytes < need) return SPSYRK_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_workspace) % ALIGN) return SPSYRK_ERR_INVALID_ARG;
    if (!d_rowptr || !d_b_rowptr || (m > 0 && !d_rperm)) return SPSYRK_ERR_INVALID_ARG;
    if (nnz > 0 && (!d_colidx || !d_vals || !d_b_colidx || !d_b_vals)) return SPSYRK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    PermuteWs w;
    carve(&w, d_workspace, m, n, nnz, sv);

    SPSYRK_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, st));
    if (m > 0) {
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.seen, 0, (size_t)m * 4, st));
        check_permutation_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(d_rperm, m, w.seen, w.err);
        note_launches(1);
    }
    if (d_cperm && n > 0) {
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.seen, 0, (size_t)n * 4, st));
        check_permutation_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(d_cperm, n, w.seen, w.err);
        note_launches(1);
    }
    if (m > 0) {
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.len, 0, (size_t)m * 4, st));
        permuted_lengths_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(d_rowptr, d_rperm, m, nnz, w.len, w.err);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.len, m, d_b_rowptr, w.partials, st));
    // a bad map or row pointer must be known before entries are moved by it
    uint32_t e = 0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, w.err, 4, cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    if (e & ERRW_BAD_ROWPTR) return SPSYRK_ERR_BAD_CSR;
    if (e) return SPSYRK_ERR_INVALID_ARG;
    if (m == 0 || nnz == 0) return SPSYRK_OK;

#define EXPAND(G)                                                                                                        \
    permute_expand_kernel<G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(d_rowptr, d_colidx, d_rperm, d_cperm, m, n, \
                                                                              w.key_a, w.pay_a, w.err)
    switch (group_width(nnz, m)) {
        case 4: EXPAND(4); break;
        case 8: EXPAND(8); break;
        case 16: EXPAND(16); break;
        default: EXPAND(32); break;
    }
#undef EXPAND
    note_launches(1);
    spsyrk_status_t s = dtype == SPSYRK_F64
                            ? permute_sort<uint64_t>(w, m, n, nnz, d_vals, d_cperm != nullptr, d_b_colidx, d_b_vals, st)
                            : permute_sort<uint32_t>(w, m, n, nnz, d_vals, d_cperm != nullptr, d_b_colidx, d_b_vals, st);
    if (s != SPSYRK_OK) return s;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, w.err, 4, cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    if (e) return SPSYRK_ERR_BAD_CSR;  // a column id outside [0, n)
    return SPSYRK_OK;
}
