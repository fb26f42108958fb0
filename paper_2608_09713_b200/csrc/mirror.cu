// Step a7: F = C_L + C_L^T - D, the full symmetric CSR from the stored lower triangle.
//
// Row j of F = row j of C_L (columns <= j) followed by the reflected entries (r, c_rj) of the
// later rows r > j that store column j, ascending in r.  That second part is a transpose of the
// strictly lower triangle, done as a stable radix sort of the entries by column id:
//   sizes   : rows are ascending, so a row stores its diagonal iff its last entry is the diagonal and
//             holds an entry above the diagonal iff its last entry is one:
//             nnz(F) = 2 nnz(C_L) - #diagonals.
//   expand  : an explicit (key, row) pair per entry, the key being the column id, or m for a
//             diagonal entry (and for an entry that should not be there) so that it sorts past the end.
//   sort    : stable LSD radix passes over (key, row, value); entries enter in ascending row order,
//             so every column's segment comes out ascending in r.  The last pass writes straight
//             into F: the s-th strictly lower entry in sorted order, of column j, lands at
//             s + l_rowptr[j + 1].  It also records where each column's segment starts and ends
//             (equal keys are adjacent in the last pass: one atomic at each end of a run), which is
//             the number of reflected entries of row j.
//   rows    : row lengths of F, scan -> f_rowptr, then the lower parts are copied into place.
#include <algorithm>
#include <mutex>

#include "mirror_rec.cuh"

using namespace spsyrk;

namespace {

constexpr size_t ALIGN = 256;

constexpr int MIRROR_RADIX_BITS = 8;

struct MirrorWs {
    uint32_t* diagf;   // m: 1 where the row stores its diagonal entry
    uint32_t* rowtot;  // m
    int64_t* dcount;   // m + 1: diagonal entries of the rows before (exclusive prefix sums of diagf)
    int64_t* fbase;    // m: l_rowptr[j + 1] - dcount[j + 1]
    // 8-byte values: the record buffer the last pass reads (nnz_l records), the tail of the buffer that lives in
    // F's value array, and digit bytes for inputs too small to keep them in F's column array
    MirrorRec *rec_keep, *rec_tail;
    uint8_t* dig_small;
    int32_t* tile_rows;  // 2 per tile
    unsigned long long* seg_start;  // m: first sorted position of column j's strictly lower entries
    unsigned long long* seg_end;    // m: one past the last
    int64_t* partials;
    uint32_t* err;
    // radix sort buffers (nnz_l entries each); buffer B's key and row arrays double as the expanded input
    uint32_t *key_a, *row_a, *key_b, *row_b;
    void *val_a, *val_b;
    uint32_t* hist;
    int64_t* offsets;
};

// Scratch inside the output.  Until the last pass writes it, F's memory is free, and the sort needs two record
// buffers of 16 nnz_l bytes each.  The buffer the last pass reads must lie outside F; the other one lives in F's
// value array, which holds 8 (2 nnz_l - D) bytes with D <= min(m, nnz_l) diagonal entries: the first
// nnz_l - ceil(min(m, nnz_l) / 2) records always fit, the few remaining ones go to a tail in the workspace.
// The digit bytes (two buffers of nnz_l bytes) live in F's column array (4 (2 nnz_l - D) bytes), which is free
// whenever a histogram reads them: the last pass, the first to write that array, starts after its histogram.
inline int mirror_passes_4byte(int64_t m) { return (bits_for((uint64_t)m) + MIRROR_RADIX_BITS - 1) / MIRROR_RADIX_BITS; }  // keys run from 0 to m
inline int64_t mirror_tail_records(int64_t m, int64_t nnz_l) { return (std::min(m, nnz_l) + 1) / 2; }
constexpr int64_t MIRROR_DIG_SMALL = 32;  // inputs of fewer entries than this keep their digit bytes in the workspace

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
    const int64_t ne = std::max<int64_t>(nnz_l, 1);
    const int64_t hist_n = (int64_t)(1 << MIRROR_RADIX_BITS) * std::max<int64_t>(sv == 8 ? mirror_groups(nnz_l) : radix_tiles(nnz_l), 1);
    MirrorWs t;
    t.diagf = (uint32_t*)take(items * 4);
    t.rowtot = (uint32_t*)take(items * 4);
    t.dcount = (int64_t*)take((items + 1) * 8);
    t.fbase = (int64_t*)take(items * 8);
    t.seg_start = (unsigned long long*)take(items * 8);
    t.seg_end = (unsigned long long*)take(items * 8);
    t.partials = (int64_t*)take(scan_partials_count(std::max<int64_t>(items + 1, hist_n)) * 8);
    t.err = (uint32_t*)take(8);  // [0] error word, [1] number of diagonal entries
    t.key_a = t.row_a = t.key_b = t.row_b = nullptr;
    t.val_a = t.val_b = nullptr;
    t.rec_keep = t.rec_tail = nullptr;
    t.dig_small = nullptr;
    t.tile_rows = nullptr;
    if (sv == 8) {
        t.rec_keep = (MirrorRec*)take(ne * sizeof(MirrorRec));
        t.rec_tail = (MirrorRec*)take((mirror_tail_records(m, nnz_l) + 1) * sizeof(MirrorRec));
        t.dig_small = (uint8_t*)take(2 * MIRROR_DIG_SMALL);
        t.tile_rows = (int32_t*)take(2 * std::max<int64_t>(mirror_tiles(nnz_l), 1) * 4);
    } else {
        // The buffer set the last pass does not read keeps its keys in F's column array and its values in F's
        // value array (4 (2 nnz_l - D) >= 4 nnz_l bytes each, free until the last pass); only its row ids need
        // workspace.  Passes alternate A, B, A, ...: the last one reads B when the number of passes is odd.
        const bool a_in_f = (mirror_passes_4byte(m) % 2) == 1;
        t.row_a = (uint32_t*)take(ne * 4);
        t.row_b = (uint32_t*)take(ne * 4);
        if (a_in_f) {
            t.key_b = (uint32_t*)take(ne * 4);
            t.val_b = take(ne * sv);
        } else {
            t.key_a = (uint32_t*)take(ne * 4);
            t.val_a = take(ne * sv);
        }
    }
    t.hist = (uint32_t*)take(hist_n * 4);
    t.offsets = (int64_t*)take((hist_n + 1) * 8);
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
    if (p1 < p0 && gl == 0) atomicOr(err, ERRW_BAD_ROWPTR);  // the row total below would wrap
    constexpr int UNR = 4;
    for (int64_t p = p0 + gl; p < p1; p += UNR * G) {
        int64_t j[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) j[u] = p + u * G < p1 ? (int64_t)l_colidx[p + u * G] : r;  // r: neither counted nor an error
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            if (j[u] > r || j[u] < 0) atomicOr(err, ERRW_UPPER);
            else if (j[u] < r) atomicAdd(&ucnt[j[u]], 1u);
        }
    }
}

__global__ void mirror_rowtot_kernel(const int64_t* __restrict__ l_rowptr, const uint32_t* __restrict__ ucnt, int64_t m,
                                     uint32_t* __restrict__ rowtot) {
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < m) rowtot[r] = (uint32_t)(l_rowptr[r + 1] - l_rowptr[r]) + ucnt[r];
}

// one thread per row: the last entry tells whether the row stores its diagonal and whether it reaches above it
// (rows are ascending); err[1] counts the diagonals
__global__ void mirror_last_entry_kernel(const int64_t* __restrict__ l_rowptr, const int32_t* __restrict__ l_colidx, int64_t m,
                                         uint32_t* err) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    bool diag = false;
    if (r < m) {
        const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
        if (p1 < p0) {
            atomicOr(err, ERRW_BAD_ROWPTR);
        } else if (p1 > p0) {
            const int64_t last = l_colidx[p1 - 1], first = l_colidx[p0];
            if (last > r || first < 0) atomicOr(err, ERRW_UPPER);
            else diag = last == r;
        }
    }
    // one atomic per warp: nearly every row of a product stores its diagonal
    const unsigned votes = __ballot_sync(FULL_MASK, diag);
    if (lane_id() == 0 && votes) atomicAdd(err + 1, (uint32_t)__popc(votes));
}

// G lanes per row: the explicit (key, row) pair of every entry
template <int G>
__global__ void __launch_bounds__(256) mirror_expand_kernel(const int64_t* __restrict__ l_rowptr, const int32_t* __restrict__ l_colidx,
                                                            int64_t m, uint32_t* __restrict__ key0, uint32_t* __restrict__ row0,
                                                            uint32_t* err) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= m) return;
    const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
    constexpr int UNR = 4;  // loads of several steps are issued before the first store
    for (int64_t p = p0 + gl; p < p1; p += UNR * G) {
        int64_t j[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) j[u] = p + u * G < p1 ? (int64_t)l_colidx[p + u * G] : r;
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int64_t pp = p + u * G;
            if (pp < p1) {
                // an entry outside the lower triangle (rows that are not ascending can hide one from the size
                // step) is keyed like a diagonal: it takes no part in the reflection
                if (j[u] > r || j[u] < 0) atomicOr(err, ERRW_UPPER);
                key0[pp] = (j[u] >= r || j[u] < 0) ? (uint32_t)m : (uint32_t)j[u];
                row0[pp] = (uint32_t)r;
            }
        }
    }
}

// G lanes per row: the lower part of row r of F is row r of C_L
template <typename V, int G>
__global__ void __launch_bounds__(256) mirror_copy_lower_kernel(const int64_t* __restrict__ l_rowptr, const int32_t* __restrict__ l_colidx,
                                                                const V* __restrict__ l_vals, int64_t m,
                                                                const int64_t* __restrict__ f_rowptr, int32_t* __restrict__ f_colidx,
                                                                V* __restrict__ f_vals) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= m) return;
    const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
    const int64_t fb = f_rowptr[r] - p0;
    constexpr int UNR = 4;
    for (int64_t p = p0 + gl; p < p1; p += UNR * G) {
        int32_t j[UNR];
        V v[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int64_t pp = p + u * G;
            if (pp < p1) {
                j[u] = l_colidx[pp];
                v[u] = l_vals[pp];
            }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int64_t pp = p + u * G;
            if (pp < p1) {
                f_colidx[fb + pp] = j[u];
                f_vals[fb + pp] = v[u];
            }
        }
    }
}

// row lengths of F: the row's own entries plus the length of its column's sorted segment
__global__ void mirror_rowlen_kernel(const int64_t* __restrict__ l_rowptr, const unsigned long long* __restrict__ seg_start,
                                     const unsigned long long* __restrict__ seg_end, int64_t m, uint32_t* __restrict__ rowtot) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= m) return;
    const unsigned long long s = seg_start[r], e = seg_end[r];
    rowtot[r] = (uint32_t)(l_rowptr[r + 1] - l_rowptr[r]) + (e > s ? (uint32_t)(e - s) : 0u);
}

template <typename V>
struct EmitMirrorFinal {
    static constexpr bool NEIGHBOURS = true;
    const int64_t* l_rowptr;
    int32_t* f_colidx;
    V* f_vals;
    unsigned long long* seg_start;
    unsigned long long* seg_end;
    uint32_t m;
    __device__ __forceinline__ void operator()(int64_t dest, uint32_t key, uint32_t row, V val, uint32_t prev, uint32_t next) const {
        if (key < m) {  // diagonal entries were keyed m and are dropped here
            const int64_t pos = dest + l_rowptr[key + 1];
            f_colidx[pos] = (int32_t)row;
            f_vals[pos] = val;
            // ends of a run of one key inside the tile; a segment that spans tiles settles through min / max
            if (prev != key) atomicMin(&seg_start[key], (unsigned long long)dest);
            if (next != key) atomicMax(&seg_end[key], (unsigned long long)dest + 1ull);
        }
    }
};

int group_width(int64_t nnz, int64_t m) {
    const double avg = m > 0 ? (double)nnz / (double)m : 0.0;
    return avg <= 4 ? 4 : avg <= 8 ? 8 : avg <= 16 ? 16 : 32;
}

template <typename V>
spsyrk_status_t mirror_fill(const MirrorWs& ws, int64_t m, int64_t nnz_l, const int64_t* l_rowptr, const int32_t* l_colidx,
                            const void* l_vals, int64_t* f_rowptr, int32_t* f_colidx, void* f_vals, cudaStream_t st) {
    constexpr int BITS = MIRROR_RADIX_BITS;
    MirrorWs w = ws;
    // the buffer set without keys and values of its own keeps them in F's arrays (see carve)
    if (!w.key_a) { w.key_a = reinterpret_cast<uint32_t*>(f_colidx); w.val_a = f_vals; }
    if (!w.key_b) { w.key_b = reinterpret_cast<uint32_t*>(f_colidx); w.val_b = f_vals; }
    const V* lv = static_cast<const V*>(l_vals);
    V* fv = static_cast<V*>(f_vals);
    const int g = group_width(nnz_l, m);
    if (m > 0) {
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.seg_start, 0xff, (size_t)m * 8, st));
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.seg_end, 0, (size_t)m * 8, st));
    }
    if (m > 0 && nnz_l > 0) {
#define EXPAND(G) mirror_expand_kernel<G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(l_rowptr, l_colidx, m, w.key_b, w.row_b, w.err)
        switch (g) {
            case 4: EXPAND(4); break;
            case 8: EXPAND(8); break;
            case 16: EXPAND(16); break;
            default: EXPAND(32); break;
        }
#undef EXPAND
        note_launches(1);
        const int npass = mirror_passes_4byte(m);
        const uint32_t* src_key = w.key_b;
        const uint32_t* src_row = w.row_b;
        const V* src_val = lv;
        for (int p = 0; p < npass; ++p) {
            const bool to_a = (p % 2) == 0;
            uint32_t* dst_key = to_a ? w.key_a : w.key_b;
            uint32_t* dst_row = to_a ? w.row_a : w.row_b;
            V* dst_val = static_cast<V*>(to_a ? w.val_a : w.val_b);
            if (p == npass - 1) {
                EmitMirrorFinal<V> emit{l_rowptr, f_colidx, fv, w.seg_start, w.seg_end, (uint32_t)m};
                SPSYRK_CUDA_TRY((radix_pass<BITS, V>(src_key, src_row, src_val, nnz_l, p * BITS, w.hist, w.offsets, w.partials, emit, w.err, st)));
            } else {
                EmitArrays<V> emit{dst_key, dst_row, dst_val};
                SPSYRK_CUDA_TRY((radix_pass<BITS, V>(src_key, src_row, src_val, nnz_l, p * BITS, w.hist, w.offsets, w.partials, emit, w.err, st)));
            }
            src_key = dst_key;
            src_row = dst_row;
            src_val = dst_val;
        }
    }
    // row pointers of F, then the lower parts
    if (m > 0) {
        mirror_rowlen_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(l_rowptr, w.seg_start, w.seg_end, m, w.rowtot);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.rowtot, m, f_rowptr, w.partials, st));
    if (m > 0 && nnz_l > 0) {
#define COPY(G) \
    mirror_copy_lower_kernel<V, G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(l_rowptr, l_colidx, lv, m, f_rowptr, f_colidx, fv)
        switch (g) {
            case 4: COPY(4); break;
            case 8: COPY(8); break;
            case 16: COPY(16); break;
            default: COPY(32); break;
        }
#undef COPY
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(cudaGetLastError());
#ifdef SPSYRK_CHECKED
    {
        uint32_t e = 0;  // the bounds-checked build reports a skipped access at once (synchronises)
        SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, w.err, 4, cudaMemcpyDeviceToHost, st));
        SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
        if (e & ERRW_INTERNAL) return SPSYRK_ERR_INTERNAL;
    }
#endif
    return SPSYRK_OK;
}

// 1 where row r stores its diagonal entry (rows are ascending: it is the last entry)
__global__ void mirror_diag_flag_kernel(const int64_t* __restrict__ l_rowptr, const int32_t* __restrict__ l_colidx, int64_t m,
                                        uint32_t* __restrict__ diagf) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= m) return;
    const int64_t p0 = l_rowptr[r], p1 = l_rowptr[r + 1];
    diagf[r] = (p1 > p0 && (int64_t)l_colidx[p1 - 1] == r) ? 1u : 0u;
}

__global__ void mirror_fbase_kernel(const int64_t* __restrict__ l_rowptr, const int64_t* __restrict__ dcount, int64_t m,
                                    int64_t* __restrict__ fbase) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < m) fbase[j] = l_rowptr[j + 1] - dcount[j + 1];
}

// row lengths of F when the sorted segments include the diagonal entries
__global__ void mirror_rowlen_diag_kernel(const int64_t* __restrict__ l_rowptr, const unsigned long long* __restrict__ seg_start,
                                          const unsigned long long* __restrict__ seg_end, const uint32_t* __restrict__ diagf, int64_t m,
                                          uint32_t* __restrict__ rowtot) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= m) return;
    const unsigned long long s = seg_start[r], e = seg_end[r];
    const uint32_t seg = e > s ? (uint32_t)(e - s) : 0u;
    rowtot[r] = (uint32_t)(l_rowptr[r + 1] - l_rowptr[r]) + (seg >= diagf[r] ? seg - diagf[r] : 0u);
}

template <bool FROM_CSR, bool FINAL>
cudaError_t launch_mirror_pass(const MirrorPassArgs& a, int64_t n, int shift, const int64_t* offsets, int64_t nt, cudaStream_t st) {
    constexpr int BITS = MIRROR_RADIX_BITS;
    auto kern = mirror_pass_kernel<BITS, FROM_CSR, FINAL>;
    const size_t smem = MirrorPassSmem<BITS>::bytes();
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)nt, MR_THREADS, smem, st>>>(a, n, shift, offsets, nt);
    note_launches(1);
    return cudaGetLastError();
}

// Measurement aid: CUDA events around every radix pass (histogram + scan + scatter) of the last record-based fill.
constexpr int MIRROR_MAX_PASSES = 4;
bool g_mirror_timing = false;
cudaEvent_t g_mirror_ev[MIRROR_MAX_PASSES + 1];
int g_mirror_passes = 0;

// 8-byte values: records, the first pass straight from C_L
spsyrk_status_t mirror_fill_rec(const MirrorWs& w, int64_t m, int64_t nnz_l, const int64_t* l_rowptr, const int32_t* l_colidx,
                                const void* l_vals, int64_t* f_rowptr, int32_t* f_colidx, void* f_vals, cudaStream_t st) {
    constexpr int BITS = MIRROR_RADIX_BITS;
    constexpr int NB = 1 << BITS;
    const uint64_t* lv = static_cast<const uint64_t*>(l_vals);
    uint64_t* fv = static_cast<uint64_t*>(f_vals);
    const int g = group_width(nnz_l, m);
    // F's arrays hold records and digit bytes during the sort: both must take 16-byte accesses
    if (nnz_l > 0 && ((reinterpret_cast<uintptr_t>(f_vals) | reinterpret_cast<uintptr_t>(f_colidx)) & 15u)) return SPSYRK_ERR_INVALID_ARG;
    if (m > 0) {
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.seg_start, 0xff, (size_t)m * 8, st));
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.seg_end, 0, (size_t)m * 8, st));
        mirror_diag_flag_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(l_rowptr, l_colidx, m, w.diagf);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.diagf, m, w.dcount, w.partials, st));
    if (m > 0 && nnz_l > 0) {
        mirror_fbase_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(l_rowptr, w.dcount, m, w.fbase);
        note_launches(1);
        const int npass = (bits_for((uint64_t)(m - 1 > 0 ? m - 1 : 1)) + BITS - 1) / BITS;  // keys are column ids below m
        const int64_t nt = mirror_groups(nnz_l);  // histogram columns and CTAs of a pass
        const int64_t ntr = mirror_tiles(nnz_l);
        mirror_tile_rows_kernel<<<(unsigned)((2 * ntr + 255) / 256), 256, 0, st>>>(l_rowptr, m, nnz_l, ntr, w.tile_rows);
        note_launches(1);
        MirrorPassArgs a{};
        a.l_rowptr = l_rowptr; a.l_colidx = l_colidx; a.l_vals = lv; a.m = m; a.tile_rows = w.tile_rows;
        a.fbase = w.fbase; a.f_colidx = f_colidx; a.f_vals = fv; a.seg_start = w.seg_start; a.seg_end = w.seg_end;
        a.dtotal = w.dcount + m; a.err = w.err;
        g_mirror_passes = 0;
        // buffers: pass p writes records X[p] and digits Y[p]; X[npass - 2] is the one the last pass reads
        MirrorRec* const alias = reinterpret_cast<MirrorRec*>(fv);
        const int64_t alias_split = nnz_l - mirror_tail_records(m, nnz_l);
        const int64_t dig_stride = (nnz_l + 15) / 16 * 16;
        uint8_t* const dig0 = nnz_l < MIRROR_DIG_SMALL ? w.dig_small : reinterpret_cast<uint8_t*>(f_colidx);
        uint8_t* const dig1 = nnz_l < MIRROR_DIG_SMALL ? w.dig_small + MIRROR_DIG_SMALL : dig0 + dig_stride;
        auto in_keep = [&](int p) { return ((npass - 2 - p) % 2) == 0; };  // does pass p write the workspace buffer?
        for (int p = 0; p < npass; ++p) {
            const bool first = p == 0, last = p == npass - 1;
            if (g_mirror_timing && p < MIRROR_MAX_PASSES) cudaEventRecord(g_mirror_ev[p], st);
            const unsigned hb = (unsigned)((nt + MR_HIST_TILES - 1) / MR_HIST_TILES);
            if (first) mirror_hist_key_kernel<BITS><<<hb, MR_THREADS, 0, st>>>(reinterpret_cast<const uint32_t*>(l_colidx), nnz_l, 0, w.hist, nt);
            else radix_hist_u8_kernel<BITS><<<hb, MR_THREADS, 0, st>>>(((p - 1) % 2) == 0 ? dig0 : dig1, nnz_l, w.hist, nt);
            note_launches(1);
            SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.hist, (int64_t)NB * nt, w.offsets, w.partials, st));
            const bool src_keep = !first && in_keep(p - 1), dst_keep = in_keep(p);
            a.src = src_keep ? w.rec_keep : alias;
            a.src_tail = w.rec_tail;
            a.src_split = src_keep ? nnz_l : alias_split;
            a.dst = dst_keep ? w.rec_keep : alias;
            a.dst_tail = w.rec_tail;
            a.dst_split = dst_keep ? nnz_l : alias_split;
            a.next_digit = (p % 2) == 0 ? dig0 : dig1;
            cudaError_t e;
            if (first && last) e = launch_mirror_pass<true, true>(a, nnz_l, p * BITS, w.offsets, nt, st);
            else if (first) e = launch_mirror_pass<true, false>(a, nnz_l, p * BITS, w.offsets, nt, st);
            else if (last) e = launch_mirror_pass<false, true>(a, nnz_l, p * BITS, w.offsets, nt, st);
            else e = launch_mirror_pass<false, false>(a, nnz_l, p * BITS, w.offsets, nt, st);
            SPSYRK_CUDA_TRY(e);
            if (g_mirror_timing && p < MIRROR_MAX_PASSES) {
                cudaEventRecord(g_mirror_ev[p + 1], st);
                g_mirror_passes = p + 1;
            }
        }
    }
    if (m > 0) {
        mirror_rowlen_diag_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(l_rowptr, w.seg_start, w.seg_end, w.diagf, m, w.rowtot);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(w.rowtot, m, f_rowptr, w.partials, st));
    if (m > 0 && nnz_l > 0) {
#define COPY(G) \
    mirror_copy_lower_kernel<uint64_t, G><<<(unsigned)((m * G + 255) / 256), 256, 0, st>>>(l_rowptr, l_colidx, lv, m, f_rowptr, f_colidx, fv)
        switch (g) {
            case 4: COPY(4); break;
            case 8: COPY(8); break;
            case 16: COPY(16); break;
            default: COPY(32); break;
        }
#undef COPY
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(cudaGetLastError());
#ifdef SPSYRK_CHECKED
    {
        uint32_t e = 0;  // the bounds-checked build reports a skipped access at once (synchronises)
        SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, w.err, 4, cudaMemcpyDeviceToHost, st));
        SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
        if (e & ERRW_INTERNAL) return SPSYRK_ERR_INTERNAL;
    }
#endif
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

    if (!d_f_colidx) {  // step 2: checks and nnz(F)
        if (!nnz_full_out) return SPSYRK_ERR_INVALID_ARG;
        SPSYRK_CUDA_TRY(cudaMemsetAsync(w.err, 0, 8, st));
        if (m > 0) {
            mirror_last_entry_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(d_l_rowptr, d_l_colidx, m, w.err);
            note_launches(1);
        }
        uint32_t e[2] = {0, 0};
        SPSYRK_CUDA_TRY(cudaMemcpyAsync(e, w.err, 8, cudaMemcpyDeviceToHost, st));
        SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
        if (e[0]) return SPSYRK_ERR_BAD_CSR;
        *nnz_full_out = 2 * nnz_l - (int64_t)e[1];
        return SPSYRK_OK;
    }
    // step 3: fill
    if (!d_f_vals || (nnz_l > 0 && !d_l_vals)) return SPSYRK_ERR_INVALID_ARG;
    switch (dtype) {
        case SPSYRK_F64: return mirror_fill_rec(w, m, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_f_rowptr, d_f_colidx, d_f_vals, st);
        default: return mirror_fill<uint32_t>(w, m, nnz_l, d_l_rowptr, d_l_colidx, d_l_vals, d_f_rowptr, d_f_colidx, d_f_vals, st);
    }
}


extern "C" spsyrk_status_t spsyrk_mirror_enable_timing(int on) {
    if (on && !g_mirror_timing) {
        for (int i = 0; i <= MIRROR_MAX_PASSES; ++i) SPSYRK_CUDA_TRY(cudaEventCreate(&g_mirror_ev[i]));
        g_mirror_passes = 0;
    } else if (!on && g_mirror_timing) {
        for (int i = 0; i <= MIRROR_MAX_PASSES; ++i) cudaEventDestroy(g_mirror_ev[i]);
    }
    g_mirror_timing = on != 0;
    return SPSYRK_OK;
}

extern "C" spsyrk_status_t spsyrk_mirror_timings(int* passes, float pass_ms[4]) {
    if (!passes || !pass_ms || !g_mirror_timing) return SPSYRK_ERR_INVALID_ARG;
    *passes = g_mirror_passes;
    for (int p = 0; p < g_mirror_passes; ++p) {
        pass_ms[p] = 0.f;
        SPSYRK_CUDA_TRY(cudaEventSynchronize(g_mirror_ev[p + 1]));
        SPSYRK_CUDA_TRY(cudaEventElapsedTime(&pass_ms[p], g_mirror_ev[p], g_mirror_ev[p + 1]));
    }
    return SPSYRK_OK;
}

// ------------------------------------------------------------------------------------------
// Allocation-free computation of F's row pointers and entry count (what steps 2 and 3 of
// spsyrk_mirror deliver between them).
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
    if (e & (ERRW_UPPER | ERRW_BAD_ROWPTR)) return SPSYRK_ERR_BAD_CSR;
    *nnz_full_out = nnz;
    return SPSYRK_OK;
}
