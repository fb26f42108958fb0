// C ABI: spsyrk_plan / spsyrk_plan_set_rows / spsyrk_symbolic / spsyrk_numeric and helpers.
// Host-side orchestration only; every step of the path runs in the kernels of the .cuh files.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "rows_cta.cuh"
#include "rows_warp.cuh"

#include <atomic>

using namespace spsyrk;

namespace spsyrk {
static std::atomic<long long> g_launches{0};
void note_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace spsyrk

namespace {

constexpr size_t ALIGN = 256;
constexpr int64_t BLOCK_CLASS_MAX_WORK = 32768;  // class 6 (block class) up to here, class 7 above
constexpr uint32_t ROW_CHUNK_BITS_MAX_NUMERIC = 1u << 18;
constexpr uint32_t ROW_CHUNK_BITS_MAX_SYMBOLIC = 1u << 20;
constexpr int TRANSPOSE_RADIX_BITS = 8;
constexpr size_t LARGE_SMEM_BUDGET = 200 * 1024;
constexpr int GLOBAL_ACC_CTAS = 160;  // upper bound of the persistent heavy-row grid (one CTA per SM)
constexpr uint32_t BLOCK_ACC_SLOTS = 4096;
constexpr int64_t MAX_PARTS = 65536;

size_t dtype_size(spsyrk_dtype_t t) { return t == SPSYRK_F64 ? 8 : 4; }

struct Carver {
    char* base;
    size_t off = 0;
    explicit Carver(void* b) : base(static_cast<char*>(b)) {}
    template <typename T>
    T* take(size_t count) {
        off = (off + ALIGN - 1) / ALIGN * ALIGN;
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += count * sizeof(T);
        return p;
    }
};

uint32_t pow2_at_least(uint64_t v, uint32_t lo, uint32_t hi) {
    uint32_t p = lo;
    while (p < hi && p < v) p <<= 1;
    return p;
}

}  // namespace

struct spsyrk_plan_s {
    PlanDev dev;
    spsyrk_dtype_t dtype;
    // Full-output mode over the whole column range is computed in two parts per row: the lower part (columns
    // <= row, this object, working exactly like the lower-triangle mode) and the upper part (columns > row, the
    // `upper` view: the rest of every column list).  The two parts of a row are sorted ranges that follow
    // each other in the output, so each is a product of half the size and the light-row kernels see rows of
    // half the work.  dev.mode is the column range the kernels of a view work on; user_mode what was asked for.
    spsyrk_mode_t user_mode;
    spsyrk_plan_s* upper;   // null in lower-triangle mode
    bool upper_active;      // the current range is computed in two parts
    uint2* desc_hi;         // descriptors of the upper parts (start after the row's own entry, rest of the column)
    int32_t* cnt_tot;       // rows: entries per row, both parts
    int64_t* hi_begin;      // rows + 1: where the upper part of every row starts in the output
    int64_t* work_sum;      // rows: work of both parts
    const int64_t* out_begin;  // set by spsyrk_numeric: where each row's part starts / ends in the output
    const int64_t* out_end;
    // spsyrk_numeric_rows: the numeric launches take only positions [sub_lo[c], sub_hi[c]) of class c's row list
    bool sub_active;
    int64_t sub_lo[NCLASS], sub_hi[NCLASS];
    // one-pass mode (spsyrk_onepass_*): per-row slot sizes (upper bounds for the light rows), their prefix sums, and
    // where the sorting numeric kernel reports the counts it finds
    int32_t* ub;
    int64_t* ub_off;
    int32_t* cnt_out;
    bool have_onepass;
    int64_t* host_pos;  // pinned, device-visible host memory the position search of spsyrk_numeric_rows writes into (4 * NCLASS)
    int64_t rows_cap;
    // workspace views
    int32_t* perm;
    uint4* hdr;  // per-row headers in class order
    uint2* desc_full;  // descriptors for the whole column range (written by the transpose)
    uint2* desc_blk;   // descriptors narrowed to the current column range
    int32_t s0, s1;    // current column range
    int32_t* cnt;
    uint8_t* cls;
    uint32_t* colcnt;
    // radix sort buffers of the transpose (nnz entries each) and its histograms
    uint32_t *rx_key_a, *rx_row_a, *rx_pos_a, *rx_key_b, *rx_row_b, *rx_pos_b;
    void *rx_val_a, *rx_val_b;
    uint32_t* rx_hist;
    int64_t* rx_offsets;
    int32_t* blockhist;
    int64_t* offsets;
    int64_t* partials;
    int64_t* class_start_dev;  // NCLASS + 1
    unsigned long long* work_total_dev;
    uint32_t* row_counter;  // row dispenser of the persistent heavy-row kernel
    double* gacc;           // its global accumulator slices (GLOBAL_ACC_CTAS x gslots, 8 bytes per slot)
    uint32_t gslots;
    uint32_t* facts;       // binary analysis (device): differs-from-one flag, heavy columns, threshold, histogram
    uint8_t* heavy_id;
    uint64_t* heavy_mask;
    int32_t* adeg;
    int64_t* itemoff;      // rows + 1, class order: where the map words of a light row start
    int64_t map_items;     // map words the current row range needs
    uint16_t* map;         // caller's item map (spsyrk_plan_lend_map), or null
    size_t map_bytes;
    bool map_filled;       // the last symbolic pass wrote the map
    int64_t* work_prefix;  // rows + 1: exclusive prefix sums of the per-row work (spsyrk_plan_partition)
    int64_t* part_bounds;  // MAX_PARTS + 1
    // host facts
    int64_t class_start[NCLASS + 1];
    int64_t work_total;
    bool have_symbolic;
    bool key64;
    bool diag;  // the light-row kernels handle the diagonal apart (lower-triangle mode, whole column range)
    int sm_count;
    // optional per-class timing of the symbolic and numeric launches
    bool timing;
    cudaEvent_t ev_sym[NCLASS + 1];
    cudaEvent_t ev_num[NCLASS + 1];
};

namespace {

size_t carve(spsyrk_plan_s* pl, spsyrk_plan_s* up, void* ws, int64_t m, int64_t n, int64_t nnz, size_t sv, bool full) {
    Carver c(ws);
    const int64_t items = std::max<int64_t>(std::max(m, n), 1);
    const int64_t nb = bin_blocks(items);
    auto colptr = c.take<int64_t>(n + 1);
    auto desc = c.take<uint2>(nnz);
    auto work = c.take<int64_t>(m);
    auto perm = c.take<int32_t>(m);
    auto hdr = c.take<uint4>(m);
    auto cnt = c.take<int32_t>(m);
    auto cls = c.take<uint8_t>(items);
    auto colcnt = c.take<uint32_t>(n);
    const int64_t rx_hist_n = (int64_t)(1 << TRANSPOSE_RADIX_BITS) * std::max<int64_t>(radix_tiles(nnz), 1);
    // The two buffer sets of the radix sort (key, row, position, value per nonzero) are reused: the set that
    // the last pass does not read receives the column lists that pass writes (row ids and records), and the
    // set it does read holds, once the sort is over, the block descriptors and the heavy-row accumulator slices.
    const uint32_t gslots = pow2_at_least((uint64_t)std::max<int64_t>(m, 1), 1024u, ROW_CHUNK_BITS_MAX_NUMERIC);
    const size_t gacc_bytes = (size_t)GLOBAL_ACC_CTAS * gslots * sizeof(double);
    const size_t set_bytes = std::max((size_t)nnz * (12 + sv) + 4 * ALIGN, (size_t)nnz * 8 + gacc_bytes + 2 * ALIGN);
    auto set_a = c.take<char>(set_bytes);
    auto set_b = c.take<char>(set_bytes);
    Carver ca(set_a), cb(set_b);
    auto rx_key_a = ca.take<uint32_t>(nnz);
    auto rx_row_a = ca.take<uint32_t>(nnz);
    auto rx_pos_a = ca.take<uint32_t>(nnz);
    auto rx_val_a = ca.take<char>(nnz * sv);
    auto rx_key_b = cb.take<uint32_t>(nnz);
    auto rx_row_b = cb.take<uint32_t>(nnz);
    auto rx_pos_b = cb.take<uint32_t>(nnz);
    auto rx_val_b = cb.take<char>(nnz * sv);
    const int npass = (bits_for((uint64_t)std::max<int64_t>(n - 1, 1)) + TRANSPOSE_RADIX_BITS - 1) / TRANSPOSE_RADIX_BITS;
    const bool last_reads_a = npass >= 2 && (npass % 2) == 0;  // pass p writes set A when p is even; one pass reads the input itself (and row ids kept in set B)
    Carver c_free(last_reads_a ? set_b : set_a), c_src(last_reads_a ? set_a : set_b);
    auto at_row = c_free.take<int32_t>(nnz + 4);  // the symbolic gathers read aligned 16-byte pieces: up to 3 entries past the end
    auto at_rec = c_free.take<char>(nnz * (sv == 8 ? 16 : 8));
    auto desc_blk = c_src.take<uint2>(nnz);
    auto gacc = c_src.take<double>((size_t)GLOBAL_ACC_CTAS * gslots);
    auto rx_hist = c.take<uint32_t>(rx_hist_n);
    auto rx_offsets = c.take<int64_t>(rx_hist_n + 1);
    auto blockhist = c.take<int32_t>(NCLASS * nb);
    auto offsets = c.take<int64_t>(NCLASS * nb + 1);
    auto partials = c.take<int64_t>(scan_partials_count(std::max<int64_t>(std::max<int64_t>(items + 1, NCLASS * nb), rx_hist_n)));
    auto class_start_dev = c.take<int64_t>(NCLASS + 1);
    auto work_total_dev = c.take<unsigned long long>(1);
    auto err = c.take<uint32_t>(1);
    auto row_counter = c.take<uint32_t>(1);
    auto work_prefix = c.take<int64_t>(items + 1);
    auto itemoff = c.take<int64_t>(items + 1);
    auto heavy_id = c.take<uint8_t>(std::max<int64_t>(n, 1));
    auto heavy_mask = c.take<uint64_t>(std::max<int64_t>(m, 1));
    auto facts = c.take<uint32_t>(64);  // [0..2] binary analysis, [32..63] its histogram
    auto adeg = c.take<int32_t>(std::max<int64_t>(m, 1));
    auto part_bounds = c.take<int64_t>(MAX_PARTS + 1);
    auto ub = c.take<int32_t>(std::max<int64_t>(m, 1));
    auto ub_off = c.take<int64_t>(items + 1);
    // full-output mode: the upper view's own per-row arrays and the second descriptor array
    uint2* desc_hi = nullptr;
    int64_t *u_work = nullptr, *u_itemoff = nullptr, *u_class_start_dev = nullptr, *hi_begin = nullptr, *work_sum = nullptr;
    int32_t *u_perm = nullptr, *u_cnt = nullptr, *cnt_tot = nullptr;
    uint4* u_hdr = nullptr;
    uint8_t* u_cls = nullptr;
    unsigned long long* u_work_total_dev = nullptr;
    if (full) {
        desc_hi = c.take<uint2>(nnz);
        u_work = c.take<int64_t>(m);
        u_perm = c.take<int32_t>(m);
        u_hdr = c.take<uint4>(m);
        u_cnt = c.take<int32_t>(m);
        u_cls = c.take<uint8_t>(items);
        u_itemoff = c.take<int64_t>(items + 1);
        u_class_start_dev = c.take<int64_t>(NCLASS + 1);
        u_work_total_dev = c.take<unsigned long long>(1);
        cnt_tot = c.take<int32_t>(m);
        hi_begin = c.take<int64_t>(items + 1);
        work_sum = c.take<int64_t>(m);
    }
    if (pl) {
        pl->desc_hi = desc_hi; pl->cnt_tot = cnt_tot; pl->hi_begin = hi_begin; pl->work_sum = work_sum;
        pl->row_counter = row_counter; pl->gacc = gacc; pl->gslots = gslots;
        pl->work_prefix = work_prefix; pl->part_bounds = part_bounds; pl->itemoff = itemoff;
        pl->ub = ub; pl->ub_off = ub_off;
        pl->dev.heavy_id = heavy_id; pl->dev.heavy_mask = heavy_mask; pl->facts = facts;
        pl->heavy_id = heavy_id; pl->heavy_mask = heavy_mask; pl->adeg = adeg; pl->dev.adeg = adeg;
        pl->dev.colptr = colptr; pl->dev.at_row = at_row; pl->dev.at_rec = at_rec; pl->dev.desc = desc;
        pl->dev.work = work; pl->dev.err = err;
        pl->desc_full = desc; pl->desc_blk = desc_blk;
        pl->perm = perm; pl->hdr = hdr; pl->cnt = cnt; pl->cls = cls; pl->colcnt = colcnt;
        pl->rx_key_a = rx_key_a; pl->rx_row_a = rx_row_a; pl->rx_pos_a = rx_pos_a; pl->rx_key_b = rx_key_b; pl->rx_row_b = rx_row_b;
        pl->rx_pos_b = rx_pos_b; pl->rx_val_a = rx_val_a; pl->rx_val_b = rx_val_b; pl->rx_hist = rx_hist; pl->rx_offsets = rx_offsets;
        pl->blockhist = blockhist; pl->offsets = offsets; pl->partials = partials;
        pl->class_start_dev = class_start_dev; pl->work_total_dev = work_total_dev;
        if (up) {
            // the upper view shares everything that describes A and the scratch space; its rows are its own
            *up = *pl;
            up->upper = nullptr;
            up->dev.desc = desc_hi; up->dev.work = u_work;
            up->perm = u_perm; up->hdr = u_hdr; up->cnt = u_cnt; up->cls = u_cls; up->itemoff = u_itemoff;
            up->class_start_dev = u_class_start_dev; up->work_total_dev = u_work_total_dev;
        }
    }
    return (c.off + ALIGN - 1) / ALIGN * ALIGN;
}

spsyrk_status_t read_err(spsyrk_plan_s* pl, cudaStream_t st) {
    uint32_t e = 0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&e, pl->dev.err, sizeof(e), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    if (e & (ERRW_BAD_ROWPTR | ERRW_BAD_COL | ERRW_UNSORTED)) return SPSYRK_ERR_BAD_CSR;
    if (e) return SPSYRK_ERR_INTERNAL;
    return SPSYRK_OK;
}

template <int G>
void launch_row_expand(spsyrk_plan_s* pl, cudaStream_t st) {
    const PlanDev& P = pl->dev;
    const int64_t threads = (int64_t)P.m * G;
    row_expand_kernel<G><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(P.rowptr, P.colidx, P.m, P.n, pl->colcnt, pl->rx_row_b, P.err);
    note_launches(1);
}

template <int G>
void launch_block_desc(spsyrk_plan_s* pl, cudaStream_t st) {
    const PlanDev& P = pl->dev;
    const int64_t threads = (int64_t)(P.r1 - P.r0) * G;
    block_desc_kernel<G><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(P, pl->desc_full, pl->user_mode == SPSYRK_FULL ? pl->desc_hi : nullptr, pl->desc_blk, pl->s0, pl->s1);
    note_launches(1);
}

template <int G>
void launch_row_work(spsyrk_plan_s* pl, cudaStream_t st) {
    const PlanDev& P = pl->dev;
    const int64_t threads = (int64_t)(P.r1 - P.r0) * G;
    const int64_t ctas = std::min<int64_t>((threads + 255) / 256, (int64_t)pl->sm_count * 16);
    row_work_kernel<G><<<(unsigned)ctas, 256, 0, st>>>(P, pl->cls, BLOCK_CLASS_MAX_WORK, pl->diag, pl->work_total_dev);
    note_launches(1);
}

int group_width(int64_t nnz, int64_t m) {
    const double avg = m > 0 ? (double)nnz / (double)m : 0.0;
    return avg <= 4 ? 4 : avg <= 8 ? 8 : avg <= 16 ? 16 : 32;
}

// stable radix sort of the nonzeros by column id; the last pass writes the column lists and descriptors.
// VB: unsigned integer of the value's width (values are only moved)
template <typename VB>
spsyrk_status_t sort_by_column(spsyrk_plan_s* pl, cudaStream_t st) {
    constexpr int BITS = TRANSPOSE_RADIX_BITS;
    const PlanDev& P = pl->dev;
    if (P.nnz == 0) return SPSYRK_OK;
    const int npass = (bits_for((uint64_t)std::max<int64_t>(P.n - 1, 1)) + BITS - 1) / BITS;
    const uint32_t* src_key = reinterpret_cast<const uint32_t*>(P.colidx);
    const uint32_t* src_row = pl->rx_row_b;
    const VB* src_val = static_cast<const VB*>(P.vals);
    const uint32_t* src_pos = nullptr;  // position in A: the element's own index in the first pass
    for (int p = 0; p < npass; ++p) {
        const bool to_a = (p % 2) == 0;
        uint32_t* dst_key = to_a ? pl->rx_key_a : pl->rx_key_b;
        uint32_t* dst_row = to_a ? pl->rx_row_a : pl->rx_row_b;
        uint32_t* dst_pos = to_a ? pl->rx_pos_a : pl->rx_pos_b;
        VB* dst_val = static_cast<VB*>(to_a ? pl->rx_val_a : pl->rx_val_b);
        if (p == npass - 1) {
            EmitTransposeFinal<VB> emit{P, pl->desc_hi};
            SPSYRK_CUDA_TRY((radix_pass3<BITS, VB>(src_key, src_row, src_val, src_pos, P.nnz, p * BITS, pl->rx_hist, pl->rx_offsets,
                                                   pl->partials, emit, P.err, st)));
        } else {
            EmitArrays3<VB> emit{dst_key, dst_row, dst_val, dst_pos};
            SPSYRK_CUDA_TRY((radix_pass3<BITS, VB>(src_key, src_row, src_val, src_pos, P.nnz, p * BITS, pl->rx_hist, pl->rx_offsets,
                                                   pl->partials, emit, P.err, st)));
        }
        src_key = dst_key;
        src_row = dst_row;
        src_val = dst_val;
        src_pos = dst_pos;
    }
    return SPSYRK_OK;
}

__global__ void add_work_kernel(const int64_t* __restrict__ a, const int64_t* __restrict__ b, int64_t rows, int64_t* __restrict__ out) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < rows) out[r] = a[r] + b[r];
}

// work estimate + binning of one view's current row range (dev.desc, dev.mode and diag are set); reads class sizes back (one sync)
spsyrk_status_t bin_view(spsyrk_plan_s* pl, cudaStream_t st) {
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    pl->have_symbolic = false;
    pl->have_onepass = false;
    const PlanDev& P = pl->dev;
    SPSYRK_CUDA_TRY(cudaMemsetAsync(pl->work_total_dev, 0, sizeof(unsigned long long), st));
    if (rows > 0) {
        switch (group_width(P.nnz, P.m)) {
            case 4: launch_row_work<4>(pl, st); break;
            case 8: launch_row_work<8>(pl, st); break;
            case 16: launch_row_work<16>(pl, st); break;
            default: launch_row_work<32>(pl, st); break;
        }
    }
    SPSYRK_CUDA_TRY(bin_items(pl->cls, rows, pl->perm, pl->class_start_dev, pl->blockhist, pl->offsets, pl->partials, st));
    if (rows > 0) {
        row_header_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(P, pl->perm, rows, pl->hdr);
        note_launches(1);
    }
    // where the item-map words of every light row start (rows in class order)
    int64_t map_items = 0;
    pl->map_filled = false;
    if (rows > 0) {
        uint32_t* items8 = reinterpret_cast<uint32_t*>(pl->cnt);  // free until the symbolic pass
        row_items_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(P, pl->hdr, pl->cls, rows, pl->diag, items8);
        note_launches(1);
        SPSYRK_CUDA_TRY(exclusive_scan_i64<uint32_t>(items8, rows, pl->itemoff, pl->partials, st));
        SPSYRK_CUDA_TRY(cudaMemcpyAsync(&map_items, pl->itemoff + rows, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    }
    unsigned long long wt = 0;
    uint32_t facts[3] = {1u, 0u, 0u};
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(facts, pl->facts, sizeof(facts), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(pl->class_start, pl->class_start_dev, sizeof(pl->class_start), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&wt, pl->work_total_dev, sizeof(wt), cudaMemcpyDeviceToHost, st));
    spsyrk_status_t s = read_err(pl, st);
    pl->work_total = (int64_t)wt;
    pl->map_items = map_items;
    pl->dev.binary = (pl->dev.nnz > 0 && facts[0] == 0) ? 1 : 0;
    pl->dev.nheavy = pl->dev.binary ? (int32_t)std::min<uint32_t>(facts[1], 64u) : 0;
    return s;
}

// descriptors, work estimate and binning of the plan's current block of output rows and columns
spsyrk_status_t estimate_and_bin(spsyrk_plan_s* pl, cudaStream_t st) {
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    const bool whole = pl->s0 <= 0 && pl->s1 >= pl->dev.m;
    pl->upper_active = false;
    if (whole) {
        pl->dev.desc = pl->desc_full;
        if (pl->user_mode == SPSYRK_FULL && pl->upper) {
            // two parts per row: this view does the lower parts like the lower-triangle mode, the upper view the rest
            pl->upper_active = true;
            pl->dev.mode = SPSYRK_TRIL;
            pl->diag = true;
            spsyrk_status_t s = bin_view(pl, st);
            if (s != SPSYRK_OK) return s;
            spsyrk_plan_s* up = pl->upper;
            up->dev.r0 = pl->dev.r0; up->dev.r1 = pl->dev.r1;
            up->dev.mode = SPSYRK_FULL;  // the upper part of row i lies in (i, m): the kernels work on the range [0, m)
            up->dev.desc = pl->desc_hi;
            up->dev.jaccard = pl->dev.jaccard;
            up->diag = false;
            s = bin_view(up, st);
            if (s != SPSYRK_OK) return s;
            if (rows > 0) {
                add_work_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(pl->dev.work, up->dev.work, rows, pl->work_sum);
                note_launches(1);
            }
            return SPSYRK_OK;
        }
        pl->dev.mode = (int32_t)pl->user_mode;
        pl->diag = pl->user_mode == SPSYRK_TRIL;
        return bin_view(pl, st);
    }
    // a column range: descriptors narrowed to [s0, s1) (cut out of the whole column lists in full-output mode)
    pl->dev.desc = pl->desc_blk;
    pl->dev.mode = (int32_t)pl->user_mode;
    pl->diag = false;
    if (rows > 0 && pl->dev.nnz > 0) {
        switch (group_width(pl->dev.nnz, pl->dev.m)) {
            case 4: launch_block_desc<4>(pl, st); break;
            case 8: launch_block_desc<8>(pl, st); break;
            case 16: launch_block_desc<16>(pl, st); break;
            default: launch_block_desc<32>(pl, st); break;
        }
    }
    return bin_view(pl, st);
}

int64_t map_items_total(const spsyrk_plan_s* pl) { return pl->map_items + (pl->upper_active ? pl->upper->map_items : 0); }

bool use_map(const spsyrk_plan_s* pl) { return pl->map && pl->map_bytes >= (size_t)map_items_total(pl) * sizeof(uint16_t); }

template <int N, bool DIAG>
spsyrk_status_t launch_symbolic_warp_d(spsyrk_plan_s* pl, int c, cudaStream_t st) {
    const int64_t count = pl->class_start[c + 1] - pl->class_start[c];
    if (count <= 0) return SPSYRK_OK;
    constexpr int G = warp_class_group(N);
    constexpr int SW = symbolic_warps(N);
    constexpr int ROWS = SW * (32 / G);  // rows a CTA works on at a time
    constexpr size_t smem = (size_t)ROWS * SymbolicWarpSmem<N>::GROUP;
    auto kern = symbolic_warp_kernel<N, G, DIAG>;
    SPSYRK_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, SW * 32, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int64_t want = (count + ROWS - 1) / ROWS;
    const int64_t cap = (int64_t)pl->sm_count * per_sm;
    kern<<<(unsigned)std::min(want, cap), SW * 32, smem, st>>>(pl->dev, pl->hdr + pl->class_start[c], count, pl->cnt);
    note_launches(1);
    return SPSYRK_OK;
}

template <int N>
spsyrk_status_t launch_symbolic_warp(spsyrk_plan_s* pl, int c, cudaStream_t st) {
    return pl->diag ? launch_symbolic_warp_d<N, true>(pl, c, st) : launch_symbolic_warp_d<N, false>(pl, c, st);
}

// the part of class c's row list (rows in ascending order) a numeric launch covers
inline int64_t numeric_first(const spsyrk_plan_s* pl, int c) { return pl->sub_active ? pl->sub_lo[c] : pl->class_start[c]; }
inline int64_t numeric_count(const spsyrk_plan_s* pl, int c) {
    return pl->sub_active ? pl->sub_hi[c] - pl->sub_lo[c] : pl->class_start[c + 1] - pl->class_start[c];
}

template <typename V, int N, typename Key, bool DIAG>
spsyrk_status_t launch_numeric_warp_d(spsyrk_plan_s* pl, int c, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    const int64_t count = numeric_count(pl, c);
    if (count <= 0) return SPSYRK_OK;
    constexpr int G = warp_class_group(N);
    constexpr int NW = numeric_warps(N);
    constexpr int ROWS = NW * (32 / G);
    constexpr size_t smem = (size_t)ROWS * NumericWarpSmem<V, N>::GROUP;
    // persistent groups: exactly as many CTAs as are resident at once, each group walks its rows with
    // a stride of the whole grid
    auto kern = numeric_warp_kernel<V, N, G, Key, DIAG>;
    SPSYRK_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NW * 32, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int64_t want = (count + ROWS - 1) / ROWS;
    const int64_t cap = (int64_t)pl->sm_count * per_sm;
    kern<<<(unsigned)std::min(want, cap), NW * 32, smem, st>>>(pl->dev, pl->hdr + numeric_first(pl, c), count, pl->out_begin, pl->out_end,
                                                               c_colidx, static_cast<V*>(c_vals), pl->cnt_out);
    note_launches(1);
    return SPSYRK_OK;
}

template <typename V, int N, typename Key>
spsyrk_status_t launch_numeric_warp(spsyrk_plan_s* pl, int c, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    return pl->diag ? launch_numeric_warp_d<V, N, Key, true>(pl, c, c_colidx, c_vals, st)
                    : launch_numeric_warp_d<V, N, Key, false>(pl, c, c_colidx, c_vals, st);
}

template <int N, typename Key, bool DIAG>
spsyrk_status_t launch_symbolic_sort_d(spsyrk_plan_s* pl, int c, cudaStream_t st) {
    const int64_t count = pl->class_start[c + 1] - pl->class_start[c];
    if (count <= 0) return SPSYRK_OK;
    constexpr int G = warp_class_group(N);
    constexpr int SW = symbolic_sort_warps(N);
    constexpr int ROWS = SW * (32 / G);
    constexpr size_t smem = (size_t)ROWS * SymbolicSortSmem<N>::GROUP;
    auto kern = symbolic_sort_warp_kernel<N, G, Key, DIAG>;
    SPSYRK_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, SW * 32, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int64_t want = (count + ROWS - 1) / ROWS;
    const int64_t cap = (int64_t)pl->sm_count * per_sm;
    kern<<<(unsigned)std::min(want, cap), SW * 32, smem, st>>>(pl->dev, pl->hdr + pl->class_start[c], pl->itemoff + pl->class_start[c],
                                                               count, pl->cnt, pl->map);
    note_launches(1);
    return SPSYRK_OK;
}

template <int N>
spsyrk_status_t launch_symbolic_sort(spsyrk_plan_s* pl, int c, cudaStream_t st) {
    if (pl->key64)
        return pl->diag ? launch_symbolic_sort_d<N, uint64_t, true>(pl, c, st) : launch_symbolic_sort_d<N, uint64_t, false>(pl, c, st);
    return pl->diag ? launch_symbolic_sort_d<N, uint32_t, true>(pl, c, st) : launch_symbolic_sort_d<N, uint32_t, false>(pl, c, st);
}

template <typename V, int N, bool DIAG>
spsyrk_status_t launch_numeric_map_d(spsyrk_plan_s* pl, int c, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    const int64_t count = numeric_count(pl, c);
    if (count <= 0) return SPSYRK_OK;
    constexpr int G = warp_class_group(N);
    constexpr int NW = numeric_map_warps(N);
    constexpr int ROWS = NW * (32 / G);
    constexpr size_t smem = (size_t)ROWS * NumericMapSmem<V, N>::GROUP;
    auto kern = numeric_map_warp_kernel<V, N, G, DIAG>;
    SPSYRK_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NW * 32, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int64_t want = (count + ROWS - 1) / ROWS;
    const int64_t cap = (int64_t)pl->sm_count * per_sm;
    kern<<<(unsigned)std::min(want, cap), NW * 32, smem, st>>>(pl->dev, pl->hdr + numeric_first(pl, c), pl->itemoff + numeric_first(pl, c),
                                                               count, pl->map, pl->out_begin, pl->out_end, c_colidx, static_cast<V*>(c_vals));
    note_launches(1);
    return SPSYRK_OK;
}

template <typename V, int N>
spsyrk_status_t launch_numeric_map(spsyrk_plan_s* pl, int c, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    return pl->diag ? launch_numeric_map_d<V, N, true>(pl, c, c_colidx, c_vals, st)
                    : launch_numeric_map_d<V, N, false>(pl, c, c_colidx, c_vals, st);
}

inline void mark(spsyrk_plan_s* pl, cudaEvent_t* ev, int i, cudaStream_t st) {
    if (pl->timing) cudaEventRecord(ev[i], st);
}

template <typename V>
void launch_numeric_map_all(spsyrk_plan_s* pl, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    mark(pl, pl->ev_num, 1, st);
    launch_numeric_map<V, 32>(pl, 1, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 2, st);
    launch_numeric_map<V, 64>(pl, 2, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 3, st);
    launch_numeric_map<V, 128>(pl, 3, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 4, st);
    launch_numeric_map<V, 256>(pl, 4, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 5, st);
    launch_numeric_map<V, 512>(pl, 5, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 6, st);
}

template <typename V, typename Key>
void launch_numeric_warp_all(spsyrk_plan_s* pl, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    mark(pl, pl->ev_num, 1, st);
    launch_numeric_warp<V, 32, Key>(pl, 1, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 2, st);
    launch_numeric_warp<V, 64, Key>(pl, 2, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 3, st);
    launch_numeric_warp<V, 128, Key>(pl, 3, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 4, st);
    launch_numeric_warp<V, 256, Key>(pl, 4, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 5, st);
    launch_numeric_warp<V, 512, Key>(pl, 5, c_colidx, c_vals, st);
    mark(pl, pl->ev_num, 6, st);
}

// bounds[p] = r0 + the smallest r in [0, rows] with prefix[r] * parts >= p * prefix[rows]
__global__ void partition_kernel(const int64_t* __restrict__ prefix, int64_t rows, int64_t parts, int64_t r0,
                                 int64_t* __restrict__ bounds) {
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p > parts) return;
    if (p == parts) { bounds[p] = r0 + rows; return; }
    const int64_t target = p * prefix[rows];
    int64_t lo = 0, hi = rows;  // prefix is non-decreasing; prefix[rows] * parts >= target always
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (prefix[mid] * parts >= target) hi = mid; else lo = mid + 1;
    }
    bounds[p] = r0 + lo;
}

uint32_t row_chunk_bits(const spsyrk_plan_s* pl, uint32_t cap) {
    const uint64_t umax = pl->dev.mode == SPSYRK_TRIL ? (uint64_t)pl->dev.r1 : (uint64_t)pl->dev.m;
    return pow2_at_least(umax, 1024u, cap);
}

template <int THREADS>
spsyrk_status_t launch_symbolic_cta(spsyrk_plan_s* pl, int c, cudaStream_t st) {
    const int64_t count = pl->class_start[c + 1] - pl->class_start[c];
    if (count <= 0) return SPSYRK_OK;
    const uint32_t cb = row_chunk_bits(pl, ROW_CHUNK_BITS_MAX_SYMBOLIC);
    const size_t smem = CtaRowSmem<int32_t, THREADS, false>::bytes(cb, 0);
    auto kern = rows_cta_kernel<int32_t, THREADS, false>;
    SPSYRK_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<(unsigned)count, THREADS, smem, st>>>(pl->dev, pl->perm + pl->class_start[c], cb, 0u, pl->cnt, nullptr, nullptr, nullptr,
                                                  nullptr, 0u, nullptr, nullptr, 0u);
    note_launches(1);
    return SPSYRK_OK;
}

template <typename V, int THREADS>
spsyrk_status_t launch_numeric_cta(spsyrk_plan_s* pl, int c, uint32_t acc_slots_or_zero, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    using Acc = typename AccOf<V>::type;
    const int64_t count = numeric_count(pl, c);
    if (count <= 0) return SPSYRK_OK;
    const int32_t* rows_of_class = pl->perm + numeric_first(pl, c);
    const uint32_t cb = row_chunk_bits(pl, ROW_CHUNK_BITS_MAX_NUMERIC);
    uint32_t slots = acc_slots_or_zero;
    if (slots == 0) {
        const size_t fixed = CtaRowSmem<V, THREADS, true>::bytes(cb, 0);
        slots = (uint32_t)((LARGE_SMEM_BUDGET - fixed) / sizeof(Acc));
        slots = std::min(slots, cb);  // a chunk never has more slots than bits
    }
    const size_t smem = CtaRowSmem<V, THREADS, true>::bytes(cb, slots);
    auto kern = rows_cta_kernel<V, THREADS, true>;
    SPSYRK_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // rows that overflow the shared-memory tile go to the persistent variant with global accumulators
    const bool use_global = acc_slots_or_zero == 0 && pl->gslots >= cb;
    const uint32_t gslots = use_global ? pl->gslots : 0u;
    kern<<<(unsigned)count, THREADS, smem, st>>>(pl->dev, rows_of_class, cb, slots, nullptr, pl->out_begin, pl->out_end,
                                                  c_colidx, static_cast<V*>(c_vals), 0u, nullptr, nullptr, gslots);
    note_launches(1);
    if (use_global) {
        auto gkern = rows_cta_kernel<V, THREADS, true, true>;
        const size_t gsmem = CtaRowSmem<V, THREADS, true>::bytes(cb, 0);
        SPSYRK_CUDA_TRY(cudaFuncSetAttribute(gkern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gsmem));
        SPSYRK_CUDA_TRY(cudaMemsetAsync(pl->row_counter, 0, sizeof(uint32_t), st));
        const unsigned grid = (unsigned)std::min<int64_t>(std::min<int64_t>(pl->sm_count, GLOBAL_ACC_CTAS), count);
        gkern<<<grid, THREADS, gsmem, st>>>(pl->dev, rows_of_class, cb, slots, nullptr, pl->out_begin, pl->out_end,
                                            c_colidx, static_cast<V*>(c_vals), (uint32_t)count, pl->row_counter,
                                            reinterpret_cast<Acc*>(pl->gacc), gslots);
        note_launches(1);
    }
    return SPSYRK_OK;
}

template <typename V>
spsyrk_status_t numeric_typed(spsyrk_plan_s* pl, int32_t* c_colidx, void* c_vals, cudaStream_t st) {
    if (pl->map_filled) launch_numeric_map_all<V>(pl, c_colidx, c_vals, st);
    else if (pl->key64) launch_numeric_warp_all<V, uint64_t>(pl, c_colidx, c_vals, st);
    else launch_numeric_warp_all<V, uint32_t>(pl, c_colidx, c_vals, st);
    spsyrk_status_t s = launch_numeric_cta<V, 512>(pl, 6, BLOCK_ACC_SLOTS, c_colidx, c_vals, st);
    if (s != SPSYRK_OK) return s;
    mark(pl, pl->ev_num, 7, st);
    s = launch_numeric_cta<V, 1024>(pl, 7, 0u, c_colidx, c_vals, st);
    if (s != SPSYRK_OK) return s;
    mark(pl, pl->ev_num, 8, st);
    SPSYRK_CUDA_TRY(cudaGetLastError());
#ifdef SPSYRK_CHECKED
    return read_err(pl, st);  // the bounds-checked build reports a skipped access at once (synchronises)
#else
    return SPSYRK_OK;
#endif
}

__global__ void add_counts_kernel(const int32_t* __restrict__ a, const int32_t* __restrict__ b, int64_t rows, int32_t* __restrict__ out) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < rows) out[r] = a[r] + b[r];
}

__global__ void upper_begin_kernel(const int64_t* __restrict__ c_rowptr, const int32_t* __restrict__ cnt_lo, int64_t rows,
                                   int64_t* __restrict__ hi_begin) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < rows) hi_begin[r] = c_rowptr[r] + cnt_lo[r];
}

// the per-class count kernels of one view (entries per row into its cnt array)
spsyrk_status_t symbolic_view(spsyrk_plan_s* pl, bool with_map, cudaStream_t st) {
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    if (rows > 0) SPSYRK_CUDA_TRY(cudaMemsetAsync(pl->cnt, 0, (size_t)rows * sizeof(int32_t), st));
    pl->map_filled = false;
    mark(pl, pl->ev_sym, 1, st);
    if (with_map) launch_symbolic_sort<32>(pl, 1, st); else launch_symbolic_warp<32>(pl, 1, st);
    mark(pl, pl->ev_sym, 2, st);
    if (with_map) launch_symbolic_sort<64>(pl, 2, st); else launch_symbolic_warp<64>(pl, 2, st);
    mark(pl, pl->ev_sym, 3, st);
    if (with_map) launch_symbolic_sort<128>(pl, 3, st); else launch_symbolic_warp<128>(pl, 3, st);
    mark(pl, pl->ev_sym, 4, st);
    if (with_map) launch_symbolic_sort<256>(pl, 4, st); else launch_symbolic_warp<256>(pl, 4, st);
    mark(pl, pl->ev_sym, 5, st);
    if (with_map) launch_symbolic_sort<512>(pl, 5, st); else launch_symbolic_warp<512>(pl, 5, st);
    mark(pl, pl->ev_sym, 6, st);
    spsyrk_status_t s = launch_symbolic_cta<256>(pl, 6, st);
    if (s != SPSYRK_OK) return s;
    mark(pl, pl->ev_sym, 7, st);
    s = launch_symbolic_cta<1024>(pl, 7, st);
    if (s != SPSYRK_OK) return s;
    mark(pl, pl->ev_sym, 8, st);
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}

}  // namespace

namespace {
// slot size of every row in the one-pass layout: light rows by the number of their partial products (an upper
// bound of their entries; with the diagonal handled apart: products without the diagonal ones, plus the diagonal
// entry), heavy rows by the count their own symbolic kernels just found
__global__ void onepass_slots_kernel(PlanDev P, const uint8_t* __restrict__ cls, const int32_t* __restrict__ cnt, bool diag, int64_t rows,
                                     int32_t* __restrict__ ub) {
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    const int c = cls[r];
    const int64_t i = P.r0 + r;
    const int64_t deg = P.rowptr[i + 1] - P.rowptr[i];
    int64_t u = 0;
    if (c >= 6) u = cnt[r];
    else if (c >= 1) u = diag ? P.work[r] - deg + (deg > 0 ? 1 : 0) : P.work[r];
    ub[r] = (int32_t)u;  // a light row has at most 512 + 32 products
}

// G lanes per row: row r moves from its slot to its place
template <typename V, int G>
__global__ void __launch_bounds__(256) onepass_compact_kernel(const int64_t* __restrict__ src_off, const int64_t* __restrict__ dst_off, int64_t rows,
                                                              const int32_t* __restrict__ s_col, const V* __restrict__ s_val,
                                                              int32_t* __restrict__ d_col, V* __restrict__ d_val) {
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (r >= rows) return;
    const int64_t s0 = src_off[r], d0 = dst_off[r], len = dst_off[r + 1] - d0;
    constexpr int UNR = 4;
    for (int64_t p = gl; p < len; p += UNR * G) {
        int32_t j[UNR];
        V v[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u)
            if (p + u * G < len) { j[u] = s_col[s0 + p + u * G]; v[u] = s_val[s0 + p + u * G]; }
#pragma unroll
        for (int u = 0; u < UNR; ++u)
            if (p + u * G < len) { d_col[d0 + p + u * G] = j[u]; d_val[d0 + p + u * G] = v[u]; }
    }
}

template <typename V>
void launch_onepass_compact(const spsyrk_plan_s* pl, const int64_t* dst_off, int64_t rows, int64_t nnz, const int32_t* s_col, const void* s_val,
                            int32_t* d_col, void* d_val, cudaStream_t st) {
    const double avg = rows > 0 ? (double)nnz / (double)rows : 0.0;
#define COMPACT(G) \
    onepass_compact_kernel<V, G><<<(unsigned)((rows * G + 255) / 256), 256, 0, st>>>(pl->ub_off, dst_off, rows, s_col, static_cast<const V*>(s_val), \
                                                                                  d_col, static_cast<V*>(d_val))
    if (avg <= 4) COMPACT(4); else if (avg <= 8) COMPACT(8); else if (avg <= 16) COMPACT(16); else COMPACT(32);
#undef COMPACT
    note_launches(1);
}
}  // namespace


extern "C" {

spsyrk_status_t spsyrk_plan(spsyrk_plan_t* plan, int64_t m, int64_t n, int64_t nnz, const int64_t* d_rowptr,
                            const int32_t* d_colidx, const void* d_vals, spsyrk_dtype_t dtype, spsyrk_mode_t mode,
                            int64_t row_begin, int64_t row_end, void* d_workspace, size_t* workspace_bytes,
                            void* cuda_stream) {
    if (!workspace_bytes || m < 0 || n < 0 || nnz < 0) return SPSYRK_ERR_INVALID_ARG;
    if (dtype != SPSYRK_F64 && dtype != SPSYRK_F32 && dtype != SPSYRK_I32) return SPSYRK_ERR_INVALID_ARG;
    if (mode != SPSYRK_TRIL && mode != SPSYRK_FULL) return SPSYRK_ERR_INVALID_ARG;
    if (row_begin < 0 || row_end < row_begin || row_end > m) return SPSYRK_ERR_INVALID_ARG;
    if (m >= (int64_t(1) << 31) - 1 || n >= (int64_t(1) << 31) - 1 || nnz >= (int64_t(1) << 31) - 1) return SPSYRK_ERR_OVERFLOW;
    const size_t sv = dtype_size(dtype);
    const bool full = mode == SPSYRK_FULL;
    const size_t need = carve(nullptr, nullptr, nullptr, m, n, nnz, sv, full);
    if (!d_workspace) {
        *workspace_bytes = need;
        return SPSYRK_OK;
    }
    if (!plan || !d_rowptr || (nnz > 0 && (!d_colidx || !d_vals))) return SPSYRK_ERR_INVALID_ARG;
    if (*workspace_bytes < need) return SPSYRK_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_workspace) % ALIGN) return SPSYRK_ERR_INVALID_ARG;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    spsyrk_plan_s* pl = new (std::nothrow) spsyrk_plan_s();
    if (!pl) return SPSYRK_ERR_INTERNAL;
    std::memset(pl, 0, sizeof(*pl));
    PlanDev& P = pl->dev;
    P.m = (int32_t)m; P.n = (int32_t)n; P.nnz = nnz; P.r0 = (int32_t)row_begin; P.r1 = (int32_t)row_end; P.mode = (int32_t)mode;
    P.rowptr = d_rowptr; P.colidx = d_colidx; P.vals = d_vals;
    pl->dtype = dtype;
    pl->user_mode = mode;
    pl->rows_cap = m;
    pl->key64 = m > (int64_t(1) << 22);
    pl->s0 = 0;
    pl->s1 = (int32_t)m;
    {
        int dev_id = 0;
        pl->sm_count = 148;
        if (cudaGetDevice(&dev_id) == cudaSuccess) cudaDeviceGetAttribute(&pl->sm_count, cudaDevAttrMultiProcessorCount, dev_id);
    }
    spsyrk_plan_s* up = nullptr;
    if (full) {
        up = new (std::nothrow) spsyrk_plan_s();
        if (!up) { delete pl; return SPSYRK_ERR_INTERNAL; }
    }
    pl->upper = up;
    carve(pl, up, d_workspace, m, n, nnz, sv, full);
    pl->upper = up;  // (the copy into the upper view happened with a null link)

    auto fail = [&](spsyrk_status_t s) { delete up; delete pl; return s; };
#define PLAN_TRY(expr) do { if ((expr) != cudaSuccess) return fail(SPSYRK_ERR_CUDA); } while (0)
    PLAN_TRY(cudaMemsetAsync(P.err, 0, sizeof(uint32_t), st));
    if (n > 0) PLAN_TRY(cudaMemsetAsync(pl->colcnt, 0, (size_t)n * sizeof(uint32_t), st));
    // 1. row pointers must be sane before anything indexes with them
    validate_rowptr_kernel<<<(unsigned)((m + 1 + 255) / 256), 256, 0, st>>>(d_rowptr, m, nnz, P.err);
    note_launches(1);
    PLAN_TRY(cudaGetLastError());
    spsyrk_status_t s = read_err(pl, st);
    if (s != SPSYRK_OK) return fail(s);
    // 2. transpose: one sweep over A for the column histogram, the explicit row ids and the checks of the column
    // ids; the histogram's scan gives colptr; stable radix sort by column
    if (nnz > 0) {
        switch (group_width(nnz, m)) {
            case 4: launch_row_expand<4>(pl, st); break;
            case 8: launch_row_expand<8>(pl, st); break;
            case 16: launch_row_expand<16>(pl, st); break;
            default: launch_row_expand<32>(pl, st); break;
        }
    }
    PLAN_TRY(exclusive_scan_i64<uint32_t>(pl->colcnt, n, P.colptr, pl->partials, st));
    s = read_err(pl, st);  // synchronises; column ids are known to be in range and rows sorted from here on
    if (s != SPSYRK_OK) return fail(s);
    s = sv == 8 ? sort_by_column<uint64_t>(pl, st) : sort_by_column<uint32_t>(pl, st);
    if (s != SPSYRK_OK) return fail(s);
    // 3. binary input: value check, heavy columns as bit masks per row
    P.binary = 0; P.nheavy = 0; P.jaccard = nullptr;
    PLAN_TRY(cudaMemsetAsync(pl->facts, 0, 64 * sizeof(uint32_t), st));
    if (m > 0) {
        row_degree_kernel<<<(unsigned)((m + 255) / 256), 256, 0, st>>>(d_rowptr, P.m, pl->adeg);
        note_launches(1);
    }
    if (nnz > 0) {
        const unsigned cb = (unsigned)std::min<int64_t>((nnz + 255) / 256, (int64_t)pl->sm_count * 16);
        switch (dtype) {
            case SPSYRK_F64: binary_check_kernel<double><<<cb, 256, 0, st>>>(static_cast<const double*>(d_vals), nnz, pl->facts); break;
            case SPSYRK_F32: binary_check_kernel<float><<<cb, 256, 0, st>>>(static_cast<const float*>(d_vals), nnz, pl->facts); break;
            default: binary_check_kernel<int32_t><<<cb, 256, 0, st>>>(static_cast<const int32_t*>(d_vals), nnz, pl->facts); break;
        }
        const unsigned hb = (unsigned)std::min<int64_t>((n + 255) / 256, (int64_t)pl->sm_count * 16);
        heavy_hist_kernel<<<hb, 256, 0, st>>>(pl->colcnt, n, pl->facts + 32);
        heavy_threshold_kernel<<<1, 32, 0, st>>>(pl->facts + 32, pl->facts);
        heavy_assign_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(pl->colcnt, n, pl->facts, pl->heavy_id);
        const unsigned mb = (unsigned)std::min<int64_t>((m * 32 + 255) / 256, (int64_t)pl->sm_count * 8);
        switch (group_width(nnz, m)) {
            case 4: heavy_mask_kernel<4><<<mb, 256, 0, st>>>(d_rowptr, d_colidx, P.m, pl->facts, pl->heavy_id, pl->heavy_mask); break;
            case 8: heavy_mask_kernel<8><<<mb, 256, 0, st>>>(d_rowptr, d_colidx, P.m, pl->facts, pl->heavy_id, pl->heavy_mask); break;
            case 16: heavy_mask_kernel<16><<<mb, 256, 0, st>>>(d_rowptr, d_colidx, P.m, pl->facts, pl->heavy_id, pl->heavy_mask); break;
            default: heavy_mask_kernel<32><<<mb, 256, 0, st>>>(d_rowptr, d_colidx, P.m, pl->facts, pl->heavy_id, pl->heavy_mask); break;
        }
        note_launches(5);
        PLAN_TRY(cudaGetLastError());
    }
    // 4. work estimate and row binning (its read-back also brings the facts above)
    s = estimate_and_bin(pl, st);
    if (s != SPSYRK_OK) return fail(s);
#undef PLAN_TRY
    *plan = pl;
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_plan_set_block(spsyrk_plan_t plan, int64_t row_begin, int64_t row_end, int64_t col_begin,
                                      int64_t col_end, void* cuda_stream) {
    if (!plan || row_begin < 0 || row_end < row_begin || row_end > plan->dev.m) return SPSYRK_ERR_INVALID_ARG;
    if (col_begin < 0 || col_end < col_begin || col_end > plan->dev.m) return SPSYRK_ERR_INVALID_ARG;
    plan->dev.r0 = (int32_t)row_begin;
    plan->dev.r1 = (int32_t)row_end;
    plan->s0 = (int32_t)col_begin;
    plan->s1 = (int32_t)col_end;
    plan->have_symbolic = false;
    return estimate_and_bin(plan, static_cast<cudaStream_t>(cuda_stream));
}

spsyrk_status_t spsyrk_plan_set_rows(spsyrk_plan_t plan, int64_t row_begin, int64_t row_end, void* cuda_stream) {
    if (!plan) return SPSYRK_ERR_INVALID_ARG;
    return spsyrk_plan_set_block(plan, row_begin, row_end, 0, plan->dev.m, cuda_stream);
}

spsyrk_status_t spsyrk_plan_partition(spsyrk_plan_t plan, int64_t parts, int64_t* bounds, void* cuda_stream) {
    if (!plan || !bounds || parts < 1 || parts > MAX_PARTS) return SPSYRK_ERR_INVALID_ARG;
    spsyrk_plan_s* pl = plan;
    const int64_t work_all = pl->work_total + (pl->upper_active ? pl->upper->work_total : 0);
    if (work_all > 0 && work_all > INT64_MAX / parts) return SPSYRK_ERR_OVERFLOW;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    SPSYRK_CUDA_TRY(exclusive_scan_i64<int64_t>(pl->upper_active ? pl->work_sum : pl->dev.work, rows, pl->work_prefix, pl->partials, st));
    partition_kernel<<<(unsigned)((parts + 1 + 255) / 256), 256, 0, st>>>(pl->work_prefix, rows, parts, pl->dev.r0, pl->part_bounds);
    note_launches(1);
    SPSYRK_CUDA_TRY(cudaGetLastError());
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(bounds, pl->part_bounds, (size_t)(parts + 1) * sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_symbolic(spsyrk_plan_t plan, int64_t* d_c_rowptr, int64_t* nnz_out, void* cuda_stream) {
    if (!plan || !d_c_rowptr || !nnz_out) return SPSYRK_ERR_INVALID_ARG;
    spsyrk_plan_s* pl = plan;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    const bool with_map = use_map(pl);
    spsyrk_status_t s = symbolic_view(pl, with_map, st);
    if (s != SPSYRK_OK) return s;
    const int32_t* counts = pl->cnt;
    if (pl->upper_active) {
        spsyrk_plan_s* up = pl->upper;
        up->map = with_map ? pl->map + pl->map_items : nullptr;  // the upper parts' words follow the lower parts'
        up->map_bytes = with_map ? (size_t)up->map_items * sizeof(uint16_t) : 0;
        s = symbolic_view(up, with_map, st);
        if (s != SPSYRK_OK) return s;
        if (rows > 0) {
            add_counts_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(pl->cnt, up->cnt, rows, pl->cnt_tot);
            note_launches(1);
        }
        counts = pl->cnt_tot;
    }
    SPSYRK_CUDA_TRY(exclusive_scan_i64<int32_t>(counts, rows, d_c_rowptr, pl->partials, st));
    if (pl->upper_active && rows > 0) {
        // the upper part of row r starts after its lower part
        upper_begin_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(d_c_rowptr, pl->cnt, rows, pl->hi_begin);
        note_launches(1);
    }
    int64_t nnz = 0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&nnz, d_c_rowptr + rows, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    s = read_err(pl, st);
    if (s != SPSYRK_OK) return s;
    *nnz_out = nnz;
    pl->have_symbolic = true;
    pl->map_filled = with_map;
    if (pl->upper_active) { pl->upper->have_symbolic = true; pl->upper->map_filled = with_map; }
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_numeric(spsyrk_plan_t plan, const int64_t* d_c_rowptr, int32_t* d_c_colidx, void* d_c_vals,
                               void* cuda_stream) {
    if (!plan || !d_c_rowptr) return SPSYRK_ERR_INVALID_ARG;
    spsyrk_plan_s* pl = plan;
    if (!pl->have_symbolic) return SPSYRK_ERR_SEQUENCE;
    const int64_t work_all = pl->work_total + (pl->upper_active ? pl->upper->work_total : 0);
    if (work_all > 0 && (!d_c_colidx || !d_c_vals)) return SPSYRK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    auto run = [&](spsyrk_plan_s* v) {
        switch (v->dtype) {
            case SPSYRK_F64: return numeric_typed<double>(v, d_c_colidx, d_c_vals, st);
            case SPSYRK_F32: return numeric_typed<float>(v, d_c_colidx, d_c_vals, st);
            default: return numeric_typed<int32_t>(v, d_c_colidx, d_c_vals, st);
        }
    };
    pl->out_begin = d_c_rowptr;
    pl->out_end = pl->upper_active ? pl->hi_begin : d_c_rowptr + 1;
    spsyrk_status_t s = run(pl);
    if (s != SPSYRK_OK || !pl->upper_active) return s;
    spsyrk_plan_s* up = pl->upper;
    up->dev.jaccard = pl->dev.jaccard;
    up->out_begin = pl->hi_begin;
    up->out_end = d_c_rowptr + 1;
    return run(up);
}

namespace {
// Pinned host blocks for the read-back of spsyrk_numeric_rows.  Allocating pinned memory takes a millisecond or
// more, so blocks of destroyed plans are kept for the next plan (a few hundred bytes each, never freed).
std::mutex g_host_pos_mutex;
std::vector<int64_t*> g_host_pos_pool;
cudaError_t host_pos_acquire(int64_t** out) {
    {
        std::lock_guard<std::mutex> lock(g_host_pos_mutex);
        if (!g_host_pos_pool.empty()) {
            *out = g_host_pos_pool.back();
            g_host_pos_pool.pop_back();
            return cudaSuccess;
        }
    }
    return cudaHostAlloc(reinterpret_cast<void**>(out), 4 * NCLASS * sizeof(int64_t), cudaHostAllocMapped | cudaHostAllocPortable);
}
void host_pos_release(int64_t* p) {
    std::lock_guard<std::mutex> lock(g_host_pos_mutex);
    g_host_pos_pool.push_back(p);
}

// out[(2 * c) + e] = first position of class c's row list (ascending local row ids) whose row is >= bound[e]
__global__ void class_positions_kernel(const int32_t* __restrict__ perm, const int64_t* __restrict__ class_start_dev, int64_t lo_row,
                                       int64_t hi_row, int64_t* __restrict__ out) {
    const int t = threadIdx.x;
    if (t >= 2 * NCLASS) return;
    const int c = t >> 1;
    const int64_t bound = (t & 1) ? hi_row : lo_row;
    int64_t lo = class_start_dev[c], hi = class_start_dev[c + 1];
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)perm[mid] < bound) lo = mid + 1; else hi = mid;
    }
    out[t] = lo;
}
}  // namespace

spsyrk_status_t spsyrk_numeric_rows(spsyrk_plan_t plan, int64_t row_begin, int64_t row_end, const int64_t* d_c_rowptr,
                                    int32_t* d_c_colidx, void* d_c_vals, void* cuda_stream) {
    if (!plan || !d_c_rowptr) return SPSYRK_ERR_INVALID_ARG;
    spsyrk_plan_s* pl = plan;
    if (!pl->have_symbolic) return SPSYRK_ERR_SEQUENCE;
    if (row_begin < pl->dev.r0 || row_end > pl->dev.r1 || row_begin > row_end) return SPSYRK_ERR_INVALID_ARG;
    if (row_begin == row_end) return SPSYRK_OK;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // where the rows of the range sit in every class's list: one small kernel per view and one read-back
    // The kernel writes straight into pinned host memory: a device-to-host copy would queue behind whatever the
    // caller is downloading at the moment (the point of this call is to overlap with such copies).
    if (!pl->host_pos) SPSYRK_CUDA_TRY(host_pos_acquire(&pl->host_pos));
    int64_t* dev_pos = nullptr;
    SPSYRK_CUDA_TRY(cudaHostGetDevicePointer(reinterpret_cast<void**>(&dev_pos), pl->host_pos, 0));
    spsyrk_plan_s* views[2] = {pl, pl->upper_active ? pl->upper : nullptr};
    for (int v = 0; v < 2; ++v) {
        if (!views[v]) continue;
        class_positions_kernel<<<1, 32, 0, st>>>(views[v]->perm, views[v]->class_start_dev, row_begin - pl->dev.r0, row_end - pl->dev.r0,
                                                 dev_pos + v * 2 * NCLASS);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(cudaGetLastError());
    SPSYRK_CUDA_TRY(cudaStreamSynchronize(st));
    const int64_t(*pos)[2 * NCLASS] = reinterpret_cast<const int64_t(*)[2 * NCLASS]>(pl->host_pos);
    for (int v = 0; v < 2; ++v) {
        if (!views[v]) continue;
        views[v]->sub_active = true;
        for (int c = 0; c < NCLASS; ++c) { views[v]->sub_lo[c] = pos[v][2 * c]; views[v]->sub_hi[c] = pos[v][2 * c + 1]; }
    }
    const spsyrk_status_t s = spsyrk_numeric(plan, d_c_rowptr, d_c_colidx, d_c_vals, cuda_stream);
    for (int v = 0; v < 2; ++v)
        if (views[v]) views[v]->sub_active = false;
    return s;
}

spsyrk_status_t spsyrk_onepass_slots(spsyrk_plan_t plan, int64_t* slot_entries, void* cuda_stream) {
    if (!plan || !slot_entries) return SPSYRK_ERR_INVALID_ARG;
    spsyrk_plan_s* pl = plan;
    if (pl->upper_active) return SPSYRK_ERR_NOT_IMPLEMENTED;  // the two-part full-output mode keeps the two-pass route
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    pl->have_onepass = false;
    if (rows > 0) SPSYRK_CUDA_TRY(cudaMemsetAsync(pl->cnt, 0, (size_t)rows * sizeof(int32_t), st));
    // heavy rows: their counts come from their own kernels (bitmaps), as in the symbolic pass
    spsyrk_status_t s = launch_symbolic_cta<256>(pl, 6, st);
    if (s != SPSYRK_OK) return s;
    s = launch_symbolic_cta<1024>(pl, 7, st);
    if (s != SPSYRK_OK) return s;
    if (rows > 0) {
        onepass_slots_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(pl->dev, pl->cls, pl->cnt, pl->diag, rows, pl->ub);
        note_launches(1);
    }
    SPSYRK_CUDA_TRY(exclusive_scan_i64<int32_t>(pl->ub, rows, pl->ub_off, pl->partials, st));
    int64_t total = 0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&total, pl->ub_off + rows, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    s = read_err(pl, st);
    if (s != SPSYRK_OK) return s;
    *slot_entries = total;
    pl->have_onepass = true;
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_onepass_numeric(spsyrk_plan_t plan, int32_t* d_slot_colidx, void* d_slot_vals, int64_t* d_c_rowptr, int64_t* nnz_out,
                                       void* cuda_stream) {
    if (!plan || !d_c_rowptr || !nnz_out) return SPSYRK_ERR_INVALID_ARG;
    spsyrk_plan_s* pl = plan;
    if (!pl->have_onepass) return SPSYRK_ERR_SEQUENCE;
    if (pl->dev.jaccard) return SPSYRK_ERR_INVALID_ARG;  // the fused similarity is written at final offsets only
    if (pl->work_total > 0 && (!d_slot_colidx || !d_slot_vals)) return SPSYRK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    // every row is computed into its slot; the light rows report their counts (the heavy ones have theirs already)
    const bool map_was = pl->map_filled;
    pl->map_filled = false;  // the kernel that sorts in the numeric pass counts as it goes
    pl->cnt_out = pl->cnt;
    pl->out_begin = pl->ub_off;
    pl->out_end = pl->ub_off + 1;
    spsyrk_status_t s;
    switch (pl->dtype) {
        case SPSYRK_F64: s = numeric_typed<double>(pl, d_slot_colidx, d_slot_vals, st); break;
        case SPSYRK_F32: s = numeric_typed<float>(pl, d_slot_colidx, d_slot_vals, st); break;
        default: s = numeric_typed<int32_t>(pl, d_slot_colidx, d_slot_vals, st); break;
    }
    pl->cnt_out = nullptr;
    pl->map_filled = map_was;
    if (s != SPSYRK_OK) return s;
    SPSYRK_CUDA_TRY(exclusive_scan_i64<int32_t>(pl->cnt, rows, d_c_rowptr, pl->partials, st));
    int64_t nnz = 0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(&nnz, d_c_rowptr + rows, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    s = read_err(pl, st);
    if (s != SPSYRK_OK) return s;
    *nnz_out = nnz;
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_onepass_row_begin(spsyrk_plan_t plan, int64_t* d_row_begin, void* cuda_stream) {
    if (!plan || !d_row_begin) return SPSYRK_ERR_INVALID_ARG;
    if (!plan->have_onepass) return SPSYRK_ERR_SEQUENCE;
    const int64_t rows = plan->dev.r1 - plan->dev.r0;
    SPSYRK_CUDA_TRY(cudaMemcpyAsync(d_row_begin, plan->ub_off, (size_t)(rows + 1) * sizeof(int64_t), cudaMemcpyDeviceToDevice,
                                    static_cast<cudaStream_t>(cuda_stream)));
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_onepass_compact(spsyrk_plan_t plan, const int64_t* d_c_rowptr, int64_t nnz, const int32_t* d_slot_colidx,
                                       const void* d_slot_vals, int32_t* d_c_colidx, void* d_c_vals, void* cuda_stream) {
    if (!plan || !d_c_rowptr || nnz < 0) return SPSYRK_ERR_INVALID_ARG;
    spsyrk_plan_s* pl = plan;
    if (!pl->have_onepass) return SPSYRK_ERR_SEQUENCE;
    if (nnz > 0 && (!d_slot_colidx || !d_slot_vals || !d_c_colidx || !d_c_vals)) return SPSYRK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int64_t rows = pl->dev.r1 - pl->dev.r0;
    if (rows > 0 && nnz > 0) {
        if (pl->dtype == SPSYRK_F64) launch_onepass_compact<uint64_t>(pl, d_c_rowptr, rows, nnz, d_slot_colidx, d_slot_vals, d_c_colidx, d_c_vals, st);
        else launch_onepass_compact<uint32_t>(pl, d_c_rowptr, rows, nnz, d_slot_colidx, d_slot_vals, d_c_colidx, d_c_vals, st);
    }
    SPSYRK_CUDA_TRY(cudaGetLastError());
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_plan_map_bytes(spsyrk_plan_t plan, size_t* bytes) {
    if (!plan || !bytes) return SPSYRK_ERR_INVALID_ARG;
    *bytes = (size_t)map_items_total(plan) * sizeof(uint16_t);
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_plan_lend_map(spsyrk_plan_t plan, void* d_map, size_t bytes) {
    if (!plan || (d_map && reinterpret_cast<uintptr_t>(d_map) % ALIGN)) return SPSYRK_ERR_INVALID_ARG;
    plan->map = static_cast<uint16_t*>(d_map);
    plan->map_bytes = d_map ? bytes : 0;
    plan->map_filled = false;
    plan->have_symbolic = false;
    if (plan->upper) { plan->upper->map_filled = false; plan->upper->have_symbolic = false; }
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_plan_set_jaccard(spsyrk_plan_t plan, float* d_jaccard) {
    if (!plan) return SPSYRK_ERR_INVALID_ARG;
    if (d_jaccard && plan->dtype != SPSYRK_I32) return SPSYRK_ERR_INVALID_ARG;
    plan->dev.jaccard = d_jaccard;
    if (plan->upper) plan->upper->dev.jaccard = d_jaccard;
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_plan_stats(spsyrk_plan_t plan, int64_t* work_total, int64_t class_rows[8]) {
    if (!plan) return SPSYRK_ERR_INVALID_ARG;
    if (work_total) *work_total = plan->work_total + (plan->upper_active ? plan->upper->work_total : 0);
    if (class_rows)
        for (int c = 0; c < NCLASS; ++c) class_rows[c] = plan->class_start[c + 1] - plan->class_start[c];
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_plan_buffers(spsyrk_plan_t plan, const int64_t** d_colptr, const int32_t** d_at_row,
                                    const void** d_at_rec, const int64_t** d_work) {
    if (!plan) return SPSYRK_ERR_INVALID_ARG;
    if (d_colptr) *d_colptr = plan->dev.colptr;
    if (d_at_row) *d_at_row = plan->dev.at_row;
    if (d_at_rec) *d_at_rec = plan->dev.at_rec;
    if (d_work) *d_work = plan->upper_active ? plan->work_sum : plan->dev.work;
    return SPSYRK_OK;
}

void spsyrk_destroy(spsyrk_plan_t plan) {
    if (!plan) return;
    if (plan->timing)
        for (int i = 0; i <= NCLASS; ++i) { cudaEventDestroy(plan->ev_sym[i]); cudaEventDestroy(plan->ev_num[i]); }
    if (plan->host_pos) host_pos_release(plan->host_pos);
    delete plan->upper;
    delete plan;
}

spsyrk_status_t spsyrk_plan_enable_timing(spsyrk_plan_t plan) {
    if (!plan) return SPSYRK_ERR_INVALID_ARG;
    if (plan->timing) return SPSYRK_OK;
    for (int i = 0; i <= NCLASS; ++i) {
        SPSYRK_CUDA_TRY(cudaEventCreate(&plan->ev_sym[i]));
        SPSYRK_CUDA_TRY(cudaEventCreate(&plan->ev_num[i]));
    }
    plan->timing = true;
    return SPSYRK_OK;
}

spsyrk_status_t spsyrk_plan_timings(spsyrk_plan_t plan, float symbolic_ms[8], float numeric_ms[8]) {
    if (!plan || !plan->timing || !symbolic_ms || !numeric_ms) return SPSYRK_ERR_INVALID_ARG;
    if (!plan->have_symbolic) return SPSYRK_ERR_SEQUENCE;
    symbolic_ms[0] = numeric_ms[0] = 0.f;
    for (int c = 1; c < NCLASS; ++c) {
        symbolic_ms[c] = numeric_ms[c] = 0.f;
        SPSYRK_CUDA_TRY(cudaEventSynchronize(plan->ev_sym[c + 1]));
        SPSYRK_CUDA_TRY(cudaEventElapsedTime(&symbolic_ms[c], plan->ev_sym[c], plan->ev_sym[c + 1]));
        if (cudaEventQuery(plan->ev_num[c + 1]) == cudaSuccess && cudaEventQuery(plan->ev_num[c]) == cudaSuccess)
            cudaEventElapsedTime(&numeric_ms[c], plan->ev_num[c], plan->ev_num[c + 1]);
    }
    cudaGetLastError();
    return SPSYRK_OK;
}

int64_t spsyrk_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

const char* spsyrk_status_string(spsyrk_status_t s) {
    switch (s) {
        case SPSYRK_OK: return "ok";
        case SPSYRK_ERR_INVALID_ARG: return "invalid argument";
        case SPSYRK_ERR_BAD_CSR: return "input is not canonical CSR";
        case SPSYRK_ERR_WORKSPACE: return "workspace too small";
        case SPSYRK_ERR_OVERFLOW: return "size exceeds the supported range";
        case SPSYRK_ERR_SEQUENCE: return "call sequence error";
        case SPSYRK_ERR_CUDA: return "CUDA runtime error";
        case SPSYRK_ERR_INTERNAL: return "internal error";
        case SPSYRK_ERR_NOT_IMPLEMENTED: return "not implemented";
    }
    return "unknown status";
}

}  // extern "C"
