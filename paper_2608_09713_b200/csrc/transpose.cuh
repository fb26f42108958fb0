// Step a1: on-device CSR transpose of A into column lists whose entries are ascending by row,
// plus the per-nonzero descriptors the row kernels consume.
//
//   colptr[n+1]        column pointers (int64)
//   at_row[q], at_rec[q]  entries of the column lists, q in [colptr[k], colptr[k+1]) ascending by row: the row ids
//                      alone (what the structure passes read) and (row id, value) records (what the value passes read)
//   desc[p] = (start, len) for nonzero p = (i, k) of A: start = colptr[k]; len = number of entries
//             of column k with row <= i (the rank of i in the list, plus one).  "Rows j <= i of
//             column k" is then at_row[start, start+len).  The full-output mode also keeps the rest of
//             the list, the rows j > i, as a second descriptor (start + len, column length - len).
//
// Method: histogram of column ids and scan for colptr; then a stable LSD radix sort of the
// nonzeros by column id with (row, value, position in A) as payload.  The nonzeros enter in row
// order, so each column's segment comes out ascending by row; the last pass writes at_row and
// at_rec and scatters the descriptor, whose length is the entry's rank inside its column.  (The
// value travels with the element because reading it in the first pass is sequential, whereas
// fetching it by position in the last pass is one random access per nonzero.)
#pragma once
#include "radix.cuh"

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
    // (the values of the column lists live in the records only)
    void* at_rec;  // the same entries as interleaved (row id, value) records: ColRec<V>[nnz]
    uint2* desc;
    int64_t* work;  // per row of the range
    uint32_t* err;
    // Binary input (every stored value is exactly one): a partial product is 1 and an entry of the
    // product is an intersection count.  Then the heaviest columns (at most 64, chosen by their number
    // of entries) are also kept as one bit per row, heavy_mask[i] bit b = row i stores heavy column b, so
    // that their share of a count is popcount(heavy_mask[i] & heavy_mask[j]) instead of one list walk each.
    int32_t binary;               // 0 / 1, valid after the plan's analysis
    int32_t nheavy;               // heavy columns in use (0: none)
    const uint8_t* heavy_id;      // [n] bit number of a heavy column, 0xff otherwise
    const uint64_t* heavy_mask;   // [m]
    float* jaccard;               // optional: the numeric pass also writes c / (|a_i| + |a_j| - c) here (int32 values)
    const int32_t* adeg;          // [m] stored entries per row of A (|a_i| of the Jaccard formula)
};

static __global__ void __launch_bounds__(256) row_degree_kernel(const int64_t* __restrict__ rowptr, int32_t m, int32_t* __restrict__ adeg) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) adeg[i] = (int32_t)(rowptr[i + 1] - rowptr[i]);
}

// ---------------------------------------------------------------------------------------------
// Analysis of a binary matrix: value check, choice of the heavy columns, the per-row bit masks.
// facts[0] = 1 if some stored value differs from one; facts[1] = heavy columns; facts[2] = threshold.
// ---------------------------------------------------------------------------------------------
template <typename V>
static __global__ void __launch_bounds__(256) binary_check_kernel(const V* __restrict__ vals, int64_t nnz, uint32_t* __restrict__ facts) {
    int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool other = false;
    for (; p < nnz; p += stride) other |= !(vals[p] == V(1));
    if (__any_sync(FULL_MASK, other) && lane_id() == 0) atomicOr(&facts[0], 1u);
}

// histogram of floor(log2(column length)) over the columns
static __global__ void __launch_bounds__(256) heavy_hist_kernel(const uint32_t* __restrict__ colcnt, int64_t n, uint32_t* __restrict__ hist32) {
    __shared__ uint32_t h[32];
    if (threadIdx.x < 32) h[threadIdx.x] = 0;
    __syncthreads();
    int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; k < n; k += stride) {
        const uint32_t d = colcnt[k];
        if (d >= 256u) atomicAdd(&h[31 - __clz(d)], 1u);  // lighter columns are never candidates
    }
    __syncthreads();
    if (threadIdx.x < 32 && h[threadIdx.x]) atomicAdd(&hist32[threadIdx.x], h[threadIdx.x]);
}

// threshold = the smallest power of two such that at most 64 columns have that many entries or more
static __global__ void heavy_threshold_kernel(const uint32_t* __restrict__ hist32, uint32_t* __restrict__ facts) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    uint32_t total = 0, thr = 0xffffffffu;
    for (int b = 31; b >= 8; --b) {
        if (total + hist32[b] > 64u) break;
        total += hist32[b];
        if (hist32[b]) thr = 1u << b;
    }
    facts[1] = 0;
    facts[2] = facts[0] ? 0xffffffffu : thr;  // no heavy columns unless the matrix is binary
}

static __global__ void __launch_bounds__(256) heavy_assign_kernel(const uint32_t* __restrict__ colcnt, int64_t n, uint32_t* __restrict__ facts,
                                                                 uint8_t* __restrict__ heavy_id) {
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= n) return;
    uint8_t id = 0xff;
    if (colcnt[k] >= facts[2]) {
        const uint32_t b = atomicAdd(&facts[1], 1u);
        if (b < 64u) id = (uint8_t)b;
    }
    heavy_id[k] = id;
}

template <int G>
static __global__ void __launch_bounds__(256) heavy_mask_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ colidx, int32_t m,
                                                               const uint32_t* __restrict__ facts, const uint8_t* __restrict__ heavy_id,
                                                               uint64_t* __restrict__ heavy_mask) {
    if (facts[1] == 0) return;  // no heavy column: nothing reads the masks (a fixed grid walks the rows, so the launch costs nothing then)
    const int gl = threadIdx.x & (G - 1);
    const int64_t groups = ((int64_t)gridDim.x * blockDim.x) / G;
    for (int64_t base = ((int64_t)blockIdx.x * blockDim.x) / G; base < m; base += groups) {  // uniform per CTA
        const int64_t gid = base + threadIdx.x / G;
        unsigned long long mk = 0;
        if (gid < m) {
            const int64_t p0 = rowptr[gid], p1 = rowptr[gid + 1];
            for (int64_t p = p0 + gl; p < p1; p += G) {
                const uint8_t id = heavy_id[colidx[p]];
                if (id != 0xff) mk |= 1ull << id;
            }
        }
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) mk |= __shfl_xor_sync(FULL_MASK, mk, o);
        if (gid < m && gl == 0) heavy_mask[gid] = mk;
    }
}

// One entry of a column list as a record: what the light-row numeric kernel gathers (one aligned
// asynchronous copy per entry, whatever the list's offset).
template <typename V> struct ColRec;
template <> struct alignas(16) ColRec<double> { int32_t j; int32_t pad; double v; };
template <> struct alignas(8) ColRec<float> { int32_t j; float v; };
template <> struct alignas(8) ColRec<int32_t> { int32_t j; int32_t v; };

static __global__ void validate_rowptr_kernel(const int64_t* __restrict__ rowptr, int64_t m, int64_t nnz, uint32_t* err) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m) {
        int64_t a = rowptr[i], b = rowptr[i + 1];
        if (a > b || a < 0 || b > nnz) atomicOr(err, ERRW_BAD_ROWPTR);
    }
    if (i == 0 && (rowptr[0] != 0 || rowptr[m] != nnz)) atomicOr(err, ERRW_BAD_ROWPTR);
}

// G lanes per row, one sweep over the nonzeros of A: the column histogram (its scan gives colptr), the explicit
// row id of every nonzero (the radix sort's first payload), and the checks that column ids are in range and
// strictly ascending inside the row.  The row pointers have been validated before.
template <int G>
static __global__ void __launch_bounds__(256) row_expand_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ colidx,
                                                                int32_t m, int32_t n, uint32_t* __restrict__ colcnt,
                                                                uint32_t* __restrict__ rowid, uint32_t* err) {
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (gid >= m) return;
    const int64_t p0 = rowptr[gid], p1 = rowptr[gid + 1];
    for (int64_t p = p0 + gl; p < p1; p += G) {
        const int32_t k = colidx[p];
        if ((uint32_t)k >= (uint32_t)n) atomicOr(err, ERRW_BAD_COL);
        else atomicAdd(&colcnt[k], 1u);
        if (p > p0 && colidx[p - 1] >= k) atomicOr(err, ERRW_UNSORTED);
        rowid[p] = (uint32_t)gid;
    }
}

// last radix pass of the transpose: the element at sorted position s is entry s of the column lists
template <typename VB>
struct EmitTransposeFinal {
    PlanDev P;
    uint2* desc_hi;  // null in lower-triangle mode
    __device__ __forceinline__ void operator()(int64_t s, uint32_t k, uint32_t row, VB val, uint32_t p) const {
        const int64_t cs = P.colptr[k];
        P.at_row[s] = (int32_t)row;
        if constexpr (sizeof(VB) == 8) static_cast<uint4*>(P.at_rec)[s] = make_uint4(row, 0u, (uint32_t)val, (uint32_t)(val >> 32));
        else static_cast<uint2*>(P.at_rec)[s] = make_uint2(row, (uint32_t)val);
        // the entries of column k with row <= i are the first rank + 1 of its list; the full-output mode also keeps
        // the rest of the list (rows > i) as a second descriptor
        const uint32_t rank1 = (uint32_t)(s - cs) + 1u;
        P.desc[p] = make_uint2((uint32_t)cs, rank1);
        if (desc_hi) desc_hi[p] = make_uint2((uint32_t)cs + rank1, (uint32_t)(P.colptr[k + 1] - cs) - rank1);
    }
};

// Restriction of the plan to output columns [s0, s1): column k's entries with row in that range are
// a contiguous piece of its (row-sorted) list, so the descriptor of every nonzero of the rows
// [r0, r1) is narrowed to that piece by two binary searches inside its full-range prefix.
template <int G>
// desc_hi (full-output mode): the rest of every column list; the block is then cut out of the whole list.
static __global__ void __launch_bounds__(256) block_desc_kernel(PlanDev P, const uint2* __restrict__ desc_full, const uint2* __restrict__ desc_hi,
                                                                uint2* __restrict__ desc_blk, int32_t s0, int32_t s1) {
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    const int gl = threadIdx.x & (G - 1);
    if (gid >= P.r1 - P.r0) return;
    const int64_t i = P.r0 + gid;
    const int64_t p0 = P.rowptr[i], p1 = P.rowptr[i + 1];
    for (int64_t p = p0 + gl; p < p1; p += G) {
        uint2 full = desc_full[p];
        if (desc_hi) full.y += desc_hi[p].y;
        const int32_t* lst = P.at_row + full.x;
        const uint32_t lo = s0 <= 0 ? 0u : lower_bound_i32(lst, full.y, s0);
        const uint32_t hi = lower_bound_i32(lst, full.y, s1);
        desc_blk[p] = make_uint2(full.x + lo, hi > lo ? hi - lo : 0u);
    }
}

// Step a2: per-row work w[i] = sum of the descriptor lengths of row i (G lanes per row), and the
// class of the row.  Rows of the range [r0, r1) only.
//   class 0: no work; 1..5: w <= 32, 64, 128, 256, 512 and at most 32 nonzeros (one warp, register sort)
//   6: w <= block_max (one 256-thread CTA, bitmap accumulator); 7: larger (one 1024-thread CTA)
template <int G>
//   diag: the light-row kernels leave the diagonal products out of their item lists (lower-triangle mode
//   over the whole column range), so a light row is classed by w minus its number of nonzeros
static __global__ void __launch_bounds__(256) row_work_kernel(PlanDev P, uint8_t* __restrict__ cls, int64_t block_max, bool diag,
                                                        unsigned long long* __restrict__ work_total) {
    const int gl = threadIdx.x & (G - 1);
    const int64_t rows = P.r1 - P.r0;
    const int64_t groups = ((int64_t)gridDim.x * blockDim.x) / G;
    unsigned long long mine = 0;  // work of the rows this thread owned
    // a fixed grid walks the rows: one atomic per CTA for the total, however many rows there are
    for (int64_t gbase = ((int64_t)blockIdx.x * blockDim.x) / G; gbase < rows; gbase += groups) {  // uniform per CTA
        const int64_t gid = gbase + threadIdx.x / G;
        int64_t w = 0, deg = 0;
        if (gid < rows) {
            const int64_t i = P.r0 + gid;
            const int64_t p0 = P.rowptr[i], p1 = P.rowptr[i + 1];
            deg = p1 - p0;
            for (int64_t p = p0 + gl; p < p1; p += G) w += P.desc[p].y;
        }
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) w += __shfl_xor_sync(FULL_MASK, w, o);
        if (gid < rows && gl == 0) {
            P.work[gid] = w;
            uint8_t c;
            const int64_t wl = diag ? w - deg : w;  // items of a light row
            if (w == 0) c = 0;
            else if (deg <= 32 && wl <= 512) c = wl <= 32 ? 1 : wl <= 64 ? 2 : wl <= 128 ? 3 : wl <= 256 ? 4 : 5;
            else c = w <= block_max ? 6 : 7;
            cls[gid] = c;
            mine += (unsigned long long)w;
        }
    }
    __shared__ unsigned long long cta_sum;
    if (threadIdx.x == 0) cta_sum = 0;
    __syncthreads();
    const unsigned long long ws = warp_reduce_sum<unsigned long long>(mine);
    if (lane_id() == 0 && ws) atomicAdd(&cta_sum, ws);
    __syncthreads();
    if (threadIdx.x == 0 && cta_sum) atomicAdd(work_total, cta_sum);
}

}  // namespace spsyrk
