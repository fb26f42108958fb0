/*
 * spsyrk.h - C ABI of the B200 local sparse SYRK library (libspsyrk.so).
 *
 * Computes the lower triangle, diagonal included, of the Gram matrix of a sparse matrix,
 *     C_L = tril(A * A^T),   A in CSR,
 * without forming the upper half, plus the optional materialisation of the full symmetric
 * matrix from the computed half and a Jaccard normalisation of intersection counts.
 *
 * Conventions
 *   - Every pointer named d_* is a DEVICE pointer, owned by the caller; h_* and plain
 *     out-parameters (int64_t *nnz_out, size_t *workspace_bytes, ...) are HOST pointers.
 *   - The library allocates no device memory except inside spsyrk_host_tril.  Scratch space
 *     is a caller-owned device workspace whose size is queried first.
 *   - CSR everywhere: int64 row pointers, int32 column ids, values of the given dtype.  Input
 *     must be canonical: column ids strictly ascending inside each row (no duplicates) and
 *     in [0, n).  Output rows are sorted ascending by column id.
 *   - Stored entries are structural: (i, j) is stored iff rows i and j of A share at least one
 *     stored column, whatever the value of the sum.  A row of A without entries gives an
 *     empty output row (no diagonal entry).
 *   - All device work is enqueued on the CUDA stream passed as `cuda_stream` (a cudaStream_t
 *     cast to void*; NULL is the default stream).  Functions that hand a value back to the
 *     host (sizes, nnz, error words) synchronise that stream; the others are asynchronous.
 *   - Every function returns a status and never throws or aborts.  On error, outputs are
 *     unspecified.  Limits: m, n < 2^31, nnz(A) < 2^31; nnz of the result is 64-bit.
 */
#ifndef SPSYRK_H
#define SPSYRK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spsyrk_plan_s *spsyrk_plan_t; /* opaque, created by spsyrk_plan, freed by spsyrk_destroy */

typedef enum {
    SPSYRK_OK = 0,
    SPSYRK_ERR_INVALID_ARG = 1,     /* null pointer, negative size, bad enum, bad row range */
    SPSYRK_ERR_BAD_CSR = 2,         /* row pointers not monotone, column ids unsorted / duplicate / out of range */
    SPSYRK_ERR_WORKSPACE = 3,       /* workspace smaller than the queried size */
    SPSYRK_ERR_OVERFLOW = 4,        /* a size exceeds the limits above */
    SPSYRK_ERR_SEQUENCE = 5,        /* numeric before symbolic, or a stale plan */
    SPSYRK_ERR_CUDA = 6,            /* a CUDA runtime call failed */
    SPSYRK_ERR_INTERNAL = 7,        /* a bounded device loop gave up (should not happen) */
    SPSYRK_ERR_NOT_IMPLEMENTED = 8
} spsyrk_status_t;

typedef enum { SPSYRK_F64 = 0, SPSYRK_F32 = 1, SPSYRK_I32 = 2 } spsyrk_dtype_t;

/* SPSYRK_TRIL keeps products a_ik * a_jk with j <= i only (Section III-A: a diagonal process
 * computes only the lower triangle; Algorithm 2, line 2).  SPSYRK_FULL removes the cut-off and
 * yields all of A * A^T with the same kernels; it exists to measure the work the symmetry saves
 * (sigma_mul = 1/2 in the cost table of Section III-C). */
typedef enum { SPSYRK_TRIL = 0, SPSYRK_FULL = 1 } spsyrk_mode_t;

/*
 * spsyrk_plan - analyse A for output rows [row_begin, row_end).
 *
 * Steps (all on the device): validate the CSR; transpose A into column lists whose entries
 * are ascending by row (the input transpose of Sections III and IV-B, done locally), so that
 * "rows j <= i of column k" is a prefix of the list; per-row work estimate
 *     w[i] = sum over nonzeros a_ik of #{entries of column k with row <= i}
 * (in FULL mode the whole column), whose total is the multiply-add count of Section III-C
 * (sum_k d_k (d_k + 1) / 2 for the half, sum_k d_k^2 for the full product); binning of the
 * rows by w into warp / block / large classes.
 *
 * Two-phase: call with d_workspace == NULL to receive *workspace_bytes (no device work, *plan
 * untouched); then call with a buffer of at least that size, 256-byte aligned.  A, the
 * workspace and the stream's device must outlive the plan; A is read, never written.
 * The second call synchronises the stream once (validation result and bin sizes).
 *
 * Row tiles: plans for disjoint row ranges are independent; concatenating their results gives
 * the untiled C_L.  (Halving a CSR matrix along rows is free, Section IV-A.)
 *
 * d_rowptr[m+1], d_colidx[nnz], d_vals[nnz] of `dtype`.  0 <= row_begin <= row_end <= m.
 * Errors: INVALID_ARG, OVERFLOW, WORKSPACE, BAD_CSR, CUDA.
 */
spsyrk_status_t spsyrk_plan(spsyrk_plan_t *plan, int64_t m, int64_t n, int64_t nnz,
                            const int64_t *d_rowptr, const int32_t *d_colidx, const void *d_vals,
                            spsyrk_dtype_t dtype, spsyrk_mode_t mode,
                            int64_t row_begin, int64_t row_end,
                            void *d_workspace, size_t *workspace_bytes, void *cuda_stream);

/*
 * spsyrk_plan_set_rows - re-target an existing plan to another row range of the same A without
 * repeating the transpose (only the work estimate and the binning are redone).  Invalidates
 * any symbolic result.  Synchronises the stream once.
 */
spsyrk_status_t spsyrk_plan_set_rows(spsyrk_plan_t plan, int64_t row_begin, int64_t row_end,
                                     void *cuda_stream);

/*
 * spsyrk_plan_set_block - re-target an existing plan to the block
 *     C[R, S] = A[R, :] * A[S, :]^T,   R = [row_begin, row_end),  S = [col_begin, col_end),
 * i.e. output rows R restricted to output columns S (rows of A again), without repeating the
 * transpose.  These are the half-block products of the local computation (Algorithm 2, lines 4
 * and 6: a row half times the other operand, or all rows times a column half; Section IV-A:
 * halving along rows is a prefix of the row pointers, halving along columns needs the transpose -
 * which the plan already holds, so a column range is a contiguous piece of every column list).
 * The plan's mode still applies: in TRIL mode only j <= i is kept (the cut matters when S overlaps
 * R: R = S gives the lower triangle of a diagonal block); in FULL mode the whole block is produced.
 * Column ids of the result stay global (in S); the row pointer is tile-local.  Invalidates any
 * symbolic result.  Synchronises the stream once.  spsyrk_plan_set_rows is the case S = [0, m).
 * Errors: INVALID_ARG, CUDA.
 */
spsyrk_status_t spsyrk_plan_set_block(spsyrk_plan_t plan, int64_t row_begin, int64_t row_end,
                                      int64_t col_begin, int64_t col_end, void *cuda_stream);

/*
 * spsyrk_plan_map_bytes / spsyrk_plan_lend_map - optional item map for the light rows.
 *
 * A light row (at most 32 nonzeros, at most 512 partial products) is computed from the list of its
 * partial products a_ik * a_jk, "items", in ascending k and j.  Producing the row sorted by j means
 * ordering the items by j; that ordering depends on the structure of A only.  If the caller lends a
 * device buffer of spsyrk_plan_map_bytes bytes (two bytes per item of the plan's current row range,
 * rows padded to eight items), spsyrk_symbolic orders the items once and records for every item the
 * output slot it adds into and its place among the items of that slot, and spsyrk_numeric only
 * gathers, multiplies and adds - also for every later spsyrk_numeric call on the same structure.
 * Without a map (or with one that is too small for the current row range) symbolic counts with a
 * hash set and numeric sorts by itself; the results are identical bit for bit either way
 * (both add the partial products of an entry in ascending k: Section II-A's dot product, left to right).
 *
 * The size is known after spsyrk_plan / spsyrk_plan_set_rows / spsyrk_plan_set_block (it changes with
 * the row range).  The buffer is caller-owned, 256-byte aligned, and must stay valid from
 * spsyrk_symbolic to the last spsyrk_numeric that uses it; lending invalidates any symbolic result.
 * d_map == NULL takes the map back.  Errors: INVALID_ARG.
 */
spsyrk_status_t spsyrk_plan_map_bytes(spsyrk_plan_t plan, size_t *bytes);
spsyrk_status_t spsyrk_plan_lend_map(spsyrk_plan_t plan, void *d_map, size_t bytes);

/*
 * spsyrk_symbolic - count the stored entries of every output row of the plan's range and
 * turn the counts into row pointers.
 *   cnt[i] = #{ j <= i : rows i and j of A share a column }   (TRIL; all j in FULL mode)
 * d_c_rowptr[rows + 1] (rows = row_end - row_begin) receives the exclusive 64-bit prefix sums,
 * starting at 0 (tile-local).  *nnz_out = d_c_rowptr[rows] is valid on return (one stream
 * synchronisation).  The lower triangle includes the diagonal (Section V-F).
 * Errors: INVALID_ARG, INTERNAL, CUDA.
 */
spsyrk_status_t spsyrk_symbolic(spsyrk_plan_t plan, int64_t *d_c_rowptr, int64_t *nnz_out,
                                void *cuda_stream);

/*
 * spsyrk_numeric - fill the rows counted by spsyrk_symbolic.
 * For each nonzero a_ik of row i and each entry (j, a_jk) of column k with j <= i:
 * acc[j] += a_ik * a_jk (row-by-row accumulation; Section II-A defines c_ij as the dot product
 * of rows i and j; Algorithm 2 line 2 restricts it to the lower triangle).  Writes
 * d_c_colidx[nnz] (global column ids, ascending inside a row) and d_c_vals[nnz] of the plan's
 * dtype (F32 input is accumulated in double and rounded once; I32 wraps modulo 2^32).
 * d_c_rowptr must be the array spsyrk_symbolic wrote for this plan.  Asynchronous.
 * Errors: INVALID_ARG, SEQUENCE, CUDA.
 */
spsyrk_status_t spsyrk_numeric(spsyrk_plan_t plan, const int64_t *d_c_rowptr,
                               int32_t *d_c_colidx, void *d_c_vals, void *cuda_stream);

/*
 * spsyrk_numeric_rows - spsyrk_numeric for the output rows [row_begin, row_end) only (global row ids inside
 * the plan's range).  The entries of these rows are written at the offsets d_c_rowptr gives them, exactly as
 * spsyrk_numeric would; the rest of d_c_colidx / d_c_vals is not touched.  Calling it over a partition of the
 * range therefore fills C_L block by block, e.g. to copy finished row blocks to the host while later ones are
 * computed (row blocks are independent: Algorithm 2 works on any row range, the halving of the rows costs
 * nothing).  Reads the positions of the range in the plan's row lists back (one stream synchronisation)
 * before it launches.  Errors: INVALID_ARG (range outside the plan's), SEQUENCE, CUDA.
 */
spsyrk_status_t spsyrk_numeric_rows(spsyrk_plan_t plan, int64_t row_begin, int64_t row_end,
                                    const int64_t *d_c_rowptr, int32_t *d_c_colidx, void *d_c_vals,
                                    void *cuda_stream);

/*
 * One-pass mode: the product of spsyrk_symbolic + spsyrk_numeric (Section II-A, Algorithm 2 line 2: the lower
 * triangle of A A^T, rows ascending in column) without a separate symbolic pass, for callers that can afford a
 * second, slightly larger output buffer.  Every light row gets a slot sized by the number of its partial products (an upper bound of its
 * entries; the heavy rows, which find their structure in bitmaps anyway, get exact slots), the numeric kernel
 * that sorts a row's products computes the row into its slot and reports its count, and the rows are then moved
 * to their places.  The column lists are gathered once instead of twice.
 *   1. spsyrk_onepass_slots: *slot_entries = entries the slot buffers need (>= nnz(C_L); synchronises).
 *   2. spsyrk_onepass_numeric: fills d_slot_colidx / d_slot_vals (slot_entries entries each), writes
 *      d_c_rowptr[rows + 1] and *nnz_out (synchronises).
 *   3. spsyrk_onepass_compact: copies the rows into d_c_colidx / d_c_vals (nnz entries).  Asynchronous.
 *      Optional: after step 2 the slot buffers already hold C_L in the four-array form of CSR (row begin and
 *      row end given separately): row r occupies [b[r], b[r] + d_c_rowptr[r + 1] - d_c_rowptr[r]) of the slot
 *      buffers with b = the rows + 1 offsets spsyrk_onepass_row_begin copies out; a consumer that accepts that
 *      form skips step 3 and the second buffer.
 * The result equals that of spsyrk_symbolic + spsyrk_numeric (same summation order for the light rows).
 * Not available for the full-output mode over the whole column range (NOT_IMPLEMENTED) nor together with
 * spsyrk_plan_set_jaccard (INVALID_ARG).  Errors: INVALID_ARG, SEQUENCE, INTERNAL, CUDA.
 */
spsyrk_status_t spsyrk_onepass_slots(spsyrk_plan_t plan, int64_t *slot_entries, void *cuda_stream);
spsyrk_status_t spsyrk_onepass_numeric(spsyrk_plan_t plan, int32_t *d_slot_colidx, void *d_slot_vals,
                                       int64_t *d_c_rowptr, int64_t *nnz_out, void *cuda_stream);
spsyrk_status_t spsyrk_onepass_row_begin(spsyrk_plan_t plan, int64_t *d_row_begin, void *cuda_stream);
spsyrk_status_t spsyrk_onepass_compact(spsyrk_plan_t plan, const int64_t *d_c_rowptr, int64_t nnz,
                                       const int32_t *d_slot_colidx, const void *d_slot_vals,
                                       int32_t *d_c_colidx, void *d_c_vals, void *cuda_stream);

/*
 * spsyrk_mirror - materialise F = C_L + C_L^T - D, the full symmetric matrix, from a complete
 * (untiled or re-assembled) lower triangle (Section III-A: the full matrix, when it is needed, is
 * obtained from the stored half by a transpose; Section V-F: C = C_L + C_L^T - D).  Row i of F is row i of C_L followed by (r, c_ri) for
 * every later row r that stores column i, ascending in r; values are bit copies, so F is
 * exactly symmetric and tril(F) == C_L.
 *
 * C_L must have its rows ascending in column, as spsyrk_numeric writes them.
 *
 * Three-step use:
 *   1. d_workspace == NULL: *workspace_bytes receives the scratch size for (m, nnz_l, dtype).
 *   2. d_f_colidx == NULL: looks at the first and last entry of every row (with ascending rows that
 *      finds any entry above the diagonal and every stored diagonal) and returns
 *      *nnz_full_out = 2 nnz_l - #diagonal entries (synchronises).  d_f_rowptr is not written yet.
 *   3. all pointers set: writes d_f_rowptr[m + 1] and fills d_f_colidx / d_f_vals (nnz_full entries).
 *      Asynchronous.  An entry above the diagonal that step 2 could not see (a row that is not
 *      ascending) is left out of the reflection; it never indexes outside the arrays.
 *      Until this step's work on the stream has completed, d_f_colidx and d_f_vals (the sizes step 2
 *      gave: nnz_full entries each) also serve as scratch of the sort, which is why the workspace is about
 *      1.5 (8-byte values) to 2.2 (4-byte values) times the bytes of C_L and not 3 times; both arrays must
 *      be 16-byte aligned and must not overlap each other, the workspace or C_L (INVALID_ARG if misaligned).
 * nnz_l = d_l_rowptr[m].  Errors: INVALID_ARG, WORKSPACE, BAD_CSR (an entry above the diagonal), CUDA.
 */
spsyrk_status_t spsyrk_mirror(int64_t m, int64_t nnz_l, spsyrk_dtype_t dtype,
                              const int64_t *d_l_rowptr, const int32_t *d_l_colidx, const void *d_l_vals,
                              int64_t *d_f_rowptr, int32_t *d_f_colidx, void *d_f_vals,
                              int64_t *nnz_full_out,
                              void *d_workspace, size_t *workspace_bytes, void *cuda_stream);

/*
 * spsyrk_column_panel - A_s = A(:, [k0, k1)) as CSR, column ids and row order unchanged.
 * The diagonal block of the product is a sum of rank-k updates, one per column panel of A
 * (Section III-A: C_ii = sum over s of SYRK(A_is)); this call cuts one panel out of a canonical
 * CSR matrix so that it can be planned and multiplied on its own.
 *
 * Three-step use:
 *   1. d_workspace == NULL: *workspace_bytes receives the scratch size for m.
 *   2. d_p_colidx == NULL: writes d_p_rowptr[m + 1] and *nnz_out (synchronises).
 *   3. all pointers set: fills d_p_colidx / d_p_vals using the d_p_rowptr of step 2.  Asynchronous.
 * All pointers are device pointers except nnz_out and workspace_bytes (host); nothing is owned
 * by the library.  nnz = d_rowptr[m].  Requires 0 <= k0 <= k1.  Errors: INVALID_ARG, WORKSPACE, CUDA.
 */
spsyrk_status_t spsyrk_column_panel(int64_t m, int64_t nnz, spsyrk_dtype_t dtype,
                                    const int64_t *d_rowptr, const int32_t *d_colidx, const void *d_vals,
                                    int64_t k0, int64_t k1,
                                    int64_t *d_p_rowptr, int32_t *d_p_colidx, void *d_p_vals,
                                    int64_t *nnz_out,
                                    void *d_workspace, size_t *workspace_bytes, void *cuda_stream);

/*
 * spsyrk_accumulate - Z = X + Y for two CSR matrices of m rows whose rows are ascending in column:
 * the "+=" of Algorithm 2 line 2 (C_local += SYRK(A_recv)), with X the running sum and Y one more
 * panel product.  The structure of Z is the union of the two structures; an entry stored in both
 * gets x + y (one rounded addition in the dtype; I32 wraps), an entry stored in one keeps its
 * value bit for bit.  Rows of Z are ascending in column.  Z must not alias X or Y.
 *
 * Three-step use:
 *   1. d_workspace == NULL: *workspace_bytes receives the scratch size for m.
 *   2. d_z_colidx == NULL: writes d_z_rowptr[m + 1] and *nnz_out (synchronises).
 *   3. all pointers set: fills d_z_colidx / d_z_vals using the d_z_rowptr of step 2.  Asynchronous.
 * All pointers are device pointers except nnz_out and workspace_bytes (host).
 * nnz_x = d_x_rowptr[m], nnz_y = d_y_rowptr[m] (they only steer how many lanes share a row).
 * Errors: INVALID_ARG, WORKSPACE, BAD_CSR (a row of X or Y not strictly ascending), CUDA.
 */
spsyrk_status_t spsyrk_accumulate(int64_t m, spsyrk_dtype_t dtype,
                                  int64_t nnz_x, const int64_t *d_x_rowptr, const int32_t *d_x_colidx, const void *d_x_vals,
                                  int64_t nnz_y, const int64_t *d_y_rowptr, const int32_t *d_y_colidx, const void *d_y_vals,
                                  int64_t *d_z_rowptr, int32_t *d_z_colidx, void *d_z_vals,
                                  int64_t *nnz_out,
                                  void *d_workspace, size_t *workspace_bytes, void *cuda_stream);

/*
 * spsyrk_permute - B = P A Q^T as canonical CSR: row i of A becomes row d_rperm[i] of B and column k
 * becomes column d_cperm[k] (d_cperm == NULL: columns stay).  With a square A and the same map
 * for rows and columns this is the symmetric random permutation that restores load balance
 * (Section III-A; the load-balance study of Section V).  Rows of B are ascending in column.
 *
 * Two-step use:
 *   1. d_workspace == NULL: *workspace_bytes receives the scratch size for (m, n, nnz, dtype).
 *   2. all pointers set: writes d_b_rowptr[m + 1], d_b_colidx[nnz], d_b_vals[nnz] (synchronises).
 * All pointers are device pointers except workspace_bytes (host); d_rperm has m entries, d_cperm n;
 * B must not alias A.  Errors: INVALID_ARG (also: a map that is
 * not a permutation), WORKSPACE, OVERFLOW, BAD_CSR (row pointers or column ids out of range), CUDA.
 */
spsyrk_status_t spsyrk_permute(int64_t m, int64_t n, int64_t nnz, spsyrk_dtype_t dtype,
                               const int64_t *d_rowptr, const int32_t *d_colidx, const void *d_vals,
                               const int32_t *d_rperm, const int32_t *d_cperm,
                               int64_t *d_b_rowptr, int32_t *d_b_colidx, void *d_b_vals,
                               void *d_workspace, size_t *workspace_bytes, void *cuda_stream);

/*
 * spsyrk_plan_partition - contiguous ranges of the plan's output rows with near-equal work, for a
 * 1-D distribution of the rows over `parts` workers (the work of the lower triangle grows with
 * the row index, so equal row counts are not equal work; Section III-A asks for balanced work).
 * bounds (HOST, parts + 1 entries) receives absolute row ids: bounds[0] = row_begin,
 * bounds[parts] = row_end, and bounds[p] is the first row at which the prefix sum of the per-row
 * work estimate reaches p/parts of the total.  Worker p then calls spsyrk_plan_set_rows with
 * [bounds[p], bounds[p + 1]).  1 <= parts <= 65536.  Synchronises.
 * Errors: INVALID_ARG, OVERFLOW (total work x parts does not fit 63 bits), CUDA.
 */
spsyrk_status_t spsyrk_plan_partition(spsyrk_plan_t plan, int64_t parts, int64_t *bounds, void *cuda_stream);

/*
 * spsyrk_symv - y = C x from the stored lower triangle alone,
 *     C x = C_L x + (x^T C_L)^T - D x        (Section V-F, Eq. 1: the triangular output is consumed
 * directly, C_L^T is never formed and the diagonal is counted once).  C_L is any lower-triangular
 * CSR (diagonal included) of F64 or F32 values; d_x[m] and d_y[m] are device vectors of the same
 * type; y is overwritten.  The reflected contributions are accumulated with atomic adds, so the
 * last bits of y can differ from run to run.  Asynchronous.  Errors: INVALID_ARG, CUDA.
 */
spsyrk_status_t spsyrk_symv(int64_t m, int64_t nnz_l, spsyrk_dtype_t dtype,
                            const int64_t *d_l_rowptr, const int32_t *d_l_colidx, const void *d_l_vals,
                            const void *d_x, void *d_y, void *cuda_stream);

/*
 * spsyrk_symm - Y = C X for a dense X from the stored lower triangle alone,
 *     C X = C_L X + (X^T C_L)^T - D X        (Section V-F, second equation: the matrix form of the
 * triangular product; unlike the vector form it cannot be replaced by A (A^T X) without possibly
 * more arithmetic than (A A^T) X, so consuming C_L directly is the form worth having).
 * C_L is any lower-triangular CSR (diagonal included) of F64 or F32 values with m rows; d_x and d_y are
 * dense row-major device matrices of the same type, m rows by p columns (element (i, c) at i * p + c);
 * Y is overwritten and must not alias X.  The reflected contributions are accumulated with atomic
 * adds, so the last bits of Y can differ from run to run.  Columns are processed eight at a time
 * (C_L is read once per eight columns of X).  Asynchronous.  Errors: INVALID_ARG, CUDA.
 */
spsyrk_status_t spsyrk_symm(int64_t m, int64_t p, int64_t nnz_l, spsyrk_dtype_t dtype,
                            const int64_t *d_l_rowptr, const int32_t *d_l_colidx, const void *d_l_vals,
                            const void *d_x, void *d_y, void *cuda_stream);

/*
 * spsyrk_mirror_rowptr_noalloc - the sizes of F = C_L + C_L^T - D, that is d_f_rowptr[m + 1] as
 * step 3 of spsyrk_mirror writes it and *nnz_full_out as step 2 returns it, for callers that can
 * neither allocate device memory nor pass a workspace.  (The paper has no counterpart: this entry
 * point exists for deployment only.)
 *
 * Who needs it: code that runs where device allocation is off limits - for instance a plug-in
 * inside a host application that has reserved the whole GPU for its own memory pool, or a service
 * loop that must not risk the device-wide synchronisation an allocation or a free can cause - and
 * that therefore has no scratch buffer to hand to spsyrk_mirror.
 *
 * How: the scratch (two 32-bit counters per row, the scan's partial sums, an error word) is a
 * fixed array inside the library image, SPSYRK_NOALLOC_MAX_ROWS rows long.  Every GPU that loads
 * the library keeps those bytes (about 8 * SPSYRK_NOALLOC_MAX_ROWS) until the process exits.
 * The call itself performs no cudaMalloc, cudaFree or any allocating library routine; the caller
 * still owns and passes d_l_rowptr[m + 1], d_l_colidx[nnz_l] and d_f_rowptr[m + 1] (device) and
 * nnz_full_out (host).
 *
 * Rules:
 *   - m > SPSYRK_NOALLOC_MAX_ROWS is rejected with SPSYRK_ERR_OVERFLOW; use spsyrk_mirror then.
 *   - The first call on a device looks up the array's device address (a one-time set-up per
 *     device, done with that device current); make that first call before any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents; the
 *     entry point clears what it accumulates into at the start of each call.  Two calls whose GPU
 *     work overlaps in time (different streams or threads) race on it: serialise them.
 *   - Synchronises the stream once (the entry count and the error word travel back).
 * The row pointers equal the ones step 3 of spsyrk_mirror writes, the count the one step 2 returns.
 * Errors: INVALID_ARG, OVERFLOW, BAD_CSR (an entry above the diagonal, a decreasing row pointer), CUDA.
 */
#define SPSYRK_NOALLOC_MAX_ROWS 1048576
spsyrk_status_t spsyrk_mirror_rowptr_noalloc(int64_t m, const int64_t *d_l_rowptr, const int32_t *d_l_colidx,
                                             int64_t *d_f_rowptr, int64_t *nnz_full_out, void *cuda_stream);

/*
 * spsyrk_jaccard - Jaccard similarity of the rows of a binary A from intersection counts,
 *     J_ij = c_ij / (|a_i| + |a_j| - c_ij),   |a_i| = stored entries of row i of A,
 * for rows [row_begin, row_begin + rows) of an int32-valued C_L with a tile-local row pointer
 * (Jaccard similarity is the application named in the abstract and Section I; the formula is
 * the standard set definition).  One single-precision division per stored entry.  Asynchronous.
 * Errors: INVALID_ARG, CUDA.
 */
spsyrk_status_t spsyrk_jaccard(int64_t m, int64_t row_begin, int64_t rows,
                               const int64_t *d_a_rowptr, const int64_t *d_c_rowptr,
                               const int32_t *d_c_colidx, const int32_t *d_c_counts,
                               float *d_jaccard, void *cuda_stream);

/*
 * spsyrk_plan_set_jaccard - fuse the Jaccard normalisation into spsyrk_numeric: while a row's counts are
 * written, J_ij = c_ij / (|a_i| + |a_j| - c_ij) is written to d_jaccard at the same offsets as d_c_vals
 * (nnz entries of float; same formula and rounding as spsyrk_jaccard, so the two agree bit for bit), and
 * the counts are not read again.  Only for I32 plans; d_jaccard == NULL switches it off.  The buffer is
 * caller-owned and must be valid during every later spsyrk_numeric call.  Errors: INVALID_ARG.
 */
spsyrk_status_t spsyrk_plan_set_jaccard(spsyrk_plan_t plan, float *d_jaccard);

/*
 * spsyrk_plan_stats - host-side facts about a plan.
 *   work_total    multiply-adds the plan's rows will perform (sum of w[i])
 *   class_rows[8] rows per class: 0 empty, 1..5 warp classes (w <= 32, 64, 128, 256, 512),
 *                 6 block class, 7 large class
 * Any out-pointer may be NULL.
 */
spsyrk_status_t spsyrk_plan_stats(spsyrk_plan_t plan, int64_t *work_total, int64_t class_rows[8]);

/*
 * spsyrk_plan_buffers - device pointers into the plan's workspace, for inspection and tests:
 * column pointers colptr[n+1] (int64), the column lists' row ids at_row[nnz] (int32), the same
 * entries as (row id, value) records at_rec[nnz] (8-byte values: int32 row id, 4 bytes of padding, the
 * value; 4-byte values: int32 row id, the value), and the per-row work w[rows] (int64).  Any may be NULL.
 */
spsyrk_status_t spsyrk_plan_buffers(spsyrk_plan_t plan, const int64_t **d_colptr, const int32_t **d_at_row,
                                    const void **d_at_rec, const int64_t **d_work);

/*
 * Measurement aids (no effect on results).
 * spsyrk_plan_enable_timing : from now on spsyrk_symbolic / spsyrk_numeric record CUDA events on
 *     the caller's stream around the launch of every row class.
 * spsyrk_plan_timings       : device milliseconds of the last symbolic and numeric call per row
 *     class (index = class, 0 unused); waits for those events.  A numeric entry is 0 if numeric
 *     has not run since timing was enabled.
 * spsyrk_launch_count       : kernels launched by this library in this process so far.
 */
spsyrk_status_t spsyrk_plan_enable_timing(spsyrk_plan_t plan);
/* spsyrk_mirror_enable_timing(1): from now on the fill step of spsyrk_mirror on 8-byte values records
 *     CUDA events around each of its sorting passes (process-wide switch, not thread-safe; 0 turns it off).
 * spsyrk_mirror_timings: *passes = sorting passes of the last such fill (at most 4) and their device
 *     milliseconds (histogram, scan and scatter of the pass); waits for those events. */
spsyrk_status_t spsyrk_mirror_enable_timing(int on);
spsyrk_status_t spsyrk_mirror_timings(int *passes, float pass_ms[4]);
spsyrk_status_t spsyrk_plan_timings(spsyrk_plan_t plan, float symbolic_ms[8], float numeric_ms[8]);
int64_t spsyrk_launch_count(void);

void spsyrk_destroy(spsyrk_plan_t plan);

const char *spsyrk_status_string(spsyrk_status_t s);

/*
 * spsyrk_host_tril - the whole path on HOST buffers: copies A to the device, runs plan,
 * symbolic and numeric, and copies C_L back.  Two calls:
 *   1. h_c_colidx == NULL: runs plan + symbolic, writes h_c_rowptr[m+1] and *nnz_out, keeps the
 *      device state in *session.
 *   2. with h_c_colidx / h_c_vals of *nnz_out entries: runs numeric, copies the result back and
 *      frees the session.  A large result is computed in up to eight row blocks of about equal
 *      numbers of entries (spsyrk_numeric_rows) and each block is copied on a second stream while
 *      the following ones are computed, so only the first block's computation is not hidden
 *      behind the download.
 * Device memory for this entry point is allocated by the library (cudaMalloc) and kept in two
 * grow-only blocks per device between calls, because allocating and freeing several GB per call
 * costs more than the computation; spsyrk_host_release_cache frees the blocks of the current
 * device that no live session uses.  A call made while another thread's session holds the blocks
 * allocates and frees its own.  Host buffers should be pinned for full copy speed.  Synchronous.
 */
typedef struct spsyrk_session_s *spsyrk_session_t;
spsyrk_status_t spsyrk_host_tril(spsyrk_session_t *session, int64_t m, int64_t n, int64_t nnz,
                                 const int64_t *h_rowptr, const int32_t *h_colidx, const void *h_vals,
                                 spsyrk_dtype_t dtype, spsyrk_mode_t mode,
                                 int64_t *h_c_rowptr, int64_t *nnz_out,
                                 int32_t *h_c_colidx, void *h_c_vals);
spsyrk_status_t spsyrk_host_release_cache(void);

#ifdef __cplusplus
}
#endif
#endif /* SPSYRK_H */
