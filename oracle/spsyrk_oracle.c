/*
 * CPU oracle for the local sparse SYRK  C_L = tril(A * A^T)  and its companions.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, single-threaded statement of
 * what the CUDA library must compute.  It shares no code with the CUDA path and is called
 * only from the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * What it follows:
 *   - Section II-A: C = A A^T, c_ij = dot product of rows i and j of A.
 *   - Section III-A (diagonal processes) and Algorithm 2 line 2: only the lower triangle
 *     is computed.  Section V-F: the stored half includes the diagonal and
 *     C = C_L + C_L^T - D.
 *   - Section III-A (C_ii = sum over s of SYRK(A_is)) and the "+=" of Algorithm 2: column panels
 *     of A and the sparse sum that accumulates their products.
 *   - Section III-C: one addition per partial product; the multiply-add count of A A^T is
 *     sum_k nnz(A(:,k))^2.
 *
 * Readings where the paper is silent (stated again in the design notes):
 *   - An entry (i, j) is stored iff rows i and j share at least one stored column, whatever
 *     its numerical value (structural nonzeros).  An empty row has no diagonal entry.
 *   - Entries of a row are emitted in ascending column order.
 *   - Partial products of an entry are added in ascending order of the shared column k,
 *     multiply and add as two separately rounded operations, in double precision.
 *     Integer and single-precision inputs are passed in as doubles (exactly representable);
 *     integer results are exact in double as long as they stay below 2^53, and the Python
 *     wrapper checks that they fit int32.
 *
 * Every function works on plain arrays: int64 row pointers, int32 column ids, double values.
 * Compile with -O2 -ffp-contract=off.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORACLE_TRIL 0
#define ORACLE_FULL 1

/* Column lists of A by counting sort (the input transpose of Section IV-B): colptr[n+1];
 * for each column the (row, value) entries in ascending row order, which falls out of
 * scanning the rows of A in order.  Returns 0. */
int oracle_transpose(int64_t m, int64_t n, const int64_t *rowptr, const int32_t *colidx,
                     const double *vals, int64_t *colptr, int32_t *at_row, double *at_val)
{
    int64_t nnz = rowptr[m];
    memset(colptr, 0, (size_t)(n + 1) * sizeof(int64_t));
    for (int64_t p = 0; p < nnz; ++p) colptr[colidx[p] + 1] += 1;
    for (int64_t k = 0; k < n; ++k) colptr[k + 1] += colptr[k];
    int64_t *next = (int64_t *)malloc((size_t)(n > 0 ? n : 1) * sizeof(int64_t));
    if (!next) return -1;
    memcpy(next, colptr, (size_t)n * sizeof(int64_t));
    for (int64_t i = 0; i < m; ++i)
        for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
            int64_t q = next[colidx[p]]++;
            at_row[q] = (int32_t)i;
            at_val[q] = vals[p];
        }
    free(next);
    return 0;
}

/* One pass of the row-by-row (Gustavson) product over output rows [r0, r1).
 *
 * For each nonzero a_ik of row i, in ascending k, walk column k's list from its start and,
 * for every entry (j, a_jk) with j <= i (TRIL) or every entry (FULL), add a_ik * a_jk to the
 * accumulator of j.  A row of the result is the set of touched j in ascending order.
 *
 * If c_colidx == NULL only counts are produced: cnt[i - r0] = stored entries of row i and
 * work[i - r0] = partial products of row i (either may be NULL).
 * Otherwise c_rowptr[r1 - r0 + 1] (tile-local, c_rowptr[0] == 0) must hold the exclusive
 * prefix sums of cnt, and c_colidx / c_vals / c_abs (c_abs may be NULL) are filled;
 * c_abs holds sum_k |a_ik * a_jk|, the scale against which rounding differences are judged.
 */
int oracle_syrk_rows(int64_t m, int64_t n, const int64_t *rowptr, const int32_t *colidx,
                     const double *vals, const int64_t *colptr, const int32_t *at_row,
                     const double *at_val, int mode, int64_t r0, int64_t r1,
                     int64_t *cnt, int64_t *work, const int64_t *c_rowptr,
                     int32_t *c_colidx, double *c_vals, double *c_abs)
{
    (void)n;
    double *acc = (double *)malloc((size_t)(m > 0 ? m : 1) * sizeof(double));
    double *absacc = (double *)malloc((size_t)(m > 0 ? m : 1) * sizeof(double));
    int64_t *mark = (int64_t *)malloc((size_t)(m > 0 ? m : 1) * sizeof(int64_t));
    int32_t *touched = (int32_t *)malloc((size_t)(m > 0 ? m : 1) * sizeof(int32_t));
    if (!acc || !absacc || !mark || !touched) { free(acc); free(absacc); free(mark); free(touched); return -1; }
    for (int64_t j = 0; j < m; ++j) mark[j] = -1;

    for (int64_t i = r0; i < r1; ++i) {
        int64_t nt = 0, nprod = 0;
        for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
            int64_t k = colidx[p];
            double aik = vals[p];
            for (int64_t q = colptr[k]; q < colptr[k + 1]; ++q) {
                int64_t j = at_row[q];
                if (mode == ORACLE_TRIL && j > i) break; /* lists are ascending in j */
                if (mark[j] != i) { mark[j] = i; acc[j] = 0.0; absacc[j] = 0.0; touched[nt++] = (int32_t)j; }
                double prod = aik * at_val[q];
                acc[j] = acc[j] + prod;
                absacc[j] = absacc[j] + fabs(prod);
                ++nprod;
            }
        }
        if (cnt) cnt[i - r0] = nt;
        if (work) work[i - r0] = nprod;
        if (c_colidx) {
            /* ascending column order: insertion sort is too slow for dense rows, so sort by
             * a pass over the marks when the row is dense enough, else a simple shell sort */
            int64_t base = c_rowptr[i - r0];
            if (nt * 8 > (mode == ORACLE_TRIL ? i + 1 : m)) {
                int64_t hi = (mode == ORACLE_TRIL) ? i + 1 : m, o = 0;
                for (int64_t j = 0; j < hi; ++j)
                    if (mark[j] == i) { touched[o++] = (int32_t)j; }
            } else {
                for (int64_t gap = nt / 2; gap > 0; gap /= 2)
                    for (int64_t a = gap; a < nt; ++a) {
                        int32_t t = touched[a]; int64_t b = a;
                        for (; b >= gap && touched[b - gap] > t; b -= gap) touched[b] = touched[b - gap];
                        touched[b] = t;
                    }
            }
            for (int64_t o = 0; o < nt; ++o) {
                int32_t j = touched[o];
                c_colidx[base + o] = j;
                c_vals[base + o] = acc[j];
                if (c_abs) c_abs[base + o] = absacc[j];
            }
        }
    }
    free(acc); free(absacc); free(mark); free(touched);
    return 0;
}

/* Mirror (materialisation, Sections III-A and V-F): F = C_L + C_L^T - D.
 * Row i of F is row i of C_L followed by (r, c_ri) for every later row r > i that stores
 * column i, in ascending r.  Phase 1 (f_colidx == NULL): fills f_rowptr[m+1].
 * Phase 2: fills f_colidx / f_vals given f_rowptr. */
int oracle_mirror(int64_t m, const int64_t *l_rowptr, const int32_t *l_colidx, const double *l_vals,
                  int64_t *f_rowptr, int32_t *f_colidx, double *f_vals)
{
    if (!f_colidx) {
        memset(f_rowptr, 0, (size_t)(m + 1) * sizeof(int64_t));
        for (int64_t r = 0; r < m; ++r)
            for (int64_t p = l_rowptr[r]; p < l_rowptr[r + 1]; ++p) {
                int64_t j = l_colidx[p];
                if (j > r) return -2;            /* not lower triangular */
                f_rowptr[r + 1] += 1;            /* the stored entry itself */
                if (j < r) f_rowptr[j + 1] += 1; /* its reflection in row j */
            }
        for (int64_t r = 0; r < m; ++r) f_rowptr[r + 1] += f_rowptr[r];
        return 0;
    }
    int64_t *next = (int64_t *)malloc((size_t)(m > 0 ? m : 1) * sizeof(int64_t));
    if (!next) return -1;
    /* lower parts first: they precede every reflected entry of the same row */
    for (int64_t r = 0; r < m; ++r) {
        int64_t o = f_rowptr[r];
        for (int64_t p = l_rowptr[r]; p < l_rowptr[r + 1]; ++p, ++o) { f_colidx[o] = l_colidx[p]; f_vals[o] = l_vals[p]; }
        next[r] = o;
    }
    for (int64_t r = 0; r < m; ++r)
        for (int64_t p = l_rowptr[r]; p < l_rowptr[r + 1]; ++p) {
            int64_t j = l_colidx[p];
            if (j < r) { int64_t o = next[j]++; f_colidx[o] = (int32_t)r; f_vals[o] = l_vals[p]; }
        }
    free(next);
    return 0;
}

/* Jaccard similarity of the rows of a binary A from intersection counts:
 * J_ij = c_ij / (|a_i| + |a_j| - c_ij), |a_i| = stored entries of row i of A; one
 * single-precision division per stored entry.  Rows [row_begin, row_begin + rows) of C_L
 * with a tile-local c_rowptr. */
int oracle_jaccard(int64_t row_begin, int64_t rows, const int64_t *a_rowptr,
                   const int64_t *c_rowptr, const int32_t *c_colidx, const int32_t *c_counts,
                   float *jac)
{
    for (int64_t t = 0; t < rows; ++t) {
        int64_t i = row_begin + t;
        int64_t na_i = a_rowptr[i + 1] - a_rowptr[i];
        for (int64_t p = c_rowptr[t]; p < c_rowptr[t + 1]; ++p) {
            int64_t j = c_colidx[p];
            int64_t na_j = a_rowptr[j + 1] - a_rowptr[j];
            int64_t c = c_counts[p];
            jac[p] = (float)c / (float)(na_i + na_j - c);
        }
    }
    return 0;
}

/* y = C x from the stored lower triangle (Section V-F, Eq. 1): C x = C_L x + (x^T C_L)^T - D x.
 * Written as the three terms of the equation, each a plain loop; abs_y receives
 * sum |c_rj x_j| over all contributions of row r, the scale for rounding comparisons. */
int oracle_symv(int64_t m, const int64_t *l_rowptr, const int32_t *l_colidx, const double *l_vals,
                const double *x, double *y, double *abs_y)
{
    for (int64_t r = 0; r < m; ++r) { y[r] = 0.0; abs_y[r] = 0.0; }
    for (int64_t r = 0; r < m; ++r)                      /* C_L x */
        for (int64_t p = l_rowptr[r]; p < l_rowptr[r + 1]; ++p) {
            y[r] += l_vals[p] * x[l_colidx[p]];
            abs_y[r] += fabs(l_vals[p] * x[l_colidx[p]]);
        }
    for (int64_t r = 0; r < m; ++r)                      /* (x^T C_L)^T */
        for (int64_t p = l_rowptr[r]; p < l_rowptr[r + 1]; ++p) {
            y[l_colidx[p]] += l_vals[p] * x[r];
            abs_y[l_colidx[p]] += fabs(l_vals[p] * x[r]);
        }
    for (int64_t r = 0; r < m; ++r)                      /* - D x */
        for (int64_t p = l_rowptr[r]; p < l_rowptr[r + 1]; ++p)
            if (l_colidx[p] == r) { y[r] -= l_vals[p] * x[r]; abs_y[r] += fabs(l_vals[p] * x[r]); }
    return 0;
}

/* Y = C X for a dense row-major X (m x p) from the stored lower triangle (Section V-F, second
 * equation): C X = C_L X + (X^T C_L)^T - D X.  Written as the three terms of the equation, each a
 * plain loop over the stored entries; abs_y receives the sum of |c_rj| |x_jq| over all
 * contributions of an output element, the scale for rounding comparisons.  Y and abs_y are
 * row-major m x p. */
int oracle_symm(int64_t m, int64_t p, const int64_t *l_rowptr, const int32_t *l_colidx, const double *l_vals,
                const double *x, double *y, double *abs_y)
{
    for (int64_t e = 0; e < m * p; ++e) { y[e] = 0.0; abs_y[e] = 0.0; }
    for (int64_t r = 0; r < m; ++r)                      /* C_L X: row r of Y += c_rj * row j of X */
        for (int64_t q = l_rowptr[r]; q < l_rowptr[r + 1]; ++q) {
            const int64_t j = l_colidx[q];
            for (int64_t c = 0; c < p; ++c) {
                y[r * p + c] += l_vals[q] * x[j * p + c];
                abs_y[r * p + c] += fabs(l_vals[q] * x[j * p + c]);
            }
        }
    for (int64_t r = 0; r < m; ++r)                      /* (X^T C_L)^T: row j of Y += c_rj * row r of X */
        for (int64_t q = l_rowptr[r]; q < l_rowptr[r + 1]; ++q) {
            const int64_t j = l_colidx[q];
            for (int64_t c = 0; c < p; ++c) {
                y[j * p + c] += l_vals[q] * x[r * p + c];
                abs_y[j * p + c] += fabs(l_vals[q] * x[r * p + c]);
            }
        }
    for (int64_t r = 0; r < m; ++r)                      /* - D X */
        for (int64_t q = l_rowptr[r]; q < l_rowptr[r + 1]; ++q)
            if (l_colidx[q] == r)
                for (int64_t c = 0; c < p; ++c) {
                    y[r * p + c] -= l_vals[q] * x[r * p + c];
                    abs_y[r * p + c] += fabs(l_vals[q] * x[r * p + c]);
                }
    return 0;
}

/* Column panel A_s = A(:, [k0, k1)) as CSR with the column ids unchanged (Section III-A: the
 * diagonal block of C is a sum over s of SYRK(A_is), one term per column panel).  Rows keep
 * their order.  First call with out_colidx == NULL fills out_rowptr[m+1]; second call fills
 * the entries.  Returns 0. */
int oracle_column_panel(int64_t m, const int64_t *rowptr, const int32_t *colidx, const double *vals,
                        int64_t k0, int64_t k1, int64_t *out_rowptr, int32_t *out_colidx, double *out_vals)
{
    int64_t o = 0;
    for (int64_t i = 0; i < m; ++i) {
        if (!out_colidx) out_rowptr[i] = o;
        for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
            if (colidx[p] < k0 || colidx[p] >= k1) continue;
            if (out_colidx) { out_colidx[o] = colidx[p]; out_vals[o] = vals[p]; }
            ++o;
        }
    }
    if (!out_colidx) out_rowptr[m] = o;
    return 0;
}

/* Z = X + Y for two CSR matrices with rows sorted by column (the "+=" of Algorithm 2 line 2:
 * the running sum X takes one more panel product Y).  The structure of Z is the union of the
 * two structures; an entry stored in both gets x + y (one rounded addition, X's value first),
 * an entry stored in one keeps its value.  Rows of Z are ascending in column.  First call with
 * z_colidx == NULL fills z_rowptr[m+1]; second call fills the entries.  Returns 0, or -2 if a
 * row of X or Y is not strictly ascending. */
int oracle_add(int64_t m, const int64_t *x_rowptr, const int32_t *x_colidx, const double *x_vals,
               const int64_t *y_rowptr, const int32_t *y_colidx, const double *y_vals,
               int64_t *z_rowptr, int32_t *z_colidx, double *z_vals)
{
    int64_t o = 0;
    for (int64_t i = 0; i < m; ++i) {
        int64_t p = x_rowptr[i], pe = x_rowptr[i + 1], q = y_rowptr[i], qe = y_rowptr[i + 1];
        for (int64_t t = p + 1; t < pe; ++t) if (x_colidx[t] <= x_colidx[t - 1]) return -2;
        for (int64_t t = q + 1; t < qe; ++t) if (y_colidx[t] <= y_colidx[t - 1]) return -2;
        if (!z_colidx) z_rowptr[i] = o;
        while (p < pe || q < qe) {
            int32_t j;
            double v;
            if (q >= qe || (p < pe && x_colidx[p] < y_colidx[q])) { j = x_colidx[p]; v = x_vals[p]; ++p; }
            else if (p >= pe || y_colidx[q] < x_colidx[p]) { j = y_colidx[q]; v = y_vals[q]; ++q; }
            else { j = x_colidx[p]; v = x_vals[p] + y_vals[q]; ++p; ++q; }
            if (z_colidx) { z_colidx[o] = j; z_vals[o] = v; }
            ++o;
        }
    }
    if (!z_colidx) z_rowptr[m] = o;
    return 0;
}

/* B = P A Q^T for permutations given as maps: row i of A becomes row rperm[i] of B and column k
 * becomes column cperm[k] (cperm == NULL: columns stay).  With a square A and cperm == rperm this
 * is the symmetric random permutation that restores load balance (Section III-A; the load
 * balance study of Section V).  Rows of B are ascending in column again.  b_rowptr[m+1],
 * b_colidx[nnz], b_vals[nnz].  Returns 0, or -2 if a map is not a permutation. */
int oracle_permute(int64_t m, int64_t n, const int64_t *rowptr, const int32_t *colidx, const double *vals,
                   const int32_t *rperm, const int32_t *cperm,
                   int64_t *b_rowptr, int32_t *b_colidx, double *b_vals)
{
    char *seen = (char *)calloc((size_t)((m > n ? m : n) + 1), 1);
    if (!seen) return -1;
    for (int64_t i = 0; i < m; ++i) {
        if (rperm[i] < 0 || rperm[i] >= m || seen[rperm[i]]) { free(seen); return -2; }
        seen[rperm[i]] = 1;
    }
    if (cperm) {
        memset(seen, 0, (size_t)((m > n ? m : n) + 1));
        for (int64_t k = 0; k < n; ++k) {
            if (cperm[k] < 0 || cperm[k] >= n || seen[cperm[k]]) { free(seen); return -2; }
            seen[cperm[k]] = 1;
        }
    }
    free(seen);
    memset(b_rowptr, 0, (size_t)(m + 1) * sizeof(int64_t));
    for (int64_t i = 0; i < m; ++i) b_rowptr[rperm[i] + 1] = rowptr[i + 1] - rowptr[i];
    for (int64_t i = 0; i < m; ++i) b_rowptr[i + 1] += b_rowptr[i];
    for (int64_t i = 0; i < m; ++i) {
        int64_t o = b_rowptr[rperm[i]], len = 0;
        for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
            int32_t c = cperm ? cperm[colidx[p]] : colidx[p];
            double v = vals[p];
            int64_t q = o + len;   /* insertion into the ascending destination row */
            while (q > o && b_colidx[q - 1] > c) { b_colidx[q] = b_colidx[q - 1]; b_vals[q] = b_vals[q - 1]; --q; }
            b_colidx[q] = c;
            b_vals[q] = v;
            ++len;
        }
    }
    return 0;
}

/* Contiguous row ranges of near-equal work for a 1-D distribution of the output rows (the work
 * of the lower triangle grows with the row index, so equal row counts are not equal work):
 * bounds[0] = 0, bounds[parts] = rows, and bounds[p] is the smallest r whose work prefix
 * sum_{i<r} work[i] reaches p/parts of the total.  Returns 0. */
int oracle_partition(int64_t rows, const int64_t *work, int64_t parts, int64_t *bounds)
{
    long double total = 0;
    for (int64_t i = 0; i < rows; ++i) total += (long double)work[i];
    int64_t r = 0;
    long double prefix = 0;   /* exact: integer values far below 2^64 */
    bounds[0] = 0;
    for (int64_t p = 1; p < parts; ++p) {
        while (r < rows && prefix * (long double)parts < (long double)p * total) { prefix += (long double)work[r]; ++r; }
        bounds[p] = r;
    }
    bounds[parts] = rows;
    return 0;
}
