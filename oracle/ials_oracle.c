/*
 * ials_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of implicit Alternating Least Squares as the
 * ALX paper (arXiv 2112.02194) defines it.  It exists to check the CUDA library
 * and to be timed as a reported CPU baseline.  The product never calls it, and it
 * shares no code, header, table or helper with the CUDA path.
 *
 * What follows the paper:
 *   - alxo_gramian        : G = sum_i h_i (x) h_i = H^T H            (Sec. 3 below Eq. 4; Alg. 1 line 2)
 *   - alxo_half_step_rows : per row, b = sum y h_i, A = alpha G + lambda I + sum h_i (x) h_i,
 *                           w = A^-1 b                               (Eq. 4; Alg. 1 lines 3-10)
 *   - alxo_loss           : the implicit objective written as printed (Eq. 3), with the
 *                           all-pairs term summed over every (u, i) explicitly
 *   - alxo_loss_gramian   : the same objective with the all-pairs term folded through the
 *                           Gramians (the identity of Sec. 3 applied to the loss)
 *   - storage rounding    : tables held in bf16 or fp32, everything else wider (Sec. 4.4)
 * What the paper leaves to the implementation and this library fixes by a written
 * integer rule (the CUDA path must reproduce these arrays bit for bit):
 *   - alxo_transpose      : CSR -> CSC, row ids ascending inside each column
 *   - alxo_degree_class / alxo_bucket_rows / alxo_chunks
 *
 * Loops are in the paper's order.  The only parallelism is over rows: "omp parallel for" over the
 * rows of the side being solved, which Alg. 2's parfor over rows licenses (a row reads only the
 * fixed table, G and its own observations), and contiguous blocks of fixed-side rows in the Gramian
 * (Alg. 2 lines 5-6: per-part Gramians added up), combined in block order.
 *
 * Pins (tests run without a GPU): brute-force stacked least squares via QR on tiny inputs,
 * closed forms (d = 1, single observation with and without the all-pairs term, orthogonal
 * fixed side), ridge regression for alpha = 0, gradient of Eq. 3 by explicit all-pairs
 * sums, monotone objective, permutation equivariance, operation counters.
 *   - alxo_cg / alxo_half_step_rows_cg : the conjugate-gradient solve of Sec. 4.5 (the solver the
 *                           paper's results use).  The paper states no start vector, iteration count or
 *                           tolerance; the reading taken here: the textbook method (Hestenes-Stiefel),
 *                           start x = 0, stop as soon as |r_k| <= tol |b| or after max_iter steps.
 *                           Pins: converges to the Cholesky answer, exact after k steps when A has k
 *                           distinct eigenvalues, error decreasing in the A-norm, residuals mutually
 *                           orthogonal.  The iterates themselves have nothing in the paper to be compared
 *                           with: parity unpinned for the iterate sequence, pinned for the limit.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ALXO_F64 = 0, ALXO_F32 = 1, ALXO_BF16 = 2 };

void alxo_row_system(int d, int64_t beg, int64_t end, const int32_t *colidx, const double *values,
                     const double *X, const double *G, double alpha, double lambda, double *A, double *b);

/* ---- storage rounding (Sec. 4.4: tables in bfloat16, solve in float32 or wider) ---- */

/* round-to-nearest-even of a double to a value with an 8-bit significand (bfloat16);
   exponent range of the inputs used here never reaches bf16's limits */
static double round_bf16(double x)
{
    if (x == 0.0 || !isfinite(x)) return x;
    int e;
    double m = frexp(x, &e);          /* x = m * 2^e, 0.5 <= |m| < 1 */
    double r = nearbyint(ldexp(m, 8)); /* 8 significant bits, ties to even */
    return ldexp(r, e - 8);
}

double alxo_round_storage(double x, int storage)
{
    if (storage == ALXO_BF16) return round_bf16(x);
    if (storage == ALXO_F32) return (double)(float)x;
    return x;
}

void alxo_round_array(double *x, int64_t n, int storage)
{
    for (int64_t i = 0; i < n; ++i) x[i] = alxo_round_storage(x[i], storage);
}

/* ---- Gramian: G = sum over ALL rows of the fixed side of h (x) h ---- */
/* The sum over rows is split into one contiguous block of rows per thread (the only parallelism: over rows),
   each block summed in row order, the blocks added in block order. */
void alxo_gramian(const double *X, int64_t N, int d, double *G)
{
    memset(G, 0, sizeof(double) * (size_t)d * d);
#pragma omp parallel
    {
        double *P = (double *)calloc((size_t)d * d, sizeof(double));
#pragma omp for schedule(static) ordered
        for (int64_t blk = 0; blk < 64; ++blk) {
            const int64_t i0 = N * blk / 64, i1 = N * (blk + 1) / 64;
            memset(P, 0, sizeof(double) * (size_t)d * d);
            for (int64_t i = i0; i < i1; ++i) {
                const double *h = X + i * d;
                for (int a = 0; a < d; ++a)
                    for (int b = 0; b < d; ++b)
                        P[a * d + b] += h[a] * h[b];
            }
#pragma omp ordered
            for (int k = 0; k < d * d; ++k) G[k] += P[k];
        }
        free(P);
    }
}

/* ---- dense SPD solve, fp64 Cholesky without pivoting + iterative refinement ---- */
/* returns 0 on success, 1 if a pivot is not positive */
static int cholesky(double *L, int d) /* in: full symmetric A; out: lower triangle = L */
{
    for (int j = 0; j < d; ++j) {
        double s = L[j * d + j];
        for (int p = 0; p < j; ++p) s -= L[j * d + p] * L[j * d + p];
        if (!(s > 0.0)) return 1;
        double ljj = sqrt(s);
        L[j * d + j] = ljj;
        for (int i = j + 1; i < d; ++i) {
            double t = L[i * d + j];
            for (int p = 0; p < j; ++p) t -= L[i * d + p] * L[j * d + p];
            L[i * d + j] = t / ljj;
        }
    }
    return 0;
}

static void chol_solve(const double *L, int d, const double *b, double *x)
{
    for (int i = 0; i < d; ++i) { /* L z = b */
        double t = b[i];
        for (int p = 0; p < i; ++p) t -= L[i * d + p] * x[p];
        x[i] = t / L[i * d + i];
    }
    for (int i = d - 1; i >= 0; --i) { /* L^T x = z */
        double t = x[i];
        for (int p = i + 1; p < d; ++p) t -= L[p * d + i] * x[p];
        x[i] = t / L[i * d + i];
    }
}

static int spd_solve(const double *A, const double *b, int d, double *x, double *work /* d*d + 2d */)
{
    double *L = work, *r = work + (size_t)d * d, *dx = r + d;
    memcpy(L, A, sizeof(double) * (size_t)d * d);
    if (cholesky(L, d)) return 1;
    chol_solve(L, d, b, x);
    for (int it = 0; it < 2; ++it) { /* refinement: x += A^-1 (b - A x) */
        for (int i = 0; i < d; ++i) {
            double t = b[i];
            for (int p = 0; p < d; ++p) t -= A[i * d + p] * x[p];
            r[i] = t;
        }
        chol_solve(L, d, r, dx);
        for (int i = 0; i < d; ++i) x[i] += dx[i];
    }
    return 0;
}

/* ---- one row of Eq. 4, exactly in Alg. 1's order (lines 4-10) ---- */
static int solve_one_row(int d, int64_t beg, int64_t end, const int32_t *colidx, const double *values,
                         const double *X, const double *G, double alpha, double lambda,
                         double *A, double *b, double *work, double *w_out, int64_t *n_outer)
{
    for (int a = 0; a < d; ++a) b[a] = 0.0;                       /* grad <- 0 */
    for (int a = 0; a < d; ++a)                                   /* hess <- alpha G + lambda I */
        for (int c = 0; c < d; ++c)
            A[a * d + c] = alpha * G[a * d + c] + (a == c ? lambda : 0.0);
    for (int64_t e = beg; e < end; ++e) {                         /* for (u, i, y) in S */
        const double *h = X + (int64_t)colidx[e] * d;
        double y = values ? values[e] : 1.0;
        for (int a = 0; a < d; ++a) b[a] += y * h[a];             /* grad += y h */
        for (int a = 0; a < d; ++a)                               /* hess += h (x) h */
            for (int c = 0; c < d; ++c)
                A[a * d + c] += h[a] * h[c];
        ++*n_outer;
    }
    if (beg == end) { /* no observation: A^-1 0 = 0 exactly */
        for (int a = 0; a < d; ++a) w_out[a] = 0.0;
        return 0;
    }
    return spd_solve(A, b, d, w_out, work);                       /* w <- hess^-1 grad */
}

/*
 * Half step over a list of rows of the solved side (row_ids == NULL: all n rows, in order).
 * CSR (rowptr, colidx, values|NULL => y = 1) is indexed by rows of the solved side and points
 * into the fixed table X[N x d] (fp64 array holding values already rounded to the storage type).
 * G must be alxo_gramian(X).  Y_out[k*d .. ] receives row row_ids[k] (or row k), rounded to
 * `storage`; Y_raw (may be NULL) receives the unrounded solution.  counters[0] += outer-product
 * updates, counters[1] += solves, counters[2] += non-SPD failures.
 */
int alxo_half_step_rows(int64_t n, int64_t N, int d, const int64_t *rowptr, const int32_t *colidx,
                        const double *values, const double *X, const double *G, double alpha,
                        double lambda, int storage, const int64_t *row_ids, int64_t n_ids,
                        double *Y_out, double *Y_raw, int64_t *counters)
{
    (void)N;
    int64_t count = row_ids ? n_ids : n;
    int64_t tot_outer = 0, tot_fail = 0;
#pragma omp parallel reduction(+ : tot_outer, tot_fail)
    {
        double *A = (double *)malloc(sizeof(double) * ((size_t)2 * d * d + 4 * (size_t)d));
        double *work = A + (size_t)d * d;
        double *b = work + (size_t)d * d + 2 * (size_t)d;
        double *w = b + d;
#pragma omp for schedule(dynamic, 16)
        for (int64_t k = 0; k < count; ++k) {
            int64_t u = row_ids ? row_ids[k] : k;
            int64_t no = 0;
            int fail = solve_one_row(d, rowptr[u], rowptr[u + 1], colidx, values, X, G, alpha, lambda,
                                     A, b, work, w, &no);
            tot_outer += no;
            tot_fail += fail;
            for (int a = 0; a < d; ++a) {
                if (Y_raw) Y_raw[k * d + a] = w[a];
                Y_out[k * d + a] = alxo_round_storage(w[a], storage);
            }
        }
        free(A);
    }
    if (counters) {
        counters[0] += tot_outer;
        counters[1] += count;
        counters[2] += tot_fail;
    }
    return tot_fail ? 1 : 0;
}

/* ---- conjugate gradients (Sec. 4.5), textbook form, fp64, x_0 = 0 ----
 * Solves A x = b for a symmetric positive definite d x d matrix.  Stops at the first k with |r_k| <= tol |b|
 * (r_k by the recurrence) or after max_iter steps; returns the number of steps taken.  When `iterates` is not
 * NULL it receives x_1 .. x_k, d values each (room for max_iter of them).  work holds 3 d doubles.
 */
int alxo_cg(int d, const double *A, const double *b, double tol, int max_iter, double *x, double *iterates,
            double *work)
{
    double *r = work, *p = work + d, *q = work + 2 * d;
    double bb = 0.0;
    for (int a = 0; a < d; ++a) { x[a] = 0.0; r[a] = b[a]; p[a] = b[a]; bb += b[a] * b[a]; }
    double rr = bb;
    if (bb == 0.0) return 0;
    int k = 0;
    while (k < max_iter && rr > tol * tol * bb) {
        double pq = 0.0;
        for (int a = 0; a < d; ++a) {                                  /* q <- A p */
            double t = 0.0;
            for (int c = 0; c < d; ++c) t += A[a * d + c] * p[c];
            q[a] = t;
            pq += p[a] * t;
        }
        const double step = rr / pq;
        double rr_new = 0.0;
        for (int a = 0; a < d; ++a) {
            x[a] += step * p[a];
            r[a] -= step * q[a];
            rr_new += r[a] * r[a];
        }
        const double beta = rr_new / rr;
        for (int a = 0; a < d; ++a) p[a] = r[a] + beta * p[a];
        rr = rr_new;
        if (iterates) memcpy(iterates + (size_t)k * d, x, sizeof(double) * (size_t)d);
        ++k;
    }
    return k;
}

/* alxo_half_step_rows with the solve of Alg. 1 line 10 done by alxo_cg; iters_out[k] (may be NULL) = steps of row k */
int alxo_half_step_rows_cg(int64_t n, int64_t N, int d, const int64_t *rowptr, const int32_t *colidx,
                           const double *values, const double *X, const double *G, double alpha,
                           double lambda, int storage, const int64_t *row_ids, int64_t n_ids, double tol,
                           int max_iter, double *Y_out, double *Y_raw, int32_t *iters_out)
{
    (void)N;
    int64_t count = row_ids ? n_ids : n;
#pragma omp parallel
    {
        double *A = (double *)malloc(sizeof(double) * ((size_t)d * d + 5 * (size_t)d));
        double *b = A + (size_t)d * d, *w = b + d, *work = w + d;
#pragma omp for schedule(dynamic, 16)
        for (int64_t k = 0; k < count; ++k) {
            int64_t u = row_ids ? row_ids[k] : k;
            alxo_row_system(d, rowptr[u], rowptr[u + 1], colidx, values, X, G, alpha, lambda, A, b);
            int it = alxo_cg(d, A, b, tol, max_iter, w, NULL, work);
            if (iters_out) iters_out[k] = it;
            for (int a = 0; a < d; ++a) {
                if (Y_raw) Y_raw[k * d + a] = w[a];
                Y_out[k * d + a] = alxo_round_storage(w[a], storage);
            }
        }
        free(A);
    }
    return 0;
}

/* normal matrix and right-hand side of one row, for residual checks of someone else's solution */
void alxo_row_system(int d, int64_t beg, int64_t end, const int32_t *colidx, const double *values,
                     const double *X, const double *G, double alpha, double lambda, double *A, double *b)
{
    for (int a = 0; a < d; ++a) b[a] = 0.0;
    for (int a = 0; a < d; ++a)
        for (int c = 0; c < d; ++c)
            A[a * d + c] = alpha * G[a * d + c] + (a == c ? lambda : 0.0);
    for (int64_t e = beg; e < end; ++e) {
        const double *h = X + (int64_t)colidx[e] * d;
        double y = values ? values[e] : 1.0;
        for (int a = 0; a < d; ++a) b[a] += y * h[a];
        for (int a = 0; a < d; ++a)
            for (int c = 0; c < d; ++c)
                A[a * d + c] += h[a] * h[c];
    }
}

/* ---- Eq. 3 as printed: observed term, all-pairs term by explicit double loop, regulariser ---- */
void alxo_loss(int64_t n_rows, int64_t n_cols, int d, const int64_t *rowptr, const int32_t *colidx,
               const double *values, const double *W, const double *H, double alpha, double lambda,
               double *components /* obs, implicit, reg */)
{
    double obs = 0.0, imp = 0.0, reg = 0.0;
    for (int64_t u = 0; u < n_rows; ++u)
        for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e) {
            const double *w = W + u * d, *h = H + (int64_t)colidx[e] * d;
            double yhat = 0.0;
            for (int a = 0; a < d; ++a) yhat += w[a] * h[a];
            double y = values ? values[e] : 1.0;
            obs += (y - yhat) * (y - yhat);
        }
    for (int64_t u = 0; u < n_rows; ++u)
        for (int64_t i = 0; i < n_cols; ++i) {
            double yhat = 0.0;
            for (int a = 0; a < d; ++a) yhat += W[u * d + a] * H[i * d + a];
            imp += yhat * yhat;
        }
    for (int64_t k = 0; k < n_rows * d; ++k) reg += W[k] * W[k];
    for (int64_t k = 0; k < n_cols * d; ++k) reg += H[k] * H[k];
    components[0] = obs;
    components[1] = alpha * imp;
    components[2] = lambda * reg;
}

/* the same objective with sum_u sum_i <w,h>^2 = <W^T W, H^T H>_F; usable at sizes where the double loop is not */
void alxo_loss_gramian(int64_t n_rows, int64_t n_cols, int d, const int64_t *rowptr, const int32_t *colidx,
                       const double *values, const double *W, const double *H, double alpha, double lambda,
                       double *components)
{
    double obs = 0.0, reg = 0.0;
#pragma omp parallel for reduction(+ : obs) schedule(dynamic, 64)
    for (int64_t u = 0; u < n_rows; ++u)
        for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e) {
            const double *w = W + u * d, *h = H + (int64_t)colidx[e] * d;
            double yhat = 0.0;
            for (int a = 0; a < d; ++a) yhat += w[a] * h[a];
            double y = values ? values[e] : 1.0;
            obs += (y - yhat) * (y - yhat);
        }
    double *GW = (double *)malloc(sizeof(double) * (size_t)d * d * 2), *GH = GW + (size_t)d * d;
    alxo_gramian(W, n_rows, d, GW);
    alxo_gramian(H, n_cols, d, GH);
    double imp = 0.0;
    for (int k = 0; k < d * d; ++k) imp += GW[k] * GH[k];
    free(GW);
    for (int64_t k = 0; k < n_rows * d; ++k) reg += W[k] * W[k];
    for (int64_t k = 0; k < n_cols * d; ++k) reg += H[k] * H[k];
    components[0] = obs;
    components[1] = alpha * imp;
    components[2] = lambda * reg;
}

/* ---- integer structures ---- */

/* CSR -> CSC by stable counting sort: inside a column, rows appear in ascending order */
void alxo_transpose(int64_t n_rows, int64_t n_cols, const int64_t *rowptr, const int32_t *colidx,
                    const float *values, int64_t *colptr, int32_t *rowidx, float *values_t)
{
    int64_t nnz = rowptr[n_rows];
    for (int64_t c = 0; c <= n_cols; ++c) colptr[c] = 0;
    for (int64_t e = 0; e < nnz; ++e) colptr[colidx[e] + 1]++;
    for (int64_t c = 0; c < n_cols; ++c) colptr[c + 1] += colptr[c];
    int64_t *cursor = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_cols > 0 ? n_cols : 1));
    for (int64_t c = 0; c < n_cols; ++c) cursor[c] = colptr[c];
    for (int64_t u = 0; u < n_rows; ++u)
        for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e) {
            int64_t q = cursor[colidx[e]]++;
            rowidx[q] = (int32_t)u;
            if (values && values_t) values_t[q] = values[e];
        }
    free(cursor);
}

/*
 * Degree class (the written rule): 0 for an empty row; otherwise the smallest c >= 1 with
 * deg <= 16 * 2^(c-1), capped at n_classes-1; a row longer than `split` entries is always in
 * the last class n_classes-1.  With split = 8192 and n_classes = 12 the bounds are
 * 16, 32, ..., 8192 and "more than 8192".
 */
int32_t alxo_degree_class(int64_t deg, int64_t split, int32_t n_classes)
{
    if (deg <= 0) return 0;
    if (deg > split) return n_classes - 1;
    int32_t c = 1;
    int64_t bound = 16;
    while (deg > bound && c < n_classes - 2) { bound *= 2; ++c; }
    return c;
}

/* rows sorted by (class, id): order[n], class_offsets[n_classes+1] */
void alxo_bucket_rows(int64_t n, const int64_t *rowptr, int64_t split, int32_t n_classes,
                      int32_t *order, int64_t *class_offsets)
{
    for (int32_t c = 0; c <= n_classes; ++c) class_offsets[c] = 0;
    for (int64_t u = 0; u < n; ++u)
        class_offsets[alxo_degree_class(rowptr[u + 1] - rowptr[u], split, n_classes) + 1]++;
    for (int32_t c = 0; c < n_classes; ++c) class_offsets[c + 1] += class_offsets[c];
    int64_t *cur = (int64_t *)malloc(sizeof(int64_t) * (size_t)n_classes);
    for (int32_t c = 0; c < n_classes; ++c) cur[c] = class_offsets[c];
    for (int64_t u = 0; u < n; ++u)
        order[cur[alxo_degree_class(rowptr[u + 1] - rowptr[u], split, n_classes)]++] = (int32_t)u;
    free(cur);
}

/*
 * Chunk descriptors of the split class: rows of the last class in ascending id order, each cut
 * into ceil(deg / split) pieces [beg + k*split, min(end, beg + (k+1)*split)).  A descriptor is
 * four int64: row, begin, end, slot; `slot` numbers the descriptors 0, 1, 2, ... in that order.
 * first_chunk[j] (j over the split rows in order, plus one sentinel) is the first slot of row j.
 * Returns the number of chunks; call with desc == NULL to size the arrays.
 */
int64_t alxo_chunks(int64_t n, const int64_t *rowptr, int64_t split, int32_t n_classes,
                    int64_t *desc, int64_t *first_chunk)
{
    int64_t slot = 0, j = 0;
    for (int64_t u = 0; u < n; ++u) {
        int64_t beg = rowptr[u], end = rowptr[u + 1];
        if (alxo_degree_class(end - beg, split, n_classes) != n_classes - 1) continue;
        if (first_chunk) first_chunk[j] = slot;
        ++j;
        for (int64_t b = beg; b < end; b += split) {
            if (desc) {
                desc[slot * 4 + 0] = u;
                desc[slot * 4 + 1] = b;
                desc[slot * 4 + 2] = (b + split < end) ? b + split : end;
                desc[slot * 4 + 3] = slot;
            }
            ++slot;
        }
    }
    if (first_chunk) first_chunk[j] = slot;
    return slot;
}
