/*
 * alx.h -- C ABI of the B200 (sm_100a) implicit-ALS half-epoch library.
 *
 * The method is implicit Alternating Least Squares as stated in "ALX: Large Scale Matrix
 * Factorization on TPUs" (arXiv 2112.02194): model Eq. 1, objective Eq. 3, row update Eq. 4,
 * order of operations Algorithm 1.  One GPU, both embedding tables and the sparse matrix
 * resident in device memory.  Every step runs in this library's own CUDA kernels.
 *
 * Conventions
 *   - Every call returns an alx_status; nothing throws across this boundary; on error the
 *     out-parameters are left untouched and alx_last_error() describes the failure.
 *   - The caller owns every pointer it passes.  Calls copy what they need; the context never
 *     keeps a caller pointer.  "on_device" arguments say whether a pointer is a device pointer
 *     (read or written on the context's stream) or a host pointer.
 *   - W is the table of the matrix's rows (n_rows x d), H the table of its columns (n_cols x d),
 *     both row-major, contiguous, in the storage type chosen at creation.
 *   - Kernels are launched asynchronously on the context's stream.  Problems a kernel detects
 *     (index out of range, non-positive pivot) set a device status word that the next
 *     synchronising call (alx_synchronize, alx_loss, alx_get_*) turns into an error code.
 *     Nothing traps or asserts on the device.
 *   - Results are run-to-run deterministic: no floating-point atomics, all partial sums are
 *     combined in a fixed order that depends only on the problem sizes.  The same sequence of calls on
 *     a fresh context gives the same bits.  (With ALX_SOLVER_AUTO a half-epoch's solver depends on what
 *     the side's previous half-epoch on that context cost, so repeating one call on a used context may
 *     give the same solution in other bits.)
 */
#ifndef ALX_H_
#define ALX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct alx_ctx alx_ctx; /* opaque; owns all device state */

typedef enum {
    ALX_OK = 0,
    ALX_ERR_INVALID_ARG = 1,
    ALX_ERR_BAD_STATE = 2,   /* call order: e.g. half-epoch before the matrix or tables are set */
    ALX_ERR_OOM = 3,
    ALX_ERR_CUDA = 4,
    ALX_ERR_BAD_CSR = 5,     /* rowptr not monotone / index out of range / row not strictly ascending */
    ALX_ERR_NOT_SPD = 6,     /* a pivot was not positive (cannot happen for lambda > 0 in exact arithmetic) */
    ALX_ERR_UNSUPPORTED = 7
} alx_status;

typedef enum { ALX_ROWS = 0, ALX_COLS = 1 } alx_side; /* which table is SOLVED; the other is held fixed */
typedef enum { ALX_F32 = 0, ALX_BF16 = 1 } alx_dtype;

typedef enum { ALX_SOLVER_AUTO = 0, ALX_SOLVER_CHOLESKY = 1 } alx_solver;
typedef enum { ALX_CG_START_STORED = 0, ALX_CG_START_ZERO = 1 } alx_cg_start;
#define ALX_DEFAULT_CG_MAX_ITER 48
#define ALX_DEFAULT_CG_TOL 1e-6f        /* fp32 tables */
#define ALX_DEFAULT_CG_TOL_BF16 3e-5f   /* bfloat16 tables */
#define ALX_DEFAULT_DUAL_COND_LIMIT 8192.f
#define ALX_DEFAULT_CG_SWITCH_PRODUCTS 28.f

/* number of degree classes and the default split threshold, see alx_get_buckets */
#define ALX_N_CLASSES 12
#define ALX_DEFAULT_SPLIT 8192

typedef void *(*alx_alloc_fn)(size_t bytes, void *user); /* returns a device pointer, 256-byte aligned, or NULL */
typedef void (*alx_free_fn)(void *ptr, void *user);

typedef struct alx_options {
    int64_t n_rows, n_cols;  /* 1 <= n < 2^31 each */
    int32_t d;               /* embedding dimension: 16, 32, 64 or 128 */
    float lambda;            /* L2 weight of Eq. 3; must be > 0 (guarantees a unique minimiser) */
    float alpha0;            /* weight of the all-pairs term of Eq. 3 (the paper's alpha); >= 0 */
    int32_t storage;         /* alx_dtype of both tables.  ALX_BF16 follows Sec. 4.4 of the paper:
                                tables in bfloat16, statistics and solve in float32, result rounded
                                to nearest even on the way back */
    int32_t device;          /* CUDA device ordinal, -1 = the current device */
    void *stream;            /* cudaStream_t all work is ordered on; NULL = the legacy default stream */
    alx_alloc_fn alloc;      /* device allocator; NULL => cudaMalloc */
    alx_free_fn free;        /* NULL => cudaFree */
    void *alloc_user;
    int64_t split;           /* rows longer than this are cut into chunks of this many entries that
                                different thread blocks accumulate; 0 => ALX_DEFAULT_SPLIT; >= 16 */
    int32_t kernels;         /* 0 = best available for (d, storage): for d = 128 with bf16 tables the tensor-core
                                kernels, rows with at most 32 observations solved in the dual (push-through) form
                                of Eq. 4 while alpha0 G + lambda I is well conditioned (see dual_cond_limit; the rows of
                                17 .. 32 observations go to the conjugate-gradient kernel instead where that is the cheaper
                                solve); for d = 64 with fp32 tables the same tensor-core kernels over bfloat16 parts of
                                the fixed table (x = x1 + x2 + x3, so to fp32 accuracy), rows with at most 16
                                observations in the dual form; every other (d, storage) the FP32-ALU kernels.
                                1 = force the plain FP32-ALU kernels (reference path inside the library; every d, every
                                storage); 2 = as 0 but every row in the primal form */
    int32_t solver;          /* how the d x d system of Eq. 4 is solved (Sec. 4.5 compares the choices):
                                ALX_SOLVER_AUTO (0): conjugate gradients where the library has them (the whole-rows
                                tensor-core kernel), started as cg_start says and stopped at |r| <= cg_tol |b|; a row that has not
                                converged after cg_max_iter steps, and every row elsewhere, is solved by Cholesky.  A side
                                whose conjugate-gradient half-epoch spent more than cg_switch_products (28) products per row on average (where
                                the in-place Cholesky is the faster solve on B200) takes Cholesky for its next half-epochs,
                                with one conjugate-gradient half-epoch in every eight to look again; the choice is made
                                on the device from the counts of the side's last run.
                                ALX_SOLVER_CHOLESKY (1): Cholesky for every row */
    int32_t cg_max_iter;     /* 0 => ALX_DEFAULT_CG_MAX_ITER */
    float cg_tol;            /* 0 => ALX_DEFAULT_CG_TOL for fp32 tables, ALX_DEFAULT_CG_TOL_BF16 for bfloat16 tables.  The error of
                                a row is bounded by cond(A) times the relative residual: bfloat16 results are rounded to 2^-9
                                anyway, so a third of the usual residual gate of 1e-4 is enough there; fp32 tables are expected
                                to be right to 1e-3, which rows with cond(A) of 10^3 only are at 1e-6.  At most 1e-2 */
    float cg_switch_products; /* the mean number of products per row beyond which a side's next half-epochs take Cholesky
                                (see solver); 0 => ALX_DEFAULT_CG_SWITCH_PRODUCTS */
    int32_t cg_start;        /* start vector of the conjugate gradients (the paper states none): ALX_CG_START_STORED (0): the
                                row's embedding as stored in the table being solved (close to the solution once training
                                is under way; costs one product for r = b - A x0, and falls back to zero when |r| > |b|);
                                ALX_CG_START_ZERO (1): x = 0, so that a row's work does not depend on the table's history */
    float dual_cond_limit;   /* 0 => ALX_DEFAULT_DUAL_COND_LIMIT.  Rows with at most 32 observations (d = 128, bfloat16 tables)
                                or 16 (d = 64, fp32 tables) are solved in the dual form of Eq. 4 while
                                ||B||_F ||B^-1||_F <= this limit, B = alpha0 G + lambda I (the form's rounding error grows
                                with the condition of B; the product is d for a multiple of the identity and about
                                sqrt(d) cond_2(B) when one direction dominates).  Beyond the limit, with solver =
                                ALX_SOLVER_AUTO and d = 128: the dual-form solutions become the start vectors of a
                                conjugate-gradient pass over those rows (alx_stats.dual_polished_rows); otherwise the
                                rows take the d x d solve like every other row */
} alx_options;

typedef struct alx_stats {
    int64_t nnz;
    int64_t rows_in_class[2][ALX_N_CLASSES]; /* [side][class] */
    int64_t n_chunks[2];                     /* chunk descriptors of the split class, per side */
    int64_t not_spd;                         /* rows whose factorisation met a non-positive pivot, so far */
    double ms_gramian, ms_rows, ms_half_epoch; /* device time of the phases of the LAST half-epoch */
    int64_t kernel_launches;                 /* kernels this context has launched so far */
    int64_t workspace_bytes;                 /* device memory the context holds */
    int32_t kernel_path[2];                  /* [side]: 0 = FP32-ALU kernels, 1 = tensor-core kernels */
    double ms_main_kernel;                   /* tensor path: device time of the whole-rows kernel of the LAST half-epoch, else 0 */
    int64_t dual_rows;                       /* rows the LAST half-epoch solved in the dual form of Eq. 4 (0: none, or the
                                                form stepped aside because alpha0 G + lambda I was ill conditioned) */
    int64_t long_rows[2];                    /* [side], tensor-core kernels only: whole rows of more than 1024 entries
                                                whose sums the chunks kernel forms (as it does for the split rows) */
    int64_t long_entries[2];                 /* [side]: the entries those rows hold */
    int64_t cg_rows;                         /* LAST half-epoch: rows the conjugate-gradient solve took, */
    int64_t cg_products;                     /* the matrix-vector products it spent on them (steps + 1 per row), */
    int64_t cg_fallbacks;                    /* and how many of those rows went on to the Cholesky solve (not converged) */
    int32_t cholesky_by_policy[2];           /* [side]: 1 if the side's LAST half-epoch took Cholesky for every row because
                                                its conjugate-gradient run before that spent too many products per row */
    int64_t dual_polished_rows;              /* LAST half-epoch: dual-form rows that went through a conjugate-gradient pass */
    int64_t dual_polish_products;            /* because B was beyond the condition limit (see dual_cond_limit), and its products */
    int64_t entries_in_class[2][ALX_N_CLASSES]; /* [side][class]: the observed entries held by the rows of each degree class
                                                   (sums to nnz over the classes of a side) */
} alx_stats;

/* Create a context for an n_rows x n_cols problem: fp32 tables, defaults for everything else.
   (Problem statement, Sec. 3: S subset of U x I x R, W in R^{U x d}, H in R^{I x d}.) */
alx_status alx_create(int64_t n_rows, int64_t n_cols, int32_t d, float lambda, float alpha0, alx_ctx **out);
alx_status alx_create_ex(const alx_options *opt, alx_ctx **out);
/* Free the context and every device buffer it owns (waits for its stream first).  NULL is accepted.
   Plumbing of this boundary: no counterpart in the paper. */
alx_status alx_destroy(alx_ctx *ctx);

/*
 * Give the observed entries S (Sec. 3) as CSR over the matrix's rows:
 * rowptr[n_rows + 1] (int64, rowptr[0] = 0, rowptr[n_rows] = nnz), colidx[nnz] (int32, strictly
 * ascending inside each row: S is a set of pairs), values[nnz] (float labels y, or NULL: y = 1).
 * The call copies the arrays, validates them on the device (ALX_ERR_BAD_CSR, never a trap), builds
 * the transpose (CSC, row ids ascending inside each column: the item-side pass of Alg. 1 line 11
 * reads the entries column by column), and for both orientations the degree-class order of the rows and the
 * chunk descriptors of the rows longer than `split`.  Integer work only; synchronises.
 */
alx_status alx_set_csr(alx_ctx *ctx, const int64_t *rowptr, const int32_t *colidx, const float *values,
                       int64_t nnz, int on_device);

/* Overwrite one table from n x d row-major data of type src_dtype (converted with round-to-nearest-even).
   The paper's counterpart is the initialisation of W and H before the first epoch (Alg. 1 takes them as given; it
   states no distribution); otherwise plumbing of this boundary.  Synchronises. */
alx_status alx_set_embeddings(alx_ctx *ctx, alx_side side, const void *src, alx_dtype src_dtype, int on_device);

/* The same for rows row_begin .. row_begin + row_count - 1 only (src holds row_count x d values).  For tables that
   are filled in slices because a second full copy would not fit beside them; the table counts as set from the
   first call on, rows no call has written hold unspecified values.  Synchronises.  (Initialisation of W and H:
   Alg. 1 takes them as given.) */
alx_status alx_set_embedding_rows(alx_ctx *ctx, alx_side side, int64_t row_begin, int64_t row_count, const void *src,
                                  alx_dtype src_dtype, int on_device);

/*
 * One half-epoch (Alg. 1 lines 2-10 for solved_side = ALX_ROWS; line 11 for ALX_COLS):
 *   G <- X^T X over ALL rows of the fixed table X            (Alg. 1 line 2; Gramian remark under Eq. 4)
 *   for every row u of the solved side:
 *       b <- sum_{(u,i,y) in S} y x_i ;  A <- alpha0 G + lambda I + sum_{(u,i,y) in S} x_i (x) x_i
 *       row u <- A^-1 b                                      (Eq. 4), rounded to the storage type
 *   rows without observations become exactly 0.
 * Asynchronous on the context's stream.
 */
alx_status alx_half_epoch(alx_ctx *ctx, alx_side solved_side);

/* alx_half_epoch(ALX_ROWS) then alx_half_epoch(ALX_COLS): the column pass sees the new W (Alg. 1). */
alx_status alx_epoch(alx_ctx *ctx);

/*
 * The same work as alx_set_csr followed by alx_set_embeddings of both tables, from HOST arrays, with the
 * copies overlapped: W (n_rows x d) and H (n_cols x d), row-major, elements of the context's STORAGE
 * type, follow S over the bus on a second stream while the integer work of alx_set_csr runs.  The
 * overlap needs page-locked host memory (pageable memory works, without overlap).  The arrays are not
 * referenced after the call returns.  Synchronises.  Errors as alx_set_csr.
 */
alx_status alx_load_host(alx_ctx *ctx, const int64_t *rowptr, const int32_t *colidx, const float *values,
                         int64_t nnz, const void *W, const void *H);

/*
 * The same work as alx_epoch followed by alx_get_embeddings of both whole tables into HOST arrays of the
 * storage type (W_dst: n_rows x d, H_dst: n_cols x d): the new W is read back on a second stream while
 * the column pass, which only reads it, runs.  Page-locked destinations overlap.  Synchronises.
 */
alx_status alx_epoch_to_host(alx_ctx *ctx, void *W_dst, void *H_dst);

/*
 * As alx_half_epoch, and additionally returns, for the k listed rows of the solved side, the
 * float32 solution BEFORE it is rounded to the storage type (x_out: k x d floats, host memory).
 * Used to check the residual |A x - b| / |b| of the solver itself.  Synchronises.
 */
alx_status alx_half_epoch_capture(alx_ctx *ctx, alx_side solved_side, const int64_t *row_ids, int64_t k,
                                  float *x_out);

/*
 * The objective of Eq. 3 at the current tables:
 *   components[0] = sum_S (y - <w_u, h_i>)^2
 *   components[1] = alpha0 * sum_u sum_i <w_u, h_i>^2   (computed as <W^T W, H^T H>_F)
 *   components[2] = lambda * (|W|_F^2 + |H|_F^2)
 * total = their sum.  Products in float32, every accumulation across entries in float64 in a fixed
 * order.  components may be NULL.  Synchronises.
 */
alx_status alx_loss(alx_ctx *ctx, double *total, double *components);

/* Copy rows [row_begin, row_begin + row_count) of one table to dst (row_count x d, dst_dtype). Synchronises.
   The tables are the method's output (W, H of Sec. 3); the call itself is plumbing with no counterpart in the paper. */
alx_status alx_get_embeddings(alx_ctx *ctx, alx_side side, void *dst, alx_dtype dst_dtype, int64_t row_begin,
                              int64_t row_count, int on_device);

/* ---- diagnostics used by tests and the benchmark ---- */

/* The Gramian the last alx_half_epoch(solved = side) or alx_loss computed for the table of `fixed_side`
   (d x d doubles, host).  ALX_ERR_BAD_STATE if none has been computed yet. */
alx_status alx_get_gramian(alx_ctx *ctx, alx_side fixed_side, double *dst);
/* Compute only the Gramian of one table now (the first step of a half-epoch) and return it. */
alx_status alx_gramian(alx_ctx *ctx, alx_side table, double *dst);

/* The transpose built by alx_set_csr: colptr[n_cols + 1], rowidx[nnz], values_t[nnz] (may be NULL). Host memory. */
alx_status alx_get_transpose(alx_ctx *ctx, int64_t *colptr, int32_t *rowidx, float *values_t);

/*
 * The degree-class structure of one orientation (side = which table's rows are ordered).
 *   class(deg) = 0 if deg = 0; ALX_N_CLASSES-1 if deg > split; otherwise the smallest c >= 1 with
 *   deg <= 16 * 2^(c-1), capped at ALX_N_CLASSES-2.
 *   order[n]              : row ids sorted by (class, id)
 *   class_offsets[13]     : start of each class inside `order`
 *   chunk_desc[4*n_chunks]: for the rows of the last class in ascending id, consecutive pieces of
 *                           `split` entries (the last one shorter): row, begin, end, slot (int64 each)
 * Pass NULL for arrays that are not wanted; *n_chunks (may be NULL) receives the descriptor count. Host memory.
 */
alx_status alx_get_buckets(alx_ctx *ctx, alx_side side, int32_t *order, int64_t *class_offsets,
                           int64_t *chunk_desc, int64_t *n_chunks);

/* Counters and device times of the context (see alx_stats).  Diagnostics: no counterpart in the paper. */
alx_status alx_get_stats(alx_ctx *ctx, alx_stats *out);

/*
 * Evaluation (Sec. 4.6; the protocol of Sec. 5; the metric of Table 2).  Not part of a training epoch.
 *
 * alx_fold_in: embeddings of rows that were not trained.  Sec. 5 obtains the embedding of a held-out source row from
 * the part of its links that is kept, through Eq. 4 with the trained column table held fixed: one more rows half-step,
 * on new rows.  rowptr[n_new + 1] / colidx[nnz] / values[nnz] (or NULL: y = 1) give the new rows as CSR over the
 * context's columns, with the rules of alx_set_csr; x_out receives n_new x d floats, the solutions after the round
 * to the storage type (the values a trained table would hold).  The arrays are host or device memory as on_device
 * says, x_out included.  The context's own matrix and tables are not touched; the call allocates what the half-step
 * needs for n_new rows, runs the same kernels as alx_half_epoch and synchronises.  A row with no entry gets 0.
 * ALX_ERR_BAD_STATE before the column table holds anything, ALX_ERR_BAD_CSR as alx_set_csr.
 */
alx_status alx_fold_in(alx_ctx *ctx, const int64_t *rowptr, const int32_t *colidx, const float *values, int64_t n_new,
                       int64_t nnz, int on_device, float *x_out);

#define ALX_MAX_TOPK 256
/*
 * alx_topk: exact Top-K retrieval (Sec. 4.6: the best k items of a user by inner product; every item is scored, no
 * approximate search).  queries: m x d floats; the items are the rows of table `items` (ALX_COLS for the protocol
 * of Sec. 5) as stored.  For query q the ids of the k largest <q, h_i> go to ids_out[q * k ..], best first; equal
 * scores are ordered by ascending id (the paper states no tie rule); scores_out (m x k, may be NULL) receives the
 * scores.  exclude_ptr[m + 1] / exclude_idx (may both be NULL) list, per query and ascending, ids that must not be
 * returned (the kept links of a fold-in row, for example; the paper does not say whether it leaves them out).  Where
 * fewer than k items qualify the row is filled with id -1 and score -inf.  1 <= k <= ALX_MAX_TOPK.
 * Scores are fp32: for d = 128 with bfloat16 tables products of bfloat16 parts summed in fp32 on the tensor cores
 * (the query as three parts, so to fp32 accuracy); otherwise fp32 FMAs.  Two items whose exact scores differ by less
 * than that rounding may come out in either order.  All arrays host or device as on_device says; synchronises.
 */
alx_status alx_topk(alx_ctx *ctx, alx_side items, const float *queries, int64_t m, int32_t k, const int64_t *exclude_ptr,
                    const int32_t *exclude_idx, int on_device, int32_t *ids_out, float *scores_out);

/*
 * alx_recall_at_k: Recall@K as Table 2 reports it, read as: for every query with at least one ground-truth id, the
 * number of ground-truth ids among its first k retrieved ids divided by the number of its ground-truth ids; the mean
 * over those queries (the paper names the metric without a formula).  ids: m rows of k_stride retrieved ids (best
 * first, -1 = none), of which the first k count; truth_ptr[m + 1] / truth_idx: ground truth per query, ascending.
 * *recall receives the mean, *n_counted (may be NULL) the number of queries it is over.  Sums in a fixed order.
 */
alx_status alx_recall_at_k(alx_ctx *ctx, const int32_t *ids, int64_t m, int32_t k_stride, int32_t k,
                           const int64_t *truth_ptr, const int32_t *truth_idx, int on_device, double *recall,
                           int64_t *n_counted);

/* Diagnostic for roofline reports: measured FP32 fused-multiply-add throughput of the device in
   TFLOP/s (a register-resident FMA loop on every SM, best of three).  No counterpart in the paper.
   Allocates and frees 256 bytes with cudaMalloc; synchronises. */
alx_status alx_fp32_peak_tflops(alx_ctx *ctx, double *tflops);

/* Wait for the context's stream and report any device-detected problem since the last check. */
alx_status alx_synchronize(alx_ctx *ctx);

/* Text of the last error on this context ("" if none).  Valid until the next call on the context. */
const char *alx_last_error(const alx_ctx *ctx);

/*
 * Gramian of a table without allocating anything (the paper has no counterpart; this is an addition for
 * callers that cannot allocate device memory when they call: inside a frozen memory pool, on a thread
 * that must not take an allocator lock, under a memory budget fixed at start-up).
 *   table   : device pointer, 16-byte aligned, n x d row-major, float32 or bfloat16 (dtype)
 *   gramian : device pointer, 8-byte aligned, d x d doubles, receives table^T table; written on `stream`
 *             (cudaStream_t, NULL = legacy default stream); the call does not synchronise
 * A pointer that is not aligned as stated is refused with ALX_ERR_INVALID_ARG before anything is launched.
 * Same kernels and the same fixed summation order as alx_gramian on a context created with kernels = 1
 * (the FP32-ALU kernels), so those results agree to the last bit.
 * The piece sums go to a fixed array inside the library image (16 MiB + 64 KiB on every GPU that loads
 * the library, held until the process exits).  Limits: d in {16, 32, 64, 128} and
 * n <= alx_gramian_noalloc_max_rows(d) = (4 Mi / d^2) * 4096 rows (1 048 576 for d = 128); larger inputs
 * are refused with ALX_ERR_UNSUPPORTED and a message in alx_noalloc_last_error().  No cudaMalloc, cudaFree
 * or other allocating routine is called.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) with that
 * device current; make that first call outside any stream capture.  The first use of the library's Gramian
 * kernels on a device is also when the driver loads the module that carries the array, so that is when the
 * 16 MiB are taken from the device: a caller whose memory is frozen later should make one warm-up call per
 * device before the freeze.  The device that owns `table` must be
 * the current device.  All calls share the one array and it keeps the previous call's contents (each call
 * overwrites every piece it later reads, so nothing needs clearing): two calls whose kernels overlap on
 * the GPU -- different streams, or different host threads -- race; order them on one stream.
 */
alx_status alx_gramian_noalloc(const void *table, alx_dtype dtype, int64_t n, int32_t d, double *gramian,
                               void *stream);
int64_t alx_gramian_noalloc_max_rows(int32_t d);
/* Message of the calling thread's last failed alx_gramian_noalloc ("" after a success). */
const char *alx_noalloc_last_error(void);

/* Library version string, e.g. "alx-b200 0.1 (sm_100a)". */
const char *alx_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ALX_H_ */
