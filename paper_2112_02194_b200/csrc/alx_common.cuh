// Shared declarations of the CUDA side of the library: device status word, storage-type helpers,
// launch descriptors.  Host entry points of each .cu file are declared at the bottom.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace alx {

constexpr int kNClasses = 12;

// bits of DevStatus::flags
enum : unsigned {
    kFlagBadRowptr = 1u,
    kFlagBadCol = 2u,
    kFlagUnsorted = 4u,
    kFlagNotSpd = 8u,
    kFlagTimeout = 16u,   // a bounded wait inside a kernel ran out
    kFlagInternal = 32u,
};

struct DevStatus {
    unsigned flags;
    unsigned pad;
    unsigned long long not_spd;   // rows whose factorisation met a non-positive pivot
    long long first_bad;          // an offending position (entry or row) for error messages
};

__device__ __forceinline__ void raise_flag(DevStatus *st, unsigned f, long long where)
{
    unsigned old = atomicOr(&st->flags, f);
    if (!(old & f)) st->first_bad = where;
}

// ---- storage types -------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_elem(float *p, float v) { *p = v; }
__device__ __forceinline__ void store_elem(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// 16-byte chunk of a table row -> floats (4 for fp32, 8 for bf16)
template <typename T> struct Chunk16;
template <> struct Chunk16<float> {
    static constexpr int kElems = 4;
    __device__ static __forceinline__ void load(const float *p, float *out)
    {
        float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct Chunk16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16 *p, float *out)
    {
        uint4 v = __ldg(reinterpret_cast<const uint4 *>(p));
        const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            out[2 * k] = __uint_as_float(w[k] << 16);
            out[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
};

// ---- what a half-epoch hands to the row kernels -------------------------------------------
struct SideView {
    const int64_t *ptr;    // [n + 1] offsets of the solved side's rows
    const int32_t *idx;    // [nnz] ids into the fixed table, ascending inside a row
    const float *val;      // [nnz] labels or nullptr (all 1)
    const int32_t *order;  // [n] rows by (class, id)
    const int64_t *chunk_desc;   // [4 * n_chunks]
    const int64_t *split_first;  // [n_split_rows + 1]
    int64_t n;
};

struct RowOut {
    void *table;             // solved table, storage type, row-major [n x d]
    const int32_t *cap_slot; // nullptr, or per-row capture slot (-1 = none)
    float *cap_out;          // [slots x d] fp32 solutions before rounding
};

// ---- host entry points (one per .cu) ----------------------------------------------------------
struct ScanScratch;

// alx_setup.cu
cudaError_t scan_exclusive(const void *in, bool in_is_i64, int64_t *out, int64_t n, int64_t *scratch,
                           int64_t scratch_elems, cudaStream_t s, int64_t *launches);
int64_t scan_scratch_elems(int64_t n);
cudaError_t launch_validate(const int64_t *rowptr, const int32_t *colidx, int64_t n_rows, int64_t n_cols,
                            int64_t nnz, DevStatus *st, cudaStream_t s, int64_t *launches);
cudaError_t launch_degrees(const int64_t *ptr, int64_t n, int32_t *deg, cudaStream_t s, int64_t *launches);
// Entry lists over a table of 2N rows (the bfloat16 parts of an fp32 table, see launch_rows_fold): row u of length L
// becomes a row of 2L entries, its L ids followed by the same ids + N (labels repeated); vptr = 2 ptr.
cudaError_t launch_double_entries(const int64_t *ptr, const int32_t *idx, const float *val, int64_t n, int64_t n_fixed,
                                  int64_t *vptr, int32_t *vidx, float *vval, cudaStream_t s, int64_t *launches);
// stable partition of a list of rows by length (see alx_setup.cu)
cudaError_t launch_partition_by_length(const int64_t *ptr, const int32_t *rows, int64_t count, int limit, int32_t *out,
                                       int64_t *block_counts, int64_t *block_offsets, int64_t *n_short_dev,
                                       int64_t *scan_scratch, int64_t scan_elems, cudaStream_t s, int64_t *launches);
// entries held by the rows of each degree class: out[kNClasses] (device), class_offs = the kNClasses + 1 offsets into order
cudaError_t launch_class_entries(const int64_t *ptr, const int32_t *order, const int64_t *class_offs_dev, int64_t n,
                                 int64_t *out, cudaStream_t s, int64_t *launches);
cudaError_t launch_sum_row_lengths(const int64_t *ptr, const int32_t *rows, int64_t count, int64_t *out, cudaStream_t s,
                                   int64_t *launches);
cudaError_t launch_count_cols(const int32_t *colidx, int64_t nnz, int32_t *counts, cudaStream_t s, int64_t *launches);
cudaError_t launch_fill_transpose(const int64_t *rowptr, const int32_t *colidx, int64_t n_rows, int64_t nnz,
                                  const int64_t *colptr, int32_t *cursor, int32_t *rowidx, cudaStream_t s,
                                  int64_t *launches);
cudaError_t launch_sort_segments(const int64_t *colptr, int32_t *rowidx, const int32_t *order,
                                 const int64_t *class_offs_host, cudaStream_t s, int64_t *launches);
cudaError_t launch_values_transpose(const int64_t *rowptr, const int32_t *colidx, const float *values,
                                    const int64_t *colptr, const int32_t *rowidx, int64_t n_cols, int64_t nnz,
                                    float *values_t, cudaStream_t s, int64_t *launches);
// order by (class, id): block_counts scratch is [kNClasses * n_blocks] int64 (+ scan scratch)
int64_t bucket_blocks(int64_t n);
cudaError_t launch_bucket(const int64_t *ptr, int64_t n, int64_t split, int64_t *block_counts,
                          int64_t *block_offsets, int64_t *scan_scratch, int64_t scan_scratch_elems,
                          int32_t *order, int64_t *class_offs_dev, cudaStream_t s, int64_t *launches);
cudaError_t launch_chunk_counts(const int64_t *ptr, const int32_t *split_rows, int64_t n_split, int64_t split,
                                int64_t *counts, cudaStream_t s, int64_t *launches);
cudaError_t launch_chunk_fill(const int64_t *ptr, const int32_t *split_rows, int64_t n_split, int64_t split,
                              const int64_t *first, int64_t *desc, cudaStream_t s, int64_t *launches);
cudaError_t launch_convert(const void *src, int src_bf16, void *dst, int dst_bf16, int64_t count, cudaStream_t s,
                           int64_t *launches);

// alx_gramian.cu
constexpr int kGramRowsPerPartial = 4096;
int64_t gramian_partials(int64_t n);
cudaError_t launch_gramian(const void *X, int bf16, int64_t n, int d, float *partials, double *G64, float *Bmat,
                           float alpha0, float lambda, cudaStream_t s, int64_t *launches);

cudaError_t launch_gramian_reduce(const float *partials, int64_t n_partials, int d, double *G64, float *Bmat,
                                  float alpha0, float lambda, cudaStream_t s, int64_t *launches);
cudaError_t measure_fp32_peak(double *tflops, cudaStream_t s);

// alx_rows.cu
cudaError_t launch_rows_simple(const SideView &sv, const int64_t *class_offs_host, int64_t n_chunks,
                               int64_t n_split_rows, const void *X, int bf16, int d, const float *Bmat,
                               float *split_partials, RowOut out, DevStatus *st, cudaStream_t s,
                               int64_t *launches);

// Tensor-core path: the first degree class whose rows (with all longer whole rows) get their sums from the chunks
// kernel instead of the rows kernel.  Classes 8 .. 10 (1025 .. 8192 observations at the default split) qualify, from
// the top, as long as they hold at most kLongRowBudget rows together (one d x d + d sum of workspace each).
constexpr int64_t kLongRowBudget = 65536;
inline int long_class_begin(const int64_t *class_offs_host)
{
    int c = kNClasses - 1;
    while (c > 8 && class_offs_host[kNClasses - 1] - class_offs_host[c - 1] <= kLongRowBudget) --c;
    return c;
}

// What the library remembers, per side, of the conjugate-gradient solve's cost, on the device (so that choosing the
// solver of a half-epoch needs no host round trip): rows and products of the side's last conjugate-gradient run, the
// choice for the run being launched, and how many half-epochs of the side have been launched.
struct CgPolicy {
    unsigned long long rows, products;
    int use_cholesky;     // this half-epoch: 1 = the in-place Cholesky takes every row of the whole-rows kernel
    int calls;
    int short_rows_by_cg; // this half-epoch: 1 = rows of 17 .. 32 observations go to the whole-rows kernel, not the dual form
    int pad_;
};
// Rows of 17 .. 32 observations: dual form, or the whole-rows kernel's conjugate gradients where those are cheap.
// Measured on the rows side of the 10M x 10M workload (1.32M such rows): with them in the whole-rows kernel the
// half-epoch takes 152.3 ms against 161.1 ms at 10.9 products per row (6.7 ns per row saved); a product costs about
// 1.8 ns per row, so the two meet near 14.5 products.  Where the side's last conjugate-gradient run stayed at or below
// this many products per row, those rows go there
constexpr float kShortRowsByCgProducts = 13.f;
// Conjugate gradients pay while a row takes fewer than about 28 products on average (measured on B200: about 2900 + 300
// per product cycles of an SM per row, against 12 600 for the in-place Cholesky; alx_options.cg_switch_products); beyond
// that the side's next half-epochs go to Cholesky, with one conjugate-gradient half-epoch every kCgReprobe to see whether
// the matrices have improved
constexpr int kCgReprobe = 8;

// conjugate-gradient solve of the whole-rows tensor-core kernel (Sec. 4.5)
struct CgOptions {
    bool enabled;
    int max_iter;                  // a row that has not converged by then is solved by the in-place Cholesky instead
    float tol;                     // stop at |r| <= tol |b|
    bool warm_start;               // start from the row's stored embedding (the solved table holds trained values)
    unsigned long long *counters;  // device, [3]: rows, matrix-vector products, rows that fell back
    int32_t *fallback_list;        // device, one entry per row of the larger side: the rows left to the Cholesky solve
    CgPolicy *policy;              // device, this side's record
    float switch_products;         // mean products per row beyond which the side's next half-epochs take Cholesky
};

// alx_umma.cu: tensor-core path, d = 128 and bf16 tables only
int64_t gramian_umma_partials();
cudaError_t launch_gramian_umma(const void *X, int64_t n, float *partials, cudaStream_t s, int64_t *launches);
// ---- evaluation (alx_eval.cu, alx_topk_umma.cu)
// slabs of items per query tile (each slab's best k are listed separately and merged)
int topk_slabs(int64_t n_items, int64_t m);
// exact Top-K of <q, h_i>: H [n_items x d] (storage type), Q [m x d] fp32; lists: [slabs][m][k] scratch;
// ids_out [m x k] (-1 where fewer than k items qualify), scores_out [m x k] or nullptr; ex_*: per-query ids to leave out
cudaError_t launch_topk(const void *H, bool bf16, int64_t n_items, int d, const float *Q, int64_t m, int k,
                        const int64_t *ex_ptr, const int32_t *ex_idx, int slabs, float *list_s, int32_t *list_id,
                        int32_t *list_cnt, int32_t *ids_out, float *scores_out, bool tensor_cores, void *scratch_q,
                        DevStatus *st, cudaStream_t s, int64_t *launches);
// the tensor-core scoring kernel (d = 128, bfloat16 table); scratch_q: topk_query_scratch_bytes(m) bytes for the queries'
// bfloat16 parts
int64_t topk_query_scratch_bytes(int64_t m);
cudaError_t launch_topk_umma(const void *H, int64_t n_items, const float *Q, int64_t m, int k, const int64_t *ex_ptr,
                             const int32_t *ex_idx, int slabs, int64_t slab, float *list_s, int32_t *list_id,
                             int32_t *list_cnt, void *scratch_q, DevStatus *st, cudaStream_t s, int64_t *launches);
cudaError_t launch_recall(const int32_t *ids, int64_t m, int k_stride, int k, const int64_t *tptr, const int32_t *tidx,
                          double *per_query, double *out2, cudaStream_t s, int64_t *launches);
cudaError_t launch_rows_fold(const SideView &sv, const int64_t *class_offs_host, int64_t n_chunks, int64_t n_split_rows,
                             const void *T, int64_t n_table, const float *Bmat, float *split_partials, RowOut out,
                             DevStatus *st, cudaStream_t s, int64_t *launches, cudaEvent_t main_begin, cudaEvent_t main_end,
                             const CgOptions &cg, const int *dual_flag);
// fp32 table [n x 64] -> bfloat16 parts [2n x 128]
cudaError_t launch_split_table(const float *X, int64_t n, void *T, cudaStream_t s, int64_t *launches);
cudaError_t launch_rows_umma(const SideView &sv, const int64_t *class_offs_host, int64_t n_chunks,
                             int64_t n_split_rows, const void *X, const float *Bmat, float *split_partials,
                             RowOut out, DevStatus *st, cudaStream_t s, int64_t *launches, cudaEvent_t main_begin,
                             cudaEvent_t main_end, const void *dual_ws, int64_t n_table, const CgOptions &cg, const int32_t *order16 = nullptr, int64_t n4 = 0, int64_t n8 = 0);

// alx_dual.cu: rows with at most 32 observations in the dual form (d = 128, bf16 tables)
size_t dual_workspace_bytes();
cudaError_t launch_dual_prepare(const float *Bmat, void *ws, float cond_limit, bool allow_start, cudaStream_t s,
                                int64_t *launches);
// fp32 tables of 64 features (alx_dual64.cu): B^-1 (fp32) + flag; rows of 1 .. 16 observations in the dual form
size_t dual64_workspace_bytes();
int *dual64_flag_ptr(void *ws);
cudaError_t launch_dual64_prepare(const float *Bmat, void *ws, float cond_limit, cudaStream_t s, int64_t *launches);
cudaError_t launch_rows_dual64(const SideView &sv, int64_t first, int64_t count, const void *X, void *ws, RowOut out,
                               cudaStream_t s, int64_t *launches);
const int *dual_flag_ptr(const void *ws);
// route: set where conjugate gradients run; the kernel of the rows of 17 .. 32 observations returns at once when it says so.
// order16 (may be null): the count16 rows of 1 .. 16 observations again, ordered by length class: the n4 rows of at most 4
// first, then those of 5 .. 8 (up to position n8), then the rest; the first two parts go to kernel instances with four and
// eight observations per row, which do four times and twice the rows per tile
cudaError_t launch_rows_dual(const SideView &sv, int64_t first16, int64_t count16, int64_t count32, const void *X,
                             const void *ws, RowOut out, DevStatus *st, const CgPolicy *route, const int32_t *order16,
                             int64_t n4, int64_t n8, cudaStream_t s, int64_t *launches);

// alx_loss.cu
int64_t loss_partials(int64_t nnz);
cudaError_t launch_loss_obs(const int64_t *rowptr, const int32_t *colidx, const float *values, int64_t n_rows,
                            int64_t nnz, const void *W, const void *H, int bf16, int d, double *partials,
                            double *result, cudaStream_t s, int64_t *launches);
cudaError_t launch_loss_finish(const double *partials, int64_t n_partials, const double *GW, const double *GH, int d,
                               double alpha0, double lambda, double *result, cudaStream_t s, int64_t *launches);

}  // namespace alx
