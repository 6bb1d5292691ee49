// C ABI of the library (declared in include/alx.h): context, argument checks, device memory,
// and the order in which the kernels of one half-epoch are launched.  No arithmetic of the method
// happens on the host.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "../../include/alx.h"
#include "alx_common.cuh"
#include <nvtx3/nvToolsExt.h>      // header-only: ranges show up in a profiler's timeline, and cost nothing without one

using namespace alx;

struct alx_ctx {
    alx_options opt{};
    int device = 0;
    cudaStream_t stream = nullptr;
    int bf16 = 0;
    size_t elem = 4;
    int64_t n[4] = {0, 0, 0, 0};   // n[ALX_ROWS] = n_rows, n[ALX_COLS] = n_cols (and again for the doubled lists, see below)
    int64_t nnz = -1;
    int64_t split = ALX_DEFAULT_SPLIT;
    bool has_values = false;
    bool have_table[2] = {false, false};
    bool have_gram[2] = {false, false};

    // per orientation: [ALX_ROWS] = CSR (rows of the matrix), [ALX_COLS] = CSC.  Slots 2 and 3 (fp32 tables of 64 features
    // on the tensor cores only): the same two orientations with every row's entry list doubled over the table of
    // bfloat16 parts, which is what that path's kernels walk; with degree classes and chunks of their own.
    int64_t *ptr[4] = {nullptr, nullptr, nullptr, nullptr};
    int32_t *idx[4] = {nullptr, nullptr, nullptr, nullptr};
    float *val[4] = {nullptr, nullptr, nullptr, nullptr};
    int32_t *order[4] = {nullptr, nullptr, nullptr, nullptr};
    int64_t *class_offs_dev[4] = {nullptr, nullptr, nullptr, nullptr};
    int64_t class_offs[4][ALX_N_CLASSES + 1] = {};
    int64_t *chunk_desc[4] = {nullptr, nullptr, nullptr, nullptr};
    int64_t *split_first[4] = {nullptr, nullptr, nullptr, nullptr};
    int64_t n_chunks[4] = {0, 0, 0, 0};
    int64_t n_split_rows[4] = {0, 0, 0, 0};
    // tensor path with the dual form: the rows of 1 .. 16 entries once more per orientation, those with at most 8 entries first
    int32_t *order16[2] = {nullptr, nullptr};
    int64_t n4[2] = {0, 0}, n8[2] = {0, 0};      // ... and those with at most 4 before them
    void *fold_table = nullptr;   // that path's fixed table: [2 N x 128] bfloat16 parts of the fp32 table, rebuilt every half-epoch

    void *table[2] = {nullptr, nullptr};
    double *G64[2] = {nullptr, nullptr};   // Gramian of table [side]
    float *Bmat = nullptr;
    float *gram_partials = nullptr;
    float *split_partials = nullptr;
    void *dual_ws = nullptr;      // tensor path: B^-1 operand tiles and the flag of the dual form
    int64_t dual_candidates = 0;  // rows of classes 1 and 2 of the last half-epoch (solved in the dual form if the flag is set)
    int dual_flag_latched = 0;
    int64_t dual_candidates32 = 0; // of them, the rows of 17 .. 32 observations (which the whole-rows kernel may have taken instead)
    CgPolicy policy_latched{};    // the side's policy record as the last half-epoch's kernels saw it    // that flag as the last half-epoch's kernels saw it (the loss and the Gramian calls rewrite it)
    double *loss_partials_buf = nullptr;
    double *loss_result = nullptr;
    DevStatus *status = nullptr;
    unsigned long long *cg_counters = nullptr;   // tensor path, last half-epoch: rows solved by conjugate gradients, products, fall-backs; dual-form rows polished, their products
    int32_t *cg_fallback_list = nullptr;         // tensor path with conjugate gradients: the rows left to the Cholesky solve
    CgPolicy *cg_policy = nullptr;               // [2]: per side, what the solver choice of its next half-epoch rests on

    // second stream for the host copies that alx_load_host / alx_epoch_to_host overlap with kernels
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t copy_ev = nullptr;
    const void *upload_after_csr[2] = {nullptr, nullptr};   // alx_load_host: tables to upload behind the upload of S

    cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    bool main_timed = false;
    alx_stats stats{};
    int64_t launches = 0;
    int64_t bytes_held = 0;
    std::vector<std::pair<void *, size_t>> owned;
    std::string err;
};

namespace {

alx_status fail(alx_ctx *c, alx_status code, const char *fmt, ...)
{
    if (c) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        c->err = buf;
    }
    return code;
}

#define ALX_CUDA(c, expr)                                                                          \
    do {                                                                                           \
        cudaError_t e_ = (expr);                                                                   \
        if (e_ != cudaSuccess)                                                                     \
            return fail((c), e_ == cudaErrorMemoryAllocation ? ALX_ERR_OOM : ALX_ERR_CUDA,         \
                        "%s failed: %s", #expr, cudaGetErrorString(e_));                           \
    } while (0)

// a named range on the profiler's timeline for as long as the object lives
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) { cudaGetDevice(&prev); if (prev != dev) cudaSetDevice(dev); else prev = -1; }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

void *dev_alloc(alx_ctx *c, size_t bytes)
{
    if (bytes == 0) bytes = 256;
    void *p = nullptr;
    if (c->opt.alloc) {
        p = c->opt.alloc(bytes, c->opt.alloc_user);
    } else if (cudaMalloc(&p, bytes) != cudaSuccess) {
        cudaGetLastError();
        p = nullptr;
    }
    if (p) {
        c->owned.emplace_back(p, bytes);
        c->bytes_held += (int64_t)bytes;
    }
    return p;
}

void dev_free(alx_ctx *c, void *p)
{
    if (!p) return;
    for (size_t k = 0; k < c->owned.size(); ++k)
        if (c->owned[k].first == p) {
            c->bytes_held -= (int64_t)c->owned[k].second;
            c->owned.erase(c->owned.begin() + k);
            break;
        }
    if (c->opt.free) c->opt.free(p, c->opt.alloc_user); else cudaFree(p);
}

template <typename T> bool alloc_into(alx_ctx *c, T *&dst, size_t count)
{
    dst = static_cast<T *>(dev_alloc(c, count * sizeof(T)));
    return dst != nullptr;
}

#define ALX_ALLOC(c, dst, count)                                                                   \
    do {                                                                                           \
        if (!alloc_into((c), (dst), (size_t)(count)))                                              \
            return fail((c), ALX_ERR_OOM, "device allocation of %zu bytes failed",                 \
                        (size_t)(count) * sizeof(*(dst)));                                         \
    } while (0)

// Temporaries of one call: whatever is still registered when the call returns, on any path, goes back to the allocator
// (after the stream has drained, since kernels in flight may still use it).
struct Scratch {
    alx_ctx *c;
    std::vector<void *> held;
    explicit Scratch(alx_ctx *ctx) : c(ctx) {}
    Scratch(const Scratch &) = delete;
    Scratch &operator=(const Scratch &) = delete;
    template <typename T> T *keep(T *p) { if (p) held.push_back(p); return p; }
    void release(void *p)
    {
        for (size_t k = 0; k < held.size(); ++k)
            if (held[k] == p) { held.erase(held.begin() + k); dev_free(c, p); return; }
    }
    ~Scratch()
    {
        if (held.empty()) return;
        cudaStreamSynchronize(c->stream);
        for (void *p : held) dev_free(c, p);
    }
};

#define ALX_TMP(c, scratch, dst, count)                                                            \
    do {                                                                                           \
        ALX_ALLOC(c, dst, count);                                                                  \
        (scratch).keep(dst);                                                                       \
    } while (0)

// read and clear the device status word (after a stream synchronise)
alx_status check_device_status(alx_ctx *c)
{
    DevStatus h;
    ALX_CUDA(c, cudaMemcpyAsync(&h, c->status, sizeof h, cudaMemcpyDeviceToHost, c->stream));
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    c->stats.not_spd += (int64_t)h.not_spd;
    if (h.flags == 0) return ALX_OK;
    ALX_CUDA(c, cudaMemsetAsync(c->status, 0, sizeof(DevStatus), c->stream));
    if (h.flags & kFlagBadRowptr) return fail(c, ALX_ERR_BAD_CSR, "rowptr is not a monotone offset array (near row %lld)", h.first_bad);
    if (h.flags & kFlagBadCol) return fail(c, ALX_ERR_BAD_CSR, "column index out of range at entry %lld", h.first_bad);
    if (h.flags & kFlagUnsorted) return fail(c, ALX_ERR_BAD_CSR, "column indices not strictly ascending inside a row at entry %lld", h.first_bad);
    // a wait that ran out leaves rows unsolved, which matters more than rows set to zero: report it first
    if (h.flags & kFlagTimeout)
        return fail(c, ALX_ERR_CUDA, "a bounded wait inside a kernel ran out (wait site %lld, block %lld)%s", h.first_bad / 1000000,
                    h.first_bad % 1000000, (h.flags & kFlagNotSpd) ? "; rows also met non-positive pivots" : "");
    if (h.flags & kFlagNotSpd) return fail(c, ALX_ERR_NOT_SPD, "%llu rows met a non-positive pivot (first: row %lld); they were set to zero", h.not_spd, h.first_bad);
    return fail(c, ALX_ERR_CUDA, "device status flags 0x%x", h.flags);
}

SideView side_view(const alx_ctx *c, int side)
{
    SideView v;
    v.ptr = c->ptr[side];
    v.idx = c->idx[side];
    v.val = c->val[side];
    v.order = c->order[side];
    v.chunk_desc = c->chunk_desc[side];
    v.split_first = c->split_first[side];
    v.n = c->n[side];
    return v;
}

// degree classes, order and chunk descriptors of one orientation
alx_status build_buckets(alx_ctx *c, int side, int64_t *scratch_a, int64_t *scratch_b, int64_t *scan_scratch,
                         int64_t scan_elems)
{
    const int64_t n = c->n[side];
    ALX_CUDA(c, launch_bucket(c->ptr[side], n, c->split, scratch_a, scratch_b, scan_scratch, scan_elems,
                              c->order[side], c->class_offs_dev[side], c->stream, &c->launches));
    ALX_CUDA(c, cudaMemcpyAsync(c->class_offs[side], c->class_offs_dev[side], sizeof(int64_t) * (ALX_N_CLASSES + 1),
                                cudaMemcpyDeviceToHost, c->stream));
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    const int64_t *offs = c->class_offs[side];
    const int64_t n_split = offs[ALX_N_CLASSES] - offs[ALX_N_CLASSES - 1];
    c->n_split_rows[side] = n_split;
    c->n_chunks[side] = 0;
    if (n_split > 0) {
        Scratch tmp(c);
        int64_t *counts = nullptr;
        ALX_TMP(c, tmp, counts, n_split);
        ALX_ALLOC(c, c->split_first[side], n_split + 1);
        const int32_t *split_rows = c->order[side] + offs[ALX_N_CLASSES - 1];
        ALX_CUDA(c, launch_chunk_counts(c->ptr[side], split_rows, n_split, c->split, counts, c->stream, &c->launches));
        ALX_CUDA(c, scan_exclusive(counts, true, c->split_first[side], n_split, scan_scratch, scan_elems, c->stream,
                                   &c->launches));
        int64_t total = 0;
        ALX_CUDA(c, cudaMemcpyAsync(&total, c->split_first[side] + n_split, sizeof total, cudaMemcpyDeviceToHost, c->stream));
        ALX_CUDA(c, cudaStreamSynchronize(c->stream));
        c->n_chunks[side] = total;
        ALX_ALLOC(c, c->chunk_desc[side], 4 * total);
        ALX_CUDA(c, launch_chunk_fill(c->ptr[side], split_rows, n_split, c->split, c->split_first[side],
                                      c->chunk_desc[side], c->stream, &c->launches));
        ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    }
    if (side < 2) {
        for (int k = 0; k < ALX_N_CLASSES; ++k) c->stats.rows_in_class[side][k] = offs[k + 1] - offs[k];
        c->stats.n_chunks[side] = c->n_chunks[side];
    }
    return ALX_OK;
}

void release_matrix(alx_ctx *c)
{
    for (int s = 0; s < 4; ++s) {
        dev_free(c, c->ptr[s]); c->ptr[s] = nullptr;
        dev_free(c, c->idx[s]); c->idx[s] = nullptr;
        dev_free(c, c->val[s]); c->val[s] = nullptr;
        dev_free(c, c->order[s]); c->order[s] = nullptr;
        dev_free(c, c->chunk_desc[s]); c->chunk_desc[s] = nullptr;
        dev_free(c, c->split_first[s]); c->split_first[s] = nullptr;
    }
    for (int s = 0; s < 2; ++s) { dev_free(c, c->order16[s]); c->order16[s] = nullptr; c->n4[s] = c->n8[s] = 0; }
    dev_free(c, c->split_partials); c->split_partials = nullptr;
    dev_free(c, c->loss_partials_buf); c->loss_partials_buf = nullptr;
    c->nnz = -1;
}

bool tensor_path(const alx_ctx *c) { return c->bf16 && c->opt.d == 128 && c->opt.kernels != 1; }
// fp32 tables of 64 features: tensor cores through bfloat16 parts and doubled entry lists (ids up to 2 N must fit int32)
bool fold_path(const alx_ctx *c)
{
    return !c->bf16 && c->opt.d == 64 && c->opt.kernels != 1 && c->n[0] < (1ll << 30) && c->n[1] < (1ll << 30);
}
bool dual_form(const alx_ctx *c) { return tensor_path(c) && c->opt.kernels == 0; }
float dual_cond_limit(const alx_ctx *c) { return c->opt.dual_cond_limit > 0.f ? c->opt.dual_cond_limit : ALX_DEFAULT_DUAL_COND_LIMIT; }
CgOptions cg_options(const alx_ctx *c, int solved_side)
{
    CgOptions o;
    // the start vector of a row is its stored embedding once that table holds something (set by the caller or solved)
    o.warm_start = c->opt.cg_start == ALX_CG_START_STORED && c->have_table[solved_side];
    o.enabled = c->opt.solver == ALX_SOLVER_AUTO;
    o.max_iter = c->opt.cg_max_iter > 0 ? c->opt.cg_max_iter : ALX_DEFAULT_CG_MAX_ITER;
    o.tol = c->opt.cg_tol > 0.f ? c->opt.cg_tol : (c->bf16 ? ALX_DEFAULT_CG_TOL_BF16 : ALX_DEFAULT_CG_TOL);
    o.counters = c->cg_counters;
    o.fallback_list = c->cg_fallback_list;
    o.policy = c->cg_policy ? c->cg_policy + solved_side : nullptr;
    o.switch_products = c->opt.cg_switch_products > 0.f ? c->opt.cg_switch_products : ALX_DEFAULT_CG_SWITCH_PRODUCTS;
    return o;
}

alx_status gramian_of(alx_ctx *c, int table_side)
{
    if (tensor_path(c)) {
        ALX_CUDA(c, launch_gramian_umma(c->table[table_side], c->n[table_side], c->gram_partials, c->stream, &c->launches));
        ALX_CUDA(c, launch_gramian_reduce(c->gram_partials, gramian_umma_partials(), c->opt.d, c->G64[table_side], c->Bmat,
                                          c->opt.alpha0, c->opt.lambda, c->stream, &c->launches));
        if (dual_form(c)) ALX_CUDA(c, launch_dual_prepare(c->Bmat, c->dual_ws, dual_cond_limit(c), c->opt.solver == ALX_SOLVER_AUTO, c->stream,
                                                         &c->launches));
        c->have_gram[table_side] = true;
        return ALX_OK;
    }
    ALX_CUDA(c, launch_gramian(c->table[table_side], c->bf16, c->n[table_side], c->opt.d, c->gram_partials,
                               c->G64[table_side], c->Bmat, c->opt.alpha0, c->opt.lambda, c->stream, &c->launches));
    if (fold_path(c) && c->dual_ws)
        ALX_CUDA(c, launch_dual64_prepare(c->Bmat, c->dual_ws, dual_cond_limit(c), c->stream, &c->launches));
    c->have_gram[table_side] = true;
    return ALX_OK;
}

alx_status half_epoch_impl(alx_ctx *c, int side, const int32_t *cap_slot, float *cap_out)
{
    if (c->nnz < 0) return fail(c, ALX_ERR_BAD_STATE, "alx_half_epoch before alx_set_csr");
    const int fixed = 1 - side;
    if (!c->have_table[fixed]) return fail(c, ALX_ERR_BAD_STATE, "the fixed table has not been set");
    NvtxRange range(side == ALX_ROWS ? "alx half-epoch: rows" : "alx half-epoch: columns");
    ALX_CUDA(c, cudaEventRecord(c->ev[0], c->stream));
    alx_status st;
    {
        NvtxRange r("alx Gramian + base matrix");
        st = gramian_of(c, fixed);
    }
    if (st != ALX_OK) return st;
    ALX_CUDA(c, cudaEventRecord(c->ev[1], c->stream));
    NvtxRange rows_range("alx rows: gather, sums, solve, store");
    RowOut out{c->table[side], cap_slot, cap_out};
    if (fold_path(c)) {
        ALX_CUDA(c, cudaMemsetAsync(c->cg_counters, 0, 5 * sizeof(unsigned long long), c->stream));
        ALX_CUDA(c, launch_split_table(static_cast<const float *>(c->table[fixed]), c->n[fixed], c->fold_table, c->stream,
                                       &c->launches));
        // rows of 1 .. 16 observations (class 1 of the entry lists as given = classes 1 and 2 of the doubled ones): dual form
        const int64_t n_dual = c->dual_ws ? c->class_offs[side][2] - c->class_offs[side][1] : 0;
        if (n_dual > 0)
            ALX_CUDA(c, launch_rows_dual64(side_view(c, side), c->class_offs[side][1], n_dual, c->table[fixed], c->dual_ws, out,
                                           c->stream, &c->launches));
        ALX_CUDA(c, launch_rows_fold(side_view(c, 2 + side), c->class_offs[2 + side], c->n_chunks[2 + side],
                                     c->n_split_rows[2 + side], c->fold_table, 2 * c->n[fixed], c->Bmat, c->split_partials,
                                     out, c->status, c->stream, &c->launches, c->ev[3], c->ev[4], cg_options(c, side),
                                     n_dual > 0 ? dual64_flag_ptr(c->dual_ws) : nullptr));
        c->stats.kernel_path[side] = 1;
        c->main_timed = true;
        c->dual_candidates = n_dual;
        c->dual_flag_latched = 0;
        if (n_dual > 0)
            ALX_CUDA(c, cudaMemcpyAsync(&c->dual_flag_latched, dual64_flag_ptr(c->dual_ws), sizeof(int), cudaMemcpyDeviceToHost,
                                        c->stream));
    } else if (tensor_path(c)) {
        ALX_CUDA(c, cudaMemsetAsync(c->cg_counters, 0, 5 * sizeof(unsigned long long), c->stream));
        ALX_CUDA(c, launch_rows_umma(side_view(c, side), c->class_offs[side], c->n_chunks[side], c->n_split_rows[side],
                                     c->table[fixed], c->Bmat, c->split_partials, out, c->status, c->stream,
                                     &c->launches, c->ev[3], c->ev[4], dual_form(c) ? c->dual_ws : nullptr, c->n[fixed],
                                     cg_options(c, side), c->order16[side], c->n4[side], c->n8[side]));
        c->stats.kernel_path[side] = 1;
        c->main_timed = true;
        c->dual_candidates = dual_form(c) ? c->class_offs[side][3] - c->class_offs[side][1] : 0;
        c->dual_candidates32 = dual_form(c) ? c->class_offs[side][3] - c->class_offs[side][2] : 0;
        c->dual_flag_latched = 0;
        c->policy_latched = CgPolicy{};
        if (c->dual_candidates > 0) {
            ALX_CUDA(c, cudaMemcpyAsync(&c->dual_flag_latched, dual_flag_ptr(c->dual_ws), sizeof(int), cudaMemcpyDeviceToHost,
                                        c->stream));
            if (c->cg_policy && c->opt.solver == ALX_SOLVER_AUTO)
                ALX_CUDA(c, cudaMemcpyAsync(&c->policy_latched, c->cg_policy + side, sizeof(CgPolicy), cudaMemcpyDeviceToHost,
                                            c->stream));
        }
    } else {
        ALX_CUDA(c, launch_rows_simple(side_view(c, side), c->class_offs[side], c->n_chunks[side],
                                       c->n_split_rows[side], c->table[fixed], c->bf16, c->opt.d, c->Bmat,
                                       c->split_partials, out, c->status, c->stream, &c->launches));
        c->stats.kernel_path[side] = 0;
        c->dual_candidates = 0;
    }
    ALX_CUDA(c, cudaEventRecord(c->ev[2], c->stream));
    c->have_table[side] = true;
    c->have_gram[side] = false;
    return ALX_OK;
}

}  // namespace

extern "C" {

const char *alx_version(void) { return "alx-b200 0.1 (sm_100a)"; }

const char *alx_last_error(const alx_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

alx_status alx_create(int64_t n_rows, int64_t n_cols, int32_t d, float lambda, float alpha0, alx_ctx **out)
{
    alx_options o;
    memset(&o, 0, sizeof o);
    o.n_rows = n_rows; o.n_cols = n_cols; o.d = d; o.lambda = lambda; o.alpha0 = alpha0;
    o.storage = ALX_F32; o.device = -1;
    return alx_create_ex(&o, out);   /* solver, cg_max_iter, cg_tol = 0: the defaults */
}

namespace {
alx_status create_impl(const alx_options *opt, const alx_ctx *parent, alx_ctx **out);
}

alx_status alx_create_ex(const alx_options *opt, alx_ctx **out) { return create_impl(opt, nullptr, out); }

namespace {
// parent: the new context borrows the parent's column table (alx_fold_in) instead of holding one of its own
alx_status create_impl(const alx_options *opt, const alx_ctx *parent, alx_ctx **out)
{
    if (!opt || !out) return ALX_ERR_INVALID_ARG;
    if (opt->n_rows < 1 || opt->n_cols < 1 || opt->n_rows >= (1ll << 31) || opt->n_cols >= (1ll << 31))
        return ALX_ERR_INVALID_ARG;
    if (opt->d != 16 && opt->d != 32 && opt->d != 64 && opt->d != 128) return ALX_ERR_UNSUPPORTED;
    if (!(opt->lambda > 0.f)) return ALX_ERR_UNSUPPORTED;   // lambda = 0: minimiser not unique
    if (!(opt->alpha0 >= 0.f)) return ALX_ERR_INVALID_ARG;
    if (opt->storage != ALX_F32 && opt->storage != ALX_BF16) return ALX_ERR_INVALID_ARG;
    if ((opt->alloc == nullptr) != (opt->free == nullptr)) return ALX_ERR_INVALID_ARG;
    if (opt->split != 0 && opt->split < 16) return ALX_ERR_INVALID_ARG;
    if (opt->solver != ALX_SOLVER_AUTO && opt->solver != ALX_SOLVER_CHOLESKY) return ALX_ERR_INVALID_ARG;
    if (opt->cg_start != ALX_CG_START_STORED && opt->cg_start != ALX_CG_START_ZERO) return ALX_ERR_INVALID_ARG;
    if (!(opt->cg_switch_products >= 0.f) || !(opt->dual_cond_limit >= 0.f)) return ALX_ERR_INVALID_ARG;
    if (opt->cg_max_iter < 0 || opt->cg_max_iter > 1024 || !(opt->cg_tol >= 0.f) || opt->cg_tol > 1e-2f) return ALX_ERR_INVALID_ARG;
    int dev = opt->device;
    if (dev < 0 && cudaGetDevice(&dev) != cudaSuccess) return ALX_ERR_CUDA;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || dev >= count) return ALX_ERR_CUDA;

    alx_ctx *c = new (std::nothrow) alx_ctx();
    if (!c) return ALX_ERR_OOM;
    c->opt = *opt;
    c->device = dev;
    c->stream = static_cast<cudaStream_t>(opt->stream);
    c->bf16 = opt->storage == ALX_BF16;
    c->elem = c->bf16 ? 2 : 4;
    c->n[ALX_ROWS] = c->n[2 + ALX_ROWS] = opt->n_rows;
    c->n[ALX_COLS] = c->n[2 + ALX_COLS] = opt->n_cols;
    c->split = opt->split ? opt->split : ALX_DEFAULT_SPLIT;
    DeviceGuard guard(dev);
    auto body = [&]() -> alx_status {
        const int d = opt->d;
        for (int s = 0; s < 2; ++s) {
            void *t = parent && s == ALX_COLS ? parent->table[s] : dev_alloc(c, (size_t)c->n[s] * d * c->elem);
            if (!t) return fail(c, ALX_ERR_OOM, "device allocation of a %lld x %d table failed", (long long)c->n[s], d);
            c->table[s] = t;
            ALX_ALLOC(c, c->G64[s], d * d);
            ALX_ALLOC(c, c->class_offs_dev[s], ALX_N_CLASSES + 1);
            if (fold_path(c)) ALX_ALLOC(c, c->class_offs_dev[2 + s], ALX_N_CLASSES + 1);
        }
        ALX_ALLOC(c, c->Bmat, d * d);
        if (dual_form(c) || (fold_path(c) && c->opt.kernels == 0)) {
            c->dual_ws = dev_alloc(c, dual_form(c) ? dual_workspace_bytes() : dual64_workspace_bytes());
            if (!c->dual_ws) return fail(c, ALX_ERR_OOM, "device allocation of the dual-form workspace failed");
        }
        const int64_t nmax = c->n[0] > c->n[1] ? c->n[0] : c->n[1];
        if (fold_path(c)) {
            c->fold_table = dev_alloc(c, (size_t)2 * nmax * 128 * 2);
            if (!c->fold_table) return fail(c, ALX_ERR_OOM, "device allocation of the table of bfloat16 parts failed");
        }
        int64_t n_part = gramian_partials(nmax);
        if (gramian_umma_partials() > n_part) n_part = gramian_umma_partials();
        ALX_ALLOC(c, c->gram_partials, n_part * d * d);
        ALX_ALLOC(c, c->loss_result, 4);
        ALX_ALLOC(c, c->status, 1);
        ALX_CUDA(c, cudaMemsetAsync(c->status, 0, sizeof(DevStatus), c->stream));
        ALX_ALLOC(c, c->cg_counters, 5);
        if (tensor_path(c) && c->opt.solver == ALX_SOLVER_AUTO) {
            ALX_ALLOC(c, c->cg_fallback_list, nmax);
            ALX_ALLOC(c, c->cg_policy, 2);
            ALX_CUDA(c, cudaMemsetAsync(c->cg_policy, 0, 2 * sizeof(CgPolicy), c->stream));
        }
        ALX_CUDA(c, cudaMemsetAsync(c->cg_counters, 0, 5 * sizeof(unsigned long long), c->stream));
        for (auto &e : c->ev) ALX_CUDA(c, cudaEventCreate(&e));
        ALX_CUDA(c, cudaStreamSynchronize(c->stream));
        return ALX_OK;
    };
    alx_status st = body();
    if (st != ALX_OK) {
        alx_destroy(c);
        return st;
    }
    *out = c;
    return ALX_OK;
}
}  // namespace

alx_status alx_destroy(alx_ctx *c)
{
    if (!c) return ALX_OK;
    DeviceGuard guard(c->device);
    cudaStreamSynchronize(c->stream);
    for (auto &e : c->ev) if (e) cudaEventDestroy(e);
    if (c->copy_stream) { cudaStreamSynchronize(c->copy_stream); cudaStreamDestroy(c->copy_stream); }
    if (c->copy_ev) cudaEventDestroy(c->copy_ev);
    std::vector<std::pair<void *, size_t>> owned = c->owned;
    for (auto &p : owned) dev_free(c, p.first);
    delete c;
    return ALX_OK;
}

alx_status alx_set_csr(alx_ctx *c, const int64_t *rowptr, const int32_t *colidx, const float *values, int64_t nnz,
                       int on_device)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!rowptr || nnz < 0 || (nnz > 0 && !colidx)) return fail(c, ALX_ERR_INVALID_ARG, "null array or negative nnz");
    DeviceGuard guard(c->device);
    NvtxRange range("alx_set_csr: validate, transpose, degree classes");
    release_matrix(c);
    const int64_t n_rows = c->n[ALX_ROWS], n_cols = c->n[ALX_COLS];
    const cudaMemcpyKind kind = on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    const size_t nz = (size_t)(nnz > 0 ? nnz : 1);
    c->has_values = values != nullptr;
    ALX_ALLOC(c, c->ptr[0], n_rows + 1);
    ALX_ALLOC(c, c->idx[0], nz);
    ALX_CUDA(c, cudaMemcpyAsync(c->ptr[0], rowptr, sizeof(int64_t) * (n_rows + 1), kind, c->stream));
    if (nnz > 0) ALX_CUDA(c, cudaMemcpyAsync(c->idx[0], colidx, sizeof(int32_t) * nnz, kind, c->stream));
    if (values) {
        ALX_ALLOC(c, c->val[0], nz);
        if (nnz > 0) ALX_CUDA(c, cudaMemcpyAsync(c->val[0], values, sizeof(float) * nnz, kind, c->stream));
    }
    if (c->upload_after_csr[0] || c->upload_after_csr[1]) {
        // alx_load_host: the tables follow S over the bus on the second stream, while the kernels below run
        ALX_CUDA(c, cudaEventRecord(c->copy_ev, c->stream));
        ALX_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->copy_ev, 0));
        for (int sd = 0; sd < 2; ++sd)
            if (c->upload_after_csr[sd])
                ALX_CUDA(c, cudaMemcpyAsync(c->table[sd], c->upload_after_csr[sd], (size_t)c->n[sd] * c->opt.d * c->elem,
                                            cudaMemcpyHostToDevice, c->copy_stream));
    }
    // validate before anything indexes with these arrays
    ALX_CUDA(c, launch_validate(c->ptr[0], c->idx[0], n_rows, n_cols, nnz, c->status, c->stream, &c->launches));
    alx_status st = check_device_status(c);
    if (st != ALX_OK) { release_matrix(c); return st; }
    c->nnz = nnz;

    // scratch shared by the scans and the bucket passes
    const int64_t nmax = n_rows > n_cols ? n_rows : n_cols;
    const int64_t nb = bucket_blocks(nmax);
    const int64_t scan_elems = scan_scratch_elems(nb * kNClasses > nmax ? nb * kNClasses : nmax) + 16;
    Scratch tmp(c);
    int64_t *scan_scratch = nullptr, *blk_counts = nullptr, *blk_offs = nullptr, *class_entries = nullptr;
    int32_t *counts = nullptr;
    ALX_TMP(c, tmp, scan_scratch, scan_elems);
    ALX_TMP(c, tmp, blk_counts, nb * kNClasses);
    ALX_TMP(c, tmp, blk_offs, nb * kNClasses + 1);
    ALX_TMP(c, tmp, counts, n_cols);
    ALX_TMP(c, tmp, class_entries, 2 * kNClasses);

    // transpose: count, prefix sum, degree classes of the columns, fill, sort each column, labels
    ALX_ALLOC(c, c->ptr[1], n_cols + 1);
    ALX_ALLOC(c, c->idx[1], nz);
    ALX_CUDA(c, cudaMemsetAsync(counts, 0, sizeof(int32_t) * n_cols, c->stream));
    ALX_CUDA(c, launch_count_cols(c->idx[0], nnz, counts, c->stream, &c->launches));
    ALX_CUDA(c, scan_exclusive(counts, false, c->ptr[1], n_cols, scan_scratch, scan_elems, c->stream, &c->launches));
    for (int s = 0; s < 2; ++s) ALX_ALLOC(c, c->order[s], c->n[s]);
    st = build_buckets(c, ALX_COLS, blk_counts, blk_offs, scan_scratch, scan_elems);
    if (st != ALX_OK) return st;
    ALX_CUDA(c, cudaMemsetAsync(counts, 0, sizeof(int32_t) * n_cols, c->stream));
    ALX_CUDA(c, launch_fill_transpose(c->ptr[0], c->idx[0], n_rows, nnz, c->ptr[1], counts, c->idx[1], c->stream,
                                      &c->launches));
    ALX_CUDA(c, launch_sort_segments(c->ptr[1], c->idx[1], c->order[1], c->class_offs[1], c->stream, &c->launches));
    if (values) {
        ALX_ALLOC(c, c->val[1], nz);
        ALX_CUDA(c, launch_values_transpose(c->ptr[0], c->idx[0], c->val[0], c->ptr[1], c->idx[1], n_cols, nnz,
                                            c->val[1], c->stream, &c->launches));
    }
    st = build_buckets(c, ALX_ROWS, blk_counts, blk_offs, scan_scratch, scan_elems);
    if (st != ALX_OK) return st;
    if (fold_path(c)) {
        // the doubled entry lists of both orientations, with degree classes and chunks of their own
        for (int s = 0; s < 2; ++s) {
            ALX_ALLOC(c, c->ptr[2 + s], c->n[s] + 1);
            ALX_ALLOC(c, c->idx[2 + s], 2 * nz);
            if (values) ALX_ALLOC(c, c->val[2 + s], 2 * nz);
            ALX_ALLOC(c, c->order[2 + s], c->n[s]);
            ALX_CUDA(c, launch_double_entries(c->ptr[s], c->idx[s], c->val[s], c->n[s], c->n[1 - s], c->ptr[2 + s],
                                              c->idx[2 + s], c->val[2 + s], c->stream, &c->launches));
            st = build_buckets(c, 2 + s, blk_counts, blk_offs, scan_scratch, scan_elems);
            if (st != ALX_OK) return st;
        }
    }
    if (dual_form(c)) {
        // the rows of 1 .. 16 entries, ordered by length class (at most 4, 5 .. 8, 9 .. 16): kernel instances with four and
        // eight observations per row take the first two parts at a quarter and half of the cost per row
        for (int s = 0; s < 2; ++s) {
            const int64_t n16 = c->class_offs[s][2] - c->class_offs[s][1];
            if (n16 <= 0) continue;
            const int64_t nb = (n16 + 1023) / 1024;
            int64_t *pc = nullptr, *po = nullptr;
            ALX_TMP(c, tmp, pc, nb + 2);
            ALX_TMP(c, tmp, po, nb + 2);
            ALX_ALLOC(c, c->order16[s], n16);
            ALX_CUDA(c, launch_partition_by_length(c->ptr[s], c->order[s] + c->class_offs[s][1], n16, 4, c->order16[s], pc, po,
                                                   class_entries + s, scan_scratch, scan_elems, c->stream, &c->launches));
            ALX_CUDA(c, cudaMemcpyAsync(&c->n4[s], class_entries + s, sizeof(int64_t), cudaMemcpyDeviceToHost, c->stream));
            ALX_CUDA(c, cudaStreamSynchronize(c->stream));
            const int64_t rest = n16 - c->n4[s];
            c->n8[s] = c->n4[s];
            if (rest > 0) {
                int32_t *part = nullptr;
                ALX_TMP(c, tmp, part, rest);
                ALX_CUDA(c, launch_partition_by_length(c->ptr[s], c->order16[s] + c->n4[s], rest, 8, part, pc, po, class_entries + s,
                                                       scan_scratch, scan_elems, c->stream, &c->launches));
                int64_t n58 = 0;
                ALX_CUDA(c, cudaMemcpyAsync(&n58, class_entries + s, sizeof(int64_t), cudaMemcpyDeviceToHost, c->stream));
                ALX_CUDA(c, cudaMemcpyAsync(c->order16[s] + c->n4[s], part, sizeof(int32_t) * rest, cudaMemcpyDeviceToDevice, c->stream));
                ALX_CUDA(c, cudaStreamSynchronize(c->stream));
                c->n8[s] += n58;
                tmp.release(part);
            }
            tmp.release(pc);
            tmp.release(po);
        }
    }
    for (int s = 0; s < 2; ++s)
        ALX_CUDA(c, launch_class_entries(c->ptr[s], c->order[s], c->class_offs_dev[s], c->n[s], class_entries + s * kNClasses,
                                         c->stream, &c->launches));
    ALX_CUDA(c, cudaMemcpyAsync(c->stats.entries_in_class, class_entries, 2 * kNClasses * sizeof(int64_t),
                                cudaMemcpyDeviceToHost, c->stream));
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    tmp.release(counts);
    tmp.release(blk_offs);
    tmp.release(blk_counts);
    tmp.release(scan_scratch);
    tmp.release(class_entries);

    const int d = c->opt.d;
    const int kb = fold_path(c) ? 2 : 0;      // the lists the row kernels walk
    const int dk = fold_path(c) ? 128 : d;    // the width of the sums they form
    int64_t sums[2] = {c->n_chunks[kb], c->n_chunks[kb + 1]};
    for (int s = 0; s < 2; ++s) c->stats.long_rows[s] = c->stats.long_entries[s] = 0;
    if (tensor_path(c) || fold_path(c)) {    // one more sum per long whole row
        int64_t *total = nullptr;
        ALX_TMP(c, tmp, total, 2);
        for (int s = 0; s < 2; ++s) {
            const int64_t *offs = c->class_offs[kb + s];
            const int64_t first = offs[long_class_begin(offs)];
            const int64_t n_long = offs[kNClasses - 1] - first;
            sums[s] += n_long;
            c->stats.long_rows[s] = n_long;
            ALX_CUDA(c, launch_sum_row_lengths(c->ptr[kb + s], c->order[kb + s] + first, n_long, total + s, c->stream, &c->launches));
        }
        ALX_CUDA(c, cudaMemcpyAsync(c->stats.long_entries, total, 2 * sizeof(int64_t), cudaMemcpyDeviceToHost, c->stream));
        ALX_CUDA(c, cudaStreamSynchronize(c->stream));
        if (fold_path(c)) for (int s = 0; s < 2; ++s) c->stats.long_entries[s] /= 2;      // (every entry is listed twice there)
        tmp.release(total);
    }
    const int64_t max_chunks = sums[0] > sums[1] ? sums[0] : sums[1];
    if (max_chunks > 0) ALX_ALLOC(c, c->split_partials, max_chunks * (int64_t)(dk * dk + dk));
    ALX_ALLOC(c, c->loss_partials_buf, loss_partials(nnz));
    c->stats.nnz = nnz;
    return ALX_OK;
}

alx_status alx_set_embeddings(alx_ctx *c, alx_side side, const void *src, alx_dtype src_dtype, int on_device)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!src || (side != ALX_ROWS && side != ALX_COLS) || (src_dtype != ALX_F32 && src_dtype != ALX_BF16))
        return fail(c, ALX_ERR_INVALID_ARG, "bad argument to alx_set_embeddings");
    DeviceGuard guard(c->device);
    const int64_t count = c->n[side] * c->opt.d;
    const size_t src_bytes = (size_t)count * (src_dtype == ALX_BF16 ? 2 : 4);
    const void *dev_src = src;
    Scratch tmp(c);
    void *staging = nullptr;
    if (!on_device) {
        if ((src_dtype == ALX_BF16) == (c->bf16 != 0)) {
            ALX_CUDA(c, cudaMemcpyAsync(c->table[side], src, src_bytes, cudaMemcpyHostToDevice, c->stream));
            ALX_CUDA(c, cudaStreamSynchronize(c->stream));
            c->have_table[side] = true;
            c->have_gram[side] = false;
            return ALX_OK;
        }
        staging = tmp.keep(dev_alloc(c, src_bytes));
        if (!staging) return fail(c, ALX_ERR_OOM, "staging allocation failed");
        ALX_CUDA(c, cudaMemcpyAsync(staging, src, src_bytes, cudaMemcpyHostToDevice, c->stream));
        dev_src = staging;
    }
    ALX_CUDA(c, launch_convert(dev_src, src_dtype == ALX_BF16, c->table[side], c->bf16, count, c->stream, &c->launches));
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    c->have_table[side] = true;
    c->have_gram[side] = false;
    return ALX_OK;
}

alx_status alx_set_embedding_rows(alx_ctx *c, alx_side side, int64_t row_begin, int64_t row_count, const void *src,
                                  alx_dtype src_dtype, int on_device)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!src || (side != ALX_ROWS && side != ALX_COLS) || (src_dtype != ALX_F32 && src_dtype != ALX_BF16) ||
        row_begin < 0 || row_count < 0 || row_begin + row_count > c->n[side])
        return fail(c, ALX_ERR_INVALID_ARG, "bad argument to alx_set_embedding_rows");
    if (row_count == 0) return ALX_OK;
    DeviceGuard guard(c->device);
    const int64_t count = row_count * c->opt.d;
    const size_t src_bytes = (size_t)count * (src_dtype == ALX_BF16 ? 2 : 4);
    char *dst = static_cast<char *>(c->table[side]) + (size_t)row_begin * c->opt.d * c->elem;
    const void *dev_src = src;
    Scratch tmp(c);
    void *staging = nullptr;
    const bool same = (src_dtype == ALX_BF16) == (c->bf16 != 0);
    if (same) {
        ALX_CUDA(c, cudaMemcpyAsync(dst, src, src_bytes, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->stream));
    } else {
        if (!on_device) {
            staging = tmp.keep(dev_alloc(c, src_bytes));
            if (!staging) return fail(c, ALX_ERR_OOM, "staging allocation failed");
            ALX_CUDA(c, cudaMemcpyAsync(staging, src, src_bytes, cudaMemcpyHostToDevice, c->stream));
            dev_src = staging;
        }
        ALX_CUDA(c, launch_convert(dev_src, src_dtype == ALX_BF16, dst, c->bf16, count, c->stream, &c->launches));
    }
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    c->have_table[side] = true;
    c->have_gram[side] = false;
    return ALX_OK;
}

alx_status alx_get_embeddings(alx_ctx *c, alx_side side, void *dst, alx_dtype dst_dtype, int64_t row_begin,
                              int64_t row_count, int on_device)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!dst || (side != ALX_ROWS && side != ALX_COLS) || (dst_dtype != ALX_F32 && dst_dtype != ALX_BF16) ||
        row_begin < 0 || row_count < 0 || row_begin + row_count > c->n[side])
        return fail(c, ALX_ERR_INVALID_ARG, "bad argument to alx_get_embeddings");
    if (!c->have_table[side]) return fail(c, ALX_ERR_BAD_STATE, "table has not been set or solved yet");
    DeviceGuard guard(c->device);
    const int d = c->opt.d;
    const int64_t count = row_count * d;
    const char *src = static_cast<const char *>(c->table[side]) + (size_t)row_begin * d * c->elem;
    const size_t dst_bytes = (size_t)count * (dst_dtype == ALX_BF16 ? 2 : 4);
    const bool same = (dst_dtype == ALX_BF16) == (c->bf16 != 0);
    if (on_device) {
        ALX_CUDA(c, launch_convert(src, c->bf16, dst, dst_dtype == ALX_BF16, count, c->stream, &c->launches));
    } else if (same) {
        ALX_CUDA(c, cudaMemcpyAsync(dst, src, dst_bytes, cudaMemcpyDeviceToHost, c->stream));
    } else {
        Scratch tmp(c);
        void *staging = tmp.keep(dev_alloc(c, dst_bytes));
        if (!staging) return fail(c, ALX_ERR_OOM, "staging allocation failed");
        ALX_CUDA(c, launch_convert(src, c->bf16, staging, dst_dtype == ALX_BF16, count, c->stream, &c->launches));
        ALX_CUDA(c, cudaMemcpyAsync(dst, staging, dst_bytes, cudaMemcpyDeviceToHost, c->stream));
        ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    }
    return check_device_status(c);
}

alx_status alx_half_epoch(alx_ctx *c, alx_side side)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (side != ALX_ROWS && side != ALX_COLS) return fail(c, ALX_ERR_INVALID_ARG, "bad side");
    DeviceGuard guard(c->device);
    return half_epoch_impl(c, side, nullptr, nullptr);
}

alx_status alx_epoch(alx_ctx *c)
{
    alx_status st = alx_half_epoch(c, ALX_ROWS);
    if (st != ALX_OK) return st;
    return alx_half_epoch(c, ALX_COLS);
}

namespace {
alx_status ensure_copy_stream(alx_ctx *c)
{
    if (!c->copy_stream) ALX_CUDA(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
    if (!c->copy_ev) ALX_CUDA(c, cudaEventCreateWithFlags(&c->copy_ev, cudaEventDisableTiming));
    return ALX_OK;
}
}  // namespace

alx_status alx_load_host(alx_ctx *c, const int64_t *rowptr, const int32_t *colidx, const float *values, int64_t nnz,
                         const void *W, const void *H)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!W || !H) return fail(c, ALX_ERR_INVALID_ARG, "null table");
    DeviceGuard guard(c->device);
    alx_status st = ensure_copy_stream(c);
    if (st != ALX_OK) return st;
    c->upload_after_csr[ALX_ROWS] = W;
    c->upload_after_csr[ALX_COLS] = H;
    st = alx_set_csr(c, rowptr, colidx, values, nnz, 0);
    c->upload_after_csr[0] = c->upload_after_csr[1] = nullptr;
    const cudaError_t e = cudaStreamSynchronize(c->copy_stream);     // whatever alx_set_csr returned, the copies have ended
    if (st != ALX_OK) return st;
    ALX_CUDA(c, e);
    for (int sd = 0; sd < 2; ++sd) {
        c->have_table[sd] = true;
        c->have_gram[sd] = false;
    }
    return ALX_OK;
}

alx_status alx_epoch_to_host(alx_ctx *c, void *W_dst, void *H_dst)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!W_dst || !H_dst) return fail(c, ALX_ERR_INVALID_ARG, "null destination");
    DeviceGuard guard(c->device);
    alx_status st = ensure_copy_stream(c);
    if (st != ALX_OK) return st;
    st = half_epoch_impl(c, ALX_ROWS, nullptr, nullptr);
    if (st != ALX_OK) return st;
    // the new W goes to the host on the second stream while the column pass (which only reads it) runs
    ALX_CUDA(c, cudaEventRecord(c->copy_ev, c->stream));
    ALX_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->copy_ev, 0));
    ALX_CUDA(c, cudaMemcpyAsync(W_dst, c->table[ALX_ROWS], (size_t)c->n[ALX_ROWS] * c->opt.d * c->elem, cudaMemcpyDeviceToHost,
                                c->copy_stream));
    st = half_epoch_impl(c, ALX_COLS, nullptr, nullptr);
    if (st == ALX_OK)
        ALX_CUDA(c, cudaMemcpyAsync(H_dst, c->table[ALX_COLS], (size_t)c->n[ALX_COLS] * c->opt.d * c->elem,
                                    cudaMemcpyDeviceToHost, c->stream));
    const cudaError_t e = cudaStreamSynchronize(c->copy_stream);
    if (st != ALX_OK) return st;
    ALX_CUDA(c, e);
    return check_device_status(c);
}

alx_status alx_half_epoch_capture(alx_ctx *c, alx_side side, const int64_t *row_ids, int64_t k, float *x_out)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if ((side != ALX_ROWS && side != ALX_COLS) || k < 0 || (k > 0 && (!row_ids || !x_out)))
        return fail(c, ALX_ERR_INVALID_ARG, "bad argument to alx_half_epoch_capture");
    for (int64_t j = 0; j < k; ++j)
        if (row_ids[j] < 0 || row_ids[j] >= c->n[side]) return fail(c, ALX_ERR_INVALID_ARG, "row id out of range");
    DeviceGuard guard(c->device);
    const int64_t n = c->n[side];
    const int d = c->opt.d;
    Scratch tmp(c);
    int32_t *slot = nullptr;
    float *cap = nullptr;
    ALX_TMP(c, tmp, slot, n);
    ALX_TMP(c, tmp, cap, (k > 0 ? k : 1) * d);
    std::vector<int32_t> h(n, -1);
    for (int64_t j = 0; j < k; ++j) h[row_ids[j]] = (int32_t)j;   // a repeated id keeps its last slot
    ALX_CUDA(c, cudaMemcpyAsync(slot, h.data(), sizeof(int32_t) * n, cudaMemcpyHostToDevice, c->stream));
    alx_status st = half_epoch_impl(c, side, slot, cap);
    if (st == ALX_OK) {
        std::vector<float> tmp((size_t)(k > 0 ? k : 1) * d);
        ALX_CUDA(c, cudaMemcpyAsync(tmp.data(), cap, sizeof(float) * k * d, cudaMemcpyDeviceToHost, c->stream));
        ALX_CUDA(c, cudaStreamSynchronize(c->stream));
        for (int64_t j = 0; j < k; ++j)
            memcpy(x_out + j * d, tmp.data() + (size_t)h[row_ids[j]] * d, sizeof(float) * d);
        st = check_device_status(c);
    } else {
        cudaStreamSynchronize(c->stream);
    }
    return st;
}

alx_status alx_gramian(alx_ctx *c, alx_side table, double *dst)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!dst || (table != ALX_ROWS && table != ALX_COLS)) return fail(c, ALX_ERR_INVALID_ARG, "bad argument");
    if (!c->have_table[table]) return fail(c, ALX_ERR_BAD_STATE, "table has not been set");
    DeviceGuard guard(c->device);
    alx_status st = gramian_of(c, table);
    if (st != ALX_OK) return st;
    return alx_get_gramian(c, table, dst);
}

alx_status alx_get_gramian(alx_ctx *c, alx_side side, double *dst)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!dst || (side != ALX_ROWS && side != ALX_COLS)) return fail(c, ALX_ERR_INVALID_ARG, "bad argument");
    if (!c->have_gram[side]) return fail(c, ALX_ERR_BAD_STATE, "no Gramian of that table is current");
    DeviceGuard guard(c->device);
    const int d = c->opt.d;
    ALX_CUDA(c, cudaMemcpyAsync(dst, c->G64[side], sizeof(double) * d * d, cudaMemcpyDeviceToHost, c->stream));
    return check_device_status(c);
}

alx_status alx_loss(alx_ctx *c, double *total, double *components)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (!total) return fail(c, ALX_ERR_INVALID_ARG, "null output");
    if (c->nnz < 0) return fail(c, ALX_ERR_BAD_STATE, "alx_loss before alx_set_csr");
    if (!c->have_table[0] || !c->have_table[1]) return fail(c, ALX_ERR_BAD_STATE, "both tables must be set");
    DeviceGuard guard(c->device);
    for (int s = 0; s < 2; ++s)
        if (!c->have_gram[s]) {
            alx_status st = gramian_of(c, s);
            if (st != ALX_OK) return st;
        }
    ALX_CUDA(c, launch_loss_obs(c->ptr[0], c->idx[0], c->val[0], c->n[0], c->nnz, c->table[0], c->table[1], c->bf16,
                                c->opt.d, c->loss_partials_buf, c->loss_result, c->stream, &c->launches));
    ALX_CUDA(c, launch_loss_finish(c->loss_partials_buf, c->nnz > 0 ? loss_partials(c->nnz) : 0, c->G64[0], c->G64[1],
                                   c->opt.d, (double)c->opt.alpha0, (double)c->opt.lambda, c->loss_result, c->stream,
                                   &c->launches));
    double h[3];
    ALX_CUDA(c, cudaMemcpyAsync(h, c->loss_result, sizeof h, cudaMemcpyDeviceToHost, c->stream));
    alx_status st = check_device_status(c);
    if (st != ALX_OK) return st;
    *total = h[0] + h[1] + h[2];
    if (components) { components[0] = h[0]; components[1] = h[1]; components[2] = h[2]; }
    return ALX_OK;
}

alx_status alx_get_transpose(alx_ctx *c, int64_t *colptr, int32_t *rowidx, float *values_t)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (c->nnz < 0) return fail(c, ALX_ERR_BAD_STATE, "alx_get_transpose before alx_set_csr");
    DeviceGuard guard(c->device);
    if (colptr) ALX_CUDA(c, cudaMemcpyAsync(colptr, c->ptr[1], sizeof(int64_t) * (c->n[1] + 1), cudaMemcpyDeviceToHost, c->stream));
    if (rowidx && c->nnz > 0) ALX_CUDA(c, cudaMemcpyAsync(rowidx, c->idx[1], sizeof(int32_t) * c->nnz, cudaMemcpyDeviceToHost, c->stream));
    if (values_t) {
        if (!c->has_values) return fail(c, ALX_ERR_BAD_STATE, "the matrix was set without labels");
        if (c->nnz > 0) ALX_CUDA(c, cudaMemcpyAsync(values_t, c->val[1], sizeof(float) * c->nnz, cudaMemcpyDeviceToHost, c->stream));
    }
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    return ALX_OK;
}

alx_status alx_get_buckets(alx_ctx *c, alx_side side, int32_t *order, int64_t *class_offsets, int64_t *chunk_desc,
                           int64_t *n_chunks)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (side != ALX_ROWS && side != ALX_COLS) return fail(c, ALX_ERR_INVALID_ARG, "bad side");
    if (c->nnz < 0) return fail(c, ALX_ERR_BAD_STATE, "alx_get_buckets before alx_set_csr");
    DeviceGuard guard(c->device);
    if (order) ALX_CUDA(c, cudaMemcpyAsync(order, c->order[side], sizeof(int32_t) * c->n[side], cudaMemcpyDeviceToHost, c->stream));
    if (class_offsets) memcpy(class_offsets, c->class_offs[side], sizeof(int64_t) * (ALX_N_CLASSES + 1));
    if (n_chunks) *n_chunks = c->n_chunks[side];
    if (chunk_desc && c->n_chunks[side] > 0)
        ALX_CUDA(c, cudaMemcpyAsync(chunk_desc, c->chunk_desc[side], sizeof(int64_t) * 4 * c->n_chunks[side], cudaMemcpyDeviceToHost, c->stream));
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    return ALX_OK;
}

alx_status alx_fold_in(alx_ctx *c, const int64_t *rowptr, const int32_t *colidx, const float *values, int64_t n_new,
                       int64_t nnz, int on_device, float *x_out)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (n_new < 0 || nnz < 0 || n_new >= (1ll << 31) || (n_new > 0 && (!rowptr || !x_out)) || (nnz > 0 && !colidx))
        return fail(c, ALX_ERR_INVALID_ARG, "bad argument to alx_fold_in");
    if (!c->have_table[ALX_COLS]) return fail(c, ALX_ERR_BAD_STATE, "the column table has not been set or solved yet");
    if (n_new == 0) return ALX_OK;
    DeviceGuard guard(c->device);
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    // a context of its own for the new rows: same options, the column table borrowed, the rows half-step of Eq. 4
    alx_options o = c->opt;
    o.n_rows = n_new;
    o.device = c->device;
    alx_ctx *k = nullptr;
    alx_status st = create_impl(&o, c, &k);
    if (st != ALX_OK) return fail(c, st, "alx_fold_in: the context for the new rows could not be created");
    k->have_table[ALX_COLS] = true;
    st = alx_set_csr(k, rowptr, colidx, values, nnz, on_device);
    if (st == ALX_OK) st = alx_half_epoch(k, ALX_ROWS);
    if (st == ALX_OK) st = alx_get_embeddings(k, ALX_ROWS, x_out, ALX_F32, 0, n_new, on_device);
    if (st == ALX_OK) st = alx_synchronize(k);
    c->launches += k->launches;
    if (st != ALX_OK) c->err = "alx_fold_in: " + k->err;
    alx_destroy(k);
    return st;
}

alx_status alx_topk(alx_ctx *c, alx_side items, const float *queries, int64_t m, int32_t k, const int64_t *exclude_ptr,
                    const int32_t *exclude_idx, int on_device, int32_t *ids_out, float *scores_out)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if ((items != ALX_ROWS && items != ALX_COLS) || m < 0 || k < 1 || k > ALX_MAX_TOPK || (m > 0 && (!queries || !ids_out)) ||
        (exclude_ptr && !exclude_idx && m > 0))
        return fail(c, ALX_ERR_INVALID_ARG, "bad argument to alx_topk");
    if (!c->have_table[items]) return fail(c, ALX_ERR_BAD_STATE, "the table has not been set or solved yet");
    if (m == 0) return ALX_OK;
    DeviceGuard guard(c->device);
    NvtxRange range("alx_topk");
    const int d = c->opt.d;
    const int64_t n_items = c->n[items];
    Scratch tmp(c);
    const float *Q = queries;
    const int64_t *ex_ptr = exclude_ptr;
    const int32_t *ex_idx = exclude_idx;
    int32_t *ids_dev = ids_out;
    float *scores_dev = scores_out;
    int64_t n_ex = 0;
    if (!on_device) {
        float *q_dev = nullptr;
        ALX_TMP(c, tmp, q_dev, m * d);
        ALX_CUDA(c, cudaMemcpyAsync(q_dev, queries, sizeof(float) * m * d, cudaMemcpyHostToDevice, c->stream));
        Q = q_dev;
        if (exclude_ptr) {
            n_ex = exclude_ptr[m];
            if (n_ex < 0) return fail(c, ALX_ERR_INVALID_ARG, "alx_topk: negative length of the exclusion lists");
            int64_t *p_dev = nullptr;
            int32_t *i_dev = nullptr;
            ALX_TMP(c, tmp, p_dev, m + 1);
            ALX_TMP(c, tmp, i_dev, n_ex > 0 ? n_ex : 1);
            ALX_CUDA(c, cudaMemcpyAsync(p_dev, exclude_ptr, sizeof(int64_t) * (m + 1), cudaMemcpyHostToDevice, c->stream));
            if (n_ex > 0) ALX_CUDA(c, cudaMemcpyAsync(i_dev, exclude_idx, sizeof(int32_t) * n_ex, cudaMemcpyHostToDevice, c->stream));
            ex_ptr = p_dev;
            ex_idx = i_dev;
        }
        ALX_TMP(c, tmp, ids_dev, m * k);
        if (scores_out) ALX_TMP(c, tmp, scores_dev, m * k);
    }
    const int slabs = topk_slabs(n_items, m);
    float *ls = nullptr;
    int32_t *li = nullptr, *lc = nullptr;
    ALX_TMP(c, tmp, ls, (int64_t)slabs * m * k);
    ALX_TMP(c, tmp, li, (int64_t)slabs * m * k);
    ALX_TMP(c, tmp, lc, (int64_t)slabs * m);
    ALX_CUDA(c, cudaMemsetAsync(lc, 0, sizeof(int32_t) * slabs * m, c->stream));
    const bool tensor_cores = c->opt.kernels != 1 && c->bf16 && d == 128;
    unsigned char *q_parts = nullptr;
    if (tensor_cores) ALX_TMP(c, tmp, q_parts, topk_query_scratch_bytes(m));
    ALX_CUDA(c, launch_topk(c->table[items], c->bf16 != 0, n_items, d, Q, m, k, ex_ptr, ex_idx, slabs, ls, li, lc, ids_dev,
                            scores_dev, tensor_cores, q_parts, c->status, c->stream, &c->launches));
    if (!on_device) {
        ALX_CUDA(c, cudaMemcpyAsync(ids_out, ids_dev, sizeof(int32_t) * m * k, cudaMemcpyDeviceToHost, c->stream));
        if (scores_out) ALX_CUDA(c, cudaMemcpyAsync(scores_out, scores_dev, sizeof(float) * m * k, cudaMemcpyDeviceToHost, c->stream));
    }
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    return check_device_status(c);
}

alx_status alx_recall_at_k(alx_ctx *c, const int32_t *ids, int64_t m, int32_t k_stride, int32_t k, const int64_t *truth_ptr,
                           const int32_t *truth_idx, int on_device, double *recall, int64_t *n_counted)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    if (m < 0 || k < 1 || k > k_stride || !recall || (m > 0 && (!ids || !truth_ptr)))
        return fail(c, ALX_ERR_INVALID_ARG, "bad argument to alx_recall_at_k");
    DeviceGuard guard(c->device);
    Scratch tmp(c);
    const int32_t *ids_dev = ids;
    const int64_t *tp = truth_ptr;
    const int32_t *ti = truth_idx;
    if (!on_device && m > 0) {
        const int64_t nt = truth_ptr[m];
        if (nt < 0 || (nt > 0 && !truth_idx)) return fail(c, ALX_ERR_INVALID_ARG, "alx_recall_at_k: bad ground-truth lists");
        int32_t *a = nullptr, *t = nullptr;
        int64_t *p = nullptr;
        ALX_TMP(c, tmp, a, m * k_stride);
        ALX_TMP(c, tmp, p, m + 1);
        ALX_TMP(c, tmp, t, nt > 0 ? nt : 1);
        ALX_CUDA(c, cudaMemcpyAsync(a, ids, sizeof(int32_t) * m * k_stride, cudaMemcpyHostToDevice, c->stream));
        ALX_CUDA(c, cudaMemcpyAsync(p, truth_ptr, sizeof(int64_t) * (m + 1), cudaMemcpyHostToDevice, c->stream));
        if (nt > 0) ALX_CUDA(c, cudaMemcpyAsync(t, truth_idx, sizeof(int32_t) * nt, cudaMemcpyHostToDevice, c->stream));
        ids_dev = a; tp = p; ti = t;
    }
    double *per_query = nullptr, *out2 = nullptr;
    ALX_TMP(c, tmp, per_query, m > 0 ? m : 1);
    ALX_TMP(c, tmp, out2, 2);
    ALX_CUDA(c, launch_recall(ids_dev, m, k_stride, k, tp, ti, per_query, out2, c->stream, &c->launches));
    double h[2] = {0.0, 0.0};
    ALX_CUDA(c, cudaMemcpyAsync(h, out2, sizeof h, cudaMemcpyDeviceToHost, c->stream));
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    *recall = h[1] > 0.0 ? h[0] / h[1] : 0.0;
    if (n_counted) *n_counted = (int64_t)h[1];
    return ALX_OK;
}

alx_status alx_get_stats(alx_ctx *c, alx_stats *out)
{
    if (!c || !out) return ALX_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->ev[0], c->ev[1]) == cudaSuccess) c->stats.ms_gramian = ms; else cudaGetLastError();
    if (cudaEventElapsedTime(&ms, c->ev[1], c->ev[2]) == cudaSuccess) c->stats.ms_rows = ms; else cudaGetLastError();
    if (cudaEventElapsedTime(&ms, c->ev[0], c->ev[2]) == cudaSuccess) c->stats.ms_half_epoch = ms; else cudaGetLastError();
    c->stats.ms_main_kernel = 0.0;
    if (c->main_timed) {
        if (cudaEventElapsedTime(&ms, c->ev[3], c->ev[4]) == cudaSuccess) c->stats.ms_main_kernel = ms; else cudaGetLastError();
    }
    c->stats.dual_rows = c->dual_candidates > 0 && c->dual_flag_latched
                             ? c->dual_candidates - (c->policy_latched.short_rows_by_cg ? c->dual_candidates32 : 0) : 0;
    {
        unsigned long long h[5] = {0, 0, 0, 0, 0};
        ALX_CUDA(c, cudaMemcpy(h, c->cg_counters, sizeof h, cudaMemcpyDeviceToHost));
        c->stats.cg_rows = (int64_t)h[0];
        c->stats.cg_products = (int64_t)h[1];
        c->stats.cg_fallbacks = (int64_t)h[2];
        c->stats.dual_polished_rows = (int64_t)h[3];
        c->stats.dual_polish_products = (int64_t)h[4];
        c->stats.cholesky_by_policy[0] = c->stats.cholesky_by_policy[1] = 0;
        if (c->cg_policy) {
            CgPolicy pol[2];
            ALX_CUDA(c, cudaMemcpy(pol, c->cg_policy, sizeof pol, cudaMemcpyDeviceToHost));
            for (int sd = 0; sd < 2; ++sd) c->stats.cholesky_by_policy[sd] = pol[sd].use_cholesky;
        }
    }
    c->stats.kernel_launches = c->launches;
    c->stats.workspace_bytes = c->bytes_held;
    *out = c->stats;
    return ALX_OK;
}

alx_status alx_fp32_peak_tflops(alx_ctx *c, double *tflops)
{
    if (!c || !tflops) return ALX_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    ALX_CUDA(c, cudaStreamSynchronize(c->stream));
    double v = 0.0;
    ALX_CUDA(c, measure_fp32_peak(&v, c->stream));
    *tflops = v;
    return ALX_OK;
}

alx_status alx_synchronize(alx_ctx *c)
{
    if (!c) return ALX_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    return check_device_status(c);
}

}  // extern "C"
