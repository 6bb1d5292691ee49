// Evaluation kernels (Sec. 4.6 and the protocol of Sec. 5): exact Top-K of <q, h_i> over every row of a table, and
// Recall@K of the retrieved ids against held-out ground truth.
//
// Top-K is exact: every item is scored and every score is looked at.  The order is total -- score descending, then
// id ascending -- so the result does not depend on how the items are divided among thread blocks: a block scans a
// contiguous slab of items in ascending id and keeps, per query, the best k it has seen (a sorted list in global
// memory: after the first few thousand items an insertion is rare); a second kernel merges the slabs' lists.
//
// Two scoring kernels feed the same selection:
//   k_topk_simple   any d, either storage type: fp32 FMAs, a thread per query with the query in registers
//   k_topk_umma     d = 128, bfloat16 tables: a 128-query x 128-item tile per tcgen05 accumulator, the fp32 query split
//                   into three bfloat16 parts (products exact, sums in fp32)
#include "alx_common.cuh"
#include "alx_ptx.cuh"
#include "alx_topk.cuh"

#include <cuda.h>
#include <cuda_bf16.h>

namespace alx {

namespace {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// grid (query tiles, slabs).  Scores: s = ((a0 + a1) + (a2 + a3)), a_j = sum over features f = j mod 4 in ascending f.
template <int DD, typename T>
__global__ void __launch_bounds__(kTopkQueries) k_topk_simple(const T *__restrict__ H, int64_t n_items,
                                                               const float *__restrict__ Q, int64_t m, int k,
                                                               const int64_t *__restrict__ ex_ptr,
                                                               const int32_t *__restrict__ ex_idx, int64_t slab,
                                                               float *__restrict__ list_s, int32_t *__restrict__ list_id,
                                                               int32_t *__restrict__ list_cnt)
{
    constexpr int kTile = 32;      // items staged per step
    __shared__ __align__(16) float tile[kTile][DD];
    const int tid = threadIdx.x;
    const int64_t q = (int64_t)blockIdx.x * kTopkQueries + tid;
    const bool live = q < m;
    float qv[DD];
#pragma unroll
    for (int f = 0; f < DD; ++f) qv[f] = live ? Q[q * DD + f] : 0.f;
    const int64_t lq = (int64_t)blockIdx.y * m + (live ? q : 0);
    TopList top{list_s + lq * k, list_id + lq * k, k, 0, 0.f, 1};
    const int64_t i0 = (int64_t)blockIdx.y * slab;
    const int64_t i1 = i0 + slab < n_items ? i0 + slab : n_items;
    for (int64_t base = i0; base < i1; base += kTile) {
        const int rows = (int)(i1 - base < kTile ? i1 - base : kTile);
        __syncthreads();
        for (int e = tid; e < rows * DD; e += kTopkQueries) tile[e / DD][e % DD] = to_f32<T>(H[base * DD + e]);
        __syncthreads();
        if (!live) continue;
        for (int j = 0; j < rows; ++j) {
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            const float4 *hp = reinterpret_cast<const float4 *>(&tile[j][0]);
#pragma unroll
            for (int f4 = 0; f4 < DD / 4; ++f4) {
                const float4 h = hp[f4];
                a0 = fmaf(qv[4 * f4], h.x, a0);
                a1 = fmaf(qv[4 * f4 + 1], h.y, a1);
                a2 = fmaf(qv[4 * f4 + 2], h.z, a2);
                a3 = fmaf(qv[4 * f4 + 3], h.w, a3);
            }
            const float v = (a0 + a1) + (a2 + a3);
            if (top.wants(v)) {
                const int32_t item = (int32_t)(base + j);
                if (!excluded(ex_ptr, ex_idx, q, item)) top.insert(v, item);
            }
        }
    }
    if (live) list_cnt[lq] = top.cnt;
}

// one thread per query: merge the slabs' lists (each sorted) into the first k by (score descending, id ascending)
__global__ void k_topk_merge(const float *__restrict__ list_s, const int32_t *__restrict__ list_id,
                             const int32_t *__restrict__ list_cnt, int64_t m, int k, int slabs,
                             int32_t *__restrict__ ids_out, float *__restrict__ scores_out)
{
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= m) return;
    constexpr int kMaxSlabs = 256;
    int head[kMaxSlabs];
    for (int s = 0; s < slabs; ++s) head[s] = 0;
    for (int r = 0; r < k; ++r) {
        int best = -1;
        float bs = 0.f;
        int32_t bi = 0;
        for (int s = 0; s < slabs; ++s) {
            const int64_t lq = (int64_t)s * m + q;
            if (head[s] >= list_cnt[lq]) continue;
            const float v = list_s[lq * k + head[s]];
            const int32_t i = list_id[lq * k + head[s]];
            if (best < 0 || v > bs || (v == bs && i < bi)) { best = s; bs = v; bi = i; }
        }
        if (best < 0) {      // fewer than k candidates: the rest of the row says so
            ids_out[q * k + r] = -1;
            if (scores_out) scores_out[q * k + r] = -INFINITY;
        } else {
            ++head[best];
            ids_out[q * k + r] = bi;
            if (scores_out) scores_out[q * k + r] = bs;
        }
    }
}

// Recall@K of one query: hits among its first k ids / number of ground-truth ids (ascending, unique); queries without
// ground truth get -1 and are left out of the mean
__global__ void k_recall_rows(const int32_t *__restrict__ ids, int64_t m, int k_stride, int k,
                              const int64_t *__restrict__ tptr, const int32_t *__restrict__ tidx,
                              double *__restrict__ per_query)
{
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= m) return;
    const int64_t t0 = tptr[q], t1 = tptr[q + 1];
    if (t1 <= t0) { per_query[q] = -1.0; return; }
    int hits = 0;
    for (int r = 0; r < k; ++r) {
        const int32_t id = ids[q * k_stride + r];
        if (id < 0) continue;
        int64_t lo = t0, hi = t1;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            const int32_t v = tidx[mid];
            if (v == id) { ++hits; break; }
            if (v < id) lo = mid + 1; else hi = mid;
        }
    }
    per_query[q] = (double)hits / (double)(t1 - t0);
}

// sum and count of the non-negative entries, in an order that depends on m only (one block)
__global__ void __launch_bounds__(1024) k_recall_mean(const double *__restrict__ per_query, int64_t m, double *__restrict__ out)
{
    __shared__ double ssum[1024];
    __shared__ long long scnt[1024];
    double s = 0.0;
    long long c = 0;
    for (int64_t q = threadIdx.x; q < m; q += 1024) {
        const double v = per_query[q];
        if (v >= 0.0) { s += v; ++c; }
    }
    ssum[threadIdx.x] = s;
    scnt[threadIdx.x] = c;
    __syncthreads();
    for (int h = 512; h > 0; h >>= 1) {
        if ((int)threadIdx.x < h) { ssum[threadIdx.x] += ssum[threadIdx.x + h]; scnt[threadIdx.x] += scnt[threadIdx.x + h]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { out[0] = ssum[0]; out[1] = (double)scnt[0]; }
}

template <int DD, typename T>
void launch_simple_t(const void *H, int64_t n_items, const float *Q, int64_t m, int k, const int64_t *ex_ptr,
                     const int32_t *ex_idx, int slabs, int64_t slab, float *ls, int32_t *li, int32_t *lc, cudaStream_t s)
{
    dim3 grid((unsigned)((m + kTopkQueries - 1) / kTopkQueries), (unsigned)slabs);
    k_topk_simple<DD, T><<<grid, kTopkQueries, 0, s>>>(static_cast<const T *>(H), n_items, Q, m, k, ex_ptr, ex_idx, slab, ls,
                                                       li, lc);
}

}  // namespace

int topk_slabs(int64_t n_items, int64_t m)
{
    // enough blocks for every SM, at most 256 slabs, at least 4096 items per slab
    const int64_t tiles = (m + kTopkQueries - 1) / kTopkQueries;
    int64_t slabs = (2 * 148 + tiles - 1) / tiles;
    const int64_t by_items = (n_items + 4095) / 4096;
    if (slabs > by_items) slabs = by_items;
    if (slabs > 256) slabs = 256;
    if (slabs < 1) slabs = 1;
    return (int)slabs;
}

cudaError_t launch_topk(const void *H, bool bf16, int64_t n_items, int d, const float *Q, int64_t m, int k,
                        const int64_t *ex_ptr, const int32_t *ex_idx, int slabs, float *list_s, int32_t *list_id,
                        int32_t *list_cnt, int32_t *ids_out, float *scores_out, bool tensor_cores, void *scratch_q,
                        DevStatus *st, cudaStream_t s, int64_t *launches)
{
    if (m <= 0) return cudaSuccess;
    int64_t slab = (n_items + slabs - 1) / slabs;
    slab = (slab + 127) / 128 * 128;
    if (tensor_cores && bf16 && d == 128) {
        cudaError_t e = launch_topk_umma(H, n_items, Q, m, k, ex_ptr, ex_idx, slabs, slab, list_s, list_id, list_cnt, scratch_q, st, s,
                                         launches);
        if (e != cudaSuccess) return e;
    } else {
#define ALX_TOPK_CASE(DD)                                                                                            \
    case DD:                                                                                                         \
        if (bf16) launch_simple_t<DD, __nv_bfloat16>(H, n_items, Q, m, k, ex_ptr, ex_idx, slabs, slab, list_s, list_id, list_cnt, s); \
        else launch_simple_t<DD, float>(H, n_items, Q, m, k, ex_ptr, ex_idx, slabs, slab, list_s, list_id, list_cnt, s);          \
        break;
        switch (d) {
            ALX_TOPK_CASE(16)
            ALX_TOPK_CASE(32)
            ALX_TOPK_CASE(64)
            ALX_TOPK_CASE(128)
            default: return cudaErrorInvalidValue;
        }
#undef ALX_TOPK_CASE
        ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    k_topk_merge<<<(unsigned)((m + 127) / 128), 128, 0, s>>>(list_s, list_id, list_cnt, m, k, slabs, ids_out, scores_out);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_recall(const int32_t *ids, int64_t m, int k_stride, int k, const int64_t *tptr, const int32_t *tidx,
                          double *per_query, double *out2, cudaStream_t s, int64_t *launches)
{
    if (m > 0) {
        k_recall_rows<<<(unsigned)((m + 255) / 256), 256, 0, s>>>(ids, m, k_stride, k, tptr, tidx, per_query);
        ++*launches;
    }
    k_recall_mean<<<1, 1024, 0, s>>>(per_query, m, out2);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace alx
