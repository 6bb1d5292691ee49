// Exact Top-K scoring on the tensor cores (Sec. 4.6) for d = 128 and bfloat16 tables.
//
// A block takes 128 queries and a slab of items.  The fp32 queries are split beforehand into three bfloat16 parts
// (q = q1 + q2 + q3 to 2^-24), so that every product is an exact product of bfloat16 values and the fp32 sums carry
// the query to fp32 accuracy.  Per tile of 128 items the MMA thread issues 3 parts x 8 K-steps of tcgen05.mma
// (128 x 128 x 16) into one of two tensor-memory accumulators; the four selection warps read the other one, a thread
// per query (= accumulator lane), and compare its 128 scores with the query's k-th best so far.
//
//   warp 5     TMA: the three query tiles once, then the item tiles through a three-stage ring
//              (2D tile loads, 128-byte swizzle, K-major: a row of the table is a row of the operand)
//   warp 4     MMA issue (one thread)
//   warps 0-3  selection (see alx_topk.cuh); an accumulator is handed back when all four warps have read it.  For
//              k <= 64 the lists are kept in shared memory while the slab is scanned (an insertion shifts a sorted list,
//              and a warp's 32 queries insert at different times: in global memory that latency was the whole run time)
//
// Every wait is bounded; a wait that gives up sets the block's abort flag, the roles leave their loops and the
// status word reports a timeout.
#include "alx_common.cuh"
#include "alx_ptx.cuh"
#include "alx_topk.cuh"

#include <cuda.h>
#include <cuda_bf16.h>

namespace alx {

using namespace ptx;

namespace {

constexpr int kD = 128;
constexpr int kTileItems = 128;
constexpr int kListMax = 64;       // lists of up to this many elements live in shared memory (beside a two-stage ring)
constexpr int kHalfTileBytes = kTileItems * 128;      // 128 rows x 64 bfloat16
constexpr int kTileBytes = 2 * kHalfTileBytes;
constexpr int kThreads = 6 * 32;

// SMEM_LISTS: the queries' lists in shared memory (k <= kListMax) and two stages of item tiles; otherwise the lists in
// global memory and three stages
template <bool SMEM_LISTS> struct __align__(1024) TopkSmem {
    static constexpr int kStages = SMEM_LISTS ? 2 : 3;
    unsigned char q[3][2][kHalfTileBytes];            // [part][feature half]: 128 queries x 64 features, swizzled
    unsigned char h[kStages][2][kHalfTileBytes];      // item tiles
    float ls[SMEM_LISTS ? kTopkQueries : 1][kListMax];         // [query][place]: a query's list is contiguous
    int32_t li[SMEM_LISTS ? kTopkQueries : 1][kListMax];
    uint64_t q_full, full[kStages], empty[kStages], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

static_assert(sizeof(TopkSmem<true>) + 1024 <= 232448 && sizeof(TopkSmem<false>) + 1024 <= 232448, "shared memory of the Top-K kernel");

// bf16 operands, fp32 accumulator, both operands K-major: D (+)= A * B^T
__host__ __device__ constexpr uint32_t idesc_bf16_k_major(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// fp32 queries -> three bfloat16 parts, [part][m_pad][128]; rows m .. m_pad - 1 are zero
__global__ void __launch_bounds__(256) k_split_queries(const float *__restrict__ Q, int64_t m, int64_t m_pad,
                                                       __nv_bfloat16 *__restrict__ P)
{
    const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= m_pad * kD) return;
    const float x = e < m * kD ? Q[e] : 0.f;
    const __nv_bfloat16 p1 = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(p1);
    const __nv_bfloat16 p2 = __float2bfloat16_rn(r1);
    const __nv_bfloat16 p3 = __float2bfloat16_rn(r1 - __bfloat162float(p2));
    P[e] = p1;
    P[m_pad * kD + e] = p2;
    P[2 * m_pad * kD + e] = p3;
}

template <bool SMEM_LISTS>
__global__ void __launch_bounds__(kThreads, 1)
k_topk_umma(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_q, int64_t n_items, int64_t m,
            int64_t m_pad, int k, const int64_t *__restrict__ ex_ptr, const int32_t *__restrict__ ex_idx, int64_t slab,
            float *__restrict__ list_s, int32_t *__restrict__ list_id, int32_t *__restrict__ list_cnt, DevStatus *st)
{
    extern __shared__ unsigned char smem_raw[];
    using SmemT = TopkSmem<SMEM_LISTS>;
    constexpr int kStages = SmemT::kStages;
    SmemT &sm = *reinterpret_cast<SmemT *>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t i0 = (int64_t)blockIdx.y * slab;
    const int64_t i1 = i0 + slab < n_items ? i0 + slab : n_items;
    const int n_tiles = i1 > i0 ? (int)((i1 - i0 + kTileItems - 1) / kTileItems) : 0;
    if (tid == 0) {
        mbar_init(&sm.q_full, 1);
        for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&sm.acc_full[a], 1); mbar_init(&sm.acc_empty[a], 4); }
        sm.abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 4) {
        tmem_alloc(&sm.tmem_base, 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (warp == 5) {
        if (lane == 0 && n_tiles > 0) {
            mbar_arrive_expect_tx(&sm.q_full, 3 * kTileBytes);
            for (int part = 0; part < 3; ++part)
                for (int half = 0; half < 2; ++half)
                    tma_tile_2d(smem_u32(&sm.q[part][half][0]), &tmap_q, 64 * half,
                                (int)(part * m_pad + (int64_t)blockIdx.x * kTopkQueries), &sm.q_full);
            for (int t = 0; t < n_tiles; ++t) {
                const int s = t % kStages;
                if (t >= kStages && !mbar_wait(&sm.empty[s], (uint32_t)((t / kStages - 1) & 1), &sm.abort_flag, 71)) break;
                mbar_arrive_expect_tx(&sm.full[s], kTileBytes);
                for (int half = 0; half < 2; ++half)
                    tma_tile_2d(smem_u32(&sm.h[s][half][0]), &tmap_h, 64 * half, (int)(i0 + (int64_t)t * kTileItems), &sm.full[s]);
            }
        }
    } else if (warp == 4) {
        if (lane == 0 && n_tiles > 0) {
            constexpr uint32_t kIdesc = idesc_bf16_k_major(128, kTileItems);
            bool ok = mbar_wait(&sm.q_full, 0, &sm.abort_flag, 72);
            for (int t = 0; ok && t < n_tiles; ++t) {
                const int s = t % kStages, a = t & 1;
                ok = mbar_wait(&sm.full[s], (uint32_t)((t / kStages) & 1), &sm.abort_flag, 73);
                if (ok && t >= 2) ok = mbar_wait(&sm.acc_empty[a], (uint32_t)((t / 2 - 1) & 1), &sm.abort_flag, 74);
                if (!ok) break;
                tc_fence_after();
                const uint32_t dcol = sm.tmem_base + (uint32_t)(a * kTileItems);
                bool first = true;
                for (int part = 0; part < 3; ++part)
                    for (int half = 0; half < 2; ++half)
                        for (int ks = 0; ks < 4; ++ks) {
                            // K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; a K step is 32 bytes along the row
                            const uint64_t adesc = smem_desc(smem_u32(&sm.q[part][half][0]) + ks * 32, 16, 1024, 2);
                            const uint64_t bdesc = smem_desc(smem_u32(&sm.h[s][half][0]) + ks * 32, 16, 1024, 2);
                            umma_f16(dcol, adesc, bdesc, kIdesc, !first);
                            first = false;
                        }
                umma_commit(&sm.empty[s]);        // the stage may be refilled once these MMAs have read it
                umma_commit(&sm.acc_full[a]);
            }
        }
    } else {
        // selection: thread = query = accumulator lane
        const int64_t q = (int64_t)blockIdx.x * kTopkQueries + tid;
        const bool live = q < m;
        const int64_t lq = (int64_t)blockIdx.y * m + (live ? q : 0);
        // lists in global memory: each thread keeps its own (alx_topk.cuh).  Lists in shared memory: a warp inserts for one
        // of its queries at a time, all 32 lanes working on that query's list -- lane l looks at elements l and l + 32,
        // two ballots give the position, every lane moves its elements one place down, the owner writes the newcomer:
        // an insertion is a dozen instructions however long the list, and no lane idles while another shifts.
        TopList top{list_s + lq * k, list_id + lq * k, k, 0, 0.f, 1};
        int cnt = 0;
        float tau = 0.f;
        for (int t = 0; t < n_tiles; ++t) {
            const int a = t & 1;
            if (!mbar_wait_warp(&sm.acc_full[a], (uint32_t)((t / 2) & 1), &sm.abort_flag, 75)) break;
            tc_fence_after();
            const uint32_t trow = sm.tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(a * kTileItems);
            const int64_t base = i0 + (int64_t)t * kTileItems;
#pragma unroll 1
            for (int cb = 0; cb < kTileItems / 16; ++cb) {
                float v[16];
                tmem_ld16(trow + 16 * cb, v);
                if constexpr (!SMEM_LISTS) {
                    if (!live) continue;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int64_t item = base + 16 * cb + j;
                        if (item < i1 && top.wants(v[j]) && !excluded(ex_ptr, ex_idx, q, (int32_t)item)) top.insert(v[j], (int32_t)item);
                    }
                } else {
                    // steady state: no query of the warp wants any of these 16 items (one ballot for the block)
                    float vmax = v[0];
#pragma unroll
                    for (int j = 1; j < 16; ++j) vmax = fmaxf(vmax, v[j]);
                    if (__ballot_sync(0xFFFFFFFFu, live && (cnt < k || vmax > tau)) == 0u) continue;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int64_t item = base + 16 * cb + j;      // (the same item for every lane: the lanes differ in the query)
                        const bool cand = live && item < i1 && (cnt < k ? (v[j] == v[j]) : v[j] > tau) &&
                                          !excluded(ex_ptr, ex_idx, q, (int32_t)item);
                        unsigned pending = __ballot_sync(0xFFFFFFFFu, cand);
                        while (pending) {
                            const int owner = __ffs(pending) - 1;
                            pending &= pending - 1;
                            const float nv = __shfl_sync(0xFFFFFFFFu, v[j], owner);
                            const int ocnt = __shfl_sync(0xFFFFFFFFu, cnt, owner);
                            float *qs = &sm.ls[warp * 32 + owner][0];
                            int32_t *qi = &sm.li[warp * 32 + owner][0];
                            const int p0 = lane, p1 = lane + 32;
                            const float e0 = p0 < ocnt ? qs[p0] : 0.f, e1 = p1 < ocnt ? qs[p1] : 0.f;
                            const int32_t d0 = p0 < ocnt ? qi[p0] : 0, d1 = p1 < ocnt ? qi[p1] : 0;
                            // elements that stay in front of the newcomer: score >= its score (their ids are smaller)
                            const int pos = __popc(__ballot_sync(0xFFFFFFFFu, p0 < ocnt && e0 >= nv)) +
                                            __popc(__ballot_sync(0xFFFFFFFFu, p1 < ocnt && e1 >= nv));
                            __syncwarp();      // every lane has read its elements
                            if (p0 >= pos && p0 < ocnt && p0 + 1 < k) { qs[p0 + 1] = e0; qi[p0 + 1] = d0; }
                            if (p1 >= pos && p1 < ocnt && p1 + 1 < k) { qs[p1 + 1] = e1; qi[p1 + 1] = d1; }
                            if (lane == owner) { qs[pos] = nv; qi[pos] = (int32_t)item; }
                            __syncwarp();
                            const int ncnt = ocnt < k ? ocnt + 1 : k;
                            const float last = qs[ncnt - 1];
                            if (lane == owner) { cnt = ncnt; tau = last; }
                            __syncwarp();
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.acc_empty[a]);
        }
        if (live) {
            if constexpr (SMEM_LISTS) {
                list_cnt[lq] = cnt;
                for (int p = 0; p < cnt; ++p) {
                    list_s[lq * k + p] = sm.ls[tid][p];
                    list_id[lq * k + p] = sm.li[tid][p];
                }
            } else {
                list_cnt[lq] = top.cnt;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(sm.tmem_base, 256);
    }
    if (tid == 0 && sm.abort_flag) raise_flag(st, kFlagTimeout, (long long)sm.abort_flag * 1000000 + blockIdx.x);
}

// 2D bfloat16 tensor [rows x 128], box 64 features x 128 rows, 128-byte swizzle; rows past the extent read as zeros
cudaError_t tile_tensor_map(const void *X, int64_t rows, CUtensorMap *tm)
{
    typedef CUresult (*Encode)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                               const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Encode encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qr;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr);
        if (e != cudaSuccess) return e;
        if (qr != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        encode = reinterpret_cast<Encode>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kD * sizeof(__nv_bfloat16)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTileItems};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(X), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

int64_t padded_queries(int64_t m) { return (m + kTopkQueries - 1) / kTopkQueries * kTopkQueries; }

}  // namespace

int64_t topk_query_scratch_bytes(int64_t m) { return 3 * padded_queries(m) * kD * (int64_t)sizeof(__nv_bfloat16); }

cudaError_t launch_topk_umma(const void *H, int64_t n_items, const float *Q, int64_t m, int k, const int64_t *ex_ptr,
                             const int32_t *ex_idx, int slabs, int64_t slab, float *list_s, int32_t *list_id,
                             int32_t *list_cnt, void *scratch_q, DevStatus *st, cudaStream_t s, int64_t *launches)
{
    const int64_t m_pad = padded_queries(m);
    __nv_bfloat16 *P = static_cast<__nv_bfloat16 *>(scratch_q);
    k_split_queries<<<(unsigned)((m_pad * kD + 255) / 256), 256, 0, s>>>(Q, m, m_pad, P);
    ++*launches;
    CUtensorMap tm_h, tm_q;
    cudaError_t e = tile_tensor_map(H, n_items, &tm_h);
    if (e != cudaSuccess) return e;
    e = tile_tensor_map(P, 3 * m_pad, &tm_q);
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)(m_pad / kTopkQueries), (unsigned)slabs);
    if (k <= kListMax) {
        const size_t smem = sizeof(TopkSmem<true>) + 1024;
        e = cudaFuncSetAttribute(k_topk_umma<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_topk_umma<true><<<grid, kThreads, smem, s>>>(tm_h, tm_q, n_items, m, m_pad, k, ex_ptr, ex_idx, slab, list_s, list_id,
                                                       list_cnt, st);
    } else {
        const size_t smem = sizeof(TopkSmem<false>) + 1024;
        e = cudaFuncSetAttribute(k_topk_umma<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_topk_umma<false><<<grid, kThreads, smem, s>>>(tm_h, tm_q, n_items, m, m_pad, k, ex_ptr, ex_idx, slab, list_s, list_id,
                                                        list_cnt, st);
    }
    ++*launches;
    return cudaGetLastError();
}

}  // namespace alx
