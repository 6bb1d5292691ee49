// Row kernels of one half-epoch, FP32-ALU version (every d, every storage type).
//
// For each row u of the solved side (Alg. 1 lines 3-10, Eq. 4):
//   gather the fixed-side rows x_i of its observations, accumulate b = sum y x_i and
//   A = sum x_i (x) x_i, add the shared base matrix alpha0 G + lambda I, factor A = L L^T,
//   solve, round to the storage type and write row u.
// Rows longer than `split` entries are cut into chunks that different thread blocks accumulate into
// a workspace; a second kernel adds a row's chunks in ascending order and solves (the role the
// paper's dense batching plays, Sec. 4.3).  Rows without observations are set to zero.
#include "alx_chol.cuh"
#include "alx_common.cuh"

namespace alx {

namespace {

// Accumulate sum x_i (x) x_i (thread tiles in registers, elements (ty + 16 a, tx + 16 b)) and sum y x_i
// over entries [beg, end) of the solved side's row.
template <int D, typename T>
__device__ __forceinline__ void accumulate_entries(const SideView &sv, int64_t beg, int64_t end,
                                                   const T *__restrict__ X, float *__restrict__ hs,
                                                   int32_t *__restrict__ idx_s, float *__restrict__ y_s,
                                                   float (&acc)[Geo<D>::TT][Geo<D>::TT], float &bsum)
{
    constexpr int TT = Geo<D>::TT, LDA = Geo<D>::LDA;
    constexpr int EL = Chunk16<T>::kElems, CH = D / EL;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    for (int64_t base = beg; base < end; base += kStage) {
        const int rc = (int)((end - base < kStage) ? end - base : kStage);
        if (tid < rc) {
            idx_s[tid] = sv.idx[base + tid];
            y_s[tid] = sv.val ? sv.val[base + tid] : 1.f;
        }
        __syncthreads();
        for (int pr = tid; pr < rc * CH; pr += kThreads) {
            const int r = pr / CH, ch = pr % CH;
            float v[EL];
            Chunk16<T>::load(X + (int64_t)idx_s[r] * D + ch * EL, v);
#pragma unroll
            for (int k = 0; k < EL; k += 4)
                *reinterpret_cast<float4 *>(&hs[r * LDA + ch * EL + k]) = make_float4(v[k], v[k + 1], v[k + 2], v[k + 3]);
        }
        __syncthreads();
        for (int r = 0; r < rc; ++r) {
            float ai[TT], bl[TT];
#pragma unroll
            for (int a = 0; a < TT; ++a) ai[a] = hs[r * LDA + ty + 16 * a];
#pragma unroll
            for (int b = 0; b < TT; ++b) bl[b] = hs[r * LDA + tx + 16 * b];
#pragma unroll
            for (int a = 0; a < TT; ++a)
#pragma unroll
                for (int b = 0; b < TT; ++b) acc[a][b] = fmaf(ai[a], bl[b], acc[a][b]);
            if (tid < D) bsum = fmaf(y_s[r], hs[r * LDA + tid], bsum);
        }
        __syncthreads();
    }
}

struct SmemView {
    float *As, *aux, *dinv, *y_s;
    int32_t *idx_s;
};

template <int D> __device__ __forceinline__ SmemView carve(unsigned char *raw)
{
    SmemView v;
    v.As = reinterpret_cast<float *>(raw);
    v.aux = v.As + Geo<D>::A_FLOATS;
    v.dinv = v.aux + Geo<D>::AUX_FLOATS;
    v.y_s = v.dinv + D;
    v.idx_s = reinterpret_cast<int32_t *>(v.y_s + kStage);
    return v;
}

// whole rows (classes 1 .. n-2): blockIdx.x counts down from the heaviest class
template <int D, typename T>
__global__ void __launch_bounds__(kThreads, 2) k_rows_simple(SideView sv, int64_t last_item, const T *__restrict__ X,
                                                             const float *__restrict__ Bmat, RowOut out,
                                                             DevStatus *st)
{
    constexpr int TT = Geo<D>::TT, LDA = Geo<D>::LDA;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemView sm = carve<D>(smem_raw);
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int64_t u = sv.order[last_item - blockIdx.x];
    const int64_t beg = sv.ptr[u], end = sv.ptr[u + 1];
    float acc[TT][TT];
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) acc[a][b] = 0.f;
    float bsum = 0.f;
    accumulate_entries<D, T>(sv, beg, end, X, sm.aux, sm.idx_s, sm.y_s, acc, bsum);
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) {
            const int i = ty + 16 * a, l = tx + 16 * b;
            sm.As[i * LDA + l] = acc[a][b] + Bmat[i * D + l];
        }
    if (tid < D) sm.As[D * LDA + tid] = bsum;
    __syncthreads();
    float xq[(D + 31) / 32];
    __shared__ int s_bad;
    const bool ok = cholesky_solve<D>(sm.As, sm.aux, sm.dinv, xq, threadIdx.x, 0, &s_bad);
    if (tid < 32) store_solution<D, T>(xq, ok, u, out, st);
}

// chunks of split rows: partial sums into the workspace, slot-major: [slot][D*D + D]
template <int D, typename T>
__global__ void __launch_bounds__(kThreads, 2) k_chunk_partials(SideView sv, const T *__restrict__ X,
                                                                float *__restrict__ partials)
{
    constexpr int TT = Geo<D>::TT;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemView sm = carve<D>(smem_raw);
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int64_t *desc = sv.chunk_desc + (int64_t)blockIdx.x * 4;
    const int64_t beg = desc[1], end = desc[2], slot = desc[3];
    float acc[TT][TT];
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) acc[a][b] = 0.f;
    float bsum = 0.f;
    accumulate_entries<D, T>(sv, beg, end, X, sm.aux, sm.idx_s, sm.y_s, acc, bsum);
    float *dst = partials + slot * (int64_t)(D * D + D);
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) dst[(ty + 16 * a) * D + tx + 16 * b] = acc[a][b];
    if (tid < D) dst[D * D + tid] = bsum;
}

// one block per split row: chunks added in ascending slot order, then the same factor / solve / store
template <int D, typename T>
__global__ void __launch_bounds__(kThreads, 2) k_split_solve(SideView sv, int64_t split_class_begin,
                                                             const float *__restrict__ partials,
                                                             const float *__restrict__ Bmat, RowOut out,
                                                             DevStatus *st)
{
    constexpr int TT = Geo<D>::TT, LDA = Geo<D>::LDA;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemView sm = carve<D>(smem_raw);
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int64_t j = blockIdx.x;
    const int64_t u = sv.order[split_class_begin + j];
    const int64_t c0 = sv.split_first[j], c1 = sv.split_first[j + 1];
    float acc[TT][TT];
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) acc[a][b] = 0.f;
    float bsum = 0.f;
    for (int64_t c = c0; c < c1; ++c) {
        const float *src = partials + c * (int64_t)(D * D + D);
#pragma unroll
        for (int a = 0; a < TT; ++a)
#pragma unroll
            for (int b = 0; b < TT; ++b) acc[a][b] += src[(ty + 16 * a) * D + tx + 16 * b];
        if (tid < D) bsum += src[D * D + tid];
    }
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) {
            const int i = ty + 16 * a, l = tx + 16 * b;
            sm.As[i * LDA + l] = acc[a][b] + Bmat[i * D + l];
        }
    if (tid < D) sm.As[D * LDA + tid] = bsum;
    __syncthreads();
    float xq[(D + 31) / 32];
    __shared__ int s_bad;
    const bool ok = cholesky_solve<D>(sm.As, sm.aux, sm.dinv, xq, threadIdx.x, 0, &s_bad);
    if (tid < 32) store_solution<D, T>(xq, ok, u, out, st);
}

// rows without observations: A^-1 0 = 0
template <typename T>
__global__ void k_zero_rows(const int32_t *__restrict__ rows, int64_t count, int d, RowOut out)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count * d) return;
    const int64_t u = rows[t / d];
    const int c = (int)(t % d);
    store_elem(reinterpret_cast<T *>(out.table) + u * d + c, 0.f);
    if (out.cap_slot) {
        const int slot = out.cap_slot[u];
        if (slot >= 0) out.cap_out[(int64_t)slot * d + c] = 0.f;
    }
}

template <int D, typename T>
cudaError_t rows_simple_dt(const SideView &sv, const int64_t *offs, int64_t n_chunks, int64_t n_split_rows,
                           const void *Xv, const float *Bmat, float *split_partials, RowOut out, DevStatus *st,
                           cudaStream_t s, int64_t *launches)
{
    const T *X = reinterpret_cast<const T *>(Xv);
    const size_t smem = Geo<D>::SMEM;
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(k_rows_simple<D, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_chunk_partials<D, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_split_solve<D, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    // longest work first: chunks of split rows, their reduction, then whole rows from the heaviest class down
    if (n_chunks > 0) {
        k_chunk_partials<D, T><<<(unsigned)n_chunks, kThreads, smem, s>>>(sv, X, split_partials);
        ++*launches;
        k_split_solve<D, T><<<(unsigned)n_split_rows, kThreads, smem, s>>>(sv, offs[kNClasses - 1], split_partials,
                                                                          Bmat, out, st);
        ++*launches;
    }
    const int64_t n_whole = offs[kNClasses - 1] - offs[1];
    if (n_whole > 0) {
        k_rows_simple<D, T><<<(unsigned)n_whole, kThreads, smem, s>>>(sv, offs[kNClasses - 1] - 1, X, Bmat, out, st);
        ++*launches;
    }
    const int64_t n_zero = offs[1] - offs[0];
    if (n_zero > 0) {
        k_zero_rows<T><<<(unsigned)((n_zero * D + 255) / 256), 256, 0, s>>>(sv.order + offs[0], n_zero, D, out);
        ++*launches;
    }
    return cudaGetLastError();
}

template <int D>
cudaError_t rows_simple_d(const SideView &sv, const int64_t *offs, int64_t n_chunks, int64_t n_split_rows,
                          const void *X, int bf16, const float *Bmat, float *split_partials, RowOut out,
                          DevStatus *st, cudaStream_t s, int64_t *launches)
{
    if (bf16)
        return rows_simple_dt<D, __nv_bfloat16>(sv, offs, n_chunks, n_split_rows, X, Bmat, split_partials, out, st, s, launches);
    return rows_simple_dt<D, float>(sv, offs, n_chunks, n_split_rows, X, Bmat, split_partials, out, st, s, launches);
}

}  // namespace

cudaError_t launch_rows_simple(const SideView &sv, const int64_t *offs, int64_t n_chunks, int64_t n_split_rows,
                               const void *X, int bf16, int d, const float *Bmat, float *split_partials,
                               RowOut out, DevStatus *st, cudaStream_t s, int64_t *launches)
{
    switch (d) {
    case 16: return rows_simple_d<16>(sv, offs, n_chunks, n_split_rows, X, bf16, Bmat, split_partials, out, st, s, launches);
    case 32: return rows_simple_d<32>(sv, offs, n_chunks, n_split_rows, X, bf16, Bmat, split_partials, out, st, s, launches);
    case 64: return rows_simple_d<64>(sv, offs, n_chunks, n_split_rows, X, bf16, Bmat, split_partials, out, st, s, launches);
    case 128: return rows_simple_d<128>(sv, offs, n_chunks, n_split_rows, X, bf16, Bmat, split_partials, out, st, s, launches);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace alx
