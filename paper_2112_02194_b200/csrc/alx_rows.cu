// Row kernels of one half-epoch, FP32-ALU version (every d, every storage type).
//
// For each row u of the solved side (Alg. 1 lines 3-10, Eq. 4):
//   gather the fixed-side rows x_i of its observations, accumulate b = sum y x_i and
//   A = sum x_i (x) x_i, add the shared base matrix alpha0 G + lambda I, factor A = L L^T,
//   solve, round to the storage type and write row u.
// Rows longer than `split` entries are cut into chunks that different thread blocks accumulate into
// a workspace; a second kernel adds a row's chunks in ascending order and solves (the role the
// paper's dense batching plays, Sec. 4.3).  Rows without observations are set to zero.
#include "alx_common.cuh"

namespace alx {

namespace {

constexpr int kThreads = 256;
constexpr int kStage = 32;   // gathered rows staged per step

template <int D> struct Geo {
    static constexpr int TT = D / 16;          // a thread owns a TT x TT tile of A
    static constexpr int LDA = D + 4;          // row stride of A in shared memory (keeps 16-byte alignment)
    static constexpr int LDP = D + 8;          // row stride of the transposed panel copy
    static constexpr int A_FLOATS = (D + 1) * LDA;   // row D holds b^T (bordered matrix)
    static constexpr int P_FLOATS = 16 * LDP;
    static constexpr int H_FLOATS = kStage * LDA;
    static constexpr int AUX_FLOATS = (P_FLOATS > H_FLOATS) ? P_FLOATS : H_FLOATS;
    static constexpr size_t SMEM = sizeof(float) * (A_FLOATS + AUX_FLOATS + D) + sizeof(int32_t) * kStage +
                                   sizeof(float) * kStage + 16;
};

// ------------------------------------------------------------------------------------------------
// Blocked right-looking Cholesky of the bordered matrix [[A, b], [b^T, .]] held in shared memory
// (lower triangle), 16 columns per step.  Afterwards rows 0..D-1 hold L and row D holds (L^-1 b)^T.
// Then warp 0 solves L^T x = L^-1 b and returns x in registers: lane holds x[q * 32 + lane] in xq[q].
// All kThreads threads must call.  Returns false (to every thread) if a pivot was not positive.
// ------------------------------------------------------------------------------------------------
template <int D>
__device__ bool cholesky_solve(float *__restrict__ As, float *__restrict__ Pt, float *__restrict__ dinv,
                               float (&xq)[(D + 31) / 32])
{
    constexpr int TT = Geo<D>::TT, LDA = Geo<D>::LDA, LDP = Geo<D>::LDP;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ty = tid >> 4, tx = tid & 15;
    __shared__ int s_bad;
    if (tid == 0) s_bad = 0;

    for (int k0 = 0; k0 < D; k0 += 16) {
        // (1) diagonal 16 x 16 block: one warp, rows in registers, columns exchanged by shuffles
        if (warp == 0) {
            const int l = lane & 15;
            float r[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) r[c] = As[(k0 + l) * LDA + k0 + c];
            float my_inv = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float pj = __shfl_sync(0xFFFFFFFFu, r[j], j);
                const bool ok = pj > 0.f;
                const float sq = ok ? __fsqrt_rn(pj) : 0.f;
                const float inv = ok ? __frcp_rn(sq) : 0.f;
                if (!ok && lane == 0) s_bad = 1;
                r[j] = (l == j) ? sq : r[j] * inv;
                if (l == j) my_inv = inv;
#pragma unroll
                for (int c = j + 1; c < 16; ++c) {
                    const float lc = __shfl_sync(0xFFFFFFFFu, r[j], c);
                    r[c] = fmaf(-r[j], lc, r[c]);
                }
            }
            if (lane < 16) {
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    if (c <= l) As[(k0 + l) * LDA + k0 + c] = r[c];
                dinv[k0 + l] = my_inv;
            }
        }
        __syncthreads();
        // (2) panel below the block (including the border row D): one thread per row, forward substitution
        const int m = D - k0 - 15;
        if (tid < m) {
            const int i = k0 + 16 + tid;
            float a[16];
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                const float4 v = *reinterpret_cast<const float4 *>(&As[i * LDA + k0 + 4 * c4]);
                a[4 * c4] = v.x; a[4 * c4 + 1] = v.y; a[4 * c4 + 2] = v.z; a[4 * c4 + 3] = v.w;
            }
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                float s = a[c];
#pragma unroll
                for (int p = 0; p < c; ++p) s = fmaf(-a[p], As[(k0 + c) * LDA + k0 + p], s);
                a[c] = s * dinv[k0 + c];
            }
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4)
                *reinterpret_cast<float4 *>(&As[i * LDA + k0 + 4 * c4]) =
                    make_float4(a[4 * c4], a[4 * c4 + 1], a[4 * c4 + 2], a[4 * c4 + 3]);
#pragma unroll
            for (int c = 0; c < 16; ++c) Pt[c * LDP + i] = a[c];
        }
        __syncthreads();
        // (3) trailing update A[i][l] -= sum_p P[i][p] P[l][p] on the lower-triangle tiles, and the border row
        const int I0 = ty * TT, L0 = tx * TT;
        if (tx <= ty && L0 >= k0 + 16) {
            float acc[TT][TT];
#pragma unroll
            for (int a = 0; a < TT; ++a)
#pragma unroll
                for (int b = 0; b < TT; ++b) acc[a][b] = 0.f;
#pragma unroll
            for (int p = 0; p < 16; ++p) {
                float ai[TT], bl[TT];
#pragma unroll
                for (int a = 0; a < TT; ++a) ai[a] = Pt[p * LDP + I0 + a];
#pragma unroll
                for (int b = 0; b < TT; ++b) bl[b] = Pt[p * LDP + L0 + b];
#pragma unroll
                for (int a = 0; a < TT; ++a)
#pragma unroll
                    for (int b = 0; b < TT; ++b) acc[a][b] = fmaf(ai[a], bl[b], acc[a][b]);
            }
#pragma unroll
            for (int a = 0; a < TT; ++a)
#pragma unroll
                for (int b = 0; b < TT; ++b) As[(I0 + a) * LDA + L0 + b] -= acc[a][b];
        }
        if (tid >= k0 + 16 && tid < D) {
            float s = 0.f;
#pragma unroll
            for (int p = 0; p < 16; ++p) s = fmaf(Pt[p * LDP + D], Pt[p * LDP + tid], s);
            As[D * LDA + tid] -= s;
        }
        __syncthreads();
    }
    // (4) back substitution L^T x = z, z = row D; one warp, column by column from the last
    constexpr int NQ = (D + 31) / 32;
    if (warp == 0) {
#pragma unroll
        for (int q = 0; q < NQ; ++q) xq[q] = (q * 32 + lane < D) ? As[D * LDA + q * 32 + lane] : 0.f;
#pragma unroll
        for (int q = NQ - 1; q >= 0; --q) {
            const int s_hi = (D - q * 32 < 32) ? D - q * 32 - 1 : 31;
            for (int s = s_hi; s >= 0; --s) {
                const int j = q * 32 + s;
                const float xj = __shfl_sync(0xFFFFFFFFu, xq[q], s) * dinv[j];
                if (lane == s) xq[q] = xj;
#pragma unroll
                for (int q2 = 0; q2 <= q; ++q2) {
                    const int i = q2 * 32 + lane;
                    if (i < j) xq[q2] = fmaf(-As[j * LDA + i], xj, xq[q2]);
                }
            }
        }
    }
    return s_bad == 0;
}

template <int D, typename T>
__device__ __forceinline__ void store_solution(const float (&xq)[(D + 31) / 32], bool ok, int64_t u, RowOut out,
                                               DevStatus *st)
{
    // called by warp 0 only
    const int lane = threadIdx.x & 31;
    T *row = reinterpret_cast<T *>(out.table) + u * D;
    const int slot = out.cap_slot ? out.cap_slot[u] : -1;
#pragma unroll
    for (int q = 0; q < (D + 31) / 32; ++q) {
        const int i = q * 32 + lane;
        if (i < D) {
            const float v = ok ? xq[q] : 0.f;
            store_elem(row + i, v);
            if (slot >= 0) out.cap_out[(int64_t)slot * D + i] = v;
        }
    }
    if (!ok && lane == 0) {
        atomicAdd(&st->not_spd, 1ull);
        raise_flag(st, kFlagNotSpd, u);
    }
}

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
    const bool ok = cholesky_solve<D>(sm.As, sm.aux, sm.dinv, xq);
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
    const bool ok = cholesky_solve<D>(sm.As, sm.aux, sm.dinv, xq);
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
