// The objective of Eq. 3 at the current tables.  The observed term is summed entry by entry
// (products and the length-d dot product in fp32, everything across entries in fp64, fixed order);
// the all-pairs term uses sum_u sum_i <w_u, h_i>^2 = <W^T W, H^T H>_F, the Gramian identity the paper
// states under Eq. 4 applied to the objective; the regulariser is the trace of the two Gramians.
#include "alx_common.cuh"

namespace alx {

namespace {

constexpr int kSpan = 128;      // entries per warp
constexpr int kWarps = 8;

__device__ __forceinline__ int64_t row_of(const int64_t *__restrict__ ptr, int64_t n, int64_t e)
{
    int64_t lo = 0, hi = n;
    while (hi - lo > 1) {
        const int64_t mid = lo + ((hi - lo) >> 1);
        if (ptr[mid] <= e) lo = mid; else hi = mid;
    }
    return lo;
}

template <int D, typename T>
__global__ void __launch_bounds__(kWarps * 32) k_loss_obs(const int64_t *__restrict__ rowptr,
                                                          const int32_t *__restrict__ colidx,
                                                          const float *__restrict__ values, int64_t n_rows,
                                                          int64_t nnz, const T *__restrict__ W,
                                                          const T *__restrict__ H, double *__restrict__ partials)
{
    constexpr int PER = (D + 31) / 32;
    __shared__ double warp_sum[kWarps];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t e0 = ((int64_t)blockIdx.x * kWarps + warp) * kSpan;
    double acc = 0.0;
    if (e0 < nnz) {
        const int64_t e1 = (e0 + kSpan < nnz) ? e0 + kSpan : nnz;
        int64_t u = row_of(rowptr, n_rows, e0);
        int64_t u_loaded = -1;
        float w[PER];
        for (int64_t e = e0; e < e1; ++e) {
            while (rowptr[u + 1] <= e) ++u;
            if (u != u_loaded) {
#pragma unroll
                for (int k = 0; k < PER; ++k) {
                    const int c = k * 32 + lane;
                    w[k] = (c < D) ? to_f32(W[u * D + c]) : 0.f;
                }
                u_loaded = u;
            }
            const int64_t i = colidx[e];
            float dot = 0.f;
#pragma unroll
            for (int k = 0; k < PER; ++k) {
                const int c = k * 32 + lane;
                if (c < D) dot = fmaf(w[k], to_f32(H[i * D + c]), dot);
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, o);
            const float y = values ? values[e] : 1.f;
            const double r = (double)y - (double)dot;
            acc += r * r;
        }
    }
    if (lane == 0) warp_sum[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int k = 0; k < kWarps; ++k) s += warp_sum[k];
        partials[blockIdx.x] = s;
    }
}

__device__ __forceinline__ double block_tree_sum(double v, double *buf)
{
    buf[threadIdx.x] = v;
    __syncthreads();
    for (int o = blockDim.x >> 1; o >= 1; o >>= 1) {
        if ((int)threadIdx.x < o) buf[threadIdx.x] += buf[threadIdx.x + o];
        __syncthreads();
    }
    const double r = buf[0];
    __syncthreads();
    return r;
}

// result[0] = observed, result[1] = alpha0 <G_W, G_H>_F, result[2] = lambda (tr G_W + tr G_H)
__global__ void __launch_bounds__(256) k_loss_finish(const double *__restrict__ partials, int64_t n_partials,
                                                     const double *__restrict__ GW, const double *__restrict__ GH,
                                                     int d, double alpha0, double lambda,
                                                     double *__restrict__ result)
{
    __shared__ double buf[256];
    double s = 0.0;
    for (int64_t p = threadIdx.x; p < n_partials; p += 256) s += partials[p];
    const double obs = block_tree_sum(s, buf);
    double f = 0.0, t = 0.0;
    for (int e = threadIdx.x; e < d * d; e += 256) {
        f += GW[e] * GH[e];
        if (e / d == e % d) t += GW[e] + GH[e];
    }
    const double imp = block_tree_sum(f, buf);
    const double tr = block_tree_sum(t, buf);
    if (threadIdx.x == 0) {
        result[0] = obs;
        result[1] = alpha0 * imp;
        result[2] = lambda * tr;
    }
}

template <int D>
cudaError_t loss_obs_d(const int64_t *rowptr, const int32_t *colidx, const float *values, int64_t n_rows,
                       int64_t nnz, const void *W, const void *H, int bf16, double *partials, cudaStream_t s)
{
    const unsigned grid = (unsigned)loss_partials(nnz);
    if (bf16)
        k_loss_obs<D, __nv_bfloat16><<<grid, kWarps * 32, 0, s>>>(rowptr, colidx, values, n_rows, nnz,
                                                                 (const __nv_bfloat16 *)W, (const __nv_bfloat16 *)H, partials);
    else
        k_loss_obs<D, float><<<grid, kWarps * 32, 0, s>>>(rowptr, colidx, values, n_rows, nnz, (const float *)W,
                                                         (const float *)H, partials);
    return cudaGetLastError();
}

}  // namespace

int64_t loss_partials(int64_t nnz)
{
    const int64_t per_block = (int64_t)kSpan * kWarps;
    const int64_t b = (nnz + per_block - 1) / per_block;
    return b > 0 ? b : 1;
}

cudaError_t launch_loss_obs(const int64_t *rowptr, const int32_t *colidx, const float *values, int64_t n_rows,
                            int64_t nnz, const void *W, const void *H, int bf16, int d, double *partials,
                            double *result, cudaStream_t s, int64_t *launches)
{
    cudaError_t e;
    switch (d) {
    case 16: e = loss_obs_d<16>(rowptr, colidx, values, n_rows, nnz, W, H, bf16, partials, s); break;
    case 32: e = loss_obs_d<32>(rowptr, colidx, values, n_rows, nnz, W, H, bf16, partials, s); break;
    case 64: e = loss_obs_d<64>(rowptr, colidx, values, n_rows, nnz, W, H, bf16, partials, s); break;
    case 128: e = loss_obs_d<128>(rowptr, colidx, values, n_rows, nnz, W, H, bf16, partials, s); break;
    default: return cudaErrorInvalidValue;
    }
    ++*launches;
    (void)result;
    return e;
}

cudaError_t launch_loss_finish(const double *partials, int64_t n_partials, const double *GW, const double *GH, int d,
                               double alpha0, double lambda, double *result, cudaStream_t s, int64_t *launches)
{
    k_loss_finish<<<1, 256, 0, s>>>(partials, n_partials, GW, GH, d, alpha0, lambda, result);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace alx
