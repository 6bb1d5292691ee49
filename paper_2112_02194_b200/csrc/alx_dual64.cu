// Rows with at most 16 observations for fp32 tables of 64 features: Eq. 4 in its dual form,
//   w = B^-1 H^T (I + H B^-1 H^T)^-1 y,   B = alpha0 G + lambda I   (the push-through identity: an exact restatement),
// a k x k system instead of a 64 x 64 one.  One warp per row, everything in fp32 on the FP32 ALUs (a row of 3 entries is
// 3 x 64 x 64 FMAs for Z = H B^-1 and a 3 x 3 solve: no tensor-core tile is worth filling):
//   gather the k rows of H into shared memory; Z = H B^-1 with lane l holding columns l and l + 32 of every row of Z
//   (B^-1 read from shared memory, conflict-free); S = I + Z H^T by per-lane partial products and halving warp
//   reductions; Cholesky of S and the two substitutions inside the warp (lane r = row r, pivots by shuffle);
//   w = Z^T t from the registers that hold Z.
// The form is used only while B is well conditioned (same rule as the d = 128 dual kernel): k_binv64_prepare computes
// B^-1 in fp64 once per half-epoch and sets a flag from ||B||_F ||B^-1||_F; with the flag clear this kernel does
// nothing and the whole-rows kernel takes these rows as well.
#include "alx_common.cuh"

namespace alx {

namespace {

constexpr int D = 64;
constexpr int kWarps = 8;

// B^-1 in fp64 by Cholesky (one block of 64 threads, thread i = row i), written in fp32
__global__ void __launch_bounds__(D, 1) k_binv64_prepare(const float *__restrict__ Bmat, float *__restrict__ Binv,
                                                         int *__restrict__ flag, double cond_limit)
{
    constexpr int LD = D + 1;
    __shared__ double A[D * LD];       // lower = L, strict upper = (L^-1)^T
    __shared__ double dinv[D], red[D];
    __shared__ int s_ok;
    const int i = threadIdx.x;
    if (i == 0) s_ok = 1;
    double fro = 0.0;
    for (int c = 0; c < D; ++c) {
        const double v = (double)Bmat[i * D + c];
        A[i * LD + c] = v;
        fro += v * v;
    }
    red[i] = fro;
    __syncthreads();
    for (int j = 0; j < D; ++j) {
        if (i == j) {
            const double p = A[j * LD + j];
            if (!(p > 0.0)) s_ok = 0;
            const double l = sqrt(p > 0.0 ? p : 1.0);
            A[j * LD + j] = l;
            dinv[j] = 1.0 / l;
        }
        __syncthreads();
        if (i > j) A[i * LD + j] *= dinv[j];
        __syncthreads();
        if (i > j) {
            const double lij = A[i * LD + j];
            for (int c = j + 1; c <= i; ++c) A[i * LD + c] -= lij * A[c * LD + j];
        }
        __syncthreads();
    }
    // column i of L^-1, stored transposed in the strict upper triangle: A[i][r] = Linv[r][i], r > i
    for (int r = i + 1; r < D; ++r) {
        double s = A[r * LD + i] * dinv[i];
        for (int k = i + 1; k < r; ++k) s += A[r * LD + k] * A[i * LD + k];
        A[i * LD + r] = -s * dinv[r];
    }
    __syncthreads();
    // row i of B^-1 = (L^-1)^T L^-1
    double fro_inv = 0.0;
    for (int c = 0; c < D; ++c) {
        const int m = i > c ? i : c;
        double s = 0.0;
        for (int k = m; k < D; ++k) {
            const double a = (k == i) ? dinv[i] : A[i * LD + k];
            const double b = (k == c) ? dinv[c] : A[c * LD + k];
            s += a * b;
        }
        fro_inv += s * s;
        Binv[i * D + c] = (float)s;
    }
    __syncthreads();
    dinv[i] = fro_inv;      // (dinv is not needed any more)
    __syncthreads();
    if (i == 0) {
        double f = 0.0, g = 0.0;
        for (int k = 0; k < D; ++k) { f += red[k]; g += dinv[k]; }
        const double cond = sqrt(f) * sqrt(g);
        *flag = (s_ok && cond <= cond_limit) ? 1 : 0;
    }
}

// sum over the 32 lanes of each of N values (N a power of two <= 16): afterwards the sum of v[c] is in v[0] of the lanes
// whose top log2(N) bits of the lane number are c
template <int N> __device__ __forceinline__ void warp_reduce_n(float (&v)[N], int lane)
{
    int width = 16;
#pragma unroll
    for (int n = N; n > 1; n >>= 1) {
        const bool up = (lane & width) != 0;
#pragma unroll
        for (int c = 0; c < n / 2; ++c) {
            const float send = up ? v[c] : v[c + n / 2];
            const float keep = up ? v[c + n / 2] : v[c];
            v[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, width);
        }
        width >>= 1;
    }
    for (; width > 0; width >>= 1) v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], width);
}

struct WarpScratch {
    float H[16][D];        // the gathered rows
    float S[16][17];       // I + Z H^T
};

// one row of at most KMAX observations (KMAX in {4, 8, 16}; KMAX a power of two)
template <int KMAX>
__device__ __forceinline__ void dual_row(const float *__restrict__ Binv_s, WarpScratch &ws, int lane, int k, float y,
                                         float &w0, float &w1)
{
    // Z = H B^-1: z0[r] = Z[r][lane], z1[r] = Z[r][lane + 32]
    float z0[KMAX], z1[KMAX];
#pragma unroll
    for (int r = 0; r < KMAX; ++r) z0[r] = z1[r] = 0.f;
#pragma unroll 2
    for (int f = 0; f < D; f += 4) {
        float b0[4], b1[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            b0[j] = Binv_s[(f + j) * D + lane];
            b1[j] = Binv_s[(f + j) * D + lane + 32];
        }
#pragma unroll
        for (int r = 0; r < KMAX; ++r) {
            const float4 h = *reinterpret_cast<const float4 *>(&ws.H[r][f]);      // (rows k .. KMAX - 1 are zero)
            z0[r] = fmaf(h.x, b0[0], z0[r]); z1[r] = fmaf(h.x, b1[0], z1[r]);
            z0[r] = fmaf(h.y, b0[1], z0[r]); z1[r] = fmaf(h.y, b1[1], z1[r]);
            z0[r] = fmaf(h.z, b0[2], z0[r]); z1[r] = fmaf(h.z, b1[2], z1[r]);
            z0[r] = fmaf(h.w, b0[3], z0[r]); z1[r] = fmaf(h.w, b1[3], z1[r]);
        }
    }
    // S = I + Z H^T, row by row: partial products over this lane's two columns, summed over the lanes
    constexpr int kShift = KMAX == 16 ? 1 : KMAX == 8 ? 2 : 3;      // the sum of value c lands in lanes c << kShift ..
    float h0[KMAX], h1[KMAX];
#pragma unroll
    for (int r = 0; r < KMAX; ++r) { h0[r] = ws.H[r][lane]; h1[r] = ws.H[r][lane + 32]; }
#pragma unroll
    for (int r = 0; r < KMAX; ++r) {
        float v[KMAX];
#pragma unroll
        for (int c = 0; c < KMAX; ++c) v[c] = fmaf(z0[r], h0[c], z1[r] * h1[c]);
        warp_reduce_n<KMAX>(v, lane);
        if ((lane & ((1 << kShift) - 1)) == 0) ws.S[r][lane >> kShift] = v[0] + ((lane >> kShift) == r ? 1.f : 0.f);
    }
    __syncwarp();
    // Cholesky of S inside the warp: lane r holds row r (rows k .. are rows of the identity: Z and H are zero there)
    float a[KMAX];
    const int rr = lane < KMAX ? lane : 0;
#pragma unroll
    for (int c = 0; c < KMAX; ++c) a[c] = ws.S[rr][c];
    float t = lane < k ? y : 0.f;      // right-hand side, carried along: t becomes L^-1 y
#pragma unroll
    for (int j = 0; j < KMAX; ++j) {
        const float ajj = __shfl_sync(0xFFFFFFFFu, a[j], j);
        const float inv = rsqrtf(ajj);       // S = I + (positive semi-definite): every pivot is at least 1
        const float lj = a[j] * inv;          // L[lane][j] (lane >= j)
        const float tj = __shfl_sync(0xFFFFFFFFu, t, j) * inv;      // (L^-1 y)[j]
        if (lane == j) t = tj;
        else if (lane > j) t = fmaf(-lj, tj, t);
        a[j] = lj;
#pragma unroll
        for (int c = j + 1; c < KMAX; ++c) {
            const float lc = __shfl_sync(0xFFFFFFFFu, lj, c);        // L[c][j]
            a[c] = fmaf(-lj, lc, a[c]);
        }
    }
    // L^T x = t, from the last row up (L through shared memory: lane c needs L[j][c], which lane j holds): lane r ends with x_r
    __syncwarp();
    if (lane < KMAX) {
#pragma unroll
        for (int c = 0; c < KMAX; ++c) ws.S[lane][c] = a[c];
    }
    __syncwarp();
#pragma unroll
    for (int j = KMAX - 1; j >= 0; --j) {
        const float xj = __shfl_sync(0xFFFFFFFFu, t, j) / ws.S[j][j];
        if (lane == j) t = xj;
        else if (lane < j) t = fmaf(-ws.S[j][lane], xj, t);
    }
    // w = Z^T x
    w0 = 0.f;
    w1 = 0.f;
#pragma unroll
    for (int r = 0; r < KMAX; ++r) {
        const float xr = __shfl_sync(0xFFFFFFFFu, t, r);
        w0 = fmaf(z0[r], xr, w0);
        w1 = fmaf(z1[r], xr, w1);
    }
}

__global__ void __launch_bounds__(kWarps * 32) k_dual64(SideView sv, int64_t first, int64_t count, const float *__restrict__ X,
                                                        const float *__restrict__ Binv, const int *__restrict__ flag, RowOut out)
{
    if (*flag == 0) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *Binv_s = reinterpret_cast<float *>(smem_raw);
    WarpScratch *scr = reinterpret_cast<WarpScratch *>(smem_raw + sizeof(float) * D * D);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int e = threadIdx.x; e < D * D; e += kWarps * 32) Binv_s[e] = Binv[e];
    __syncthreads();
    WarpScratch &ws = scr[warp];
    const int64_t n_warps = (int64_t)gridDim.x * kWarps;
    for (int64_t t = (int64_t)blockIdx.x * kWarps + warp; t < count; t += n_warps) {
        const int64_t u = sv.order[first + t];
        const int64_t beg = sv.ptr[u];
        const int k = (int)(sv.ptr[u + 1] - beg);      // 1 .. 16
        const int kmax = k <= 4 ? 4 : k <= 8 ? 8 : 16;
        int32_t col = 0;
        float y = 0.f;
        if (lane < k) {
            col = sv.idx[beg + lane];
            y = sv.val ? sv.val[beg + lane] : 1.f;
        }
        __syncwarp();
        // gather: two rows per pass (16 lanes x 16 bytes each); rows k .. kmax - 1 are zero
        for (int r0 = 0; r0 < kmax; r0 += 2) {
            const int r = r0 + (lane >> 4);
            const int32_t c = __shfl_sync(0xFFFFFFFFu, col, r);
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r < k) v = *reinterpret_cast<const float4 *>(X + (int64_t)c * D + 4 * (lane & 15));
            *reinterpret_cast<float4 *>(&ws.H[r][4 * (lane & 15)]) = v;
        }
        __syncwarp();
        float w0, w1;
        if (kmax == 4) dual_row<4>(Binv_s, ws, lane, k, y, w0, w1);
        else if (kmax == 8) dual_row<8>(Binv_s, ws, lane, k, y, w0, w1);
        else dual_row<16>(Binv_s, ws, lane, k, y, w0, w1);
        float *dst = reinterpret_cast<float *>(out.table) + u * D;
        dst[lane] = w0;
        dst[lane + 32] = w1;
        if (out.cap_slot) {
            const int cs = out.cap_slot[u];
            if (cs >= 0) {
                out.cap_out[(int64_t)cs * D + lane] = w0;
                out.cap_out[(int64_t)cs * D + lane + 32] = w1;
            }
        }
    }
}

}  // namespace

size_t dual64_workspace_bytes() { return sizeof(float) * D * D + 256; }
int *dual64_flag_ptr(void *ws) { return reinterpret_cast<int *>(static_cast<unsigned char *>(ws) + sizeof(float) * D * D); }

cudaError_t launch_dual64_prepare(const float *Bmat, void *ws, float cond_limit, cudaStream_t s, int64_t *launches)
{
    k_binv64_prepare<<<1, D, 0, s>>>(Bmat, static_cast<float *>(ws), dual64_flag_ptr(ws), (double)cond_limit);
    ++*launches;
    return cudaGetLastError();
}

// rows sv.order[first .. first + count): the rows of 1 .. 16 observations of the REAL entry lists (degree class 1)
cudaError_t launch_rows_dual64(const SideView &sv, int64_t first, int64_t count, const void *X, void *ws, RowOut out,
                               cudaStream_t s, int64_t *launches)
{
    if (count <= 0) return cudaSuccess;
    const size_t smem = sizeof(float) * D * D + kWarps * sizeof(WarpScratch);
    cudaError_t e = cudaFuncSetAttribute(k_dual64, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int64_t blocks = (count + kWarps - 1) / kWarps;
    if (blocks > 148 * 6) blocks = 148 * 6;
    k_dual64<<<(unsigned)blocks, kWarps * 32, smem, s>>>(sv, first, count, static_cast<const float *>(X),
                                                         static_cast<const float *>(ws), dual64_flag_ptr(ws), out);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace alx
