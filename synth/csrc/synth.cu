// Device twin of the seeded input generators in synth/graphs.py: the same integer recipe, so both
// produce identical bits.  Inputs only: no arithmetic of the factorisation method lives here, and
// this file is built into its own shared object.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

typedef unsigned long long u64;

__host__ __device__ inline u64 mix64(u64 z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__host__ __device__ inline u64 hash2(u64 key, u64 a, u64 b) { return mix64(mix64(key ^ a) + b * 0x9E3779B97F4A7C15ull); }

constexpr int kQtBits = 16;
constexpr int kNtBits = 12;
constexpr int kNtFracBits = 20;

__device__ inline u64 g_fixed(const u64 *__restrict__ qt, u64 j, u64 k)
{
    const u64 pos = (j << 32) / k;
    u64 idx = pos >> (32 - kQtBits);
    const u64 frac = pos & ((1ull << (32 - kQtBits)) - 1);
    const u64 T = 1ull << kQtBits;
    if (idx > T) idx = T;
    const u64 nxt = (idx + 1 < T) ? idx + 1 : T;
    const u64 q0 = qt[idx], q1 = qt[nxt];
    return q0 + (((q1 - q0) * frac) >> (32 - kQtBits));
}

__device__ inline u64 quantile_bound(const u64 *__restrict__ qt, u64 N, u64 j, u64 k)
{
    return j + (((N - k) * g_fixed(qt, j, k)) >> 32);
}

__device__ inline u64 uniform_bound(u64 j, u64 k, u64 M) { return (j * M) / (k ? k : 1); }

struct EdgeParams {
    int law;              // 0 quantile, 1 local
    long long n_rows, n_cols;
    u64 key;
    const u64 *qtable;    // [2^16 + 1]
    long long delta, local_num, local_den;
};

__device__ inline long long row_of(const long long *__restrict__ ptr, long long n, long long e)
{
    long long lo = 0, hi = n;
    while (hi - lo > 1) {
        const long long mid = lo + ((hi - lo) >> 1);
        if (ptr[mid] <= e) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ inline int32_t column_of(const EdgeParams &p, long long u, long long kdeg, long long jj)
{
    const u64 j = (u64)jj, k = (u64)kdeg;
    if (p.law == 0) {
        const u64 lo = quantile_bound(p.qtable, (u64)p.n_cols, j, k);
        const u64 hi = quantile_bound(p.qtable, (u64)p.n_cols, j + 1, k);
        return (int32_t)(lo + hash2(p.key, (u64)u, j) % (hi - lo));
    }
    const long long N = p.n_cols, wsz = 2 * p.delta + 1, M = N - wsz;
    long long kloc = (kdeg * p.local_num + p.local_den / 2) / p.local_den;
    if (kloc > wsz) kloc = wsz;
    const long long kfar = kdeg - kloc;
    long long wlo = u - p.delta;
    if (wlo < 0) wlo = 0;
    if (wlo > N - wsz) wlo = N - wsz;
    long long cbelow = 0;
    if (kfar > 0) {
        long long t = ((wlo + 1) * kfar - 1) / M;
        if (t > kfar) t = kfar;
        const long long js = t;   // (count of strata starting at or below wlo) - 1
        cbelow = js;
        if (js < kfar) {
            const u64 f0 = uniform_bound((u64)js, (u64)kfar, (u64)M), f1 = uniform_bound((u64)js + 1, (u64)kfar, (u64)M);
            const u64 span = (f1 > f0) ? f1 - f0 : 1;
            const u64 ts = f0 + hash2(p.key, (u64)u, (u64)js + (1ull << 40)) % span;
            if ((long long)ts < wlo) cbelow += 1;
        }
    }
    if (jj >= cbelow && jj < cbelow + kloc) {
        const u64 jl = (u64)(jj - cbelow);
        const u64 l0 = uniform_bound(jl, (u64)kloc, (u64)wsz), l1 = uniform_bound(jl + 1, (u64)kloc, (u64)wsz);
        const u64 span = (l1 > l0) ? l1 - l0 : 1;
        return (int32_t)((u64)wlo + l0 + hash2(p.key, (u64)u, jl) % span);
    }
    const u64 jf = (u64)((jj < cbelow) ? jj : jj - kloc);
    const u64 g0 = uniform_bound(jf, (u64)kfar, (u64)M), g1 = uniform_bound(jf + 1, (u64)kfar, (u64)M);
    const u64 span = (g1 > g0) ? g1 - g0 : 1;
    const u64 t = g0 + hash2(p.key, (u64)u, jf + (1ull << 40)) % span;
    return (int32_t)(((long long)t < wlo) ? t : t + (u64)wsz);
}

constexpr int kPerThread = 8;

__global__ void k_edges(EdgeParams p, const long long *__restrict__ rowptr, long long nnz, int32_t *__restrict__ colidx)
{
    const long long e0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * kPerThread;
    if (e0 >= nnz) return;
    long long u = row_of(rowptr, p.n_rows, e0);
    const long long e1 = (e0 + kPerThread < nnz) ? e0 + kPerThread : nnz;
    for (long long e = e0; e < e1; ++e) {
        while (rowptr[u + 1] <= e) ++u;
        colidx[e] = column_of(p, u, rowptr[u + 1] - rowptr[u], e - rowptr[u]);
    }
}

template <typename T>
__global__ void k_normal(u64 key, const long long *__restrict__ table, long long start, long long count, double scale,
                         T *__restrict__ out)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const u64 h = hash2(key, (u64)(start + i), 0);
    const long long cell = (long long)(h >> (64 - kNtBits));
    const long long frac = (long long)((h >> (64 - kNtBits - kNtFracBits)) & ((1ull << kNtFracBits) - 1));
    const long long t0 = table[cell], t1 = table[cell + 1];
    const long long v = t0 + (((t1 - t0) * frac) >> kNtFracBits);
    const double x = (double)v * scale;
    const float f = (float)x;   // round to nearest even, as numpy's astype(float32)
    if (sizeof(T) == 4) reinterpret_cast<float *>(out)[i] = f;
    else reinterpret_cast<__nv_bfloat16 *>(out)[i] = __float2bfloat16_rn(f);
}

}  // namespace

extern "C" {

// colidx[nnz] <- columns of every row; rowptr, qtable and colidx are device pointers. Returns a cudaError_t.
int synth_edges(int law, long long n_rows, long long n_cols, unsigned long long key, const void *qtable,
                long long delta, long long local_num, long long local_den, const void *rowptr, long long nnz,
                void *colidx, void *stream)
{
    if (nnz <= 0) return 0;
    EdgeParams p{law, n_rows, n_cols, key, (const u64 *)qtable, delta, local_num, local_den};
    const long long threads = (nnz + kPerThread - 1) / kPerThread;
    k_edges<<<(unsigned)((threads + 255) / 256), 256, 0, (cudaStream_t)stream>>>(p, (const long long *)rowptr, nnz,
                                                                             (int32_t *)colidx);
    return (int)cudaGetLastError();
}

// out[count] <- normal draws (element indices start .. start+count-1) times scale, as float32 or bfloat16
int synth_normal(unsigned long long key, const void *table, long long start, long long count, double scale, int bf16,
                 void *out, void *stream)
{
    if (count <= 0) return 0;
    const unsigned grid = (unsigned)((count + 255) / 256);
    if (bf16)
        k_normal<__nv_bfloat16><<<grid, 256, 0, (cudaStream_t)stream>>>(key, (const long long *)table, start, count, scale, (__nv_bfloat16 *)out);
    else
        k_normal<float><<<grid, 256, 0, (cudaStream_t)stream>>>(key, (const long long *)table, start, count, scale, (float *)out);
    return (int)cudaGetLastError();
}

}  // extern "C"
