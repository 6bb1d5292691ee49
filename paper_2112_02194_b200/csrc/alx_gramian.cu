// Gramian of the fixed table, G = X^T X over all of its rows (Alg. 1 line 2; the remark under Eq. 4
// that sum_i h_i (x) h_i does not depend on the row being solved), and the base matrix
// alpha0 G + lambda I that every row's normal matrix starts from (Alg. 1 line 5).
//
// The table is cut into pieces of kGramRowsPerPartial rows (a function of the table size only); each
// piece is summed in fp32 by one thread block, and the pieces are added in ascending order in fp64,
// so the result does not depend on how blocks are scheduled.
#include <mutex>
#include <string>

#include "../../include/alx.h"
#include "alx_common.cuh"

namespace alx {

namespace {

constexpr int kStageRows = 32;

// FP32-ALU version: works for every d in {16, 32, 64, 128} and both storage types
template <int D, typename T>
__global__ void __launch_bounds__(256) k_gramian_simple(const T *__restrict__ X, int64_t n,
                                                        float *__restrict__ partials)
{
    constexpr int TT = D / 16;
    constexpr int LDS = D + 4;
    constexpr int CH = D / Chunk16<T>::kElems;   // 16-byte chunks per row
    __shared__ __align__(16) float hs[kStageRows * LDS];
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int64_t r0 = (int64_t)blockIdx.x * kGramRowsPerPartial;
    const int64_t r1 = (r0 + kGramRowsPerPartial < n) ? r0 + kGramRowsPerPartial : n;
    float acc[TT][TT];
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) acc[a][b] = 0.f;

    for (int64_t base = r0; base < r1; base += kStageRows) {
        const int rc = (int)((r1 - base < kStageRows) ? r1 - base : kStageRows);
        for (int pr = tid; pr < rc * CH; pr += 256) {
            const int r = pr / CH, ch = pr % CH;
            float v[Chunk16<T>::kElems];
            Chunk16<T>::load(X + (base + r) * D + ch * Chunk16<T>::kElems, v);
#pragma unroll
            for (int k = 0; k < Chunk16<T>::kElems; ++k) hs[r * LDS + ch * Chunk16<T>::kElems + k] = v[k];
        }
        __syncthreads();
        // two-level sum: a fresh accumulator per staged batch keeps the fp32 error near sqrt(rows) * 2^-24
        float part[TT][TT];
#pragma unroll
        for (int a = 0; a < TT; ++a)
#pragma unroll
            for (int b = 0; b < TT; ++b) part[a][b] = 0.f;
        for (int r = 0; r < rc; ++r) {
            float ai[TT], bl[TT];
#pragma unroll
            for (int a = 0; a < TT; ++a) ai[a] = hs[r * LDS + ty + 16 * a];
#pragma unroll
            for (int b = 0; b < TT; ++b) bl[b] = hs[r * LDS + tx + 16 * b];
#pragma unroll
            for (int a = 0; a < TT; ++a)
#pragma unroll
                for (int b = 0; b < TT; ++b) part[a][b] = fmaf(ai[a], bl[b], part[a][b]);
        }
#pragma unroll
        for (int a = 0; a < TT; ++a)
#pragma unroll
            for (int b = 0; b < TT; ++b) acc[a][b] += part[a][b];
        __syncthreads();
    }
    float *out = partials + (int64_t)blockIdx.x * D * D;
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < TT; ++b) out[(ty + 16 * a) * D + tx + 16 * b] = acc[a][b];
}

// pieces added in ascending order in fp64; also writes alpha0 G + lambda I in fp32
__global__ void k_gramian_reduce(const float *__restrict__ partials, int64_t n_partials, int d,
                                 double *__restrict__ G64, float *__restrict__ Bmat, float alpha0, float lambda)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= d * d) return;
    double s = 0.0;
    for (int64_t p = 0; p < n_partials; ++p) s += (double)partials[p * d * d + e];
    G64[e] = s;
    const int i = e / d, l = e % d;
    Bmat[e] = (float)((double)alpha0 * s + (i == l ? (double)lambda : 0.0));
}

template <int D>
cudaError_t gramian_simple_d(const void *X, int bf16, int64_t n, float *partials, cudaStream_t s)
{
    const unsigned grid = (unsigned)gramian_partials(n);
    if (bf16)
        k_gramian_simple<D, __nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16 *)X, n, partials);
    else
        k_gramian_simple<D, float><<<grid, 256, 0, s>>>((const float *)X, n, partials);
    return cudaGetLastError();
}

}  // namespace

int64_t gramian_partials(int64_t n) { return (n + kGramRowsPerPartial - 1) / kGramRowsPerPartial; }

cudaError_t launch_gramian_reduce(const float *partials, int64_t n_partials, int d, double *G64, float *Bmat,
                                  float alpha0, float lambda, cudaStream_t s, int64_t *launches)
{
    k_gramian_reduce<<<(d * d + 255) / 256, 256, 0, s>>>(partials, n_partials, d, G64, Bmat, alpha0, lambda);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_gramian(const void *X, int bf16, int64_t n, int d, float *partials, double *G64, float *Bmat,
                           float alpha0, float lambda, cudaStream_t s, int64_t *launches)
{
    cudaError_t e;
    switch (d) {
    case 16: e = gramian_simple_d<16>(X, bf16, n, partials, s); break;
    case 32: e = gramian_simple_d<32>(X, bf16, n, partials, s); break;
    case 64: e = gramian_simple_d<64>(X, bf16, n, partials, s); break;
    case 128: e = gramian_simple_d<128>(X, bf16, n, partials, s); break;
    default: return cudaErrorInvalidValue;
    }
    ++*launches;
    if (e != cudaSuccess) return e;
    k_gramian_reduce<<<(d * d + 255) / 256, 256, 0, s>>>(partials, gramian_partials(n), d, G64, Bmat, alpha0, lambda);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace alx

// ---- FP32 FMA throughput probe (diagnostic; gives the denominator of the ALU roofline) ------------
namespace alx {
namespace {
__global__ void __launch_bounds__(256) k_ffma_probe(float *out, int iters)
{
    float a[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) a[k] = 1.0f + 1e-3f * (float)(threadIdx.x + k);
    const float m = 0.999999f, c = 1e-7f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int k = 0; k < 16; ++k) a[k] = fmaf(a[k], m, c);
    }
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < 16; ++k) s += a[k];
    if (s == 12345.678f) out[0] = s;   // keeps the loop alive; practically never taken
}
}  // namespace

cudaError_t measure_fp32_peak(double *tflops, cudaStream_t s)
{
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    float *out = nullptr;
    cudaError_t e = cudaMalloc(&out, 256);
    if (e != cudaSuccess) return e;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const int iters = 1 << 16, grid = sms * 8;
    double best = 0.0;
    for (int rep = 0; rep < 4; ++rep) {
        cudaEventRecord(e0, s);
        k_ffma_probe<<<grid, 256, 0, s>>>(out, iters);
        cudaEventRecord(e1, s);
        cudaEventSynchronize(e1);
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double fl = 2.0 * 16.0 * (double)iters * 256.0 * (double)grid;
        if (rep > 0 && ms > 0.f && fl / (ms * 1e-3) * 1e-12 > best) best = fl / (ms * 1e-3) * 1e-12;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(out);
    *tflops = best;
    return cudaGetLastError();
}
}  // namespace alx

// ---- Gramian without any allocation ---------------------------------------------------------------
// For callers that must not allocate device memory at the time of the call: code running inside a
// memory pool that has been frozen, a host thread that may not take the allocator's lock, a service
// whose memory budget was fixed at start-up.  The piece sums that the context-based path keeps in a
// buffer it allocates live here in a fixed array that is part of the library image, so every GPU that
// loads the library carries kNoAllocScratchFloats * 4 bytes (16 MiB + 64 KiB) until the process exits.
namespace alx {
namespace {

constexpr int64_t kNoAllocPieceFloats = 4ll << 20;                       // room for the piece sums
constexpr int64_t kNoAllocScratchFloats = kNoAllocPieceFloats + 128 * 128;  // + one d x d fp32 by-product
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocScratchFloats];

constexpr int kNoAllocMaxDevices = 64;
float *g_noalloc_ptr[kNoAllocMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_noalloc_mutex;
thread_local std::string g_noalloc_error;

alx_status noalloc_fail(alx_status code, const std::string &msg)
{
    g_noalloc_error = msg;
    return code;
}

}  // namespace
}  // namespace alx

extern "C" {

int64_t alx_gramian_noalloc_max_rows(int32_t d)
{
    if (d != 16 && d != 32 && d != 64 && d != 128) return 0;
    return (alx::kNoAllocPieceFloats / ((int64_t)d * d)) * alx::kGramRowsPerPartial;
}

const char *alx_noalloc_last_error(void) { return alx::g_noalloc_error.c_str(); }

alx_status alx_gramian_noalloc(const void *table, alx_dtype dtype, int64_t n, int32_t d, double *gramian,
                               void *stream)
{
    using namespace alx;
    if (!table || !gramian || n < 1 || (dtype != ALX_F32 && dtype != ALX_BF16))
        return noalloc_fail(ALX_ERR_INVALID_ARG, "alx_gramian_noalloc: null pointer, n < 1 or unknown dtype");
    if (d != 16 && d != 32 && d != 64 && d != 128)
        return noalloc_fail(ALX_ERR_UNSUPPORTED, "alx_gramian_noalloc: d must be 16, 32, 64 or 128");
    // the kernels read the table in 16-byte pieces and write doubles: a pointer that is not aligned for that would
    // fault on the device instead of being refused here
    if ((reinterpret_cast<uintptr_t>(table) & 15u) != 0 || (reinterpret_cast<uintptr_t>(gramian) & 7u) != 0)
        return noalloc_fail(ALX_ERR_INVALID_ARG,
                            "alx_gramian_noalloc: table must be 16-byte aligned and gramian 8-byte aligned");
    const int64_t max_rows = alx_gramian_noalloc_max_rows(d);
    if (n > max_rows)
        return noalloc_fail(ALX_ERR_UNSUPPORTED,
                            "alx_gramian_noalloc: " + std::to_string(n) + " rows exceed the fixed scratch array (at most " +
                                std::to_string(max_rows) + " rows for d = " + std::to_string(d) +
                                "); use a context and alx_gramian instead");
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices)
        return noalloc_fail(ALX_ERR_CUDA, "alx_gramian_noalloc: no current CUDA device");
    float *scratch = nullptr;
    {
        // set-up, once per device, with that device current: the array's name is only a handle in host
        // code; the kernels need its device address
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_ptr[dev]) {
            void *p = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (e != cudaSuccess || !p)
                return noalloc_fail(ALX_ERR_CUDA, std::string("alx_gramian_noalloc: cudaGetSymbolAddress failed: ") +
                                                      cudaGetErrorString(e));
            g_noalloc_ptr[dev] = static_cast<float *>(p);
        }
        scratch = g_noalloc_ptr[dev];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float *pieces = scratch, *base_out = scratch + kNoAllocPieceFloats;
    cudaError_t e;
    const int bf16 = dtype == ALX_BF16;
    switch (d) {
    case 16: e = gramian_simple_d<16>(table, bf16, n, pieces, s); break;
    case 32: e = gramian_simple_d<32>(table, bf16, n, pieces, s); break;
    case 64: e = gramian_simple_d<64>(table, bf16, n, pieces, s); break;
    default: e = gramian_simple_d<128>(table, bf16, n, pieces, s); break;
    }
    if (e == cudaSuccess) {
        // every piece the reduction reads was written in full by the launch above: nothing has to start at zero
        k_gramian_reduce<<<(d * d + 255) / 256, 256, 0, s>>>(pieces, gramian_partials(n), d, gramian, base_out, 0.f, 0.f);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess)
        return noalloc_fail(ALX_ERR_CUDA, std::string("alx_gramian_noalloc: launch failed: ") + cudaGetErrorString(e));
    g_noalloc_error.clear();
    return ALX_OK;
}

}  // extern "C"
