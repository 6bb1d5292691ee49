// Rows with at most 32 observations, d = 128, bfloat16 tables: Eq. 4 solved in its dual form.
//
// With B = alpha0 G + lambda I (the same for every row, Alg. 1 line 5) and H_u the k x d matrix of the row's
// observed fixed-side embeddings, the push-through identity gives
//     w_u = (B + H_u^T H_u)^-1 H_u^T y_u = B^-1 H_u^T (I_k + H_u B^-1 H_u^T)^-1 y_u ,
// an exact restatement of Eq. 4 whose linear system is k x k instead of d x d.  B^-1 is computed once per
// half-step (fp64, one block), the k x d products Z_u = H_u B^-1 of 8 (or 4) rows at a time are one
// 128 x 128 x 128 tensor-core product (rows padded to 16 (or 32) observations with zero embeddings, B^-1 split
// into three bfloat16 parts), and per row: S_u = I + Z_u H_u^T (FP32 FMAs), S_u t = y_u by the in-warp Cholesky
// the primal kernel uses for its diagonal blocks (padding rows are rows of the identity), w_u = Z_u^T t.
// Four instances: rows of 1 .. 4 observations (eight rows per warp), 5 .. 8 (four), 9 .. 16 (two) and 17 .. 32 (one row per warp).
// The form is used only while B is well conditioned (its error grows with cond(B), which the primal form
// avoids): k_binv_prepare sets a flag from ||B||_F ||B^-1||_F, the dual kernel does nothing when it is clear,
// and the primal kernel then takes these rows as well.
//
// One persistent block per SM; three tiles of 128 padded observations in flight (shared-memory tile + 128 tensor-memory
// columns each); roles as in the primal kernel: 4 producer warps (gather, 16-byte cp.async into the K-major,
// 128-byte-swizzled operand layout), 1 MMA warp, 3 solver groups of 128 threads (thread = tensor-memory lane =
// one padded observation).  Every wait is bounded; a block that gives up sets a status flag and returns.
#include "alx_common.cuh"
#include "alx_ptx.cuh"

namespace alx {

namespace {

using namespace ptx;

constexpr int D = 128;
constexpr int kMaxTileRows = 32;              // matrix rows per tile at most: 128 / (observations per row after padding)
constexpr int kSlots = 3;                     // tiles in flight
constexpr int kTileBytes = 128 * D * 2;       // 128 padded observations x 128 features, bf16: two 64-feature panels
constexpr int kPanelBytes = kTileBytes / 2;
constexpr int kBinvBytes = 3 * kTileBytes;    // three bfloat16 parts of B^-1
constexpr int kProducerWarps = 4;
constexpr int kGroupThreads = 128;
constexpr int kSolverThreads = kSlots * kGroupThreads;
constexpr int kMmaWarp = kSolverThreads / 32;
constexpr int kBlockThreads = kSolverThreads + 32 + kProducerWarps * 32;

// byte offset of element (row, feature) inside a K-major tile with 128-byte swizzle: rows of 64 features
// (128 bytes), groups of 8 rows (1024 bytes), the 16-byte chunk index XORed with the row's index in its group
__host__ __device__ constexpr uint32_t tile_offset(int row, int feature)
{
    return (uint32_t)((feature >> 6) * kPanelBytes + (row >> 3) * 1024 + (row & 7) * 128 +
                      ((((feature & 63) >> 3) ^ (row & 7)) << 4) + (feature & 7) * 2);
}

// bf16 operands, fp32 accumulator, both operands K-major
__host__ __device__ constexpr uint32_t idesc_bf16_k_major(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------------------
// B^-1 in fp64 by Cholesky (one block of 128 threads, thread i = row i), written as three bfloat16 parts in the
// operand layout of the dual kernel; flag = 1 if B is positive definite and ||B||_F ||B^-1||_F <= cond_limit,
// 2 if it is positive definite but beyond the limit and the caller can use the dual solutions as start vectors, else 0
// (the product is 128 for a multiple of the identity).
__global__ void __launch_bounds__(128, 1) k_binv_prepare(const float *__restrict__ Bmat, unsigned char *__restrict__ tiles,
                                                         int *__restrict__ flag, double cond_limit, int allow_start)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *A = reinterpret_cast<double *>(smem_raw);          // [128][129]: lower = L, strict upper = (L^-1)^T
    double *dinv = A + D * (D + 1);                            // [128]: 1 / L[i][i]
    double *red = dinv + D;                                    // [128]
    __shared__ int s_ok;
    constexpr int LD = D + 1;
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
    // right-looking Cholesky, lower triangle
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
    // column i of L^-1 (stored transposed in the strict upper triangle: A[i][r] = Linv[r][i], r > i)
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
        const float v = (float)s;
        // three bfloat16 parts: the first rounds to nearest, the others keep the leading 8 bits of what is left
        const __nv_bfloat16 p1 = __float2bfloat16_rn(v);
        const float r1 = v - __bfloat162float(p1);
        const uint32_t m2 = __float_as_uint(r1) & 0xFFFF0000u;
        const float r2 = r1 - __uint_as_float(m2);
        const uint32_t m3 = __float_as_uint(r2) & 0xFFFF0000u;
        const uint32_t off = tile_offset(i, c);        // operand row n = i, K index = c  (B^-1 is symmetric)
        *reinterpret_cast<__nv_bfloat16 *>(tiles + off) = p1;
        *reinterpret_cast<unsigned short *>(tiles + kTileBytes + off) = (unsigned short)(m2 >> 16);
        *reinterpret_cast<unsigned short *>(tiles + 2 * kTileBytes + off) = (unsigned short)(m3 >> 16);
    }
    __syncthreads();
    dinv[i] = fro_inv;       // dinv is no longer needed
    __syncthreads();
    if (i == 0) {
        double a = 0.0, b = 0.0;
        for (int k = 0; k < D; ++k) { a += red[k]; b += dinv[k]; }
        *flag = !s_ok ? 0 : (sqrt(a) * sqrt(b) <= cond_limit) ? 1 : (allow_start ? 2 : 0);
    }
}

// ---------------------------------------------------------------------------------------------------------
struct DualParams {
    SideView sv;
    const __nv_bfloat16 *X;        // fixed table [N x 128]
    const unsigned char *binv;     // three operand tiles of B^-1
    const int *flag;
    const CgPolicy *route;         // rows of 17 .. 32 observations: nothing to do when the whole-rows kernel takes them
    int64_t first;                 // position in sv.order of the first row of the class
    int64_t count;                 // rows of the class
    int64_t n_tiles;
    RowOut out;
    DevStatus *st;
};

struct __align__(1024) DualSmem {
    unsigned char binv[kBinvBytes];
    unsigned char h[kSlots][kTileBytes];     // after a tile's S matrices are formed: scratch of its solver group
    uint64_t full[kSlots], empty[kSlots], acc_full[kSlots], acc_empty[kSlots];
    // KP = 16: scratch of a solver group's factorisation (exchange buffers and L), apart from the tile, so that the
    // tile's slot is refilled while the group factors, solves and forms w (KP = 32 needs 18 KB per group, which does
    // not fit: there the scratch takes the tile's place after the S products, and the slot is released at the end)
    float scratch16[kSlots][8 * 64 + 8 * 256];
    uint32_t tmem_base;
    int abort_flag;
    int stop[kSlots];
    int row_u[kSlots][kMaxTileRows];         // matrix row ids of the tile (-1: none)
    int row_k[kSlots][kMaxTileRows];         // their numbers of observations
    float y[kSlots][128];                    // labels of the padded observations (0 for padding)
};

__device__ __forceinline__ float rsqrt_fast(float x)
{
    float r;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// Cholesky of a KP x KP matrix held one row per lane (KP = 16: row l = lane & 15 in d[0 .. l], both half-warps of
// the warp at once on their own matrices; KP = 32: row l = lane); b is carried along as one more column.  Two
// pivots per round; the two new columns go through shared memory (xch: 4 KP floats per matrix, double buffered).
// On return lane l holds row l of L in d[0 .. l], its component of L^-1 b in b and 1 / L[l][l] in my_inv.
template <int KP> __device__ __forceinline__ bool factor_rows(float (&d)[KP], float &b, float &my_inv, int lane, float *xch)
{
    const int hb = lane & (32 - KP), l = lane & (KP - 1);      // first lane of my matrix, my row of it
    bool all_ok = true;
#pragma unroll
    for (int j = 0; j < KP; j += 2) {
        const float p00 = __shfl_sync(0xFFFFFFFFu, d[j], hb + j);
        const float p10 = __shfl_sync(0xFFFFFFFFu, d[j], hb + j + 1);
        const float p11 = __shfl_sync(0xFFFFFFFFu, d[j + 1], hb + j + 1);
        const float bj = __shfl_sync(0xFFFFFFFFu, b, hb + j);
        const float bj1 = __shfl_sync(0xFFFFFFFFu, b, hb + j + 1);
        const bool ok0 = p00 > 0.f;
        const float inv0 = ok0 ? rsqrt_fast(p00) : 0.f;
        const float l10 = p10 * inv0;
        const float q11 = fmaf(-l10, l10, p11);
        const bool ok1 = q11 > 0.f;
        const float inv1 = ok1 ? rsqrt_fast(q11) : 0.f;
        all_ok = all_ok && ok0 && ok1;
        const float zj = bj * inv0;
        const float zj1 = fmaf(-l10, zj, bj1) * inv1;
        const float x0 = d[j] * inv0;
        const float x1 = fmaf(-x0, l10, d[j + 1]) * inv1;
        const bool below = l > j + 1;
        d[j] = (l == j) ? p00 * inv0 : ((l == j + 1) ? l10 : x0);
        d[j + 1] = (l == j + 1) ? q11 * inv1 : x1;
        my_inv = (l == j) ? inv0 : ((l == j + 1) ? inv1 : my_inv);
        const float m0 = below ? x0 : 0.f, m1 = below ? x1 : 0.f;
        const float bdown = fmaf(-m1, zj1, fmaf(-m0, zj, b));
        b = (l == j) ? zj : ((l == j + 1) ? zj1 : bdown);
        if (j < KP - 2) {
            float *xb = &xch[(j & 2) * KP];
            xb[l] = x0;
            xb[KP + l] = x1;
            __syncwarp();
#pragma unroll
            for (int q4 = (j + 2) / 4; q4 < KP / 4; ++q4) {
                const float4 u4 = *reinterpret_cast<const float4 *>(&xb[4 * q4]);
                const float4 v4 = *reinterpret_cast<const float4 *>(&xb[KP + 4 * q4]);
                const float c0[4] = {u4.x, u4.y, u4.z, u4.w}, c1[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int c = 4 * q4 + e;
                    if (c >= j + 2) d[c] = fmaf(-m1, c1[e], fmaf(-m0, c0[e], d[c]));
                }
            }
        }
    }
    return all_ok;
}

// sum over the 16 lanes of a half-warp of v[c], for 16 values at once: lane l (of its half-warp) returns column l
__device__ __forceinline__ float halfwarp_reduce16(float (&v)[16], int lane)
{
    float t8[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const bool up = (lane & 8) != 0;
        const float send = up ? v[c] : v[c + 8];
        const float keep = up ? v[c + 8] : v[c];
        t8[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
    }
    float t4[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const bool up = (lane & 4) != 0;
        const float send = up ? t8[c] : t8[c + 4];
        const float keep = up ? t8[c + 4] : t8[c];
        t4[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
    }
    float t2[2];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const bool up = (lane & 2) != 0;
        const float send = up ? t4[c] : t4[c + 2];
        const float keep = up ? t4[c + 2] : t4[c];
        t2[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 2);
    }
    const bool up = (lane & 1) != 0;
    const float send = up ? t2[0] : t2[1];
    const float keep = up ? t2[1] : t2[0];
    return keep + __shfl_xor_sync(0xFFFFFFFFu, send, 1);
}

// sum over 4 lanes of v[c], for 16 values at once: lane l (of its four) returns columns 4 l .. 4 l + 3
__device__ __forceinline__ void eighthwarp_reduce16(float (&v)[16], int lane, float (&r)[4])
{
    float t8[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const bool up = (lane & 2) != 0;
        const float send = up ? v[c] : v[c + 8];
        const float keep = up ? v[c + 8] : v[c];
        t8[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 2);
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const bool up = (lane & 1) != 0;
        const float send = up ? t8[c] : t8[c + 4];
        const float keep = up ? t8[c + 4] : t8[c];
        r[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 1);
    }
}

// sum over the 8 lanes of a quarter-warp of v[c], for 16 values at once: lane l (of its eight) returns columns 2 l, 2 l + 1
__device__ __forceinline__ void quarterwarp_reduce16(float (&v)[16], int lane, float &r0, float &r1)
{
    float t8[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const bool up = (lane & 4) != 0;
        const float send = up ? v[c] : v[c + 8];
        const float keep = up ? v[c + 8] : v[c];
        t8[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
    }
    float t4[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const bool up = (lane & 2) != 0;
        const float send = up ? t8[c] : t8[c + 4];
        const float keep = up ? t8[c + 4] : t8[c];
        t4[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 2);
    }
    float t2[2];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const bool up = (lane & 1) != 0;
        const float send = up ? t4[c] : t4[c + 2];
        const float keep = up ? t4[c + 2] : t4[c];
        t2[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 1);
    }
    r0 = t2[0];
    r1 = t2[1];
}

// Producer warp pw fills padded observations 32 pw .. 32 pw + 31 of every tile.  The index loads of a tile form a
// chain of three dependent loads (row id from the order, its offsets, its column ids); they are issued one, two
// and three tiles ahead, so that none of them is waited for.  A tile is announced once the next one has been
// issued (or at once when the warp would otherwise block).
template <int KP> __device__ void dual_producer(const DualParams &p, DualSmem &sm, int pw, int lane)
{
    constexpr int kTileRows = 128 / KP;
    const int mr = (32 * pw + lane) / KP, j = lane & (KP - 1);     // my matrix row of the tile, my observation of it
    const int c = lane & 15;                                        // 16-byte chunk of the 256-byte embedding
    const int64_t stride = gridDim.x;
    // pipeline registers: tile t+1 (ids loaded), tile t+2 (offsets loaded), tile t+3 (row id loaded)
    int32_t u1 = -1, idx1 = -1, u2 = -1, u3 = -1;
    int k1 = 0;
    float y1 = 0.f;
    int64_t beg2 = 0, end2 = 0;
    auto load_u = [&](int64_t t) -> int32_t {
        const int64_t r = t * kTileRows + mr;
        return (t < p.n_tiles && r < p.count) ? p.sv.order[p.first + r] : -1;
    };
    auto load_ptr = [&](int32_t u, int64_t &beg, int64_t &end) {
        beg = end = 0;
        if (u >= 0) { beg = p.sv.ptr[u]; end = p.sv.ptr[u + 1]; }
    };
    auto load_idx = [&](int32_t u, int64_t beg, int64_t end, int32_t &idx, float &y, int &k) {
        k = (int)(end - beg);
        idx = -1;
        y = 0.f;
        if (u >= 0 && j < k) {
            idx = p.sv.idx[beg + j];
            y = p.sv.val ? p.sv.val[beg + j] : 1.f;
        }
    };
    {   // fill the pipeline for the first tile of this block
        const int64_t t0 = blockIdx.x;
        u1 = load_u(t0);
        int64_t b1, e1;
        load_ptr(u1, b1, e1);
        load_idx(u1, b1, e1, idx1, y1, k1);
        u2 = load_u(t0 + stride);
        load_ptr(u2, beg2, end2);
        u3 = load_u(t0 + 2 * stride);
    }
    int64_t it = 0;
    int pending = -1;      // slot of the tile issued but not yet announced
    for (int64_t t = blockIdx.x; t < p.n_tiles; t += stride, ++it) {
        const int slot = (int)(it % kSlots);
        const uint32_t ph = (uint32_t)((it / kSlots) & 1);
        // this tile's values, then advance the pipeline by one tile (nothing loaded here is used before the next trip)
        const int32_t u = u1, my_idx = idx1;
        const int k = k1;
        const float my_y = y1;
        u1 = u2;
        load_idx(u2, beg2, end2, idx1, y1, k1);
        u2 = u3;
        load_ptr(u3, beg2, end2);
        u3 = load_u(t + 3 * stride);

        {
            int free_now = 1;
            if (lane == 0) free_now = mbar_test_wait(&sm.empty[slot], ph ^ 1u) ? 1 : 0;
            free_now = __shfl_sync(0xFFFFFFFFu, free_now, 0);
            if (!free_now && pending >= 0) {
                cp_async_wait<0>();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.full[pending]);
                pending = -1;
            }
        }
        if (!mbar_wait_parked_warp(&sm.empty[slot], ph ^ 1u, &sm.abort_flag, 110)) break;
        sm.y[slot][32 * pw + lane] = my_y;
        if (j == 0) { sm.row_u[slot][mr] = u; sm.row_k[slot][mr] = k; }
        const uint32_t tile = smem_u32(&sm.h[slot][0]);
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int rr = 2 * q + (lane >> 4);   // observation inside this warp's 32
            const int32_t src = __shfl_sync(0xFFFFFFFFu, my_idx, rr);
            const uint32_t dst = tile + tile_offset(32 * pw + rr, 8 * c);
            if (src >= 0) cp_async16(dst, p.X + (int64_t)src * D + c * 8);
            else st_shared_zero16(dst);
        }
        cp_async_commit();
        if (pending >= 0) {
            cp_async_wait<1>();
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.full[pending]);
        }
        pending = slot;
    }
    cp_async_wait<0>();
    if (pending >= 0) {
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.full[pending]);
    }
}

__device__ void dual_mma(const DualParams &p, DualSmem &sm, int lane)
{
    constexpr uint32_t kIdesc = idesc_bf16_k_major(128, 128);
    int64_t it = 0;
    for (int64_t t = blockIdx.x; t < p.n_tiles; t += gridDim.x, ++it) {
        const int slot = (int)(it % kSlots);
        const uint32_t ph = (uint32_t)((it / kSlots) & 1);
        if (!mbar_wait_parked_warp(&sm.full[slot], ph, &sm.abort_flag, 120)) break;
        if (!mbar_wait_parked_warp(&sm.acc_empty[slot], ph ^ 1u, &sm.abort_flag, 121)) break;    // the slot's accumulator is free
        tc_fence_after();
        if (lane == 0) {
            const uint32_t hb = smem_u32(&sm.h[slot][0]);
            const uint32_t bb = smem_u32(&sm.binv[0]);
            const uint32_t d_tmem = sm.tmem_base + slot * D;
            bool first = true;
            for (int q = 0; q < 3; ++q) {
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t koff = (uint32_t)((ks >> 2) * kPanelBytes + (ks & 3) * 32);
                    const uint64_t adesc = smem_desc(hb + koff, 16, 1024, 2);
                    const uint64_t bdesc = smem_desc(bb + q * kTileBytes + koff, 16, 1024, 2);
                    umma_f16(d_tmem, adesc, bdesc, kIdesc, !first);
                    first = false;
                }
            }
            umma_commit(&sm.acc_full[slot]);
        }
        __syncwarp();
    }
}

template <int KP> __device__ void dual_solver(const DualParams &p, DualSmem &sm, int g, int tid)
{
    const int lane = tid & 31, w = tid >> 5;
    const int m = tid;                         // my padded observation = tensor-memory lane
    const int mr = m / KP, j = m & (KP - 1);   // matrix row of the tile, observation of that row
    const int bar_id = 1 + g;
    const uint32_t trow = sm.tmem_base + ((uint32_t)(w * 32) << 16) + g * D;
    int64_t it = 0;
    for (int64_t t = blockIdx.x; t < p.n_tiles; t += gridDim.x, ++it) {
        if ((int)(it % kSlots) != g) continue;
        const uint32_t ph = (uint32_t)((it / kSlots) & 1);
        if (tid == 0) sm.stop[g] = mbar_wait_parked(&sm.acc_full[g], ph, &sm.abort_flag, 130) ? 0 : 1;
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        if (sm.stop[g]) break;
        tc_fence_after();
        const int u = sm.row_u[g][mr];
        const int k_u = sm.row_k[g][mr];
        int kmax = k_u;                                       // warp-uniform: the longest of this warp's rows
#pragma unroll
        for (int o = KP; o < 32; o <<= 1) {
            const int k_other = __shfl_xor_sync(0xFFFFFFFFu, kmax, o);
            kmax = kmax > k_other ? kmax : k_other;
        }
        // S row: s[j'] = sum_f Z[me][f] H[row mr, observation j'][f]
        float s[KP];
#pragma unroll
        for (int c = 0; c < KP; ++c) s[c] = 0.f;
        // rows of my matrix row start at a multiple of 8 rows: the swizzle term of row KP mr + jj is jj & 7, known
        // at compile time, and the row's offset is one runtime base plus constants
        const unsigned char *tile = &sm.h[g][0] + (KP * mr / 8) * 1024;
        const int rsub = (KP < 8) ? (KP * mr) & 7 : 0;      // four observations per row: two rows share a group of 8 tile rows
        float z[16], zn[16];
        tmem_ld16(trow, z);
        // not unrolled: the body is KP dot products of 16 terms; eight copies of it would not fit the instruction cache
#pragma unroll 1
        for (int cf = 0; cf < D / 16; ++cf) {
            if (cf + 1 < D / 16) tmem_ld16_nowait(trow + 16 * (cf + 1), zn);      // lands while this chunk is used
            if constexpr (KP <= 32) {      // (every instance; the one-observation-per-trip form below is kept for reference)
#pragma unroll
                for (int jj = 0; jj < KP; jj += 2) {
                    // two observations per trip and two partial sums each: four independent chains of packed FMAs (one
                    // chain of eight per observation left the warp waiting on its own results); an odd kmax spends one
                    // product on a padding row, which holds zeros
                    if (jj < kmax) {
                        float2 acc[2][2];
#pragma unroll
                        for (int t = 0; t < 2; ++t) {
                            const int jt = jj + t;
                            const int jr = jt + rsub;      // (row of the observation inside its group of 8 tile rows, for KP < 8)
                            const int base = (cf >> 2) * kPanelBytes + (jr >> 3) * 1024 + (jr & 7) * 128;
                            const int c0 = (cf & 3) * 2;
                            const uint4 h0 = *reinterpret_cast<const uint4 *>(tile + base + ((c0 ^ (jr & 7)) << 4));
                            const uint4 h1 = *reinterpret_cast<const uint4 *>(tile + base + (((c0 + 1) ^ (jr & 7)) << 4));
                            const uint32_t hw[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
                            // packed FP32 FMAs: even features in .x, odd features in .y (a bfloat16 pair unpacks to exactly that)
                            acc[t][0] = make_float2(s[jt], 0.f);
                            acc[t][1] = make_float2(0.f, 0.f);
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                acc[t][e & 1] = __ffma2_rn(make_float2(z[2 * e], z[2 * e + 1]),
                                                           make_float2(__uint_as_float(hw[e] << 16), __uint_as_float(hw[e] & 0xFFFF0000u)),
                                                           acc[t][e & 1]);
                        }
#pragma unroll
                        for (int t = 0; t < 2; ++t) s[jj + t] = (acc[t][0].x + acc[t][1].x) + (acc[t][0].y + acc[t][1].y);
                    }
                }
            } else {
#pragma unroll
                for (int jj = 0; jj < KP; ++jj) {
                    if (jj < kmax) {
                        const int base = (cf >> 2) * kPanelBytes + (jj >> 3) * 1024 + (jj & 7) * 128;
                        const int c0 = (cf & 3) * 2;
                        const uint4 h0 = *reinterpret_cast<const uint4 *>(tile + base + ((c0 ^ (jj & 7)) << 4));
                        const uint4 h1 = *reinterpret_cast<const uint4 *>(tile + base + (((c0 + 1) ^ (jj & 7)) << 4));
                        const uint32_t hw[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
                        // packed FP32 FMAs: even features in .x, odd features in .y (a bfloat16 pair unpacks to exactly that)
                        float2 acc = make_float2(s[jj], 0.f);
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            acc = __ffma2_rn(make_float2(z[2 * e], z[2 * e + 1]),
                                             make_float2(__uint_as_float(hw[e] << 16), __uint_as_float(hw[e] & 0xFFFF0000u)), acc);
                        s[jj] = acc.x + acc.y;
                    }
                }
            }
            if (cf + 1 < D / 16) {
                tmem_ld_wait16(zn);
#pragma unroll
                for (int c = 0; c < 16; ++c) z[c] = zn[c];
            }
        }
        // S = I + (the k x k block); padding observations are rows of the identity with a zero label
        float d[KP];
        const bool mine = j < k_u;
#pragma unroll
        for (int c = 0; c < KP; ++c) d[c] = ((mine && c < k_u) ? s[c] : 0.f) + ((c == j) ? 1.f : 0.f);
        float b = sm.y[g][m];
        float my_inv = 0.f;
        // every thread of the group is past its reads of the tile: its memory now serves as scratch
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        if (KP <= 16 && tid == 0) mbar_arrive(&sm.empty[g]);    // the tile, its labels and row ids are not read again
        float *scratch = (KP <= 16) ? &sm.scratch16[g][0] : reinterpret_cast<float *>(&sm.h[g][0]);
        float *xch = scratch + mr * (4 * KP);                   // per matrix row
        float *Lrow = scratch + (128 / KP) * (4 * KP) + mr * (KP * KP);       // per matrix row: L, row-major
        const bool ok = factor_rows<KP>(d, b, my_inv, lane, xch);
        // back substitution L^T t = z, column by column from the end
#pragma unroll
        for (int q4 = 0; q4 < KP / 4; ++q4)
            *reinterpret_cast<float4 *>(&Lrow[j * KP + 4 * q4]) = make_float4(d[4 * q4], d[4 * q4 + 1], d[4 * q4 + 2], d[4 * q4 + 3]);
        __syncwarp();
        float tj = 0.f;
        const int hb = lane & (32 - KP);
#pragma unroll
        for (int c = KP - 1; c >= 0; --c) {
            const float tc = __shfl_sync(0xFFFFFFFFu, b * my_inv, hb + c);
            if (j == c) tj = tc;
            if (j < c) b = fmaf(-Lrow[c * KP + j], tc, b);
        }
        // w = sum over my row's observations of t * Z[observation][:]
        const bool row_ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, hb) != 0;    // the same for the lanes of a row
        const bool store = (u >= 0);
#pragma unroll 1
        for (int cf = 0; cf < D / 16; ++cf) {
            float z[16];
            tmem_ld16(trow + 16 * cf, z);
#pragma unroll
            for (int c = 0; c < 16; ++c) z[c] *= tj;
            if (KP == 32) {
                // the two halves of the row's 32 observations, lower half first
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const float other = __shfl_xor_sync(0xFFFFFFFFu, z[c], 16);
                    z[c] = (lane & 16) ? other + z[c] : z[c] + other;
                }
            }
            if constexpr (KP == 4) {
                // four observations per row: the row's four lanes end with four features each
                float w4[4];
                eighthwarp_reduce16(z, lane, w4);              // features 16 cf + 4 (lane & 3) .. + 3 of row u
                if (store) {
                    const int f = 16 * cf + 4 * (lane & 3);
#pragma unroll
                    for (int e = 0; e < 4; ++e) w4[e] = row_ok ? w4[e] : 0.f;
                    __nv_bfloat162 *dst = reinterpret_cast<__nv_bfloat162 *>(reinterpret_cast<__nv_bfloat16 *>(p.out.table) + (int64_t)u * D + f);
                    dst[0] = __floats2bfloat162_rn(w4[0], w4[1]);
                    dst[1] = __floats2bfloat162_rn(w4[2], w4[3]);
                    if (p.out.cap_slot) {
                        const int cs = p.out.cap_slot[u];
                        if (cs >= 0) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) p.out.cap_out[(int64_t)cs * D + f + e] = w4[e];
                        }
                    }
                }
            } else if constexpr (KP == 8) {
                // eight observations per row: the row's eight lanes end with two features each
                float w0, w1;
                quarterwarp_reduce16(z, lane, w0, w1);         // features 16 cf + 2 (lane & 7) and the next of row u
                if (store) {
                    const int f = 16 * cf + 2 * (lane & 7);
                    const float v0 = row_ok ? w0 : 0.f, v1 = row_ok ? w1 : 0.f;
                    *reinterpret_cast<__nv_bfloat162 *>(reinterpret_cast<__nv_bfloat16 *>(p.out.table) + (int64_t)u * D + f) =
                        __floats2bfloat162_rn(v0, v1);
                    if (p.out.cap_slot) {
                        const int cs = p.out.cap_slot[u];
                        if (cs >= 0) {
                            p.out.cap_out[(int64_t)cs * D + f] = v0;
                            p.out.cap_out[(int64_t)cs * D + f + 1] = v1;
                        }
                    }
                }
            } else {
            const float wr = halfwarp_reduce16(z, lane);       // feature 16 cf + (lane & 15) of row u
            const float wv = row_ok ? wr : 0.f;
            if (store && (KP == 16 || lane < 16)) {
                const int f = 16 * cf + (lane & 15);
                reinterpret_cast<__nv_bfloat16 *>(p.out.table)[(int64_t)u * D + f] = __float2bfloat16_rn(wv);
                if (p.out.cap_slot) {
                    const int cs = p.out.cap_slot[u];
                    if (cs >= 0) p.out.cap_out[(int64_t)cs * D + f] = wv;
                }
            }
            }
        }
        if (!row_ok && u >= 0 && j == 0) {
            atomicAdd(&p.st->not_spd, 1ull);
            raise_flag(p.st, kFlagNotSpd, u);
        }
        // the tile's shared memory and tensor-memory columns are free again
        tc_fence_before();
        asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
        if (tid == 0) {
            mbar_arrive(&sm.acc_empty[g]);
            if (KP > 16) mbar_arrive(&sm.empty[g]);
        }
    }
}

template <int KP> __global__ void __launch_bounds__(kBlockThreads, 1) k_dual(DualParams p)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *aligned = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    DualSmem &sm = *reinterpret_cast<DualSmem *>(aligned);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (*p.flag == 0) return;       // the primal kernel takes these rows (block-uniform)
    if (KP == 32 && p.route && p.route->short_rows_by_cg) return;

    if (tid == 0) {
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(&sm.full[s], kProducerWarps);
            mbar_init(&sm.empty[s], 1);
            mbar_init(&sm.acc_full[s], 1);
            mbar_init(&sm.acc_empty[s], 1);
            sm.stop[s] = 0;
        }
        sm.abort_flag = 0;
        mbar_fence_init();
    }
    for (int k = tid; k < kBinvBytes / 16; k += kBlockThreads)
        reinterpret_cast<uint4 *>(sm.binv)[k] = reinterpret_cast<const uint4 *>(p.binv)[k];
    fence_proxy_async();
    if (warp == kMmaWarp) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (warp < kMmaWarp) dual_solver<KP>(p, sm, warp / (kGroupThreads / 32), tid % kGroupThreads);
    else if (warp == kMmaWarp) dual_mma(p, sm, lane);
    else dual_producer<KP>(p, sm, warp - kMmaWarp - 1, lane);

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(sm.tmem_base, 512);
    }
    if (tid == 0 && sm.abort_flag) raise_flag(p.st, kFlagTimeout, (long long)sm.abort_flag * 1000000 + blockIdx.x);
}

static_assert(sizeof(DualSmem) + 1024 <= 232448, "shared memory of one block exceeds what an SM offers");

template <int KP> cudaError_t launch_dual_instance(DualParams p, int sms, cudaStream_t s, int64_t *launches)
{
    if (p.count <= 0) return cudaSuccess;
    p.n_tiles = (p.count + 128 / KP - 1) / (128 / KP);
    const size_t smem = sizeof(DualSmem) + 1024;
    cudaError_t e = cudaFuncSetAttribute(k_dual<KP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int grid = (int)(p.n_tiles < sms ? p.n_tiles : (sms > 0 ? sms : 1));
    k_dual<KP><<<grid, kBlockThreads, smem, s>>>(p);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace

size_t dual_workspace_bytes() { return (size_t)kBinvBytes + 256; }

// B^-1 (three operand tiles at `ws`) and the flag (at ws + kBinvBytes) for the dual kernel
cudaError_t launch_dual_prepare(const float *Bmat, void *ws, float cond_limit, bool allow_start, cudaStream_t s,
                                int64_t *launches)
{
    const size_t smem = sizeof(double) * (D * (D + 1) + 2 * D);
    cudaError_t e = cudaFuncSetAttribute(k_binv_prepare, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    unsigned char *w = static_cast<unsigned char *>(ws);
    k_binv_prepare<<<1, 128, smem, s>>>(Bmat, w, reinterpret_cast<int *>(w + kBinvBytes), (double)cond_limit, allow_start ? 1 : 0);
    ++*launches;
    return cudaGetLastError();
}

const int *dual_flag_ptr(const void *ws) { return reinterpret_cast<const int *>(static_cast<const unsigned char *>(ws) + kBinvBytes); }

// rows order[first16 .. first16 + count16) of the solved side have 1 .. 16 observations each, the count32 rows after
// them 17 .. 32
cudaError_t launch_rows_dual(const SideView &sv, int64_t first16, int64_t count16, int64_t count32, const void *X,
                             const void *ws, RowOut out, DevStatus *st, const CgPolicy *route, const int32_t *order16,
                             int64_t n4, int64_t n8, cudaStream_t s, int64_t *launches)
{
    DualParams p{};
    p.route = route;
    p.sv = sv;
    p.X = reinterpret_cast<const __nv_bfloat16 *>(X);
    p.binv = static_cast<const unsigned char *>(ws);
    p.flag = dual_flag_ptr(ws);
    p.out = out;
    p.st = st;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaError_t e;
    if (order16) {
        // the rows of at most 4 and of 5 .. 8 observations (32 and 16 rows per tile), then the rest of the class
        p.sv.order = order16;
        p.first = 0;
        p.count = n4;
        e = launch_dual_instance<4>(p, sms, s, launches);
        if (e != cudaSuccess) return e;
        p.first = n4;
        p.count = n8 - n4;
        e = launch_dual_instance<8>(p, sms, s, launches);
        if (e != cudaSuccess) return e;
        p.first = n8;
        p.count = count16 - n8;
        e = launch_dual_instance<16>(p, sms, s, launches);
        if (e != cudaSuccess) return e;
        p.sv.order = sv.order;
    } else {
        p.first = first16;
        p.count = count16;
        e = launch_dual_instance<16>(p, sms, s, launches);
        if (e != cudaSuccess) return e;
    }
    p.first = first16 + count16;
    p.count = count32;
    return launch_dual_instance<32>(p, sms, s, launches);
}

}  // namespace alx
