// Factor-and-solve of one row's bordered normal matrix in shared memory, shared by the FP32-ALU row
// kernels and the tensor-core row kernels (Eq. 4; Alg. 1 line 10).  A group of kThreads threads that
// synchronise on a named barrier works on one matrix, so several groups can live in one block.
#pragma once

#include "alx_common.cuh"

namespace alx {

constexpr int kThreads = 256;   // threads per solver group
constexpr int kStage = 32;      // gathered rows staged per step (FP32-ALU path)

__device__ __forceinline__ void group_sync(int bar_id)
{
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(kThreads) : "memory");
}

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
// All kThreads threads of the group must call (tid = index inside the group, bar_id = the group's named
// barrier).  Returns false (to every thread) if a pivot was not positive.
// ------------------------------------------------------------------------------------------------
template <int D>
__device__ bool cholesky_solve(float *__restrict__ As, float *__restrict__ Pt, float *__restrict__ dinv,
                               float (&xq)[(D + 31) / 32], int tid, int bar_id, volatile int *s_bad_ptr)
{
    constexpr int TT = Geo<D>::TT, LDA = Geo<D>::LDA, LDP = Geo<D>::LDP;
    const int lane = tid & 31, warp = tid >> 5;
    const int ty = tid >> 4, tx = tid & 15;
    volatile int &s_bad = *s_bad_ptr;
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
                float inv = ok ? rsqrtf(pj) : 0.f;
                inv = inv * fmaf(-0.5f * pj * inv, inv, 1.5f);   // one Newton step: full fp32 accuracy
                const float sq = pj * inv;
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
        group_sync(bar_id);
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
        group_sync(bar_id);
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
        group_sync(bar_id);
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
    const int lane = threadIdx.x & 31;   // the caller is the first warp of its solver group
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

}  // namespace alx
