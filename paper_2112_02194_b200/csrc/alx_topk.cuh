// Selection shared by the Top-K scoring kernels (see alx_eval.cu).
#pragma once
#include <cstdint>

namespace alx {

constexpr int kTopkQueries = 128;      // queries per block (= threads of the selection)

__device__ __forceinline__ bool excluded(const int64_t *ex_ptr, const int32_t *ex_idx, int64_t q, int32_t id)
{
    if (!ex_ptr) return false;
    int64_t lo = ex_ptr[q], hi = ex_ptr[q + 1];
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        const int32_t v = ex_idx[mid];
        if (v == id) return true;
        if (v < id) lo = mid + 1; else hi = mid;
    }
    return false;
}

// One query's list of the best k so far, sorted by (score descending, id ascending).  Items arrive in ascending id, so a
// newcomer goes behind every element of equal score.
// (stride: distance between consecutive elements of the list, 1 in global memory; in shared memory the lists of a
// block's 128 queries are interleaved, element p of query t at p * 128 + t, so that no two threads share a bank)
struct TopList {
    float *s;
    int32_t *id;
    int k, cnt;
    float tau;      // score of the k-th element once the list is full
    int stride;
    __device__ __forceinline__ bool wants(float v) const { return cnt < k ? (v == v) : v > tau; }
    __device__ __forceinline__ void insert(float v, int32_t item)
    {
        int pos = cnt < k ? cnt : k - 1;
        while (pos > 0 && s[(pos - 1) * stride] < v) {
            s[pos * stride] = s[(pos - 1) * stride];
            id[pos * stride] = id[(pos - 1) * stride];
            --pos;
        }
        s[pos * stride] = v;
        id[pos * stride] = item;
        if (cnt < k) ++cnt;
        if (cnt == k) tau = s[(k - 1) * stride];
    }
};


}  // namespace alx
