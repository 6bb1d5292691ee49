// Integer set-up kernels: CSR validation, transpose (CSR -> CSC with ascending row ids inside a
// column), degree-class ordering of rows, chunk descriptors of long rows, prefix sums, and the
// storage-type conversion used when tables are copied in or out.
//
// The paper gives S as per-row histories; the item-side pass of Alg. 1 line 11 reads the same entries column by
// column, which needs the transpose; its dense batching (Sec. 4.3) tames the long tail
// of row lengths, which here is the job of the degree classes and the chunk descriptors.
#include "alx_common.cuh"

namespace alx {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;

__device__ __forceinline__ int64_t block_exclusive_scan(int64_t v, int64_t *total)
{
    // exclusive prefix of v over the 256 threads of the block
    __shared__ int64_t warp_sums[kScanThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int64_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int64_t base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kScanThreads / 32; ++w) {
        int64_t s = warp_sums[w];
        if (w < warp) base += s;
        tot += s;
    }
    __syncthreads();
    *total = tot;
    return base + incl - v;
}

template <typename Tin>
__global__ void __launch_bounds__(kScanThreads) k_scan_tile_sums(const Tin *__restrict__ in, int64_t n,
                                                                 int64_t *__restrict__ sums)
{
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int64_t s = 0;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k)
        if (base + k < n) s += (int64_t)in[base + k];
    int64_t tot;
    block_exclusive_scan(s, &tot);
    if (threadIdx.x == 0) sums[blockIdx.x] = tot;
}

// out[i] = sum of in[0 .. i-1] for i in [0, n]; tile_offsets may be nullptr when there is one tile
template <typename Tin>
__global__ void __launch_bounds__(kScanThreads) k_scan_apply(const Tin *__restrict__ in, int64_t n,
                                                             const int64_t *__restrict__ tile_offsets,
                                                             int64_t *__restrict__ out)
{
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanItems;
    int64_t v[kScanItems];
    int64_t s = 0;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        v[k] = (base + k < n) ? (int64_t)in[base + k] : 0;
        s += v[k];
    }
    int64_t tot;
    int64_t run = block_exclusive_scan(s, &tot) + (tile_offsets ? tile_offsets[blockIdx.x] : 0);
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        if (base + k <= n) out[base + k] = run;   // position n receives the grand total
        run += v[k];
    }
}

// ---- validation -----------------------------------------------------------------------------
__global__ void k_validate_rowptr(const int64_t *__restrict__ rowptr, int64_t n, int64_t nnz, DevStatus *st)
{
    const int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= n) return;
    const int64_t a = rowptr[u], b = rowptr[u + 1];
    if (a > b || a < 0 || b > nnz || b - a > 0x7FFFFFFFll) raise_flag(st, kFlagBadRowptr, u);
    if (u == 0 && a != 0) raise_flag(st, kFlagBadRowptr, 0);
    if (u == n - 1 && b != nnz) raise_flag(st, kFlagBadRowptr, n);
}

// largest u in [0, n) with ptr[u] <= e (ptr non-decreasing, ptr[0] = 0 <= e)
__device__ __forceinline__ int64_t row_of_entry(const int64_t *__restrict__ ptr, int64_t n, int64_t e)
{
    int64_t lo = 0, hi = n;   // answer in [lo, hi)
    while (hi - lo > 1) {
        const int64_t mid = lo + ((hi - lo) >> 1);
        if (ptr[mid] <= e) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void k_validate_cols(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                                int64_t n_rows, int64_t n_cols, int64_t nnz, DevStatus *st)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= nnz) return;
    const int32_t c = colidx[e];
    if (c < 0 || c >= n_cols) { raise_flag(st, kFlagBadCol, e); return; }
    if (e > 0 && colidx[e - 1] >= c) {
        // legal only if e is the first entry of a row
        const int64_t u = row_of_entry(rowptr, n_rows, e);
        if (rowptr[u] != e) raise_flag(st, kFlagUnsorted, e);
    }
}

__global__ void k_degrees(const int64_t *__restrict__ ptr, int64_t n, int32_t *__restrict__ deg)
{
    const int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (u < n) deg[u] = (int32_t)(ptr[u + 1] - ptr[u]);
}

// ---- transpose ---------------------------------------------------------------------------------
__global__ void k_count_cols(const int32_t *__restrict__ colidx, int64_t nnz, int32_t *__restrict__ counts)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < nnz) atomicAdd(&counts[colidx[e]], 1);
}

constexpr int kFillPerThread = 8;

__global__ void k_fill_transpose(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                                 int64_t n_rows, int64_t nnz, const int64_t *__restrict__ colptr,
                                 int32_t *__restrict__ cursor, int32_t *__restrict__ rowidx)
{
    const int64_t e0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kFillPerThread;
    if (e0 >= nnz) return;
    int64_t u = row_of_entry(rowptr, n_rows, e0);
    const int64_t e1 = (e0 + kFillPerThread < nnz) ? e0 + kFillPerThread : nnz;
    for (int64_t e = e0; e < e1; ++e) {
        while (rowptr[u + 1] <= e) ++u;
        const int32_t c = colidx[e];
        const int32_t k = atomicAdd(&cursor[c], 1);   // slot inside the column, any order; sorted afterwards
        rowidx[colptr[c] + k] = (int32_t)u;
    }
}

// Sorting network in which every comparator puts the smaller key at the lower index, so positions
// at or beyond `len` behave as +infinity without being stored (any len, in place).
template <typename SyncFn>
__device__ __forceinline__ void sort_network(int32_t *a, int64_t len, int tid, int nthreads, SyncFn sync)
{
    int64_t P = 1;
    while (P < len) P <<= 1;
    const int64_t half = P >> 1;
    for (int64_t k = 2; k <= P; k <<= 1) {
        const int64_t hk = k >> 1;
        for (int64_t t = tid; t < half; t += nthreads) {
            const int64_t i = (t / hk) * k + (t % hk);
            const int64_t j = i ^ (k - 1);
            if (j < len) {
                const int32_t x = a[i], y = a[j];
                if (x > y) { a[i] = y; a[j] = x; }
            }
        }
        sync();
        for (int64_t s = k >> 2; s >= 1; s >>= 1) {
            for (int64_t t = tid; t < half; t += nthreads) {
                const int64_t i = (t / s) * (2 * s) + (t % s);
                const int64_t j = i + s;
                if (j < len) {
                    const int32_t x = a[i], y = a[j];
                    if (x > y) { a[i] = y; a[j] = x; }
                }
            }
            sync();
        }
    }
}

// columns of at most 32 entries: one warp each, rank by counting (row ids in a column are distinct)
__global__ void k_sort_small(const int64_t *__restrict__ colptr, int32_t *__restrict__ rowidx,
                             const int32_t *__restrict__ cols, int64_t n_cols_in_class)
{
    const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_cols_in_class) return;
    const int32_t c = cols[w];
    const int64_t beg = colptr[c];
    const int len = (int)(colptr[c + 1] - beg);
    if (len <= 1) return;
    const int32_t v = (lane < len) ? rowidx[beg + lane] : 0x7FFFFFFF;
    int rank = 0;
    for (int o = 0; o < len; ++o) {
        const int32_t other = __shfl_sync(0xFFFFFFFFu, v, o);
        rank += (other < v) ? 1 : 0;
    }
    if (lane < len) rowidx[beg + rank] = v;
}

// columns of 33 .. 128 entries (classes 3 and 4): one warp each, four keys per lane, rank by counting over shuffles
// (about 1200 warp instructions per column; a block-wide network with a barrier per stage took ten times as long)
__global__ void k_sort_warp128(const int64_t *__restrict__ colptr, int32_t *__restrict__ rowidx,
                               const int32_t *__restrict__ cols, int64_t n_cols_in_class)
{
    const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_cols_in_class) return;
    const int32_t c = cols[w];
    const int64_t beg = colptr[c];
    const int len = (int)(colptr[c + 1] - beg);
    int32_t v[4];
    int rank[4] = {0, 0, 0, 0};
#pragma unroll
    for (int q = 0; q < 4; ++q) v[q] = (32 * q + lane < len) ? rowidx[beg + 32 * q + lane] : 0x7FFFFFFF;
#pragma unroll
    for (int q2 = 0; q2 < 4; ++q2) {
        if (32 * q2 < len) {            // warp-uniform
#pragma unroll 8
            for (int o = 0; o < 32; ++o) {
                const int32_t other = __shfl_sync(0xFFFFFFFFu, v[q2], o);
#pragma unroll
                for (int q = 0; q < 4; ++q) rank[q] += (other < v[q]) ? 1 : 0;
            }
        }
    }
    // every lane has read its keys before any lane writes (the shuffles above need all lanes); ids are distinct
#pragma unroll
    for (int q = 0; q < 4; ++q)
        if (32 * q + lane < len) rowidx[beg + rank[q]] = v[q];
}

constexpr int kSortMediumMax = 4096;

__global__ void __launch_bounds__(256) k_sort_medium(const int64_t *__restrict__ colptr,
                                                     int32_t *__restrict__ rowidx,
                                                     const int32_t *__restrict__ cols)
{
    __shared__ int32_t buf[kSortMediumMax];
    const int32_t c = cols[blockIdx.x];
    const int64_t beg = colptr[c];
    const int64_t len = colptr[c + 1] - beg;
    if (len > kSortMediumMax) return;   // not reached: the launcher routes longer columns elsewhere
    for (int64_t t = threadIdx.x; t < len; t += blockDim.x) buf[t] = rowidx[beg + t];
    __syncthreads();
    sort_network(buf, len, threadIdx.x, blockDim.x, [] { __syncthreads(); });
    for (int64_t t = threadIdx.x; t < len; t += blockDim.x) rowidx[beg + t] = buf[t];
}

__global__ void __launch_bounds__(1024) k_sort_large(const int64_t *__restrict__ colptr,
                                                     int32_t *__restrict__ rowidx,
                                                     const int32_t *__restrict__ cols)
{
    const int32_t c = cols[blockIdx.x];
    const int64_t beg = colptr[c];
    const int64_t len = colptr[c + 1] - beg;
    sort_network(rowidx + beg, len, threadIdx.x, blockDim.x, [] { __syncthreads(); });
}

// labels of the transpose: the entry (r, c) sits in row r of the CSR at the position of c, found by
// bisection because a row's columns are strictly ascending
__global__ void k_values_transpose(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                                   const float *__restrict__ values, const int64_t *__restrict__ colptr,
                                   const int32_t *__restrict__ rowidx, int64_t n_cols, int64_t nnz,
                                   float *__restrict__ values_t)
{
    const int64_t q0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * kFillPerThread;
    if (q0 >= nnz) return;
    int64_t c = row_of_entry(colptr, n_cols, q0);
    const int64_t q1 = (q0 + kFillPerThread < nnz) ? q0 + kFillPerThread : nnz;
    for (int64_t q = q0; q < q1; ++q) {
        while (colptr[c + 1] <= q) ++c;
        const int32_t r = rowidx[q];
        int64_t lo = rowptr[r], hi = rowptr[r + 1] - 1;
        while (lo < hi) {
            const int64_t mid = lo + ((hi - lo) >> 1);
            if (colidx[mid] < (int32_t)c) lo = mid + 1; else hi = mid;
        }
        values_t[q] = values[lo];
    }
}

// ---- degree classes ------------------------------------------------------------------------------
__device__ __forceinline__ int degree_class(int64_t deg, int64_t split)
{
    if (deg <= 0) return 0;
    if (deg > split) return kNClasses - 1;
    if (deg <= 16) return 1;
    const int ceil_log2 = 64 - __clzll((unsigned long long)(deg - 1));
    const int c = ceil_log2 - 3;
    return c < kNClasses - 2 ? c : kNClasses - 2;
}

constexpr int kBucketThreads = 256;

template <bool kScatter>
__global__ void __launch_bounds__(kBucketThreads) k_bucket(const int64_t *__restrict__ ptr, int64_t n,
                                                           int64_t split, int64_t n_blocks,
                                                           int64_t *__restrict__ block_counts,
                                                           const int64_t *__restrict__ block_offsets,
                                                           int32_t *__restrict__ order)
{
    __shared__ int warp_counts[kBucketThreads / 32][kNClasses];
    const int64_t u = (int64_t)blockIdx.x * kBucketThreads + threadIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cls = (u < n) ? degree_class(ptr[u + 1] - ptr[u], split) : -1;
    int rank_in_warp = 0;
#pragma unroll
    for (int c = 0; c < kNClasses; ++c) {
        const unsigned m = __ballot_sync(0xFFFFFFFFu, cls == c);
        if (cls == c) rank_in_warp = __popc(m & ((1u << lane) - 1u));
        if (lane == 0) warp_counts[warp][c] = __popc(m);
    }
    __syncthreads();
    if (!kScatter) {
        if (threadIdx.x < kNClasses) {
            int s = 0;
            for (int w = 0; w < kBucketThreads / 32; ++w) s += warp_counts[w][threadIdx.x];
            block_counts[(int64_t)threadIdx.x * n_blocks + blockIdx.x] = s;
        }
    } else if (cls >= 0) {
        int before = 0;
        for (int w = 0; w < warp; ++w) before += warp_counts[w][cls];
        order[block_offsets[(int64_t)cls * n_blocks + blockIdx.x] + before + rank_in_warp] = (int32_t)u;
    }
}

__global__ void k_class_offsets(const int64_t *__restrict__ block_offsets, int64_t n_blocks, int64_t n,
                                int64_t *__restrict__ class_offs)
{
    const int c = threadIdx.x;
    if (c < kNClasses) class_offs[c] = block_offsets[(int64_t)c * n_blocks];
    if (c == kNClasses) class_offs[c] = n;
}

__global__ void k_chunk_counts(const int64_t *__restrict__ ptr, const int32_t *__restrict__ split_rows,
                               int64_t n_split, int64_t split, int64_t *__restrict__ counts)
{
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n_split) return;
    const int32_t u = split_rows[j];
    counts[j] = (ptr[u + 1] - ptr[u] + split - 1) / split;
}

__global__ void k_chunk_fill(const int64_t *__restrict__ ptr, const int32_t *__restrict__ split_rows,
                             int64_t n_split, int64_t split, const int64_t *__restrict__ first,
                             int64_t *__restrict__ desc)
{
    const int64_t j = blockIdx.x;
    if (j >= n_split) return;
    const int32_t u = split_rows[j];
    const int64_t beg = ptr[u], end = ptr[u + 1], s0 = first[j], cnt = first[j + 1] - s0;
    for (int64_t k = threadIdx.x; k < cnt; k += blockDim.x) {
        const int64_t b = beg + k * split;
        int64_t *d = desc + (s0 + k) * 4;
        d[0] = u;
        d[1] = b;
        d[2] = (b + split < end) ? b + split : end;
        d[3] = s0 + k;
    }
}

// ---- storage conversion -----------------------------------------------------------------------
template <typename Tsrc, typename Tdst>
__global__ void k_convert(const Tsrc *__restrict__ src, Tdst *__restrict__ dst, int64_t count)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) store_elem(dst + i, to_f32(src[i]));
}

inline unsigned grid_for(int64_t n, int threads) { return (unsigned)((n + threads - 1) / threads); }

}  // namespace

// ---- host launchers -------------------------------------------------------------------------------
int64_t scan_scratch_elems(int64_t n)
{
    // per level: tile sums [T] and their exclusive scan [T + 1], T = tiles covering n + 1 outputs
    int64_t total = 0;
    int64_t tiles = (n + 1 + kScanTile - 1) / kScanTile;
    while (tiles > 1) {
        total += 2 * tiles + 1;
        tiles = (tiles + 1 + kScanTile - 1) / kScanTile;
    }
    return total + 2;
}

cudaError_t scan_exclusive(const void *in, bool in_is_i64, int64_t *out, int64_t n, int64_t *scratch,
                           int64_t scratch_elems, cudaStream_t s, int64_t *launches)
{
    if (n <= 0) return cudaMemsetAsync(out, 0, sizeof(int64_t), s);
    const int64_t tiles = (n + 1 + kScanTile - 1) / kScanTile;   // out has n + 1 positions
    const int64_t *tile_offsets = nullptr;
    if (tiles > 1) {
        if (scratch_elems < 2 * tiles + 1) return cudaErrorInvalidValue;
        int64_t *sums = scratch, *offs = scratch + tiles;
        if (in_is_i64)
            k_scan_tile_sums<int64_t><<<(unsigned)tiles, kScanThreads, 0, s>>>((const int64_t *)in, n, sums);
        else
            k_scan_tile_sums<int32_t><<<(unsigned)tiles, kScanThreads, 0, s>>>((const int32_t *)in, n, sums);
        ++*launches;
        cudaError_t e = scan_exclusive(sums, true, offs, tiles, scratch + 2 * tiles + 1,
                                       scratch_elems - (2 * tiles + 1), s, launches);
        if (e != cudaSuccess) return e;
        tile_offsets = offs;
    }
    if (in_is_i64)
        k_scan_apply<int64_t><<<(unsigned)tiles, kScanThreads, 0, s>>>((const int64_t *)in, n, tile_offsets, out);
    else
        k_scan_apply<int32_t><<<(unsigned)tiles, kScanThreads, 0, s>>>((const int32_t *)in, n, tile_offsets, out);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_validate(const int64_t *rowptr, const int32_t *colidx, int64_t n_rows, int64_t n_cols,
                            int64_t nnz, DevStatus *st, cudaStream_t s, int64_t *launches)
{
    k_validate_rowptr<<<grid_for(n_rows, 256), 256, 0, s>>>(rowptr, n_rows, nnz, st);
    ++*launches;
    if (nnz > 0) {
        k_validate_cols<<<grid_for(nnz, 256), 256, 0, s>>>(rowptr, colidx, n_rows, n_cols, nnz, st);
        ++*launches;
    }
    return cudaGetLastError();
}

// total length of the listed rows (one block; a few ten thousand rows at most)
__global__ void k_sum_row_lengths(const int64_t *__restrict__ ptr, const int32_t *__restrict__ rows, int64_t count,
                                  int64_t *__restrict__ out)
{
    __shared__ long long part[256];
    long long s = 0;
    for (int64_t k = threadIdx.x; k < count; k += 256) {
        const int32_t u = rows[k];
        s += ptr[u + 1] - ptr[u];
    }
    part[threadIdx.x] = s;
    __syncthreads();
    for (int h = 128; h > 0; h >>= 1) {
        if ((int)threadIdx.x < h) part[threadIdx.x] += part[threadIdx.x + h];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = part[0];
}

// Stable two-way partition of a list of rows by length (at most `limit` entries first, the others after them, both in
// their old order): per-block counts, a scan of the counts, then a block-wide scatter.  Blocks of 1024 positions.
constexpr int kPartBlock = 1024;
__global__ void __launch_bounds__(256) k_part_count(const int64_t *__restrict__ ptr, const int32_t *__restrict__ rows, int64_t count,
                                                    int limit, int64_t *__restrict__ block_counts)
{
    __shared__ int warp_sums[8];
    const int64_t base = (int64_t)blockIdx.x * kPartBlock;
    int mine = 0;
    for (int k = threadIdx.x; k < kPartBlock; k += 256) {
        const int64_t i = base + k;
        if (i < count) {
            const int32_t u = rows[i];
            mine += (ptr[u + 1] - ptr[u] <= limit) ? 1 : 0;
        }
    }
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, o);
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < 8; ++w) t += warp_sums[w];
        block_counts[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(256) k_part_scatter(const int64_t *__restrict__ ptr, const int32_t *__restrict__ rows, int64_t count,
                                                      int limit, const int64_t *__restrict__ block_offsets, int64_t n_blocks,
                                                      int32_t *__restrict__ out)
{
    __shared__ int warp_short[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t base = (int64_t)blockIdx.x * kPartBlock;
    const int64_t n_short_total = block_offsets[n_blocks];
    int64_t short_at = block_offsets[blockIdx.x];              // next free place among the short rows
    int64_t long_at = n_short_total + (base - short_at);       // ... and among the others (every earlier row is in one of the two)
    for (int round = 0; round < kPartBlock / 256; ++round) {
        const int64_t i = base + round * 256 + threadIdx.x;
        const bool live = i < count;
        int32_t u = 0;
        bool is_short = false;
        if (live) {
            u = rows[i];
            is_short = ptr[u + 1] - ptr[u] <= limit;
        }
        const unsigned m_short = __ballot_sync(0xFFFFFFFFu, live && is_short);
        const unsigned m_live = __ballot_sync(0xFFFFFFFFu, live);
        if (lane == 0) warp_short[warp] = __popc(m_short);
        __syncthreads();
        int short_before = 0, short_round = 0;
        for (int w = 0; w < 8; ++w) {
            if (w < warp) short_before += warp_short[w];
            short_round += warp_short[w];
        }
        const int live_before = warp * 32;                      // (a round's live threads are a prefix of the block)
        const unsigned below = (1u << lane) - 1u;
        if (live) {
            if (is_short) out[short_at + short_before + __popc(m_short & below)] = u;
            else out[long_at + (live_before - short_before) + __popc(m_live & ~m_short & below)] = u;
        }
        int live_round = 0;
        {
            const int64_t left = count - (base + round * 256);
            live_round = left >= 256 ? 256 : (left > 0 ? (int)left : 0);
        }
        short_at += short_round;
        long_at += live_round - short_round;
        __syncthreads();
    }
}

// out[0 .. count): the rows of `rows` with at most `limit` entries, then the others; *n_short_dev receives the number of the
// former (device; block_counts and block_offsets: count / 1024 + 2 int64 each)
cudaError_t launch_partition_by_length(const int64_t *ptr, const int32_t *rows, int64_t count, int limit, int32_t *out,
                                       int64_t *block_counts, int64_t *block_offsets, int64_t *n_short_dev,
                                       int64_t *scan_scratch, int64_t scan_elems, cudaStream_t s, int64_t *launches)
{
    if (count <= 0) return cudaMemsetAsync(n_short_dev, 0, sizeof(int64_t), s);
    const int64_t nb = (count + kPartBlock - 1) / kPartBlock;
    k_part_count<<<(unsigned)nb, 256, 0, s>>>(ptr, rows, count, limit, block_counts);
    ++*launches;
    cudaError_t e = scan_exclusive(block_counts, true, block_offsets, nb, scan_scratch, scan_elems, s, launches);
    if (e != cudaSuccess) return e;
    k_part_scatter<<<(unsigned)nb, 256, 0, s>>>(ptr, rows, count, limit, block_offsets, nb, out);
    ++*launches;
    e = cudaMemcpyAsync(n_short_dev, block_offsets + nb, sizeof(int64_t), cudaMemcpyDeviceToDevice, s);
    return e != cudaSuccess ? e : cudaGetLastError();
}

// doubled entry lists: one warp per row
__global__ void __launch_bounds__(256) k_double_entries(const int64_t *__restrict__ ptr, const int32_t *__restrict__ idx,
                                                        const float *__restrict__ val, int64_t n, int64_t n_fixed,
                                                        int64_t *__restrict__ vptr, int32_t *__restrict__ vidx,
                                                        float *__restrict__ vval)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * 8;
    for (int64_t u = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); u <= n; u += warps) {
        const int64_t beg = ptr[u];
        if (lane == 0) vptr[u] = 2 * beg;
        if (u == n) break;
        const int64_t len = ptr[u + 1] - beg;
        for (int64_t j = lane; j < len; j += 32) {
            const int32_t c = idx[beg + j];
            vidx[2 * beg + j] = c;
            vidx[2 * beg + len + j] = (int32_t)(c + n_fixed);
            if (val) {
                const float y = val[beg + j];
                vval[2 * beg + j] = y;
                vval[2 * beg + len + j] = y;
            }
        }
    }
}

cudaError_t launch_double_entries(const int64_t *ptr, const int32_t *idx, const float *val, int64_t n, int64_t n_fixed,
                                  int64_t *vptr, int32_t *vidx, float *vval, cudaStream_t s, int64_t *launches)
{
    const int64_t blocks = (n + 1 + 7) / 8;
    k_double_entries<<<(unsigned)(blocks < 148 * 16 ? blocks : 148 * 16), 256, 0, s>>>(ptr, idx, val, n, n_fixed, vptr, vidx, vval);
    ++*launches;
    return cudaGetLastError();
}

// entries per degree class: position k of `order` belongs to the class whose offset range holds k
__global__ void __launch_bounds__(256) k_class_entries(const int64_t *__restrict__ ptr, const int32_t *__restrict__ order,
                                                       const int64_t *__restrict__ class_offs, int64_t n,
                                                       unsigned long long *__restrict__ out)
{
    __shared__ unsigned long long part[kNClasses];
    __shared__ int64_t offs[kNClasses + 1];
    if (threadIdx.x <= kNClasses) offs[threadIdx.x] = class_offs[threadIdx.x];
    if (threadIdx.x < kNClasses) part[threadIdx.x] = 0;
    __syncthreads();
    for (int64_t k = (int64_t)blockIdx.x * 256 + threadIdx.x; k < n; k += (int64_t)gridDim.x * 256) {
        int c = 0;
        while (c + 1 < kNClasses && k >= offs[c + 1]) ++c;
        const int32_t u = order[k];
        const unsigned long long len = (unsigned long long)(ptr[u + 1] - ptr[u]);
        if (len) atomicAdd(&part[c], len);
    }
    __syncthreads();
    if (threadIdx.x < kNClasses && part[threadIdx.x]) atomicAdd(&out[threadIdx.x], part[threadIdx.x]);
}

cudaError_t launch_class_entries(const int64_t *ptr, const int32_t *order, const int64_t *class_offs_dev, int64_t n,
                                 int64_t *out, cudaStream_t s, int64_t *launches)
{
    cudaError_t e = cudaMemsetAsync(out, 0, sizeof(int64_t) * kNClasses, s);
    if (e != cudaSuccess) return e;
    const int64_t blocks = (n + 255) / 256;
    k_class_entries<<<(unsigned)(blocks < 1184 ? (blocks > 0 ? blocks : 1) : 1184), 256, 0, s>>>(
        ptr, order, class_offs_dev, n, reinterpret_cast<unsigned long long *>(out));
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_sum_row_lengths(const int64_t *ptr, const int32_t *rows, int64_t count, int64_t *out, cudaStream_t s,
                                   int64_t *launches)
{
    k_sum_row_lengths<<<1, 256, 0, s>>>(ptr, rows, count, out);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_degrees(const int64_t *ptr, int64_t n, int32_t *deg, cudaStream_t s, int64_t *launches)
{
    k_degrees<<<grid_for(n, 256), 256, 0, s>>>(ptr, n, deg);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_count_cols(const int32_t *colidx, int64_t nnz, int32_t *counts, cudaStream_t s,
                              int64_t *launches)
{
    if (nnz == 0) return cudaSuccess;
    k_count_cols<<<grid_for(nnz, 256), 256, 0, s>>>(colidx, nnz, counts);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_fill_transpose(const int64_t *rowptr, const int32_t *colidx, int64_t n_rows, int64_t nnz,
                                  const int64_t *colptr, int32_t *cursor, int32_t *rowidx, cudaStream_t s,
                                  int64_t *launches)
{
    if (nnz == 0) return cudaSuccess;
    const int64_t threads = (nnz + kFillPerThread - 1) / kFillPerThread;
    k_fill_transpose<<<grid_for(threads, 256), 256, 0, s>>>(rowptr, colidx, n_rows, nnz, colptr, cursor, rowidx);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_sort_segments(const int64_t *colptr, int32_t *rowidx, const int32_t *order,
                                 const int64_t *offs, cudaStream_t s, int64_t *launches)
{
    // classes 1-2: at most 32 entries; 3-4: at most 128; 5-9: at most 4096; 10-11: anything longer (class 11 starts at
    // split + 1, which a small split can put below 4096: the global-memory network handles any length)
    const int64_t n_small = offs[3] - offs[1];
    const int64_t n_warp = offs[5] - offs[3];        // classes 3 and 4: 33 .. 128 entries
    const int64_t n_medium = offs[10] - offs[5];
    const int64_t n_large = offs[12] - offs[10];
    if (n_small > 0) {
        k_sort_small<<<grid_for(n_small * 32, 256), 256, 0, s>>>(colptr, rowidx, order + offs[1], n_small);
        ++*launches;
    }
    if (n_warp > 0) {
        k_sort_warp128<<<grid_for(n_warp * 32, 256), 256, 0, s>>>(colptr, rowidx, order + offs[3], n_warp);
        ++*launches;
    }
    if (n_medium > 0) {
        k_sort_medium<<<(unsigned)n_medium, 256, 0, s>>>(colptr, rowidx, order + offs[5]);
        ++*launches;
    }
    if (n_large > 0) {
        k_sort_large<<<(unsigned)n_large, 1024, 0, s>>>(colptr, rowidx, order + offs[10]);
        ++*launches;
    }
    return cudaGetLastError();
}

cudaError_t launch_values_transpose(const int64_t *rowptr, const int32_t *colidx, const float *values,
                                    const int64_t *colptr, const int32_t *rowidx, int64_t n_cols, int64_t nnz,
                                    float *values_t, cudaStream_t s, int64_t *launches)
{
    if (nnz == 0) return cudaSuccess;
    const int64_t threads = (nnz + kFillPerThread - 1) / kFillPerThread;
    k_values_transpose<<<grid_for(threads, 256), 256, 0, s>>>(rowptr, colidx, values, colptr, rowidx, n_cols, nnz,
                                                             values_t);
    ++*launches;
    return cudaGetLastError();
}

int64_t bucket_blocks(int64_t n) { return (n + kBucketThreads - 1) / kBucketThreads; }

cudaError_t launch_bucket(const int64_t *ptr, int64_t n, int64_t split, int64_t *block_counts,
                          int64_t *block_offsets, int64_t *scan_scratch, int64_t scan_elems, int32_t *order,
                          int64_t *class_offs_dev, cudaStream_t s, int64_t *launches)
{
    const int64_t nb = bucket_blocks(n);
    k_bucket<false><<<(unsigned)nb, kBucketThreads, 0, s>>>(ptr, n, split, nb, block_counts, nullptr, nullptr);
    ++*launches;
    cudaError_t e = scan_exclusive(block_counts, true, block_offsets, nb * kNClasses, scan_scratch, scan_elems, s,
                                   launches);
    if (e != cudaSuccess) return e;
    k_bucket<true><<<(unsigned)nb, kBucketThreads, 0, s>>>(ptr, n, split, nb, nullptr, block_offsets, order);
    ++*launches;
    k_class_offsets<<<1, 32, 0, s>>>(block_offsets, nb, n, class_offs_dev);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_chunk_counts(const int64_t *ptr, const int32_t *split_rows, int64_t n_split, int64_t split,
                                int64_t *counts, cudaStream_t s, int64_t *launches)
{
    if (n_split == 0) return cudaSuccess;
    k_chunk_counts<<<grid_for(n_split, 256), 256, 0, s>>>(ptr, split_rows, n_split, split, counts);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_chunk_fill(const int64_t *ptr, const int32_t *split_rows, int64_t n_split, int64_t split,
                              const int64_t *first, int64_t *desc, cudaStream_t s, int64_t *launches)
{
    if (n_split == 0) return cudaSuccess;
    k_chunk_fill<<<(unsigned)n_split, 128, 0, s>>>(ptr, split_rows, n_split, split, first, desc);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_convert(const void *src, int src_bf16, void *dst, int dst_bf16, int64_t count, cudaStream_t s,
                           int64_t *launches)
{
    if (count == 0) return cudaSuccess;
    const unsigned g = grid_for(count, 256);
    if (src_bf16 && dst_bf16)
        return cudaMemcpyAsync(dst, src, count * 2, cudaMemcpyDeviceToDevice, s);
    if (!src_bf16 && !dst_bf16)
        return cudaMemcpyAsync(dst, src, count * 4, cudaMemcpyDeviceToDevice, s);
    if (src_bf16)
        k_convert<__nv_bfloat16, float><<<g, 256, 0, s>>>((const __nv_bfloat16 *)src, (float *)dst, count);
    else
        k_convert<float, __nv_bfloat16><<<g, 256, 0, s>>>((const float *)src, (__nv_bfloat16 *)dst, count);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace alx
