// Tensor-core (tcgen05 / tensor memory) kernels for d = 128 with bfloat16 tables (and, through bfloat16 parts of the
// table and doubled entry lists, for d = 64 with fp32 tables: kModeRowsFold below):
//   - the Gramian X^T X of the fixed table                                   (Alg. 1 line 2)
//   - per row: sum x_i (x) x_i and sum y x_i over the row's observations      (Alg. 1 lines 6-9),
//     then the solve of Eq. 4 and the store                                   (Alg. 1 line 10)
//   - partial sums of the chunks of rows longer than `split`
//
// One persistent block per SM, three roles:
//   producer warps   gather the fixed-side rows of an item into a ring of shared-memory stages, already in the
//                    operand layout the tensor core reads: "MN-major, 128-byte swizzle" - a gathered row is one
//                    K index, its 128 features are the M (and N) index, split into two 64-feature halves of 128
//                    bytes.  By TMA row gathers (chunks, Gramian, conjugate-gradient rows kernel) or 16-byte
//                    cp.async (Cholesky rows kernel);
//   one MMA thread   issues tcgen05.mma 128 x 128 x 16 (A = B = the staged tile) into one of the fp32
//                    accumulators in tensor memory (four of 128 columns in the rows modes, two of 256 otherwise);
//                    chunks also get a 128 x 16 x 16 product with a two-column (high / low bfloat16 parts of
//                    the label) tile that yields sum y x_i (whole rows: the producer warps sum it);
//   solver groups    rows: four groups of 128 threads, one per accumulator.  The matrix never leaves tensor
//                    memory.  kModeRowsCg (the default): conjugate gradients, the matrix read through the 16x128b
//                    tensor-memory shape for every product (Sec. 4.5: the paper's solver); a row that does not
//                    converge is left to a second launch.  kModeRows: thread i owns row i, the group adds
//                    alpha0 G + lambda I on first touch and factors in place with a blocked right-looking
//                    Cholesky (tcgen05.ld / tcgen05.st of 16-column row segments, trailing updates on the
//                    tensor core), solves and stores the row.  kModeRowsFold: the group folds the 64 x 64 system out
//                    of its accumulator into registers and solves it there (conjugate gradients, or Cholesky in
//                    shared memory).  Gramian pieces and chunks: two groups of 256 threads copy the sums out.
// Stage and accumulator hand-over is by mbarriers; every wait is bounded and a block that gives up
// sets a status flag, releases its tensor memory and returns.
#include "alx_chol.cuh"
#include "alx_common.cuh"
#include "alx_ptx.cuh"
#include <cstring>
#include <type_traits>
#include <cuda.h>      // CUtensorMap and its enumerations (types only: the encoder is looked up at run time)

namespace alx {

namespace {

using namespace ptx;



constexpr int D = 128;
constexpr int kStageRows = 32;
// ring of stages: rows mode shares shared memory with the solver groups' scratch and alpha0 G + lambda I, the two
// streaming modes (chunks, Gramian) use that space for a deeper ring, which is what keeps HBM busy
// (and stages of 64 gathered rows instead of 32: half the per-stage waits and commits of the MMA thread)
template <int MODE> struct Ring {
    static constexpr int kRows = (MODE == 0) ? 32 : 64;   // gathered rows per stage
    // (the conjugate-gradient rows kernel needs no operand tiles for a factorisation: their space goes to its ring)
    static constexpr int kNStage = (MODE == 0 || MODE >= 3) ? 8 : 12;
    static constexpr int kHalfBytes = kRows * 128;        // one 64-feature half of a stage
    static constexpr int kStageHBytes = 2 * kHalfBytes;
    static constexpr int kStageYBytes = 2 * kRows * 16;   // label tile, two 8-column chunks
    // rows modes: ring of per-item right-hand sides.  A slot is read when a solver group starts its item j; by then the
    // MMA warp is at item j + 3 at most (item j + 4 needs the accumulator of j) and the producers at most one ring of
    // stages, hence as many items, further: slots j .. j + kNStage + 3 are live at most
    static constexpr int kBRing = kNStage + 4;
};
constexpr int kHalfBytes = kStageRows * 128;          // rows mode: one 64-feature half of a stage
constexpr int kProducerWarps = 4;
constexpr int kTmemCols = 512;
constexpr int kMaxGroups = 4;
constexpr int kGramSubRows = 256;                     // rows per tensor-memory accumulation of the Gramian (the
                                                      // accumulator truncates: fewer steps, smaller bias)
constexpr int kGramBlocks = 148;                      // fixed, so that the order of sums depends on sizes only

// kModeRowsCg: whole rows as kModeRows, solved by conjugate gradients instead of the in-place Cholesky
// kModeRowsFold: the feed of kModeRowsCg for fp32 tables of 64 features.  The fixed table is given as 2N rows of 128
//                bfloat16 values, [x1 | x2] and [x1 | x3] with x = x1 + x2 + x3 to 2^-24, and every row's entry list names
//                both rows of each of its entries; the 128 x 128 sums S then hold the 64 x 64 sum of outer products as
//                S11 / 2 + S12 + S21 + S22 (and the right-hand side as s1 / 2 + s2), which the solver folds and solves.
enum Mode { kModeRows = 0, kModeChunks = 1, kModeGramian = 2, kModeRowsCg = 3, kModeRowsFold = 4 };
__host__ __device__ constexpr bool is_cg(int mode) { return mode == kModeRowsCg || mode == kModeRowsFold; }
__host__ __device__ constexpr bool is_rows(int mode) { return mode == kModeRows || is_cg(mode); }

// thread layout per mode: solver groups (one accumulator each), then one MMA warp, then the producer warps
template <int MODE> struct Cfg {
    static constexpr int kGroups = is_rows(MODE) ? 4 : 2;
    static constexpr int kGroupThreads = is_rows(MODE) ? 128 : 256;
    static constexpr int kAccStride = is_rows(MODE) ? 128 : 256;   // accumulator a: columns a * stride ..
    static constexpr int kSolverThreads = kGroups * kGroupThreads;
    static constexpr int kMmaWarp = kSolverThreads / 32;
    static constexpr int kFirstProducerWarp = kMmaWarp + 1;
    // rows mode: the four producer warps share every stage (8 rows each, by cp.async; their partial right-hand sides
    // are summed in a fixed order); streaming modes: four producer warps, each fills whole stages of its own by TMA
    // row gathers
    static constexpr int kProducers = is_rows(MODE) ? kProducerWarps : 4;
    static constexpr int kFullArrivals = (MODE == kModeRows) ? kProducerWarps : 1;
    // a stage is free again when the tensor core has read it -- and, in the conjugate-gradient rows kernel, when the
    // producer warp that gathered it has summed y x over its rows
    static constexpr int kEmptyArrivals = is_cg(MODE) ? 2 : 1;
    static constexpr int kBlockThreads = kSolverThreads + 32 + kProducers * 32;
};

struct Params {
    SideView sv;
    const __nv_bfloat16 *X;      // fixed table [N x 128]
    int64_t n_items;             // rows of classes 1 .. 10 / chunk descriptors / 1024-row sub-pieces
    int64_t last_item;           // rows mode: position in sv.order of item 0 (items walk downwards)
    int64_t n_fixed;             // Gramian mode: rows of the table
    int64_t n_table;             // rows of the fixed table (= the first row coordinate that a row gather fills with zeros)
    int64_t n_chunks;            // chunks mode: chunk descriptors; the items after them are the long whole rows
    int64_t long_end;            // chunks mode and solve-from-sums: one past the position in sv.order of the last long row
    int64_t split_begin;         // solve-from-sums: position in sv.order of the first split row
    int64_t n_split_rows;        // solve-from-sums: split rows (items 0 .. n_split_rows - 1), then the long whole rows
    const float *Bmat;           // alpha0 G + lambda I
    const int *dual_flag;        // rows mode: set when the rows of classes 1 and 2 are solved in the dual form elsewhere
    int64_t n_items_primal;      // rows mode: items without the rows of classes 1 and 2 (the last ones of the walk)
    float *partials;             // chunks: [slot][D*D + D]; Gramian: [2 * kGramBlocks][D*D]
    RowOut out;
    DevStatus *st;
    const int32_t *item_list;    // rows mode, second launch: the rows to solve (instead of the walk through sv.order) ...
    const unsigned long long *item_count;   // ... and how many of them (device)
    int32_t *fallback_list;      // conjugate gradients: rows that did not converge are appended here (any order) ...
    unsigned long long *fallback_count;     // ... and counted here; a second launch solves them by Cholesky
    const CgPolicy *policy;      // rows modes: the side's solver choice for this half-epoch (nullptr: none, the launch decides)
    int solver;                  // rows mode: 0 = in-place Cholesky, 1 = conjugate gradients
    int cg_max_iter;             // conjugate gradients: steps after which a row goes to the Cholesky solve instead
    float cg_tol2;               // conjugate gradients: stop at |r|^2 <= cg_tol2 |b|^2
    int cg_warm;                 // conjugate gradients: start from the row's stored embedding instead of zero
    unsigned long long *cg_counters;   // [3]: rows solved by conjugate gradients, their matrix-vector products, rows that fell back
    const int *polish_flag;      // set: this launch only runs while the flag reads 2 (the dual-form rows need a polish, see launch_rows_umma)
    const CgPolicy *route;       // set where conjugate gradients run: whether the rows of 17 .. 32 observations are this kernel's
    int64_t n_class2;            // how many rows those are (they follow the longer rows in the walk)
};

constexpr int kLdB = D + 4;
// conjugate gradients on the folded 64 x 64 system: a row that needed this many products has its true residual b - A x
// checked once before it is accepted (|b - A x| <= kCgVerifySlack * tol * |b|), else it goes to the direct solve
constexpr int kCgVerifyProducts = 24;
constexpr float kCgVerifySlack = 2.f;
// conjugate gradients read the matrix with the 16x128b tensor-memory shape (a thread holds four rows, every fourth
// column): the vector of a product is kept in shared memory by column class (column mod 4), 36 floats per class so
// that the four classes of a quarter-warp's 16-byte loads fall into different banks
constexpr int kQStride = 36;
constexpr int kLdBq = 4 * kQStride;      // floats reserved per row of alpha0 G + lambda I in the rows kernels' shared memory
struct __align__(128) RowGroupSmem {   // scratch of one tensor-memory solver group
    // Panel of the current block step as tensor-core operands: row i = what thread i computed, split into
    // three bfloat16 parts (p = p1 + p2 + p3 to 2^-24), each part a K-major 128 x 16 tile without swizzle:
    // groups of 8 rows take 256 bytes, the two 8-element K halves of a group are 128 bytes apart.
    unsigned char pop[3][D * 32];
    uint64_t trail_bar;     // completion of the trailing update of the current block step (operand tiles free again)
    alignas(16) float Lt[16][16];    // transpose of the diagonal block's factor: Lt[p][c] = L[c][p] (read as float4)
    alignas(16) float xch[64];       // the two new columns of a diagonal-block step, double buffered
    alignas(16) float dinv[16];
    alignas(16) float z[16];   // the block's part of L^-1 b
    float red[2][4][16];    // per-warp partial sums of the back substitution (double buffered)
    int bad;
    int stop;               // set by the polling thread when a wait gave up; read by the group after its barrier
};

// scratch of one conjugate-gradient solver group: the vector of the next product by column class, the four warps' partial
// sums of a step's reduction, and the flags the group shares
struct __align__(128) CgGroupSmem {
    alignas(16) float pop[1][4 * 36 + 16];
    int bad;
    int stop;
};

template <int MODE> struct __align__(1024) SmemT {
    static constexpr int kNStage = Ring<MODE>::kNStage;
    unsigned char h[kNStage][Ring<MODE>::kStageHBytes];
    unsigned char y[is_rows(MODE) ? 1 : kNStage][Ring<MODE>::kStageYBytes];      // label tiles (chunks mode only)
    uint64_t full[kNStage], empty[kNStage], acc_full[kMaxGroups], acc_empty[kMaxGroups];
    uint64_t rhs_done[is_cg(MODE) ? Ring<MODE>::kBRing : 1];   // conjugate-gradient rows kernel: an item's right-hand side is written
    uint32_t tmem_base;
    int abort_flag;
    // rows modes: the producer warps also sum y x_i of the rows they staged.  kModeRows: the four warps share every stage
    // (four partial sums per item); kModeRowsCg: a warp gathers whole items (one sum per item)
    static constexpr int kRhsParts = is_cg(MODE) ? 1 : kProducerWarps;
    float ylab[kNStage][Ring<MODE>::kRows];      // labels of the staged rows
    int stage_meta[kNStage];                     // K steps of the stage (1 or 2) | 4 if it ends its item; -1: no more work
    int rows_staged[kProducerWarps][kNStage];    // kModeRows, per producer warp: how many of its 8 rows of the stage are defined
    int last_of_item[kProducerWarps][kNStage];   // kModeRows, per producer warp: 1 + ring index of the item whose last stage this is, else 0
    int own_queue[kProducerWarps][kNStage];      // kModeRowsCg, per producer warp: its stages in flight (slot, rows, last-of-item mark)
    alignas(16) float bpart[is_rows(MODE) ? Ring<MODE>::kBRing : 1][kRhsParts][D];
};

template <int MODE> __device__ __forceinline__ void item_range(const Params &p, int64_t t, int64_t &u, int64_t &beg,
                                                               int64_t &end, int64_t &slot)
{
    if (is_rows(MODE)) {
        u = p.item_list ? p.item_list[t] : p.sv.order[p.last_item - t];
        beg = p.sv.ptr[u];
        end = p.sv.ptr[u + 1];
        slot = 0;
    } else if (MODE == kModeChunks) {
        if (t < p.n_chunks) {
            const int64_t *d = p.sv.chunk_desc + 4 * t;
            u = d[0]; beg = d[1]; end = d[2]; slot = d[3];
        } else {      // a long whole row, longest class first: one sum of its own, stored after the chunks' sums
            u = p.sv.order[p.long_end - 1 - (t - p.n_chunks)];
            beg = p.sv.ptr[u];
            end = p.sv.ptr[u + 1];
            slot = t;
        }
    } else {
        u = 0; slot = t;
        beg = t * kGramSubRows;
        end = (beg + kGramSubRows < p.n_fixed) ? beg + kGramSubRows : p.n_fixed;
    }
}

// ---------------------------------------------------------------------------------------------------------
// rows mode: sum y x over this warp's 8 rows of a landed stage (lane = features 4*lane .. 4*lane+3)
using Smem = SmemT<0>;       // rows mode

template <class SmemRows>
__device__ __forceinline__ void stage_rhs(SmemRows &sm, int slot, int pw, int lane, float (&bacc)[4])
{
    const int f = 4 * lane;
    const int half = f >> 6, cc = (f & 63) >> 3, inner = (f & 7) * 2;
    const unsigned char *base = &sm.h[slot][0] + half * kHalfBytes + pw * 1024;
    const int nrows = sm.rows_staged[pw][slot];      // rows of this warp that hold data or zeros
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (j < nrows) {
            const uint2 v = *reinterpret_cast<const uint2 *>(base + j * 128 + ((cc ^ j) << 4) + inner);
            const float y = sm.ylab[slot][pw * 8 + j];
            bacc[0] = fmaf(y, __uint_as_float(v.x << 16), bacc[0]);
            bacc[1] = fmaf(y, __uint_as_float(v.x & 0xFFFF0000u), bacc[1]);
            bacc[2] = fmaf(y, __uint_as_float(v.y << 16), bacc[2]);
            bacc[3] = fmaf(y, __uint_as_float(v.y & 0xFFFF0000u), bacc[3]);
        }
    }
}

template <int MODE> __device__ __forceinline__ void producer_signal(SmemT<MODE> &sm, int64_t signalled, int pw, int lane,
                                                                   float (&bacc)[4])
{
    constexpr int kNStage = Ring<MODE>::kNStage;
    const int slot = (int)(signalled % kNStage);
    if constexpr (is_rows(MODE)) {
        __syncwarp();      // every lane's copies of this stage have landed (each lane waited for its own)
        stage_rhs(sm, slot, pw, lane, bacc);
        const int last = sm.last_of_item[pw][slot];
        if (last) {
            *reinterpret_cast<float4 *>(&sm.bpart[last - 1][pw][4 * lane]) = make_float4(bacc[0], bacc[1], bacc[2], bacc[3]);
            bacc[0] = bacc[1] = bacc[2] = bacc[3] = 0.f;
        }
    }
    fence_proxy_async();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.full[slot]);
}

// Rows modes: the offsets of the block's next 32 items, one item per lane, fetched together every 32 items (a row's
// offsets hang on a chain of dependent loads, order -> ptr; walked item by item, that latency would be paid per item,
// which rows of a hundred entries cannot afford).  Item `it` of the block is row order[last_item - (blockIdx.x + it grid)].
struct ItemWindow {
    int64_t beg = 0, end = 0;      // this lane's item of the window (empty range past the last item)
    __device__ __forceinline__ void load(const Params &p, int64_t it0, int lane)
    {
        const int64_t t = (int64_t)blockIdx.x + (it0 + lane) * gridDim.x;
        beg = end = 0;
        if (t < p.n_items) {
            const int64_t u = p.item_list ? p.item_list[t] : p.sv.order[p.last_item - t];
            beg = p.sv.ptr[u];
            end = p.sv.ptr[u + 1];
        }
    }
    __device__ __forceinline__ void get(int k, int64_t &b, int64_t &e) const
    {
        b = __shfl_sync(0xFFFFFFFFu, beg, k);
        e = __shfl_sync(0xFFFFFFFFu, end, k);
    }
};

template <int MODE> __device__ void producer_role(const Params &p, SmemT<MODE> &sm, int pw, int lane)
{
    constexpr int kNStage = Ring<MODE>::kNStage, kLag = 6;      // kLag: stages of cp.async copies in flight per producer warp
    int64_t g = 0, signalled = 0, it = 0;
    const int c = lane & 15;                 // 16-byte chunk of the 256-byte row
    const int half = c >> 3, cc = c & 7;
    float bacc[4] = {0.f, 0.f, 0.f, 0.f};
    bool alive = true;
    ItemWindow win;
    // ids (and labels) of this warp's 8 rows of a stage are fetched one stage ahead by lanes 0..7; those of an item's
    // first stage while the item before it is gathered (except across a window's end)
    int32_t pre_idx = -1;
    float pre_y = 0.f;
    bool have_pre = false;
    auto first_ids = [&](int64_t beg, int64_t end, int32_t &idx, float &y) {
        idx = -1;
        y = 0.f;
        const int64_t e = beg + pw * 8 + (lane & 7);
        if (lane < 8 && e < end) {
            idx = p.sv.idx[e];
            y = p.sv.val ? p.sv.val[e] : 1.f;
        }
    };
    for (int64_t t = blockIdx.x; t < p.n_items && alive; t += gridDim.x, ++it) {
        if ((it & 31) == 0) win.load(p, it, lane);
        int64_t beg, end;
        win.get((int)(it & 31), beg, end);
        int32_t nxt_idx;
        float nxt_y;
        if (have_pre) { nxt_idx = pre_idx; nxt_y = pre_y; }
        else first_ids(beg, end, nxt_idx, nxt_y);
        have_pre = (it & 31) != 31;
        if (have_pre) {
            int64_t nbeg, nend;
            win.get((int)(it & 31) + 1, nbeg, nend);
            first_ids(nbeg, nend, pre_idx, pre_y);
        }
        for (int64_t e0 = beg; e0 < end; e0 += kStageRows) {
            const int slot = (int)(g % kNStage);
            const uint32_t ph = (uint32_t)((g / kNStage) & 1);
            const int32_t my_idx = nxt_idx;
            const float my_y = nxt_y;
            {
                const int64_t e = e0 + kStageRows + pw * 8 + (lane & 7);
                nxt_idx = -1;
                nxt_y = 0.f;
                if (lane < 8 && e < end) {
                    nxt_idx = (MODE == kModeGramian) ? (int32_t)e : p.sv.idx[e];
                    nxt_y = (MODE == kModeGramian) ? 0.f : (p.sv.val ? p.sv.val[e] : 1.f);
                }
            }
            // No free slot yet: the copies in flight have time to land, so hand over every stage issued so far
            // before blocking (otherwise up to kLag landed stages would stay unannounced until the next issue).
            {
                int free_now = 1;
                if (lane == 0) free_now = mbar_test_wait(&sm.empty[slot], ph ^ 1u) ? 1 : 0;
                free_now = __shfl_sync(0xFFFFFFFFu, free_now, 0);
                if (!free_now && signalled < g) {
                    cp_async_wait<0>();
                    for (; signalled < g; ++signalled) producer_signal<MODE>(sm, signalled, pw, lane, bacc);
                }
            }
            if (!mbar_wait_warp(&sm.empty[slot], ph ^ 1u, &sm.abort_flag, 10 + MODE)) { alive = false; break; }
            const int rc = (int)((end - e0 < kStageRows) ? end - e0 : kStageRows);
            const int rc16 = (rc + 15) & ~15;
            if (is_rows(MODE)) {
                if (lane < 8) sm.ylab[slot][pw * 8 + lane] = my_y;
                if (lane == 0) {
                    sm.last_of_item[pw][slot] = (e0 + kStageRows >= end) ? 1 + (int)(it % Ring<MODE>::kBRing) : 0;
                    const int mine = rc16 - pw * 8;
                    sm.rows_staged[pw][slot] = mine < 0 ? 0 : (mine > 8 ? 8 : mine);
                }
            }
            const uint32_t hbase = smem_u32(&sm.h[slot][0]) + half * kHalfBytes + pw * 1024;
            const uint32_t ybase = smem_u32(&sm.y[slot][0]) + pw * 128;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int j = (lane >> 4) + 2 * q;          // row inside this warp's group of 8
                const int r = pw * 8 + j;                   // row inside the stage
                const int32_t src = __shfl_sync(0xFFFFFFFFu, my_idx, j);
                const float yv = __shfl_sync(0xFFFFFFFFu, my_y, j);
                const uint32_t dst = hbase + j * 128 + ((cc ^ j) << 4);
                if (src >= 0) cp_async16(dst, p.X + (int64_t)src * D + c * 8);
                else if (r < rc16) st_shared_zero16(dst);
                if (MODE == kModeChunks && c == 0 && r < rc16) {
                    const __nv_bfloat16 yhi = __float2bfloat16_rn(yv);
                    const __nv_bfloat16 ylo = __float2bfloat16_rn(yv - __bfloat162float(yhi));
                    const uint32_t packed = (uint32_t)__bfloat16_as_ushort(yhi) | ((uint32_t)__bfloat16_as_ushort(ylo) << 16);
                    st_shared_v4(ybase + j * 16, packed, 0u, 0u, 0u);
                }
            }
            cp_async_commit();
            ++g;
            if (g - signalled > kLag) {     // the oldest unannounced stage is kLag issues back: its copies have landed
                cp_async_wait<kLag>();
                producer_signal<MODE>(sm, signalled, pw, lane, bacc);
                ++signalled;
            }
        }
    }
    cp_async_wait<0>();
    for (; signalled < g; ++signalled) producer_signal<MODE>(sm, signalled, pw, lane, bacc);
}

// Producer of the conjugate-gradient rows kernel.  Producer warp pw gathers every fourth item of the block, whole: all its
// stages of 64 rows, by TMA row gathers (four rows of one 64-feature half per instruction, written with the 128-byte
// swizzle the tensor core reads; lanes 0 .. 15 issue them, the stage's mbarrier counts the bytes, rows past the item's end
// take a row coordinate past the end of the table and are filled with zeros).  The four warps thus work on four items at
// a time: what bounds a gather of short rows is the chain of loads, waits and hand-overs per stage, and four chains run
// side by side.  Every warp walks all items (their offsets come in windows of 32) to number the stages: stage g of the
// block sits in slot g mod ring, whichever warp fills it; the MMA warp takes the stages in that order.
// Stages are ISSUED in order too: a warp issues stage g after stage g - 1 has been issued (a counter in shared memory
// passes the turn).  An mbarrier tells its phases apart by parity only; a warp that jumped ahead by a lap of the ring
// would take a slot's release of two laps ago for the one it needs.  With the turn, the slot of stage g is in one of two
// states when its warp looks: stage g - ring released, or not yet.  The turn covers only the wait for the slot and the
// copy instructions; the index loads before and the sums after run in parallel.
// Once a stage has landed its warp adds the rows' y x to the item's right-hand side and releases the slot (a slot is
// free again after the tensor core and that warp are done with it); after an item's last stage it publishes the sum
// and arrives on the item's right-hand-side barrier, which the solver group waits for.
template <int MODE>
__device__ void producer_role_items(const Params &p, const CUtensorMap *tmap, SmemT<MODE> &sm, int pw, int lane)
{
    constexpr int kNStage = Ring<MODE>::kNStage, kRows = Ring<MODE>::kRows, kBRing = Ring<MODE>::kBRing;
    static_assert(kRows == 64, "two rows per lane, sixteen groups of four rows");
    const int32_t past_end = (int32_t)p.n_table;
    volatile int *turn = &sm.stage_meta[0];  // stages issued so far by the four warps together
    int g_run = 0;                           // stages of the items walked so far (the same count in every warp)
    int head = 0, tail = 0;                  // this warp's stages handed over / issued
    uint32_t q_parity = 0;                   // bit k: parity of the `full` phase of this warp's stage number k (modulo 32)
    float bacc[4] = {0.f, 0.f, 0.f, 0.f};
    bool alive = true;
    ItemWindow win;
    const int f = 4 * lane;                  // this lane's four features in the sums of y x
    const int fhalf = f >> 6, fcc = (f & 63) >> 3, finner = (f & 7) * 2;
    // the oldest stage of this warp not handed over yet has landed (the caller made sure): sum y x over its rows, release it
    auto hand_over = [&]() {
        const int e = sm.own_queue[pw][head % kNStage];
        const int slot = e & 0xFF, nrows = (e >> 8) & 0xFF, last = e >> 16;
        // every lane reads the copied rows, so every lane observes the completed phase itself
        for (int k = 0; k < 64 && !mbar_test_wait(&sm.full[slot], (q_parity >> (head & 31)) & 1u); ++k) { }
        const unsigned char *base = &sm.h[slot][0] + fhalf * Ring<MODE>::kHalfBytes;
        if (p.sv.val) {
#pragma unroll 4
            for (int j = 0; j < nrows; ++j) {
                const uint2 v = *reinterpret_cast<const uint2 *>(base + j * 128 + ((fcc ^ (j & 7)) << 4) + finner);
                const float y = sm.ylab[slot][j];
                bacc[0] = fmaf(y, __uint_as_float(v.x << 16), bacc[0]);
                bacc[1] = fmaf(y, __uint_as_float(v.x & 0xFFFF0000u), bacc[1]);
                bacc[2] = fmaf(y, __uint_as_float(v.y << 16), bacc[2]);
                bacc[3] = fmaf(y, __uint_as_float(v.y & 0xFFFF0000u), bacc[3]);
            }
        } else {        // every label is 1: eight rows (one 1024-byte group of the tile) per trip, loads first
            for (int j0 = 0; j0 < nrows; j0 += 8) {
                uint2 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = *reinterpret_cast<const uint2 *>(base + (j0 + j) * 128 + ((fcc ^ j) << 4) + finner);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    bacc[0] += __uint_as_float(v[j].x << 16);
                    bacc[1] += __uint_as_float(v[j].x & 0xFFFF0000u);
                    bacc[2] += __uint_as_float(v[j].y << 16);
                    bacc[3] += __uint_as_float(v[j].y & 0xFFFF0000u);
                }
            }
        }
        if (last) {
            *reinterpret_cast<float4 *>(&sm.bpart[last - 1][0][f]) = make_float4(bacc[0], bacc[1], bacc[2], bacc[3]);
            bacc[0] = bacc[1] = bacc[2] = bacc[3] = 0.f;
        }
        __syncwarp();
        if (lane == 0) {
            if (last) mbar_arrive(&sm.rhs_done[last - 1]);
            mbar_arrive(&sm.empty[slot]);
        }
        ++head;
    };
    // has this warp's oldest stage in flight landed?  (lane 0 looks, the warp follows)
    auto oldest_landed = [&]() {
        int yes = 0;
        if (lane == 0)
            yes = mbar_test_wait(&sm.full[sm.own_queue[pw][head % kNStage] & 0xFF], (q_parity >> (head & 31)) & 1u) ? 1 : 0;
        return __shfl_sync(0xFFFFFFFFu, yes, 0) != 0;
    };
    auto wait_oldest = [&]() {
        return mbar_wait_parked_warp(&sm.full[sm.own_queue[pw][head % kNStage] & 0xFF], (q_parity >> (head & 31)) & 1u,
                                     &sm.abort_flag, 20);
    };
    int64_t it = 0;
    for (int64_t t = blockIdx.x; t < p.n_items && alive; t += gridDim.x, ++it) {
        if ((it & 31) == 0) win.load(p, it, lane);
        int64_t beg, end;
        win.get((int)(it & 31), beg, end);
        const int nst = (int)((end - beg + kRows - 1) / kRows);
        const int g0 = g_run;
        g_run += nst;
        if ((int)(it & 3) != pw) continue;
        // ids and labels of a stage's rows: this lane's two rows (lane and 32 + lane), fetched one stage ahead
        int32_t nxt_idx[2];
        float nxt_y[2];
        auto fetch_ids = [&](int64_t e0) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int64_t e = e0 + 32 * k + lane;
                nxt_idx[k] = past_end;
                nxt_y[k] = 0.f;
                if (e < end) {
                    nxt_idx[k] = p.sv.idx[e];
                    nxt_y[k] = p.sv.val ? p.sv.val[e] : 1.f;
                }
            }
        };
        fetch_ids(beg);
        for (int s = 0; s < nst && alive; ++s) {
            const int g = g0 + s;
            const int64_t e0 = beg + (int64_t)s * kRows;
            const int slot = g % kNStage;
            const uint32_t ph = (uint32_t)((g / kNStage) & 1);
            const int32_t my_idx[2] = {nxt_idx[0], nxt_idx[1]};
            const float my_y[2] = {nxt_y[0], nxt_y[1]};
            if (s + 1 < nst) fetch_ids(e0 + kRows);
            // (1) wait for the turn; the hand-overs fill the wait (one stage at a time, the turn is looked at first: while this
            // warp holds the turn the other three wait for it)
            for (uint32_t spin = 0;; ++spin) {
                int mine = 0;
                if (lane == 0) mine = (*turn >= g) ? 1 : 0;
                if (__shfl_sync(0xFFFFFFFFu, mine, 0)) break;
                if (head < tail && oldest_landed()) {
                    hand_over();
                    spin = 0;
                    continue;
                }
                if (spin > (1u << 22) || ((spin & 63u) == 63u && sm.abort_flag)) {
                    if (lane == 0 && sm.abort_flag == 0) sm.abort_flag = 12;
                    alive = false;
                    break;
                }
                if (spin > 8u) __nanosleep(spin < 128u ? 64u : 256u);
            }
            if (!alive) break;
            // (2) the slot: stage g - ring must have been released.  While it is not, this warp's own stages in flight go
            // first (their release may be what the ring's turn-over waits for), then the warp waits suspended.
            for (;;) {
                int free_now = 0;
                if (lane == 0) free_now = mbar_test_wait(&sm.empty[slot], ph ^ 1u) ? 1 : 0;
                if (__shfl_sync(0xFFFFFFFFu, free_now, 0)) break;
                if (head < tail) {
                    if (!wait_oldest()) { alive = false; break; }
                    hand_over();
                } else {
                    if (!mbar_wait_parked_warp(&sm.empty[slot], ph ^ 1u, &sm.abort_flag, 10)) alive = false;
                    break;
                }
            }
            if (!alive) break;
            // (3) issue the stage and pass the turn on
            const int rc = (int)((end - e0 < kRows) ? end - e0 : kRows);
            const int rc16 = (rc + 15) & ~15;
            if (p.sv.val) {
                sm.ylab[slot][lane] = my_y[0];
                sm.ylab[slot][32 + lane] = my_y[1];
            }
            if (lane == 0) sm.own_queue[pw][tail % kNStage] = slot | (rc16 << 8) | ((s + 1 == nst) ? ((1 + (int)(it % kBRing)) << 16) : 0);
            q_parity = (q_parity & ~(1u << (tail & 31))) | (ph << (tail & 31));
            // rows 4 * lane .. 4 * lane + 3 of the stage (lanes 0 .. 15)
            int32_t r4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int32_t v0 = __shfl_sync(0xFFFFFFFFu, my_idx[0], (4 * lane + j) & 31);
                const int32_t v1 = __shfl_sync(0xFFFFFFFFu, my_idx[1], (4 * lane + j) & 31);
                r4[j] = (lane < 8) ? v0 : v1;
            }
            __syncwarp();
            const int ngroups = rc16 >> 2;        // groups of four rows the tensor core will read
            if (lane == 0) mbar_arrive_expect_tx(&sm.full[slot], (uint32_t)ngroups * 1024u);
            if (lane < ngroups) {
                const uint32_t dst = smem_u32(&sm.h[slot][0]) + lane * 512;
                tma_gather4(dst, tmap, 0, r4[0], r4[1], r4[2], r4[3], &sm.full[slot]);
                tma_gather4(dst + Ring<MODE>::kHalfBytes, tmap, 64, r4[0], r4[1], r4[2], r4[3], &sm.full[slot]);
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                *turn = g + 1;
            }
            ++tail;
        }
    }
    while (alive && head < tail) {
        if (!wait_oldest()) break;
        hand_over();
    }
}

// Streaming modes (chunks, Gramian pieces): producer warp pw fills the stages whose running number is pw modulo the
// number of producer warps, whole stages of 64 rows each.  The rows come by TMA row gathers (four rows of one
// 64-feature half per instruction, written with the 128-byte swizzle the tensor core reads), issued by lanes 0 .. 15 for
// the 16 groups of four rows; the stage's mbarrier counts the bytes.  Rows past the end of the item take a row
// coordinate past the end of the table, which the copy fills with zeros.  The Gramian's rows are consecutive: there a
// stage is two tile loads of 64 rows, issued by one lane.
template <int MODE>
__device__ void stream_producer_role(const Params &p, const CUtensorMap *tmap, SmemT<MODE> &sm, int pw, int lane)
{
    constexpr int kNStage = Ring<MODE>::kNStage, kRows = Ring<MODE>::kRows, P = Cfg<MODE>::kProducers;
    static_assert(kRows == 64, "two rows per lane, sixteen groups of four rows");
    int64_t g = 0;                        // running number of the stage over all items of this block
    int ring_slot = 0;                    // ring position and phase of stage g
    uint32_t ring_ph = 0;
    const int32_t past_end = (int32_t)p.n_table;
    bool alive = true;
    for (int64_t t = blockIdx.x; t < p.n_items && alive; t += gridDim.x) {
        int64_t u, beg, end, slot_unused;
        item_range<MODE>(p, t, u, beg, end, slot_unused);
        for (int64_t e0 = beg; e0 < end; e0 += kRows, ++g) {
            const int slot = ring_slot;
            const uint32_t ph = ring_ph;
            if (++ring_slot == kNStage) { ring_slot = 0; ring_ph ^= 1u; }
            if ((int)(g % P) != pw) continue;
            if constexpr (MODE == kModeGramian) {
                // consecutive rows of the table: one tile load per 64-feature half (the same lines and swizzle as the
                // row gathers leave; the tensor map of this launch has boxes of 64 rows)
                if (!mbar_wait_warp(&sm.empty[slot], ph ^ 1u, &sm.abort_flag, 10 + MODE)) { alive = false; break; }
                if (lane == 0) {
                    const uint32_t dst = smem_u32(&sm.h[slot][0]);
                    mbar_arrive_expect_tx(&sm.full[slot], 2u * (uint32_t)Ring<MODE>::kHalfBytes);
                    tma_tile_2d(dst, tmap, 0, (int)e0, &sm.full[slot]);
                    tma_tile_2d(dst + Ring<MODE>::kHalfBytes, tmap, 64, (int)e0, &sm.full[slot]);
                }
                __syncwarp();
                continue;
            }
            // this lane's two rows of the stage (lane and 32 + lane)
            int32_t my_idx[2] = {past_end, past_end};
            float my_y[2] = {0.f, 0.f};
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int64_t e = e0 + 32 * k + lane;
                if (e < end) {
                    my_idx[k] = (MODE == kModeGramian) ? (int32_t)e : p.sv.idx[e];
                    my_y[k] = (MODE == kModeGramian) ? 0.f : (p.sv.val ? p.sv.val[e] : 1.f);
                }
            }
            // rows 4 * lane .. 4 * lane + 3 of the stage (lanes 0 .. 15)
            int32_t r4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int32_t v0 = __shfl_sync(0xFFFFFFFFu, my_idx[0], (4 * lane + j) & 31);
                const int32_t v1 = __shfl_sync(0xFFFFFFFFu, my_idx[1], (4 * lane + j) & 31);
                r4[j] = (lane < 8) ? v0 : v1;
            }
            if (!mbar_wait_warp(&sm.empty[slot], ph ^ 1u, &sm.abort_flag, 10 + MODE)) { alive = false; break; }
            const int rc = (int)((end - e0 < kRows) ? end - e0 : kRows);
            const int rc16 = (rc + 15) & ~15;
            if (MODE == kModeChunks) {
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    if (32 * k + lane < rc16) {
                        const __nv_bfloat16 yhi = __float2bfloat16_rn(my_y[k]);
                        const __nv_bfloat16 ylo = __float2bfloat16_rn(my_y[k] - __bfloat162float(yhi));
                        const uint32_t packed = (uint32_t)__bfloat16_as_ushort(yhi) | ((uint32_t)__bfloat16_as_ushort(ylo) << 16);
                        st_shared_v4(smem_u32(&sm.y[slot][0]) + (32 * k + lane) * 16, packed, 0u, 0u, 0u);
                    }
                }
                fence_proxy_async();
            }
            __syncwarp();
            const int ngroups = rc16 >> 2;        // groups of four rows the tensor core will read
            if (lane == 0) mbar_arrive_expect_tx(&sm.full[slot], (uint32_t)ngroups * 1024u);
            if (lane < ngroups) {
                const uint32_t dst = smem_u32(&sm.h[slot][0]) + lane * 512;
                tma_gather4(dst, tmap, 0, r4[0], r4[1], r4[2], r4[3], &sm.full[slot]);
                tma_gather4(dst + Ring<MODE>::kHalfBytes, tmap, 64, r4[0], r4[1], r4[2], r4[3], &sm.full[slot]);
            }
            __syncwarp();
        }
    }
}

template <int MODE> __device__ void mma_role(const Params &p, SmemT<MODE> &sm, int lane, uint32_t base_smem = 0)
{
    constexpr int kNStage = Ring<MODE>::kNStage, kRows = Ring<MODE>::kRows;
    constexpr uint32_t kIdescMain = idesc_bf16_mn_major(128, 128);
    constexpr uint32_t kIdescY = idesc_bf16_mn_major(128, 16);
    const uint32_t tmem = sm.tmem_base;
    const uint64_t base_desc = smem_desc(base_smem, 128, 256, 0);      // (conjugate-gradient rows kernel: alpha0 G + lambda I)
    int slot = 0;             // ring position and phase of the next stage
    uint32_t ph = 0;
    bool alive = true;
    // one stage: wait for it, issue its K steps of 16 rows, release it when they have completed
    auto stage = [&](uint32_t d_main, int nk, bool &first) -> bool {
        if (!mbar_wait_parked_warp(&sm.full[slot], ph, &sm.abort_flag, 30 + MODE)) return false;
        tc_fence_after();
        if (lane == 0) {
            const uint32_t hb = smem_u32(&sm.h[slot][0]);
            const uint32_t yb = smem_u32(&sm.y[slot][0]);
            for (int ks = 0; ks < nk; ++ks) {
                // 16 gathered rows = two groups of 8 rows of 128 bytes; halves are kHalfBytes apart
                const uint64_t adesc = smem_desc(hb + ks * 2048, Ring<MODE>::kHalfBytes, 1024, 2);
                umma_f16(d_main, adesc, adesc, kIdescMain, !first);
                if (MODE == kModeChunks) {
                    const uint64_t ydesc = smem_desc(yb + ks * 256, 128, kRows * 16, 0);
                    umma_f16(d_main + D, adesc, ydesc, kIdescY, !first);
                }
                first = false;
            }
            umma_commit(&sm.empty[slot]);
        }
        if (++slot == kNStage) { slot = 0; ph ^= 1u; }
        return true;
    };
    if constexpr (is_rows(MODE)) {
        // rows modes: all this warp needs of an item is its number of stages and the K steps of the last one; they come
        // for 32 items at a time, one item per lane (the offsets hang on a chain of dependent loads, see ItemWindow)
        const int n_mine = (int)((p.n_items - blockIdx.x + gridDim.x - 1) / gridDim.x);      // items of this block
        int info = 0;
        for (int it = 0; it < n_mine && alive; ++it) {
            if ((it & 31) == 0) {
                ItemWindow win;
                win.load(p, it, lane);
                const int len = (int)(win.end - win.beg);
                const int nst = (len + kRows - 1) / kRows;
                const int tail_rows = len - (nst - 1) * kRows;
                info = (nst << 8) | ((tail_rows + 15) >> 4);
            }
            const int mine = __shfl_sync(0xFFFFFFFFu, info, it & 31);
            const int nst = mine >> 8, nk_last = mine & 0xFF;
            const int a = it % Cfg<MODE>::kGroups;
            const uint32_t aph = (uint32_t)((it / Cfg<MODE>::kGroups) & 1);
            if (!mbar_wait_parked_warp(&sm.acc_empty[a], aph ^ 1u, &sm.abort_flag, 40 + MODE)) break;
            tc_fence_after();
            const uint32_t d_main = tmem + a * Cfg<MODE>::kAccStride;
            bool first = true;
            if constexpr (MODE == kModeRowsCg) {
                // the accumulator starts as alpha0 G + lambda I (copied from shared memory by the tensor pipe, in
                // order with the products that follow): the solver finds the complete matrix of Eq. 4
                if (lane == 0) {
                    // (the address field of the descriptor counts 16-byte units: 4096 bytes per block of 8 columns)
#pragma unroll 1
                    for (int c8 = 0; c8 < D / 8; ++c8) tmem_cp_128x256b(d_main + 8 * c8, base_desc + (uint64_t)(c8 * 256));
                }
                first = false;
            }
            for (int s = 0; s < nst; ++s)
                if (!stage(d_main, s + 1 < nst ? kRows / 16 : nk_last, first)) { alive = false; break; }
            if (alive && lane == 0) umma_commit(&sm.acc_full[a]);
            __syncwarp();
        }
    } else {
        int64_t it = 0;
        for (int64_t t = blockIdx.x; t < p.n_items && alive; t += gridDim.x, ++it) {
            int64_t u, beg, end, slot_unused;
            item_range<MODE>(p, t, u, beg, end, slot_unused);
            const int a = (int)(it % Cfg<MODE>::kGroups);
            const uint32_t aph = (uint32_t)((it / Cfg<MODE>::kGroups) & 1);
            if (!mbar_wait_parked_warp(&sm.acc_empty[a], aph ^ 1u, &sm.abort_flag, 40 + MODE)) break;
            tc_fence_after();
            const uint32_t d_main = tmem + a * Cfg<MODE>::kAccStride;
            bool first = true;
            for (int64_t e0 = beg; e0 < end; e0 += kRows) {
                const int rc = (int)((end - e0 < kRows) ? end - e0 : kRows);
                if (!stage(d_main, (rc + 15) >> 4, first)) { alive = false; break; }
            }
            if (alive && lane == 0) umma_commit(&sm.acc_full[a]);
            __syncwarp();
        }
    }
}

template <int MODE>
__device__ void copyout_role(const Params &p, SmemT<MODE> &sm, int gidx, int tid)
{
    constexpr int kAccStride = Cfg<MODE>::kAccStride;
    const int lane = tid & 31, w = tid >> 5;
    const int q = w & 3, hh = w >> 2;            // lane quarter of tensor memory, column half
    const int i = q * 32 + lane;                 // row of the matrix this thread reads back
    const int bar_id = 1 + gidx;
    const uint32_t tmem = sm.tmem_base;
    float run[(MODE == kModeGramian) ? 64 : 1];
    if (MODE == kModeGramian) {
#pragma unroll
        for (int k = 0; k < 64; ++k) run[k] = 0.f;
    }
    int64_t it = 0;
    for (int64_t t = blockIdx.x; t < p.n_items; t += gridDim.x, ++it) {
        if ((it & 1) != gidx) continue;
        int64_t u, beg, end, slot;
        item_range<MODE>(p, t, u, beg, end, slot);
        const uint32_t aph = (uint32_t)((it >> 1) & 1);
        if (!mbar_wait_warp(&sm.acc_full[gidx], aph, &sm.abort_flag, 50 + MODE)) break;
        tc_fence_after();
        const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + gidx * kAccStride + hh * 64;
        uint32_t v0[32], v1[32];
        tmem_ld32(taddr, v0);
        tmem_ld32(taddr + 32, v1);
        tmem_ld_wait();
        if (MODE == kModeGramian) {
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                run[k] += __uint_as_float(v0[k]);
                run[32 + k] += __uint_as_float(v1[k]);
            }
        } else if (MODE == kModeChunks) {
            float *dst = p.partials + slot * (int64_t)(D * D + D) + (int64_t)i * D + hh * 64;
#pragma unroll
            for (int k = 0; k < 32; k += 4) {
                *reinterpret_cast<float4 *>(dst + k) = make_float4(__uint_as_float(v0[k]), __uint_as_float(v0[k + 1]),
                                                                   __uint_as_float(v0[k + 2]), __uint_as_float(v0[k + 3]));
                *reinterpret_cast<float4 *>(dst + 32 + k) = make_float4(__uint_as_float(v1[k]), __uint_as_float(v1[k + 1]),
                                                                        __uint_as_float(v1[k + 2]), __uint_as_float(v1[k + 3]));
            }
        }
        if (MODE != kModeGramian && hh == 0) {
            uint32_t bv[4];
            tmem_ld4(tmem + ((uint32_t)(q * 32) << 16) + gidx * kAccStride + D, bv);
            tmem_ld_wait();
            const float b = __uint_as_float(bv[0]) + __uint_as_float(bv[1]);   // high and low parts of the labels
            p.partials[slot * (int64_t)(D * D + D) + D * D + i] = b;
        }
        tc_fence_before();
        group_sync(bar_id);
        if (tid == 0) mbar_arrive(&sm.acc_empty[gidx]);
    }
    if (MODE == kModeGramian) {
        float *dst = p.partials + ((int64_t)blockIdx.x * Cfg<MODE>::kGroups + gidx) * (D * D) + (int64_t)i * D + hh * 64;
#pragma unroll
        for (int k = 0; k < 64; k += 4)
            *reinterpret_cast<float4 *>(dst + k) = make_float4(run[k], run[k + 1], run[k + 2], run[k + 3]);
    }
}


// ---------------------------------------------------------------------------------------------------------
// Rows mode: factor and solve in place in tensor memory.  128 threads, thread i = row i = tensor-memory lane i.
// Blocked right-looking Cholesky, 16 columns per step:
//   (1) the warp that holds the diagonal block waits for the previous step's tensor-core update, reads its 16 panel
//       values (adding alpha0 G + lambda I) and factors the block with shuffles, two pivots per round, b carried
//       along as a 17th column; the rows after the block in the same warp get their forward substitution in the
//       same rounds;
//   (2) after the group's barrier the other live rows read their panel values, those after the block do their
//       forward substitution against the block (from shared memory) and
//       fold the block's part of L^-1 b into their b; every row after the block publishes its panel row as three
//       bfloat16 parts in the operand tiles and writes it back to tensor memory (back substitution reads it);
//   (3) trailing update A22 -= P P^T on the tensor core, in place in tensor memory: six tcgen05.mma
//       128 x N x 16 (N = all columns right of the block) over the three-way bfloat16 split of P
//       (p1p1 + p1p2 + p2p1 + p1p3 + p3p1 + p2p2, the dropped terms are below 2^-26 relative),
//       A operand negated by the instruction descriptor, issued by one thread of a warp that does not hold the
//       next diagonal block;
//   (4) after the last step every thread computes its column of the inverse of its own diagonal block (the
//       eight blocks go through shared memory at once);
//   (5) back substitution block by block from the end: per-block partial sums over the rows below are
//       reduced in a fixed order (warp butterfly, then four warps in order), the diagonal threads apply
//       their inverse columns.
// alpha0 G + lambda I is added from shared memory when a panel is read (every element of the lower triangle
// is read as part of a panel exactly once; the tensor-core updates commute with that addition).
__device__ __forceinline__ void warp_reduce16(float (&v)[16], int lane)
{
    // after the call, lane 2c (and 2c+1) holds the sum over the 32 lanes of v[c], in v[0]
    float t8[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const bool up = (lane & 16) != 0;
        const float send = up ? v[c] : v[c + 8];
        const float keep = up ? v[c + 8] : v[c];
        t8[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 16);
    }
    float t4[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const bool up = (lane & 8) != 0;
        const float send = up ? t8[c] : t8[c + 4];
        const float keep = up ? t8[c + 4] : t8[c];
        t4[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
    }
    float t2[2];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const bool up = (lane & 4) != 0;
        const float send = up ? t4[c] : t4[c + 2];
        const float keep = up ? t4[c + 2] : t4[c];
        t2[c] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
    }
    {
        const bool up = (lane & 2) != 0;
        const float send = up ? t2[0] : t2[1];
        const float keep = up ? t2[1] : t2[0];
        v[0] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 2);
    }
    v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 1);
}

// one MUFU instruction, about 2 ulp: the factor absorbs it as a relative perturbation of 2^-22 of the pivot
__device__ __forceinline__ float rsqrt_fast(float x)
{
    float r;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ void group128_sync(int bar_id)
{
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");
}


// The in-place factor / solve of one matrix held in tensor memory (steps (1) .. (5) above); returns x_i.  add_b: alpha0 G +
// lambda I is still to be added (from shared memory, as the panels are read); b: my component of the right-hand side.
// A wait that gave up leaves gs.stop set (the caller leaves its loop); a non-positive pivot leaves gs.bad set.
template <class SmemRows>
__device__ __forceinline__ float chol_in_tmem(SmemRows &sm, RowGroupSmem &gs, const float *Brow, uint32_t trow, uint32_t d_base,
                                              int bar_id, int tid, float b, bool add_b, uint32_t &trail_parity)
{
    const int lane = tid & 31, w = tid >> 5;
    const int i = tid, pos = tid, wpos = pos & ~31;
    float lrow[16];          // my row of my diagonal block's factor (kept for the block inverse at the end)
    float my_dinv = 0.f;     // 1 / L[i][i]
#pragma unroll
    for (int c = 0; c < 16; ++c) lrow[c] = 0.f;

    for (int k = 0; k < D / 16; ++k) {
        const int k0 = 16 * k;
        const int ck = k0;                                     // tensor-memory columns of this block
        float a[16];
        const bool warp_live = (wpos + 31 >= k0);              // some row of my warp is at or after the block
        const bool diag_warp = (wpos == (k0 & ~31));
        auto load_panel = [&]() {
            tmem_ld16(trow + ck, a);
#pragma unroll
            for (int c = 0; c < 16; c += 4) {
                if (!add_b) break;
                const float4 bb = *reinterpret_cast<const float4 *>(Brow + ck + c);
                const float2 s01 = __fadd2_rn(make_float2(a[c], a[c + 1]), make_float2(bb.x, bb.y));
                const float2 s23 = __fadd2_rn(make_float2(a[c + 2], a[c + 3]), make_float2(bb.z, bb.w));
                a[c] = s01.x; a[c + 1] = s01.y; a[c + 2] = s23.x; a[c + 3] = s23.y;
            }
        };
        if (diag_warp) {
            // the previous step's tensor-core update has landed: only the warp that holds the diagonal block waits
            // for it (a wait that gives up only sets the group's stop flag; the group leaves together after the
            // block loop); the other warps follow through the barrier below, at no cost in issue slots
            if (k > 0) {
                if (!mbar_wait_warp(&gs.trail_bar, trail_parity ^ 1u, &sm.abort_flag, 70) && lane == 0) gs.stop = 1;
                tc_fence_after();
            }
            load_panel();
        }
        // (1) diagonal block
        if (diag_warp) {
            const int hb = k0 & 16;
            const int l = lane - hb;      // place relative to the block: < 0 eliminated earlier, 0 .. 15 the block,
                                          // >= 16 the 16 rows after the block (when it is the first of its warp)
            const bool is_diag = (l >= 0 && l < 16);
            float my_inv = 0.f;
            bool all_ok = true;
            // Two pivots per round, no masks on the matrix entries: a row that is done only ever overwrites
            // entries of its upper triangle (never read), and the rows after the block that share this warp get
            // their forward substitution against the block for free (the same arithmetic in the same order as
            // the substitution step below, which they then skip).  Only b needs guarding: rows that are done
            // keep their component of L^-1 b.
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
                const float p00 = __shfl_sync(0xFFFFFFFFu, a[j], hb + j);
                const float p10 = __shfl_sync(0xFFFFFFFFu, a[j], hb + j + 1);
                const float p11 = __shfl_sync(0xFFFFFFFFu, a[j + 1], hb + j + 1);
                const float bj = __shfl_sync(0xFFFFFFFFu, b, hb + j);
                const float bj1 = __shfl_sync(0xFFFFFFFFu, b, hb + j + 1);
                // a pivot <= 0 turns into NaN or infinity here and stays visible in 1 / L[row][row] (checked below)
                const float inv0 = rsqrt_fast(p00);
                const float l10 = p10 * inv0;
                const float q11 = fmaf(-l10, l10, p11);
                const float inv1 = rsqrt_fast(q11);
                const float zj = bj * inv0;
                const float zj1 = fmaf(-l10, zj, bj1) * inv1;
                const float x0 = a[j] * inv0;                       // L[row][j]   (row j itself: sqrt of the pivot)
                const float x1 = fmaf(-x0, l10, a[j + 1]) * inv1;   // L[row][j+1] (row j+1 itself: sqrt of the second pivot)
                a[j] = x0;
                a[j + 1] = x1;
                my_inv = (l == j) ? inv0 : ((l == j + 1) ? inv1 : my_inv);
                const float bdown = fmaf(-x1, zj1, fmaf(-x0, zj, b));
                b = (l > j + 1) ? bdown : ((l == j + 1) ? zj1 : ((l == j) ? zj : b));
                // the two new columns go through shared memory (shuffles are the slower path for 2 x 14 values)
                float *xb = &gs.xch[(j & 2) * 16];
                if (is_diag) { xb[l] = x0; xb[16 + l] = x1; }
                __syncwarp();
                float c0[16], c1[16];
#pragma unroll
                for (int q4 = (j + 2) / 4; q4 < 4; ++q4) {
                    const float4 u4 = *reinterpret_cast<const float4 *>(&xb[4 * q4]);
                    const float4 v4 = *reinterpret_cast<const float4 *>(&xb[16 + 4 * q4]);
                    c0[4 * q4] = u4.x; c0[4 * q4 + 1] = u4.y; c0[4 * q4 + 2] = u4.z; c0[4 * q4 + 3] = u4.w;
                    c1[4 * q4] = v4.x; c1[4 * q4 + 1] = v4.y; c1[4 * q4 + 2] = v4.z; c1[4 * q4 + 3] = v4.w;
                }
#pragma unroll
                for (int c = j + 2; c < 16; c += 2) {
                    float2 r = __ffma2_rn(make_float2(-x0, -x0), make_float2(c0[c], c0[c + 1]), make_float2(a[c], a[c + 1]));
                    r = __ffma2_rn(make_float2(-x1, -x1), make_float2(c1[c], c1[c + 1]), r);
                    a[c] = r.x;
                    a[c + 1] = r.y;
                }
            }
            all_ok = __all_sync(0xFFFFFFFFu, !is_diag || (my_inv > 0.f && my_inv <= 3.0e38f));
            if (!all_ok && lane == 0) gs.bad = 1;
            if (is_diag) {
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const float v = (c <= l) ? a[c] : 0.f;
                    gs.Lt[c][l] = v;
                    lrow[c] = v;
                }
                gs.dinv[l] = my_inv;
                gs.z[l] = b;
                my_dinv = my_inv;
            }
        }
        tc_fence_before();
        group128_sync(bar_id);
        if (warp_live && !diag_warp) {
            tc_fence_after();
            load_panel();
        }
        // (2) rows after the block: forward substitution, split, operand tiles
        if (pos >= k0 + 16) {
          if (wpos != (k0 & ~31)) {      // (the rows after the block in its own warp are already done, see above)
            float dv[16];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const float4 v = *reinterpret_cast<const float4 *>(&gs.dinv[4 * q4]);
                dv[4 * q4] = v.x; dv[4 * q4 + 1] = v.y; dv[4 * q4 + 2] = v.z; dv[4 * q4 + 3] = v.w;
            }
            // column-oriented: once a[pp] is final it is eliminated from the later entries, which are
            // independent of each other
#pragma unroll
            for (int pp = 0; pp < 16; ++pp) {
                float lt[16];
#pragma unroll
                for (int q4 = (pp + 1) / 4; q4 < 4; ++q4) {
                    const float4 v = *reinterpret_cast<const float4 *>(&gs.Lt[pp][4 * q4]);
                    lt[4 * q4] = v.x; lt[4 * q4 + 1] = v.y; lt[4 * q4 + 2] = v.z; lt[4 * q4 + 3] = v.w;
                }
                a[pp] *= dv[pp];
                // packed FP32 FMAs on pairs of columns: half the issue slots, which the chains of the other
                // groups on this sub-partition need
                const float mneg = -a[pp];
                if ((pp + 1) & 1) a[pp + 1] = fmaf(mneg, lt[pp + 1], a[pp + 1]);
#pragma unroll
                for (int c = (pp + 2) & ~1; c < 16; c += 2) {
                    const float2 r = __ffma2_rn(make_float2(mneg, mneg), make_float2(lt[c], lt[c + 1]), make_float2(a[c], a[c + 1]));
                    a[c] = r.x;
                    a[c + 1] = r.y;
                }
            }
            float2 acc2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const float4 zz = *reinterpret_cast<const float4 *>(&gs.z[4 * q4]);
                acc2 = __ffma2_rn(make_float2(a[4 * q4], a[4 * q4 + 1]), make_float2(zz.x, zz.y), acc2);
                acc2 = __ffma2_rn(make_float2(a[4 * q4 + 2], a[4 * q4 + 3]), make_float2(zz.z, zz.w), acc2);
            }
            b -= acc2.x + acc2.y;
          }
            uint32_t w1[8], w2[8], w3[8];
#pragma unroll
            for (int c = 0; c < 16; c += 2) {
                // part 1 rounds to nearest (one packed conversion); parts 2 and 3 keep the leading 8 bits of
                // what is left, so p1 + p2 + p3 = p up to 2^-24
                const __nv_bfloat162 hpair = __floats2bfloat162_rn(a[c], a[c + 1]);
                const uint32_t hw = *reinterpret_cast<const uint32_t *>(&hpair);
                // (packed arithmetic: x - y as fma(y, -1, x) on both lanes; the upper halves of two words are
                // gathered by one byte permutation)
                const float2 minus1 = make_float2(-1.f, -1.f);
                const float2 r = __ffma2_rn(make_float2(__uint_as_float(hw << 16), __uint_as_float(hw & 0xFFFF0000u)), minus1,
                                            make_float2(a[c], a[c + 1]));
                const uint32_t m0 = __float_as_uint(r.x) & 0xFFFF0000u, m1 = __float_as_uint(r.y) & 0xFFFF0000u;
                const float2 sres = __ffma2_rn(make_float2(__uint_as_float(m0), __uint_as_float(m1)), minus1, r);
                w1[c >> 1] = hw;
                w2[c >> 1] = __byte_perm(m0, m1, 0x7632);
                w3[c >> 1] = __byte_perm(__float_as_uint(sres.x), __float_as_uint(sres.y), 0x7632);
            }
            const uint32_t roff = (uint32_t)((i >> 3) * 256 + (i & 7) * 16);
            const uint32_t b1 = smem_u32(&gs.pop[0][0]) + roff, b2 = smem_u32(&gs.pop[1][0]) + roff,
                           b3 = smem_u32(&gs.pop[2][0]) + roff;
            st_shared_v4(b1, w1[0], w1[1], w1[2], w1[3]); st_shared_v4(b1 + 128, w1[4], w1[5], w1[6], w1[7]);
            st_shared_v4(b2, w2[0], w2[1], w2[2], w2[3]); st_shared_v4(b2 + 128, w2[4], w2[5], w2[6], w2[7]);
            st_shared_v4(b3, w3[0], w3[1], w3[2], w3[3]); st_shared_v4(b3 + 128, w3[4], w3[5], w3[6], w3[7]);
            fence_proxy_async();
        }
        if (warp_live) {
            tmem_st16(trow + ck, a);      // L (rows before the block rewrite what they read)
            tmem_st_wait();
        }
        tc_fence_before();
        group128_sync(bar_id);
        // (3) trailing update on the tensor core.  The issuing thread changes with the step: lane 0 of the warp two
        // blocks of 32 rows further on (cyclically), which never holds the next diagonal block.  It
        // issues the update and commits it to the group's mbarrier (a tcgen05.mma takes the issuing thread about
        // 50 cycles); the next step's diagonal warp waits for it.
        const bool issuer = (lane == 0) && (wpos == ((k0 + 16 + 64) & 96));
        uint64_t da[3] = {0, 0, 0};
        // columns [c_lo, c_lo + n) of the matrix (= panel rows c_lo ..) -= P P^T restricted to them
        auto update = [&](int c_lo, int n) {
            const uint32_t idesc = idesc_bf16_k_major_negA(128, n);
            uint64_t db[3];
#pragma unroll
            for (int q = 0; q < 3; ++q) db[q] = smem_desc(smem_u32(&gs.pop[q][0]) + (uint32_t)(c_lo * 32), 128, 256, 0);
            umma_f16(d_base + c_lo, da[0], db[0], idesc, true);
            umma_f16(d_base + c_lo, da[0], db[1], idesc, true);
            umma_f16(d_base + c_lo, da[1], db[0], idesc, true);
            umma_f16(d_base + c_lo, da[0], db[2], idesc, true);
            umma_f16(d_base + c_lo, da[2], db[0], idesc, true);
            umma_f16(d_base + c_lo, da[1], db[1], idesc, true);
        };
        if (k < D / 16 - 1 && issuer) {
            tc_fence_after();
#pragma unroll
            for (int q = 0; q < 3; ++q) da[q] = smem_desc(smem_u32(&gs.pop[q][0]), 128, 256, 0);
            // all trailing columns in one set of six instructions: the tensor pipe takes about 50 cycles per
            // instruction whatever its width, and it is shared by the four groups and the gather
            update(k0 + 16, D - k0 - 16);
            umma_commit(&gs.trail_bar);
        }
        if (k < D / 16 - 1) trail_parity ^= 1u;
    }
    group128_sync(bar_id);
    if (gs.stop) return 0.f;
    // my column of the inverse of my diagonal block.  The eight blocks go through shared memory, in the operand
    // tiles: every trailing update has completed (the last one was waited for before the last block step).
    float yinv[16];
    {
        float *Lall = reinterpret_cast<float *>(&gs.pop[0][0]);      // [8 blocks][16][16], transposed
        float *dall = Lall + 8 * 256;                                 // [128] reciprocals of the diagonal
        float *Lb = Lall + (pos >> 4) * 256;
        const int l = pos & 15;
#pragma unroll
        for (int c = 0; c < 16; ++c) Lb[c * 16 + l] = lrow[c];
        dall[pos] = my_dinv;
        __syncwarp();
        const float *dvb = dall + (pos & ~15);
        float tacc[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) tacc[c] = 0.f;
#pragma unroll
        for (int cp = 0; cp < 16; ++cp) {
            // y[cp] of the solve L y = e_l
            const float ycp = (cp < l) ? 0.f : ((cp == l) ? dvb[cp] : -tacc[cp] * dvb[cp]);
            yinv[cp] = ycp;
            float lt[16];
#pragma unroll
            for (int q4 = (cp + 1) / 4; q4 < 4; ++q4) {
                const float4 v = *reinterpret_cast<const float4 *>(&Lb[cp * 16 + 4 * q4]);
                lt[4 * q4] = v.x; lt[4 * q4 + 1] = v.y; lt[4 * q4 + 2] = v.z; lt[4 * q4 + 3] = v.w;
            }
            if ((cp + 1) & 1) tacc[cp + 1] = fmaf(lt[cp + 1], ycp, tacc[cp + 1]);
#pragma unroll
            for (int c = (cp + 2) & ~1; c < 16; c += 2) {
                const float2 r = __ffma2_rn(make_float2(lt[c], lt[c + 1]), make_float2(ycp, ycp), make_float2(tacc[c], tacc[c + 1]));
                tacc[c] = r.x;
                tacc[c + 1] = r.y;
            }
        }
    }
    // (4) back substitution L^T x = z; b now holds z_i
    float x = 0.f;
    for (int k = D / 16 - 1; k >= 0; --k) {
        const int k0 = 16 * k;
        const int ck = k0;
        float wv[16];
        if (wpos + 31 >= k0 + 16) {
            tmem_ld16(trow + ck, wv);
            const float xm = (pos >= k0 + 16) ? x : 0.f;
#pragma unroll
            for (int c = 0; c < 16; c += 2) {
                const float2 r = __fmul2_rn(make_float2(wv[c], wv[c + 1]), make_float2(xm, xm));
                wv[c] = (pos >= k0 + 16) ? r.x : 0.f;
                wv[c + 1] = (pos >= k0 + 16) ? r.y : 0.f;
            }
            warp_reduce16(wv, lane);
        } else {
            wv[0] = 0.f;
        }
        if ((lane & 1) == 0) gs.red[k & 1][w][lane >> 1] = wv[0];
        group128_sync(bar_id);
        if (wpos == (k0 & ~31)) {
            const int hb = k0 & 16;
            const int l = lane - hb;
            const bool is_diag = (l >= 0 && l < 16);
            float rhs = 0.f;
            if (is_diag) rhs = b - (((gs.red[k & 1][0][l] + gs.red[k & 1][1][l]) + gs.red[k & 1][2][l]) + gs.red[k & 1][3][l]);
            float acc = 0.f;
#pragma unroll
            for (int cp = 0; cp < 16; ++cp) {
                const float r = __shfl_sync(0xFFFFFFFFu, rhs, hb + cp);
                acc = fmaf(yinv[cp], r, acc);     // yinv[cp] = Linv[cp][l], zero for cp < l
            }
            if (is_diag) x = acc;
        }
    }
    return x;
}

// Sums of two values over the warp with five shuffles instead of ten: the first exchange leaves the pair sum of `a` in
// the even lanes and of `b` in the odd lanes, four more rounds complete them.  Returns the total of `a` in even lanes,
// of `b` in odd lanes (a fixed order of additions).
__device__ __forceinline__ float warp_sum_pair(float a, float b, int lane)
{
    const bool odd = (lane & 1) != 0;
    float m = (odd ? b : a) + __shfl_xor_sync(0xFFFFFFFFu, odd ? a : b, 1);
#pragma unroll
    for (int o = 2; o < 32; o <<= 1) m += __shfl_xor_sync(0xFFFFFFFFu, m, o);
    return m;
}

// The 16x128b tensor-memory shape as the conjugate-gradient solve uses it: thread (g, q) = (lane / 4, lane % 4) of warp w
// sees rows 32w + g + 8k (k = 0 .. 3) of the matrix at the columns of its class, q + 4j.  One load brings 32 columns by
// 16 lanes: cur[2j] = (row k = 2h, column 32cb + q + 4j), cur[2j + 1] = (row k = 2h + 1, same column), j = 0 .. 7.
//
// Partial sums of the product A v for this thread's four rows over its column class: acc01 = rows k = 0, 1; acc23 =
// rows k = 2, 3.  The next load is in flight while the current one is multiplied.  vq: the vector by column class,
// vq[q * kQStride + j] = v[q + 4j].
__device__ __forceinline__ void cg_matvec(uint32_t twarp, const float *vq, int q, float2 &acc01, float2 &acc23)
{
    float a[2][16];
    float2 vv[8];
    float2 s01[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)}, s23[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
    tmem_ld_16x128b_x8_nowait(twarp, a[0]);
#pragma unroll
    for (int step = 0; step < 8; ++step) {
        const int h = step & 1, cb = step >> 1;         // lane half (rows k = 2h, 2h + 1), block of 32 columns
        float (&cur)[16] = a[step & 1];
        float (&nxt)[16] = a[(step + 1) & 1];
        if (h == 0) {       // the eight vector entries of this block of columns serve both lane halves
            const float4 v0 = *reinterpret_cast<const float4 *>(vq + q * kQStride + 8 * cb);
            const float4 v1 = *reinterpret_cast<const float4 *>(vq + q * kQStride + 8 * cb + 4);
            vv[0] = make_float2(v0.x, v0.x); vv[1] = make_float2(v0.y, v0.y); vv[2] = make_float2(v0.z, v0.z);
            vv[3] = make_float2(v0.w, v0.w); vv[4] = make_float2(v1.x, v1.x); vv[5] = make_float2(v1.y, v1.y);
            vv[6] = make_float2(v1.z, v1.z); vv[7] = make_float2(v1.w, v1.w);
        }
        tmem_ld_wait16(cur);
        if (step + 1 < 8)
            tmem_ld_16x128b_x8_nowait(twarp + ((uint32_t)(((step + 1) & 1) * 16) << 16) + 32 * ((step + 1) >> 1), nxt);
        float2 (&dst)[2] = h ? s23 : s01;
#pragma unroll
        for (int j = 0; j < 8; ++j)
            dst[j & 1] = __ffma2_rn(make_float2(cur[2 * j], cur[2 * j + 1]), vv[j], dst[j & 1]);
    }
    acc01 = __fadd2_rn(s01[0], s01[1]);
    acc23 = __fadd2_rn(s23[0], s23[1]);
}

// Conjugate gradients on (A' + alpha0 G + lambda I) x = b with the matrix in tensor memory (Sec. 4.5: the solver of the
// paper's results).  Start: x = 0, or (cg_warm) the row's stored embedding x0 -- one more product for r = b - A x0, taken
// back to x = 0 when |r| > |b|.  The matrix is read through the 16x128b shape: thread (g, q) = (lane / 4, lane % 4) of
// warp w multiplies rows 32w + g + 8k (k = 0 .. 3) by the vector's entries of its column class q, the four threads of a
// quad exchange their partial sums so that thread (g, q) ends up with the product's component of row 32w + g + 8q: the
// row it owns (component of x, r, p and A p).  The vector of the next product goes through shared memory, stored by
// column class.  One fused reduction per step: the recurrences are arranged so that the product is taken with the
// residual (w = A r; p and s = A p follow by recurrence), and |r|^2 and r.w are reduced together (warp butterfly, then
// the four warps in order: a fixed order).  The accumulator started as alpha0 G + lambda I (the MMA warp copies it in
// before the item's outer products), so the matrix in tensor memory is complete.
// Returns true with the owned component of x when
// |r| <= tol |b|; false when the step limit is reached or a step length is not positive (the matrix is left complete
// in tensor memory, and the caller solves it directly).
__device__ __forceinline__ bool cg_in_tmem(const Params &p, CgGroupSmem &gs, uint32_t twarp, int bar_id,
                                           int tid, float b, float x0, float &x_out, int &matvecs)
{
    const int lane = tid & 31, w = tid >> 5, g = lane >> 2, q = lane & 3;
    const int own = 32 * w + g + 8 * q;                          // the row this thread owns
    float *vq = reinterpret_cast<float *>(&gs.pop[0][0]);       // the vector of the next product
    float *red = vq + 4 * kQStride;                              // [3 sums][4 warps]
    float *vslot = vq + (own & 3) * kQStride + (own >> 2);
    // product with the vector in shared memory; this thread's component of the result
    auto product = [&]() {
        float2 acc01, acc23;
        cg_matvec(twarp, vq, q, acc01, acc23);
        // quad exchange: after two rounds thread q holds the sum over the quad of the partial sums of row k = q
        const bool hi = (q & 2) != 0;                           // keeps rows 2, 3 and sends rows 0, 1
        const float send0 = hi ? acc01.x : acc23.x, send1 = hi ? acc01.y : acc23.y;
        const float keep0 = hi ? acc23.x : acc01.x, keep1 = hi ? acc23.y : acc01.y;
        const float t0 = keep0 + __shfl_xor_sync(0xFFFFFFFFu, send0, 2);
        const float t1 = keep1 + __shfl_xor_sync(0xFFFFFFFFu, send1, 2);
        const bool odd = (q & 1) != 0;                          // keeps the odd row of its pair
        const float send = odd ? t0 : t1, keep = odd ? t1 : t0;
        return keep + __shfl_xor_sync(0xFFFFFFFFu, send, 1);
    };
    bool warm = p.cg_warm != 0;
    float x = warm ? x0 : 0.f, r = b, pdir = 0.f, sdir = 0.f;
    float rg_old = 0.f, inv_alpha_old = 0.f, bb = 0.f;
    int products = 0;
    *vslot = warm ? x0 : b;
    group128_sync(bar_id);
    if (warm) {                 // r = b - A x0
        r = b - product();
        ++products;
        group128_sync(bar_id);  // every thread has read the vector
        *vslot = r;
        group128_sync(bar_id);
    }
    bool ok = false;
    for (int it = 0;; ++it) {
        const float wv = product();
        ++products;
        // |r|^2 and r.w of the warp with one butterfly: after the first exchange the even lanes carry |r|^2, the odd
        // lanes r.w (red: [4 warps] of |r|^2, then of r.w, then of |b|^2)
        float gsum, dl;
        {
            const float mine = warp_sum_pair(r * r, r * wv, lane);
            if (lane < 2) red[4 * lane + w] = mine;
            if (it == 0) {
                float bsum = b * b;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) bsum += __shfl_xor_sync(0xFFFFFFFFu, bsum, o);
                if (lane == 0) red[8 + w] = bsum;
            }
        }
        group128_sync(bar_id);
        {
            const float4 g4 = *reinterpret_cast<const float4 *>(red), d4 = *reinterpret_cast<const float4 *>(red + 4);
            gsum = ((g4.x + g4.y) + g4.z) + g4.w;
            dl = ((d4.x + d4.y) + d4.z) + d4.w;
            if (it == 0) {
                const float4 b4 = *reinterpret_cast<const float4 *>(red + 8);
                bb = ((b4.x + b4.y) + b4.z) + b4.w;
            }
        }
        if (it == 0 && warm && !(gsum <= bb)) {
            // the start vector is further from the solution than zero is (tables not trained yet): start again from zero
            warm = false;
            x = 0.f;
            r = b;
            group128_sync(bar_id);
            *vslot = r;
            group128_sync(bar_id);
            it = -1;
            continue;
        }
        if (gsum <= p.cg_tol2 * bb) { ok = true; break; }        // (also b = 0: x = 0)
        if (it >= p.cg_max_iter) break;
        const float rg = __fdividef(1.f, gsum);
        const float beta = gsum * rg_old;                        // 0 at the first step
        const float inv_alpha = dl * rg - beta * inv_alpha_old;  // p.A p / |r|^2
        if (!(inv_alpha > 0.f) || !(inv_alpha <= 3.0e38f)) break;
        const float alpha = __fdividef(1.f, inv_alpha);
        pdir = fmaf(beta, pdir, r);
        sdir = fmaf(beta, sdir, wv);
        x = fmaf(alpha, pdir, x);
        r = fmaf(-alpha, sdir, r);
        rg_old = rg;
        inv_alpha_old = inv_alpha;
        *vslot = r;
        group128_sync(bar_id);
    }
    // (every thread took the same branches: the reduced values are the same in all of them)
    matvecs = products;
    x_out = x;
    return ok;
}

// FROM_SUMS: the items are rows whose sums were formed by the chunks kernel (split rows: several chunks, added here
// in ascending order; long whole rows: one sum each); the group loads them into its accumulator itself, no producer
// or MMA warp takes part.
template <bool FROM_SUMS, bool CG, class SmemRows, class GroupSmem>
__device__ void solver_rows_tmem(const Params &p, SmemRows &sm, GroupSmem &gs, const float *__restrict__ Bs, int gidx,
                                 int tid)
{
    static_assert(!(FROM_SUMS && CG), "the rows whose sums come from the chunks kernel are solved directly");
    constexpr int kGroups = Cfg<kModeRows>::kGroups, kAccStride = Cfg<kModeRows>::kAccStride;
    const int lane = tid & 31, w = tid >> 5;     // w = lane quarter of tensor memory (= the SM sub-partition)
    const int i = tid;                           // my row of the matrix (= feature index = tensor-memory lane)
    const int wpos = i & ~31;                    // first row of my warp
    const int bar_id = 1 + gidx;
    const uint32_t trow = sm.tmem_base + ((uint32_t)(w * 32) << 16) + gidx * kAccStride;
    const float *Brow = Bs + i * kLdB;
    // (CG: Bs holds alpha0 G + lambda I as the MMA warp's copy source; the solver does not read it)
    const int own_cg = 32 * w + (lane >> 2) + 8 * (lane & 3);
    uint32_t trail_parity = 0;
    unsigned cg_rows = 0, cg_matvecs = 0;      // thread 0 of the group counts (per block: far below 2^32)
    for (int it = gidx;; it += kGroups) {      // this group's items: every fourth of the block's
        const int64_t t = (int64_t)blockIdx.x + (int64_t)it * gridDim.x;
        if (t >= p.n_items) break;
        int64_t u, beg, end, slot;
        float b, x0 = 0.f;
        if constexpr (FROM_SUMS) {
            int64_t c0, c1;      // the row's sums: slots c0 .. c1 - 1 of the workspace
            if (t < p.n_split_rows) {
                u = p.sv.order[p.split_begin + t];
                c0 = p.sv.split_first[t];
                c1 = p.sv.split_first[t + 1];
            } else {
                const int64_t j = t - p.n_split_rows;
                u = p.sv.order[p.long_end - 1 - j];
                c0 = p.n_chunks + j;
                c1 = c0 + 1;
            }
            if (tid == 0) { gs.stop = 0; gs.bad = 0; }
            // my row of the lower triangle (16-column blocks up to my own) and my component of the right-hand side
            constexpr int64_t kSum = (int64_t)D * D + D;
            const float *base = p.partials + c0 * kSum;
            b = 0.f;
            for (int64_t c = c0; c < c1; ++c) b += p.partials[c * kSum + D * D + i];
#pragma unroll 1
            for (int cb = 0; cb <= (wpos + 31) / 16; ++cb) {
                float acc[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) acc[e] = 0.f;
                const float *src = base + (int64_t)i * D + 16 * cb;
                for (int64_t c = c0; c < c1; ++c, src += kSum) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const float4 v = *reinterpret_cast<const float4 *>(src + 4 * q4);
                        acc[4 * q4] += v.x; acc[4 * q4 + 1] += v.y; acc[4 * q4 + 2] += v.z; acc[4 * q4 + 3] += v.w;
                    }
                }
                tmem_st16(trow + 16 * cb, acc);
            }
            tmem_st_wait();
            tc_fence_before();
            group128_sync(bar_id);
            tc_fence_after();
        } else {
            item_range<CG ? kModeRowsCg : kModeRows>(p, t, u, beg, end, slot);
            if constexpr (CG) {       // the start vector: the row's stored embedding (read before the wait for the sums)
                if (p.cg_warm) x0 = __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p.out.table)[u * D + own_cg]);
            }
            const uint32_t aph = (uint32_t)((it / kGroups) & 1);
            // one thread polls, the group follows through its barrier (a failed wait sets the block's abort flag)
            if (tid == 0) {
                bool ok = mbar_wait_parked(&sm.acc_full[gidx], aph, &sm.abort_flag, 60);
                if constexpr (CG) {       // (the right-hand side follows the stages' landing on a barrier of its own)
                    constexpr int kBRing = Ring<kModeRowsCg>::kBRing;
                    ok = ok && mbar_wait_parked(&sm.rhs_done[it % kBRing], (uint32_t)((it / kBRing) & 1), &sm.abort_flag, 61);
                }
                gs.stop = ok ? 0 : 1;
                gs.bad = 0;
            }
            group128_sync(bar_id);
            if (gs.stop) break;
            tc_fence_after();
            if constexpr (CG) {
                b = sm.bpart[it % Ring<kModeRowsCg>::kBRing][0][own_cg];
            } else {      // right-hand side: the four producer warps' partial sums, in order
                const float *bp = &sm.bpart[it % Ring<kModeRows>::kBRing][0][i];
                b = ((bp[0] + bp[D]) + bp[2 * D]) + bp[3 * D];
            }
        }
        float x = 0.f;
        int own = i;                  // the row whose solution this thread holds at the end
        bool solved = true;
        if constexpr (CG) {
            int matvecs = 0;
            solved = cg_in_tmem(p, gs, sm.tmem_base + ((uint32_t)(w * 32) << 16) + gidx * kAccStride, bar_id, tid, b, x0,
                                x, matvecs);
            own = own_cg;
            if (tid == 0) {
                ++cg_rows;
                cg_matvecs += matvecs;
                if (!solved) p.fallback_list[atomicAdd(p.fallback_count, 1ull)] = (int32_t)u;    // left to the direct solve
            }
        } else {
            x = chol_in_tmem(sm, gs, Brow, trow, sm.tmem_base + gidx * kAccStride, bar_id, tid, b, true, trail_parity);
            if (gs.stop) break;
        }
        // tensor memory is free again for the next item of this accumulator
        tc_fence_before();
        group128_sync(bar_id);
        if (!FROM_SUMS && tid == 0) mbar_arrive(&sm.acc_empty[gidx]);
        const bool ok = gs.bad == 0;
        const float xo = ok ? x : 0.f;
        if (solved) {
            reinterpret_cast<__nv_bfloat16 *>(p.out.table)[u * D + own] = __float2bfloat16_rn(xo);
            if (p.out.cap_slot) {
                const int cs = p.out.cap_slot[u];
                if (cs >= 0) p.out.cap_out[(int64_t)cs * D + own] = xo;
            }
        }
        if (!ok && tid == 0) {
            atomicAdd(&p.st->not_spd, 1ull);
            raise_flag(p.st, kFlagNotSpd, u);
        }
        group128_sync(bar_id);      // gs.bad is reset at the top of the next item
    }
    if (tid == 0 && cg_rows && p.cg_counters) {
        atomicAdd(&p.cg_counters[0], (unsigned long long)cg_rows);
        atomicAdd(&p.cg_counters[1], (unsigned long long)cg_matvecs);
    }
}



// ---------------------------------------------------------------------------------------------------------
// kModeRowsFold: the 64 x 64 system of an fp32 table of 64 features (Eq. 4), folded out of the 128 x 128 sums.
// A solver group's 128 threads hold the folded matrix in registers: thread (i, h) = (tid & 63, tid >> 6) has columns
// 32 h .. 32 h + 31 of row i.  Conjugate gradients (Sec. 4.5) run on it with the vector in shared memory (two named
// barriers per step); a row that does not converge, and every row under the Cholesky option, is factored in shared
// memory column by column.
constexpr int kFoldD = 64;
constexpr int kFoldLd = 65;                              // row stride of the matrix in shared memory (bank = row + column)
struct __align__(128) FoldGroupSmem {
    float M[kFoldD * 66];                                // the exchange buffers of the fold, then the matrix of the direct solve
    alignas(16) float vec[kFoldD];                       // the vector of the next product
    float ws[2][kFoldD];                                 // the two column halves' parts of a product
    alignas(16) float red[4][4];                         // per-warp sums of a step
    float dinv[kFoldD];
    float zs[kFoldD];
    int bad;
    int stop;
};
static_assert(kMaxGroups * sizeof(FoldGroupSmem) <= sizeof(float) * D * kLdBq + kMaxGroups * sizeof(CgGroupSmem),
              "the fold's scratch takes the place of the 128-feature solver's");

// Conjugate gradients on the folded matrix: a[k] = A[i][32 h + k], b and x0 = this row's components.  Same recurrences,
// start rule and stopping rule as cg_in_tmem.  Returns true with x_i when |r| <= tol |b|.
__device__ __forceinline__ bool fold_cg(const Params &p, FoldGroupSmem &gs, const float (&a)[32], int bar_id, int tid,
                                        float b, float x0, float &x_out, int &matvecs)
{
    const int lane = tid & 31, w = tid >> 5, i = tid & 63, h = tid >> 6;
    // product with the vector in gs.vec: my half row's part, with this thread's share of r.w (v = the vector's own
    // component); the parts and the warps' sums go through shared memory behind one barrier
    auto product_and_sums = [&](float v, float bb_term, bool want_b, float &gsum, float &dl, float &bsum) {
        float acc0 = 0.f, acc1 = 0.f;
        const float4 *vp = reinterpret_cast<const float4 *>(gs.vec + 32 * h);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float4 q = vp[k];
            acc0 = fmaf(a[4 * k], q.x, acc0);
            acc1 = fmaf(a[4 * k + 1], q.y, acc1);
            acc0 = fmaf(a[4 * k + 2], q.z, acc0);
            acc1 = fmaf(a[4 * k + 3], q.w, acc1);
        }
        const float part = acc0 + acc1;
        gs.ws[h][i] = part;
        // (red: [3 sums][4 warps]; |v|^2 and |b|^2 come from the warps of the first column half alone)
        const float m = warp_sum_pair(h == 0 ? v * v : 0.f, v * part, lane);
        if (lane < 2) gs.red[lane][w] = m;
        if (want_b) {
            float s2 = h == 0 ? bb_term : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
            if (lane == 0) gs.red[2][w] = s2;
        }
        group128_sync(bar_id);
        const float4 g4 = *reinterpret_cast<const float4 *>(&gs.red[0][0]), d4 = *reinterpret_cast<const float4 *>(&gs.red[1][0]);
        gsum = g4.x + g4.y;
        dl = ((d4.x + d4.y) + d4.z) + d4.w;
        bsum = want_b ? gs.red[2][0] + gs.red[2][1] : 0.f;
        return gs.ws[0][i] + gs.ws[1][i];
    };
    bool warm = p.cg_warm != 0;
    float x = warm ? x0 : 0.f, r = b, pdir = 0.f, sdir = 0.f;
    float rg_old = 0.f, inv_alpha_old = 0.f, bb = 0.f;
    int products = 0;
    if (h == 0) gs.vec[i] = warm ? x0 : b;
    group128_sync(bar_id);
    if (warm) {                 // r = b - A x0
        float g0, d0, b0;
        r = b - product_and_sums(x0, 0.f, false, g0, d0, b0);
        ++products;
        // (the vector was read before the barrier inside the product; the parts and sums are read before the next one)
        if (h == 0) gs.vec[i] = r;
        group128_sync(bar_id);
    }
    bool ok = false;
    for (int it = 0;; ++it) {
        float gsum, dl, bsum;
        const float wv = product_and_sums(r, b * b, it == 0, gsum, dl, bsum);
        ++products;
        if (it == 0) bb = bsum;
        if (it == 0 && warm && !(gsum <= bb)) {
            // the start vector is further from the solution than zero is: start again from zero
            warm = false;
            x = 0.f;
            r = b;
            if (h == 0) gs.vec[i] = r;
            group128_sync(bar_id);
            it = -1;
            continue;
        }
        if (gsum <= p.cg_tol2 * bb) { ok = true; break; }        // (also b = 0: x = 0)
        if (it >= p.cg_max_iter) break;
        const float rg = __fdividef(1.f, gsum);
        const float beta = gsum * rg_old;                        // 0 at the first step
        const float inv_alpha = dl * rg - beta * inv_alpha_old;  // p.A p / |r|^2
        if (!(inv_alpha > 0.f) || !(inv_alpha <= 3.0e38f)) break;
        const float alpha = __fdividef(1.f, inv_alpha);
        pdir = fmaf(beta, pdir, r);
        sdir = fmaf(beta, sdir, wv);
        x = fmaf(alpha, pdir, x);
        r = fmaf(-alpha, sdir, r);
        rg_old = rg;
        inv_alpha_old = inv_alpha;
        if (h == 0) gs.vec[i] = r;
        group128_sync(bar_id);
    }
    group128_sync(bar_id);          // (the scratch is free for whatever follows)
    if (ok && products >= kCgVerifyProducts) {
        // After many steps the residual of the recurrence can have drifted away from b - A x (its rounding errors add up
        // with the condition of the matrix): look at the true residual once, with one more product, and leave the row to
        // the direct solve if it is not what the recurrence says.  (The 128-feature kernel does not do this: there the
        // check costs 1.5-3 % of the kernel's time for rows that, with its step limit and the per-side policy, have
        // always passed their residual gate.)
        if (h == 0) gs.vec[i] = x;
        group128_sync(bar_id);
        float g0, d0, b0;
        const float rt = b - product_and_sums(x, 0.f, false, g0, d0, b0);
        ++products;
        group128_sync(bar_id);      // the sums of the product have been read
        float tsum = h == 0 ? rt * rt : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tsum += __shfl_xor_sync(0xFFFFFFFFu, tsum, o);
        if (lane == 0) gs.red[w][0] = tsum;
        group128_sync(bar_id);
        tsum = gs.red[0][0] + gs.red[1][0];
        if (!(tsum <= kCgVerifySlack * kCgVerifySlack * p.cg_tol2 * bb)) ok = false;
        group128_sync(bar_id);
    }
    matvecs = products;
    x_out = x;
    return ok;
}

// Direct solve of the folded system: the matrix goes to shared memory, Cholesky column by column, then the two
// substitutions, one column per step.  Returns x_i; a non-positive pivot sets gs.bad.
__device__ __forceinline__ float fold_cholesky(FoldGroupSmem &gs, const float (&a)[32], int bar_id, int tid, float b)
{
    const int i = tid & 63, h = tid >> 6;
    float *M = gs.M;
#pragma unroll
    for (int k = 0; k < 32; ++k) M[i * kFoldLd + 32 * h + k] = a[k];
    group128_sync(bar_id);
    for (int k = 0; k < kFoldD; ++k) {
        const float piv = M[k * kFoldLd + k];
        if (!(piv > 0.f)) {             // (every thread reads the same value)
            if (tid == 0) gs.bad = 1;
            return 0.f;
        }
        const float inv = rsqrtf(piv);
        if (tid == 0) gs.dinv[k] = inv;
        if (h == 0 && i > k) M[i * kFoldLd + k] *= inv;
        group128_sync(bar_id);
        // trailing update of the lower triangle: row i, columns k + 1 .. i, every second one per half
        if (i > k) {
            const float lik = M[i * kFoldLd + k];
            for (int c = k + 1 + h; c <= i; c += 2) M[i * kFoldLd + c] = fmaf(-lik, M[c * kFoldLd + k], M[i * kFoldLd + c]);
        }
        group128_sync(bar_id);
    }
    // L z = b, then L^T x = z: the thread of row i carries its component; column k is final at step k
    float v = b;
    for (int k = 0; k < kFoldD; ++k) {
        if (tid == k) gs.zs[k] = v * gs.dinv[k];
        group128_sync(bar_id);
        if (i > k) v = fmaf(-M[i * kFoldLd + k], gs.zs[k], v);
    }
    group128_sync(bar_id);
    v = gs.zs[i];
    group128_sync(bar_id);
    for (int k = kFoldD - 1; k >= 0; --k) {
        if (tid == k) gs.zs[k] = v * gs.dinv[k];
        group128_sync(bar_id);
        if (i < k) v = fmaf(-M[k * kFoldLd + i], gs.zs[k], v);
    }
    group128_sync(bar_id);
    const float x = gs.zs[i];
    group128_sync(bar_id);
    return x;
}

// Adds alpha0 G + lambda I (64 x 64, from global memory: 16 KB that stay in L1) to the folded half row, solves, stores.
__device__ __forceinline__ void fold_solve_store(const Params &p, FoldGroupSmem &gs, float (&a)[32], int bar_id, int tid,
                                                 int64_t u, float b, float x0, bool use_cg, unsigned &cg_rows,
                                                 unsigned &cg_matvecs, unsigned &cg_fallbacks)
{
    const int i = tid & 63, h = tid >> 6;
    const float4 *Bp = reinterpret_cast<const float4 *>(p.Bmat + i * kFoldD + 32 * h);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const float4 q = __ldg(Bp + k);
        a[4 * k] += q.x; a[4 * k + 1] += q.y; a[4 * k + 2] += q.z; a[4 * k + 3] += q.w;
    }
    float x = 0.f;
    bool solved = false;
    if (use_cg) {
        int matvecs = 0;
        solved = fold_cg(p, gs, a, bar_id, tid, b, x0, x, matvecs);
        if (tid == 0) {
            ++cg_rows;
            cg_matvecs += matvecs;
            if (!solved) ++cg_fallbacks;
        }
    }
    if (!solved) x = fold_cholesky(gs, a, bar_id, tid, b);
    group128_sync(bar_id);
    const bool ok = gs.bad == 0;
    const float xo = ok ? x : 0.f;
    if (h == 0) {
        reinterpret_cast<float *>(p.out.table)[u * kFoldD + i] = xo;
        if (p.out.cap_slot) {
            const int cs = p.out.cap_slot[u];
            if (cs >= 0) p.out.cap_out[(int64_t)cs * kFoldD + i] = xo;
        }
    }
    if (!ok && tid == 0) {
        atomicAdd(&p.st->not_spd, 1ull);
        raise_flag(p.st, kFlagNotSpd, u);
    }
    group128_sync(bar_id);
    if (tid == 0) gs.bad = 0;
}

// solver group of the kModeRowsFold kernel
template <class SmemRows>
__device__ void solver_rows_fold(const Params &p, SmemRows &sm, FoldGroupSmem &gs, int gidx, int tid)
{
    constexpr int kGroups = Cfg<kModeRows>::kGroups, kAccStride = Cfg<kModeRows>::kAccStride;
    constexpr int kBRing = Ring<kModeRowsFold>::kBRing;
    const int w = tid >> 5;
    const int i = tid & 63, h = tid >> 6;
    const int bar_id = 1 + gidx;
    const uint32_t trow = sm.tmem_base + ((uint32_t)(w * 32) << 16) + gidx * kAccStride;   // my lane (= row tid of the sums)
    float *xbuf = gs.M + (1 - h) * (kFoldD * 33);      // where my half sends: [0] rows 0..63 -> the other half, [1] the reverse
    const float *rbuf = gs.M + h * (kFoldD * 33);
    const float scale = h == 0 ? 0.5f : 1.f;           // S11 / 2 + S12 in rows 0..63, S21 + S22 in rows 64..127
    unsigned cg_rows = 0, cg_matvecs = 0, cg_fallbacks = 0;
    if (tid == 0) gs.bad = 0;
    for (int it = gidx;; it += kGroups) {
        const int64_t t = (int64_t)blockIdx.x + (int64_t)it * gridDim.x;
        if (t >= p.n_items) break;
        int64_t u, beg, end, slot;
        item_range<kModeRowsFold>(p, t, u, beg, end, slot);
        const float x0 = p.cg_warm ? reinterpret_cast<const float *>(p.out.table)[u * kFoldD + i] : 0.f;
        const uint32_t aph = (uint32_t)((it / kGroups) & 1);
        if (tid == 0) {
            bool ok = mbar_wait_parked(&sm.acc_full[gidx], aph, &sm.abort_flag, 62);
            ok = ok && mbar_wait_parked(&sm.rhs_done[it % kBRing], (uint32_t)((it / kBRing) & 1), &sm.abort_flag, 63);
            gs.stop = ok ? 0 : 1;
        }
        group128_sync(bar_id);
        if (gs.stop) break;
        tc_fence_after();
        const float *bp = &sm.bpart[it % kBRing][0][0];
        const float b = 0.5f * bp[i] + bp[kFoldD + i];
        // fold: the half that goes to the other half's threads first (through shared memory), then the half I keep
        float a[32];
        {
            const int send0 = 32 * (1 - h);            // first of the 32 folded columns I send
            float lo[16], hi[16];
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                tmem_ld16(trow + send0 + 16 * part, lo);
                tmem_ld16(trow + kFoldD + send0 + 16 * part, hi);
#pragma unroll
                for (int k = 0; k < 16; ++k) xbuf[i * 33 + 16 * part + k] = fmaf(scale, lo[k], hi[k]);
            }
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                tmem_ld16(trow + 32 * h + 16 * part, lo);
                tmem_ld16(trow + kFoldD + 32 * h + 16 * part, hi);
#pragma unroll
                for (int k = 0; k < 16; ++k) a[16 * part + k] = fmaf(scale, lo[k], hi[k]);
            }
        }
        // the sums have been read: the accumulator is free for the MMA warp's next item
        tc_fence_before();
        group128_sync(bar_id);
        if (tid == 0) mbar_arrive(&sm.acc_empty[gidx]);
#pragma unroll
        for (int k = 0; k < 32; ++k) a[k] += rbuf[i * 33 + k];
        group128_sync(bar_id);      // the exchange buffers are free (the direct solve reuses them)
        fold_solve_store(p, gs, a, bar_id, tid, u, b, x0, p.solver != 0, cg_rows, cg_matvecs, cg_fallbacks);
    }
    if (tid == 0 && p.cg_counters) {
        if (cg_rows) atomicAdd(&p.cg_counters[0], (unsigned long long)cg_rows);
        if (cg_matvecs) atomicAdd(&p.cg_counters[1], (unsigned long long)cg_matvecs);
        if (cg_fallbacks) atomicAdd(&p.cg_counters[2], (unsigned long long)cg_fallbacks);
    }
}

// The conjugate-gradient variant runs 24 warps: the 21 of the roles and three idle ones that complete the last
// warpgroup, so that registers can move between warpgroups (setmaxnreg): the four producer warps form one warpgroup
// (64 registers per thread), the MMA warp and the idle warps the next (32), and the solver warps take 96 (their
// matrix-vector product holds two loads of 16 matrix entries, 8 duplicated vector entries and four packed sums).
template <int MODE> constexpr int block_threads() { return is_cg(MODE) ? 768 : Cfg<MODE>::kBlockThreads; }

template <int MODE>
__global__ void __launch_bounds__(block_threads<MODE>(), 1) k_umma(Params p, const __grid_constant__ CUtensorMap tmap)
{
    using C = Cfg<MODE>;
    constexpr bool CG = is_cg(MODE), FOLD = MODE == kModeRowsFold;
    // which rows this launch takes (block-uniform decisions, before any barrier or allocation)
    const bool short_rows_here = is_rows(MODE) && p.route && p.route->short_rows_by_cg;
    if (is_rows(MODE) && p.polish_flag) {
        if (*p.polish_flag != 2) return;
        if (short_rows_here) { p.n_items -= p.n_class2; p.last_item -= p.n_class2; }      // (those rows are not dual-form rows then)
    }
    if (MODE == kModeRowsCg && p.policy && p.policy->use_cholesky) return;      // the Cholesky launch takes them all
    if (MODE == kModeRows && p.item_count && !(p.policy && p.policy->use_cholesky)) {
        p.n_items = (int64_t)*p.item_count;                 // the rows conjugate gradients left over
        if ((int64_t)blockIdx.x >= p.n_items) return;
    } else {
        if (MODE == kModeRows) p.item_list = nullptr;       // (every row: the walk through the degree classes)
        if (is_rows(MODE) && p.dual_flag && *p.dual_flag) p.n_items = p.n_items_primal + (short_rows_here ? p.n_class2 : 0);
        if (is_rows(MODE) && (int64_t)blockIdx.x >= p.n_items) return;
    }
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment for the swizzled stages; plain offset arithmetic on the shared array, so that the
    // compiler keeps every access below in the shared address space (no generic loads)
    unsigned char *aligned = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int kNStage = Ring<MODE>::kNStage;
    SmemT<MODE> &sm = *reinterpret_cast<SmemT<MODE> *>(aligned);
    float *Bs = reinterpret_cast<float *>(aligned + sizeof(SmemT<MODE>));
    using GroupSmem = typename std::conditional<CG, CgGroupSmem, RowGroupSmem>::type;
    GroupSmem *rgs = reinterpret_cast<GroupSmem *>(aligned + sizeof(SmemT<MODE>) + sizeof(float) * D * kLdBq);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kNStage; ++s) { mbar_init(&sm.full[s], C::kFullArrivals); mbar_init(&sm.empty[s], C::kEmptyArrivals); }
        if (CG) for (int s = 0; s < Ring<MODE>::kBRing; ++s) mbar_init(&sm.rhs_done[s], 1);
        for (int a = 0; a < kMaxGroups; ++a) { mbar_init(&sm.acc_full[a], 1); mbar_init(&sm.acc_empty[a], 1); }
        sm.abort_flag = 0;
        sm.stage_meta[0] = 0;      // (conjugate-gradient rows kernel: the producers' turn counter)
        mbar_fence_init();
    }
    // label tiles start finite (all zero): rows beyond an item's end multiply zeros, never stale NaNs
    constexpr int kThreads = block_threads<MODE>();
    for (int k = tid; k < (int)sizeof(sm.y) / 16; k += kThreads)
        st_shared_zero16(smem_u32(&sm.y[0][0]) + k * 16);
    for (int k = tid; k < (int)sizeof(sm.h) / 16; k += kThreads)
        st_shared_zero16(smem_u32(&sm.h[0][0]) + k * 16);
    if constexpr (FOLD) {
        // (alpha0 G + lambda I is 64 x 64 here and read from global memory; the space holds the groups' scratch)
    } else if constexpr (CG) {
        // alpha0 G + lambda I as the source of the tensor-memory copies that start every accumulator: sixteen blocks
        // of 8 columns, each 128 rows x 32 bytes in the layout tmem_cp_128x256b reads (offsets 128 and 256 bytes)
        for (int e = tid; e < D * D; e += kThreads) {
            const int r = e >> 7, c = e & (D - 1);
            Bs[(c >> 3) * 1024 + (r >> 3) * 64 + ((c & 7) >> 2) * 32 + (r & 7) * 4 + (c & 3)] = p.Bmat[e];
        }
    } else if constexpr (MODE == kModeRows) {
        for (int e = tid; e < D * D; e += kThreads) Bs[(e >> 7) * kLdB + (e & (D - 1))] = p.Bmat[e];
        for (int g = 0; g < C::kGroups; ++g) {
            if (tid == 0) mbar_init(&rgs[g].trail_bar, 1);
            for (int k = tid; k < 3 * D * 32 / 16; k += kThreads)
                st_shared_zero16(smem_u32(&rgs[g].pop[0][0]) + k * 16);
        }
        if (tid == 0) mbar_fence_init();
    }
    fence_proxy_async();
    // Roles by warp.  The conjugate-gradient variant puts the producers (one warpgroup), then the MMA warp with three idle
    // warps (the next warpgroup), in front of the sixteen solver warps: the warp scheduler favours low warp numbers when
    // several warps are ready, and the few instructions of the roles that feed the solvers must not queue behind them.
    // `rw` is the warp's number in the order solvers, MMA / producers as the other modes have it.
    constexpr int kMmaWarp = CG ? C::kFirstProducerWarp + C::kProducers - 1 : C::kMmaWarp;      // CG: after the producers
    constexpr int kFirstProducerWarp = CG ? C::kMmaWarp : C::kFirstProducerWarp;
    const int rw = CG ? (warp < 8 ? warp + C::kMmaWarp : warp - 8) : warp;
    const int rtid = rw * 32 + lane;
    if (rw == kMmaWarp) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (rw < C::kMmaWarp) {
        const int gidx = rw / (C::kGroupThreads / 32);
        if constexpr (CG) setmaxnreg_inc<96>();
        if constexpr (FOLD) solver_rows_fold(p, sm, reinterpret_cast<FoldGroupSmem *>(Bs)[gidx], gidx, rtid - gidx * C::kGroupThreads);
        else if constexpr (is_rows(MODE)) solver_rows_tmem<false, CG>(p, sm, rgs[gidx], Bs, gidx, rtid - gidx * C::kGroupThreads);
        else copyout_role<MODE>(p, sm, gidx, rtid - gidx * C::kGroupThreads);
    } else if (CG && rw > kMmaWarp) {
        setmaxnreg_dec<32>();       // idle warps of the last warpgroup
    } else if (rw == kMmaWarp) {
        if constexpr (CG) setmaxnreg_dec<32>();
        mma_role<MODE>(p, sm, lane, smem_u32(Bs));
    } else {
        if constexpr (CG) setmaxnreg_dec<64>();
        if constexpr (CG) producer_role_items<MODE>(p, &tmap, sm, rw - kFirstProducerWarp, lane);
        else if constexpr (is_rows(MODE)) producer_role<MODE>(p, sm, rw - kFirstProducerWarp, lane);
        else stream_producer_role<MODE>(p, &tmap, sm, rw - kFirstProducerWarp, lane);
    }

    tc_fence_before();
    __syncthreads();
    if (rw == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(sm.tmem_base, kTmemCols);
    }
    if (tid == 0 && sm.abort_flag) raise_flag(p.st, kFlagTimeout, (long long)sm.abort_flag * 1000000 + blockIdx.x);
}

// Before a side's whole-rows launches: choose the solver from the side's last conjugate-gradient run.
__global__ void k_cg_policy(CgPolicy *pol, float switch_products)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const int calls = pol->calls++;
    int use = 0;
    if (pol->rows > 0 && (float)pol->products > switch_products * (float)pol->rows) use = 1;
    if (use && (calls % kCgReprobe) == kCgReprobe - 1) use = 0;
    pol->use_cholesky = use;
    pol->short_rows_by_cg = (!use && pol->rows > 0 && (float)pol->products <= kShortRowsByCgProducts * (float)pol->rows) ? 1 : 0;
}
// After them: keep the run's counts (they are cleared at the start of every half-epoch).
__global__ void k_cg_record(CgPolicy *pol, const unsigned long long *counters)
{
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    if (!pol->use_cholesky) {
        pol->rows = counters[0];
        pol->products = counters[1];
    }
}

__global__ void k_zero_rows_bf16(const int32_t *__restrict__ rows, int64_t count, RowOut out)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= count * D) return;
    const int64_t u = rows[t / D];
    const int c = (int)(t % D);
    reinterpret_cast<__nv_bfloat16 *>(out.table)[u * D + c] = __float2bfloat16_rn(0.f);
    if (out.cap_slot) {
        const int slot = out.cap_slot[u];
        if (slot >= 0) out.cap_out[(int64_t)slot * D + c] = 0.f;
    }
}

// Split rows and long whole rows: their sums come from the chunks kernel; four groups of 128 threads load them into
// tensor memory (a split row's chunks added in ascending order) and factor / solve / store as in rows mode.
__global__ void __launch_bounds__(4 * 128, 1) k_solve_sums(Params p)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *aligned = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    Smem &sm = *reinterpret_cast<Smem *>(aligned);
    float *Bs = reinterpret_cast<float *>(aligned + sizeof(Smem));
    RowGroupSmem *rgs = reinterpret_cast<RowGroupSmem *>(aligned + sizeof(Smem) + sizeof(float) * D * kLdBq);
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) sm.abort_flag = 0;
    for (int e = tid; e < D * D; e += blockDim.x) Bs[(e >> 7) * kLdB + (e & (D - 1))] = p.Bmat[e];
    for (int g = 0; g < kMaxGroups; ++g) {
        if (tid == 0) mbar_init(&rgs[g].trail_bar, 1);
        for (int k = tid; k < 3 * D * 32 / 16; k += blockDim.x) st_shared_zero16(smem_u32(&rgs[g].pop[0][0]) + k * 16);
    }
    if (tid == 0) mbar_fence_init();
    fence_proxy_async();
    if (warp == 0) {
        tmem_alloc(&sm.tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    solver_rows_tmem<true, false>(p, sm, rgs[warp >> 2], Bs, warp >> 2, tid & 127);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(sm.tmem_base, kTmemCols);
    }
    if (tid == 0 && sm.abort_flag) raise_flag(p.st, kFlagTimeout, (long long)sm.abort_flag * 1000000 + blockIdx.x);
}

// kModeRowsFold: rows whose sums the chunks kernel formed (split rows: their chunks in ascending order; long whole rows:
// one sum each), folded straight from the workspace.  Four groups of 128 threads per block, no tensor memory.
__global__ void __launch_bounds__(4 * 128) k_solve_sums_fold(Params p)
{
    extern __shared__ unsigned char smem_raw[];
    FoldGroupSmem *groups = reinterpret_cast<FoldGroupSmem *>(smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u));
    const int tid = threadIdx.x & 127, gidx = threadIdx.x >> 7;
    FoldGroupSmem &gs = groups[gidx];
    const int i = tid & 63, h = tid >> 6, bar_id = 1 + gidx;
    if (tid == 0) { gs.bad = 0; gs.stop = 0; }
    group128_sync(bar_id);
    unsigned cg_rows = 0, cg_matvecs = 0, cg_fallbacks = 0;
    constexpr int64_t kSum = (int64_t)D * D + D;
    for (int64_t t = (int64_t)blockIdx.x * 4 + gidx; t < p.n_items; t += (int64_t)gridDim.x * 4) {
        int64_t u, c0, c1;
        if (t < p.n_split_rows) {
            u = p.sv.order[p.split_begin + t];
            c0 = p.sv.split_first[t];
            c1 = p.sv.split_first[t + 1];
        } else {
            const int64_t j = t - p.n_split_rows;
            u = p.sv.order[p.long_end - 1 - j];
            c0 = p.n_chunks + j;
            c1 = c0 + 1;
        }
        float a[32];
#pragma unroll
        for (int k = 0; k < 32; ++k) a[k] = 0.f;
        float b = 0.f;
        for (int64_t c = c0; c < c1; ++c) {
            const float *S = p.partials + c * kSum;
            const float *r0 = S + (int64_t)i * D + 32 * h, *r1 = S + (int64_t)(kFoldD + i) * D + 32 * h;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float4 q11 = *reinterpret_cast<const float4 *>(r0 + 4 * k), q12 = *reinterpret_cast<const float4 *>(r0 + kFoldD + 4 * k);
                const float4 q21 = *reinterpret_cast<const float4 *>(r1 + 4 * k), q22 = *reinterpret_cast<const float4 *>(r1 + kFoldD + 4 * k);
                a[4 * k] += (fmaf(0.5f, q11.x, q12.x) + q21.x) + q22.x;
                a[4 * k + 1] += (fmaf(0.5f, q11.y, q12.y) + q21.y) + q22.y;
                a[4 * k + 2] += (fmaf(0.5f, q11.z, q12.z) + q21.z) + q22.z;
                a[4 * k + 3] += (fmaf(0.5f, q11.w, q12.w) + q21.w) + q22.w;
            }
            b += fmaf(0.5f, S[D * D + i], S[D * D + kFoldD + i]);
        }
        const float x0 = p.cg_warm ? reinterpret_cast<const float *>(p.out.table)[u * kFoldD + i] : 0.f;
        fold_solve_store(p, gs, a, bar_id, tid, u, b, x0, p.solver != 0, cg_rows, cg_matvecs, cg_fallbacks);
    }
    if (tid == 0 && p.cg_counters) {
        if (cg_rows) atomicAdd(&p.cg_counters[0], (unsigned long long)cg_rows);
        if (cg_matvecs) atomicAdd(&p.cg_counters[1], (unsigned long long)cg_matvecs);
        if (cg_fallbacks) atomicAdd(&p.cg_counters[2], (unsigned long long)cg_fallbacks);
    }
}

// fp32 table of 64 features -> 2N rows of 128 bfloat16: row i = [x1 | x2], row N + i = [x1 | x3], x = x1 + x2 + x3 with
// every part the nearest bfloat16 of what the parts before it leave (the remainders are exact in fp32)
__global__ void __launch_bounds__(256) k_split_table(const float *__restrict__ X, int64_t n, __nv_bfloat16 *__restrict__ T)
{
    const int64_t e = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 4;      // four features of one row
    if (e >= n * kFoldD) return;
    const int64_t row = e / kFoldD;
    const int f = (int)(e % kFoldD);
    const float4 x = *reinterpret_cast<const float4 *>(X + e);
    const float xs[4] = {x.x, x.y, x.z, x.w};
    __nv_bfloat16 p1[4], p2[4], p3[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        p1[k] = __float2bfloat16_rn(xs[k]);
        const float r1 = xs[k] - __bfloat162float(p1[k]);
        p2[k] = __float2bfloat16_rn(r1);
        p3[k] = __float2bfloat16_rn(r1 - __bfloat162float(p2[k]));
    }
    __nv_bfloat16 *t1 = T + row * D + f, *t2 = T + (n + row) * D + f;
    *reinterpret_cast<uint2 *>(t1) = *reinterpret_cast<const uint2 *>(p1);
    *reinterpret_cast<uint2 *>(t1 + kFoldD) = *reinterpret_cast<const uint2 *>(p2);
    *reinterpret_cast<uint2 *>(t2) = *reinterpret_cast<const uint2 *>(p1);
    *reinterpret_cast<uint2 *>(t2 + kFoldD) = *reinterpret_cast<const uint2 *>(p3);
}

__global__ void k_zero_rows_f32x64(const int32_t *__restrict__ rows, int64_t count, RowOut out)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= count * kFoldD) return;
    const int64_t u = rows[e / kFoldD];
    const int f = (int)(e % kFoldD);
    reinterpret_cast<float *>(out.table)[u * kFoldD + f] = 0.f;
    if (out.cap_slot) {
        const int cs = out.cap_slot[u];
        if (cs >= 0) out.cap_out[(int64_t)cs * kFoldD + f] = 0.f;
    }
}

template <int MODE> size_t smem_bytes()
{
    // a large request in every mode (more than half of what an SM offers): at most one block per SM, so two
    // blocks never compete for the SM's 512 tensor-memory columns
    size_t b = sizeof(SmemT<MODE>) + 1024;
    if (MODE == kModeRows) b += sizeof(float) * D * kLdBq + kMaxGroups * sizeof(RowGroupSmem);
    if (is_cg(MODE)) b += sizeof(float) * D * kLdBq + kMaxGroups * sizeof(CgGroupSmem);
    return b;
}
static_assert(sizeof(SmemT<1>) + 1024 <= 232448 && sizeof(SmemT<1>) > 116224, "ring depth of the streaming modes");
static_assert(sizeof(SmemT<0>) + 1024 + sizeof(float) * D * kLdBq + kMaxGroups * sizeof(RowGroupSmem) <= 232448, "rows mode");
static_assert(sizeof(SmemT<3>) + 1024 + sizeof(float) * D * kLdBq + kMaxGroups * sizeof(CgGroupSmem) <= 232448, "rows mode, CG");
static_assert(sizeof(SmemT<4>) == sizeof(SmemT<3>), "the fold kernel has the conjugate-gradient kernel's feed");

// Tensor map of a bfloat16 table [n x 128]: boxes of 64 features (128 bytes) by one row for the row gathers, by a stage's
// 64 rows for the tile loads of the Gramian; 128-byte swizzle.
// (The encoder is a driver entry point, looked up through the runtime so that the library needs no driver at link time.)
cudaError_t table_tensor_map(const void *X, int64_t n, CUtensorMap *tm, int box_rows = 1)
{
    typedef CUresult (*Encode)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                               const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Encode encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (e != cudaSuccess) return e;
        if (q != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        encode = reinterpret_cast<Encode>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)n};
    const cuuint64_t strides[1] = {(cuuint64_t)D * sizeof(__nv_bfloat16)};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(X), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int MODE> cudaError_t launch_mode(const Params &p, int grid, cudaStream_t s)
{
    const size_t smem = smem_bytes<MODE>();
    cudaError_t e = cudaFuncSetAttribute(k_umma<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    CUtensorMap tm;
    e = table_tensor_map(p.X, p.n_table, &tm, MODE == kModeGramian ? Ring<MODE>::kRows : 1);
    if (e != cudaSuccess) return e;
    k_umma<MODE><<<grid, block_threads<MODE>(), smem, s>>>(p, tm);
    return cudaGetLastError();
}

int sm_count()
{
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms > 0 ? sms : 1;
}

}  // namespace


int64_t gramian_umma_partials() { return (int64_t)kGramBlocks * Cfg<kModeGramian>::kGroups; }

// Gramian of a bf16 table with d = 128 on the tensor cores; partials must hold gramian_umma_partials() * d * d floats
cudaError_t launch_gramian_umma(const void *X, int64_t n, float *partials, cudaStream_t s, int64_t *launches)
{
    Params p{};
    p.X = reinterpret_cast<const __nv_bfloat16 *>(X);
    p.n_fixed = n;
    p.n_table = n;
    p.n_items = (n + kGramSubRows - 1) / kGramSubRows;
    p.partials = partials;
    cudaError_t e = launch_mode<kModeGramian>(p, kGramBlocks, s);
    ++*launches;
    return e;
}

cudaError_t launch_rows_umma(const SideView &sv, const int64_t *offs, int64_t n_chunks, int64_t n_split_rows,
                             const void *X, const float *Bmat, float *split_partials, RowOut out, DevStatus *st,
                             cudaStream_t s, int64_t *launches, cudaEvent_t main_begin, cudaEvent_t main_end,
                             const void *dual_ws, int64_t n_table, const CgOptions &cg, const int32_t *order16, int64_t n4, int64_t n8)
{
    const int sms = sm_count();
    Params p{};
    p.sv = sv;
    p.X = reinterpret_cast<const __nv_bfloat16 *>(X);
    p.n_table = n_table;
    p.Bmat = Bmat;
    p.partials = split_partials;
    p.out = out;
    p.st = st;
    cudaError_t e;
    // Rows of more than 1024 observations (as many classes from the top as the workspace budget allows) do not go
    // through the rows kernel, whose gather holds 64 KB in flight per SM: the chunks kernel (192 KB in flight)
    // forms their sums, one per row, behind the sums of the split rows' chunks.
    const int c_long = long_class_begin(offs);
    const int64_t n_long = offs[kNClasses - 1] - offs[c_long];
    if (n_chunks + n_long > 0) {
        p.n_chunks = n_chunks;
        p.long_end = offs[kNClasses - 1];
        p.n_items = n_chunks + n_long;
        e = launch_mode<kModeChunks>(p, (int)(p.n_items < sms ? p.n_items : sms), s);
        ++*launches;
        if (e != cudaSuccess) return e;
        p.split_begin = offs[kNClasses - 1];
        p.n_split_rows = n_split_rows;
        p.n_items = n_split_rows + n_long;
        const size_t smem = smem_bytes<kModeRows>();
        e = cudaFuncSetAttribute(k_solve_sums, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_solve_sums<<<(int)(p.n_items < sms ? p.n_items : sms), 4 * 128, smem, s>>>(p);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const int64_t n_whole = offs[c_long] - offs[1];
    if (cg.enabled && n_whole > 0) {
        // solver of this half-epoch: conjugate gradients unless the side's last run took too many products; and where the
        // rows of 17 .. 32 observations go
        k_cg_policy<<<1, 32, 0, s>>>(cg.policy, cg.switch_products);
        ++*launches;
        p.route = cg.policy;
        p.n_class2 = offs[3] - offs[2];
    }
    if (dual_ws && offs[3] > offs[1]) {
        // rows with 1 .. 32 observations (classes 1 and 2): dual form, if the flag (set on the device) allows it
        e = launch_rows_dual(sv, offs[1], offs[2] - offs[1], offs[3] - offs[2], X, dual_ws, out, st, p.route, order16, n4, n8, s, launches);
        if (e != cudaSuccess) return e;
        p.dual_flag = dual_flag_ptr(dual_ws);
        p.n_items_primal = offs[c_long] - offs[3];
    }
    if (n_whole > 0) {
        p.n_items = n_whole;
        p.last_item = offs[c_long] - 1;
        p.solver = cg.enabled ? 1 : 0;
        p.cg_max_iter = cg.max_iter;
        p.cg_tol2 = cg.tol * cg.tol;
        p.cg_warm = cg.warm_start ? 1 : 0;
        p.cg_counters = cg.counters;
        p.fallback_list = cg.fallback_list;
        p.fallback_count = cg.counters + 2;
        const int grid = (int)(n_whole < sms ? n_whole : sms);
        if (main_begin) cudaEventRecord(main_begin, s);
        if (cg.enabled && p.dual_flag) {
            // The dual form beyond its condition limit (flag 2): its solutions, already in the table, are the start
            // vectors of a conjugate-gradient pass over the same rows, which works on the d x d system itself and stops
            // at the same residual as every other row (a few products instead of a solve from scratch); rows that do
            // not converge get the Cholesky solve.  With the flag at 1 (or 0) both launches return at once.
            Params q = p;
            q.n_items = offs[3] - offs[1];
            q.last_item = offs[3] - 1;
            q.dual_flag = nullptr;
            q.polish_flag = p.dual_flag;
            q.cg_warm = 1;
            q.cg_counters = cg.counters + 3;
            const int grid_q = (int)(q.n_items < sms ? q.n_items : sms);
            e = launch_mode<kModeRowsCg>(q, grid_q, s);
            if (e != cudaSuccess) return e;
            q.item_list = cg.fallback_list;
            q.item_count = cg.counters + 2;
            e = launch_mode<kModeRows>(q, grid_q, s);
            if (e != cudaSuccess) return e;
            *launches += 2;
        }
        if (cg.enabled) {
            p.policy = cg.policy;
            e = launch_mode<kModeRowsCg>(p, grid, s);
            if (e != cudaSuccess) return e;
            k_cg_record<<<1, 32, 0, s>>>(cg.policy, cg.counters);
            // the Cholesky kernel: the rows conjugate gradients did not finish (none, as a rule: its blocks then return at
            // once), or every row when the choice above fell on it
            p.item_list = cg.fallback_list;
            p.item_count = cg.counters + 2;
            e = launch_mode<kModeRows>(p, grid, s);
            *launches += 3;
        } else {
            e = launch_mode<kModeRows>(p, grid, s);
            ++*launches;
        }
        if (e != cudaSuccess) return e;
        if (main_end) cudaEventRecord(main_end, s);
    }
    const int64_t n_zero = offs[1] - offs[0];
    if (n_zero > 0) {
        k_zero_rows_bf16<<<(unsigned)((n_zero * D + 255) / 256), 256, 0, s>>>(sv.order + offs[0], n_zero, out);
        ++*launches;
    }
    return cudaGetLastError();
}

// Whole half-epoch of the rows of an fp32 table of 64 features on the tensor cores: sv is the doubled entry list over the
// 2N-row bfloat16 table T (see kModeRowsFold), offs its degree classes.
cudaError_t launch_rows_fold(const SideView &sv, const int64_t *offs, int64_t n_chunks, int64_t n_split_rows, const void *T,
                             int64_t n_table, const float *Bmat, float *split_partials, RowOut out, DevStatus *st,
                             cudaStream_t s, int64_t *launches, cudaEvent_t main_begin, cudaEvent_t main_end,
                             const CgOptions &cg, const int *dual_flag)
{
    const int sms = sm_count();
    Params p{};
    p.sv = sv;
    p.X = reinterpret_cast<const __nv_bfloat16 *>(T);
    p.n_table = n_table;
    p.Bmat = Bmat;
    p.partials = split_partials;
    p.out = out;
    p.st = st;
    p.solver = cg.enabled ? 1 : 0;
    p.cg_max_iter = cg.max_iter;
    p.cg_tol2 = cg.tol * cg.tol;
    p.cg_warm = cg.warm_start ? 1 : 0;
    p.cg_counters = cg.counters;
    cudaError_t e;
    const int c_long = long_class_begin(offs);
    const int64_t n_long = offs[kNClasses - 1] - offs[c_long];
    if (n_chunks + n_long > 0) {
        p.n_chunks = n_chunks;
        p.long_end = offs[kNClasses - 1];
        p.n_items = n_chunks + n_long;
        e = launch_mode<kModeChunks>(p, (int)(p.n_items < sms ? p.n_items : sms), s);
        ++*launches;
        if (e != cudaSuccess) return e;
        p.split_begin = offs[kNClasses - 1];
        p.n_split_rows = n_split_rows;
        p.n_items = n_split_rows + n_long;
        const size_t smem = 4 * sizeof(FoldGroupSmem) + 128;
        e = cudaFuncSetAttribute(k_solve_sums_fold, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        const int64_t blocks = (p.n_items + 3) / 4;
        k_solve_sums_fold<<<(int)(blocks < 2 * sms ? blocks : 2 * sms), 4 * 128, smem, s>>>(p);
        ++*launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const int64_t n_whole = offs[c_long] - offs[1];
    if (dual_flag && offs[3] > offs[1]) {
        // rows of at most 32 doubled entries (16 observations) are solved in the dual form elsewhere while the flag is set
        p.dual_flag = dual_flag;
        p.n_items_primal = offs[c_long] - offs[3];
    }
    if (n_whole > 0) {
        p.n_items = n_whole;
        p.last_item = offs[c_long] - 1;
        if (main_begin) cudaEventRecord(main_begin, s);
        e = launch_mode<kModeRowsFold>(p, (int)(n_whole < sms ? n_whole : sms), s);
        ++*launches;
        if (e != cudaSuccess) return e;
        if (main_end) cudaEventRecord(main_end, s);
    }
    const int64_t n_zero = offs[1] - offs[0];
    if (n_zero > 0) {
        k_zero_rows_f32x64<<<(unsigned)((n_zero * kFoldD + 255) / 256), 256, 0, s>>>(sv.order + offs[0], n_zero, out);
        ++*launches;
    }
    return cudaGetLastError();
}

cudaError_t launch_split_table(const float *X, int64_t n, void *T, cudaStream_t s, int64_t *launches)
{
    if (n <= 0) return cudaSuccess;
    k_split_table<<<(unsigned)((n * kFoldD / 4 + 255) / 256), 256, 0, s>>>(X, n, reinterpret_cast<__nv_bfloat16 *>(T));
    ++*launches;
    return cudaGetLastError();
}

}  // namespace alx
