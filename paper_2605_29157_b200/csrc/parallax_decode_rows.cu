// Multi-token decode step with up to 64 rows per KV head, 32 per CTA (a handful to a few dozen new tokens per sequence
// times the query heads of a GQA group) on the tcgen05 tensor cores, with the KEYS on the TMEM lanes.
//
// The row-major multi-token kernel computes a 128-row tile whatever the number of rows, and the mma.sync decode
// kernel is bound by its SM work from about ten rows on.  Here the work follows the rows present (NR = 16 or 32;
// head dimension 128 or 64):
//   S^T [128 keys x 2 NR]  = K_c [Q; R]^T                      one product per 128-key tile (Algorithm 1: S1, S2)
//   O^T [D x 4 NR]        += V_c^T [P1 | P1 res | P2 | P2 res]^T  one product: A = the V tile read MN-major (head
//                                                                dimension on M), B = the four weight tiles side by side
// so K/V is read from HBM once per KV head for all its rows and both branches, the V tile is read from shared
// memory once per tile, and the element-wise work is 128 x NR weights per tile.  P1, P2 reach the tensor cores as
// bf16 plus their bf16 rounding residuals, as everywhere in the library; the two halves are added in the epilogue.
// The price of keys on the lanes is that a row's maximum lives across 128 threads.  The reference exponent of a row
// therefore moves lazily: a tile in which no visible score exceeds the reference by more than 2^8 (one OR over
// the element-wise warps) is exponentiated against the reference as it stands; otherwise the tile's maxima are
// formed (a register transpose inside each warp, one exchange through shared memory), the references of the rows
// that need it move, and the accumulators are rescaled in TMEM.
//
// Output: rows finished in place (one split), or the decode path's partial records
// (m ln 2, d1, d2, 0, O1[D], O2[D]) per (row, split), merged by the decode path's combine kernel.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "parallax.h"
#include "plx_common.cuh"
#include "plx_internal.h"
#include "plx_tcgen05.cuh"

#ifndef PLX_DEBUG_CHECKS
#define PLX_DEBUG_CHECKS 0  // 1: page ids are verified against the pool before they are followed
#endif

// Cycle accounting for experiments (-DPLX_TRACE=1; never part of the shipped build): CTA 0 accumulates the cycles
// its element-wise thread 0, its issuing thread and its producer thread spend in each phase of a tile.
#ifndef PLX_TRACE
#define PLX_TRACE 0
#endif
#if PLX_TRACE
__device__ long long g_rows_trace[32];
#define ROWS_T0 long long tr_t = clock64(), tr_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}
#define ROWS_T(i)                           \
    do {                                    \
        const long long tr_now = clock64(); \
        tr_acc[(i) & 7] += tr_now - tr_t;   \
        tr_t = tr_now;                      \
    } while (0)
#define ROWS_STAMP(i)                                                              \
    do {                                                                           \
        if (blockIdx.x == 0 && threadIdx.x == 0) {                                 \
            unsigned long long tr_g;                                               \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tr_g));               \
            g_rows_trace[24 + (i)] = static_cast<long long>(tr_g);                 \
        }                                                                          \
    } while (0)
#define ROWS_FLUSH(base_index)                                                    \
    do {                                                                          \
        if (blockIdx.x == 0)                                                      \
            for (int tr_i = 0; tr_i < 8; ++tr_i) g_rows_trace[(base_index) + tr_i] = tr_acc[tr_i]; \
    } while (0)
#else
#define ROWS_T0
#define ROWS_T(i)
#define ROWS_STAMP(i)
#define ROWS_FLUSH(base_index)
#endif

namespace {

constexpr int BK = 128;  // keys per tile = TMEM lanes
constexpr int kMaxRows = 64;  // per KV head; more than 32 are worked as two parts (two items that share their K/V through L2)
constexpr int kRowsPerThread = 8;              // rows per element-wise thread: NR / 8 threads share a key
constexpr int kBoxKV = BK * 128;       // [128 keys x 64 columns] bf16 box: 16 KiB (a K or V tile is HD / 64 of them)
constexpr int kBlockP = BK * 128;      // [128 keys x 64 columns of the stacked weights] bf16: 16 KiB
constexpr int kMaxStages = 4;
enum : int { kBarQRFull = 0, kBarQRFree = 2, kBarKFull = 4, kBarKFree = 8, kBarVFull = 12, kBarVFree = 16, kBarSFull = 20,
             kBarSFree = 22, kBarPFull = 24, kBarPvDone = 25, kBarFinal = 26, kBarOFree = 27, kBarItemFull = 28, kBarItemFree = 30,
             kNumBars = 32 };
constexpr float kRowsLazyThreshold = 8.0f;       // log2 units
constexpr float kLn2 = 0.6931471805599453f;

// NR: rows of a KV head per CTA (the N extent of the weight tiles; fewer rows are padded); HD: head dimension
template <int NR, int HD>
struct RowsCfg {
    static_assert(NR == 16 || NR == 32, "rows per KV head");
    static_assert(HD == 64 || HD == 128, "head dimension");
    static constexpr int kBoxes = HD / 64;                // 64-column boxes per row of Q, R, K, V
    static constexpr int kTileKV = kBoxes * kBoxKV;       // K or V tile
    static constexpr int REC = 2 * HD + 4;                // floats of a split record
    static constexpr int RPT = kRowsPerThread;
    static constexpr int kParts = NR / RPT;               // element-wise threads per key (2 or 4)
    static constexpr int kEwWarps = 4 * kParts;           // four warps cover the 128 keys (TMEM lanes) of a tile
    static constexpr int kEwThreads = kEwWarps * 32;
    static constexpr int kMmaWarp = kEwWarps, kPvWarp = kEwWarps + 1, kTmaWarp = kEwWarps + 2;
    static constexpr int kThreads = (kEwWarps + 3) * 32;
    // ring depths by measurement (64 x 8192 keys, head dimension 64, 16 / 32 rows): K / V stages 4 / 4: 218 / 307 us, 3 / 3: 252 /
    // 301, 2 / 3: 251 / 356, 6 / 6 (5 / 6 at 32 rows): 233 / 323 -- deeper rings than these are slower, not faster
    static constexpr int kStagesK = HD == 64 ? (NR == 16 ? 4 : 3) : NR == 16 ? 3 : 2, kStagesV = HD == 64 ? (NR == 16 ? 4 : 3) : 3;
    static constexpr int kBoxQR = 2 * NR * 128;           // [Q rows; R rows] x 64 columns: the N = 2 NR operand of the score product
    static constexpr int kTileQR = kBoxes * kBoxQR;
    static constexpr int kPBlocks = 4 * NR / 64;          // 64-wide blocks of [P1 | P1 res | P2 | P2 res]
    static constexpr int kTileP = kPBlocks * kBlockP;
    static constexpr int kOffQR = 0;
    static constexpr int kOffK = kOffQR + 2 * kTileQR;    // two [Q; R] tiles: the next item's is fetched under the current one
    static constexpr int kOffV = kOffK + kStagesK * kTileKV;
    static constexpr int kOffP = kOffV + kStagesV * kTileKV;
    static constexpr int kOffBar = kOffP + kTileP;
    static constexpr int kOffTmemSlot = kOffBar + kNumBars * 8;
    static constexpr int kOffRef = kOffTmemSlot + 16;     // float [NR]: reference exponent of each row (log2 units)
    static constexpr int kOffAlpha = kOffRef + NR * 4;    // float [NR]: rescale factors of a tile that moves references
    static constexpr int kOffWmax = kOffAlpha + NR * 4;   // float [element-wise warps][RPT]: per-warp tile maxima
    static constexpr int kOffItems = kOffWmax + kEwWarps * RPT * 4;  // int [2]: the items handed from the producer to the other roles
    static constexpr int kOffDsum = kOffItems + 16;  // float [element-wise warps][RPT][2] per-warp row sums, then [NR][2] totals
    static constexpr int kSmemBytes = kOffDsum + (kEwWarps * RPT * 2 + NR * 2) * 4;
    static_assert(kSmemBytes <= 232448, "shared-memory budget of one CTA");
    static_assert(kOffK % 1024 == 0 && kOffBar % 8 == 0 && kOffRef % 16 == 0, "alignment of the tiles, barriers and references");
    static constexpr uint32_t kColS = 0;                  // two score buffers of 2 NR fp32 columns: S1^T | S2^T
    static constexpr uint32_t kColO = 4 * NR;             // O1 | O1 res | O2 | O2 res, NR columns each
    static constexpr uint32_t kTmemCols = 8 * NR;         // 128 or 256
};

struct RowsParams {
    const int32_t* seqlens;
    void* out;
    float* partials;   // nullptr: one split, rows finished here
    int32_t* status;
    int B, Hq, Hkv, Lq, T_max;
    int rows;          // (Hq / Hkv) * Lq rows of a KV head, contiguous in [B, Hq, Lq, D]
    int parts, rows_per_part;  // the rows of a KV head are worked in `parts` items of at most rows_per_part <= NR rows
    int num_splits, tiles_per_split;
    int n_items;       // B * Hkv * num_splits * parts (sequence, KV head, key split, part) items; parts of a split are neighbours
    // Device int32, zero between calls: the next item to hand out (the CTAs of a grid smaller than n_items draw their
    // items from it; the last draw of a launch sets it back to zero).  nullptr: one CTA per item.
    int32_t* ticket;
    float scale_log2e;
    int out_dtype;
    // paged cache: int32 [B, max_pages] page ids (else nullptr); pools [num_pages, Hkv, page_size, D]; page_size
    // divides 128 or is a multiple of it, so a 128-key tile is a whole number of boxes of `page_box` keys
    const int32_t* block_table;
    int page_size, max_pages, page_box;
    long long pool_rows;
};

template <int kEwThreads>
__device__ __forceinline__ void ew_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEwThreads) : "memory"); }
// barrier among the element-wise warps that also ORs a predicate over them
template <int kEwThreads>
__device__ __forceinline__ bool ew_barrier_or(bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\tbar.red.or.pred p, 2, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(static_cast<uint32_t>(pred)), "n"(kEwThreads)
        : "memory");
    return r != 0;
}

// N values per lane in, one out: every lane ends up with the reduction over the warp's 32 lanes of value
// (lane mod N).  Each round sends half of the remaining values to the partner lane and keeps the other half.
template <int N, bool kMax>
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[N], int lane)
{
#pragma unroll
    for (int off = N / 2; off >= 1; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < off; ++i) {
            const float keep = up ? v[i + off] : v[i];
            const float send = up ? v[i] : v[i + off];
            const float recv = __shfl_xor_sync(0xffffffffu, send, off);
            v[i] = kMax ? fmaxf(keep, recv) : keep + recv;
        }
    }
#pragma unroll
    for (int off = N; off < 32; off <<= 1) {
        const float recv = __shfl_xor_sync(0xffffffffu, v[0], off);
        v[0] = kMax ? fmaxf(v[0], recv) : v[0] + recv;
    }
    return v[0];
}

__device__ __forceinline__ void ld_cols(uint32_t taddr, uint32_t (&r)[8]) { tmem_ld8(taddr, r); }
__device__ __forceinline__ void st_cols(uint32_t taddr, const uint32_t (&r)[8]) { tmem_st8(taddr, r); }

__device__ __forceinline__ void store_value(void* out, size_t idx, float v, int out_dtype)
{
    if (out_dtype == PLX_OUT_F32)
        static_cast<float*>(out)[idx] = v;
    else
        static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------
// Kernel: item = (sequence, KV head, key split); a CTA works through the items it draws
// ---------------------------------------------------------------------------
// With one item per CTA nothing overlaps a CTA's set-up, first fetch and epilogue (one CTA per SM).  Given a ticket
// word, the host launches at most one CTA per SM and each CTA draws items until none is left: the rings, the score
// buffers and the weight tile carry on across items (stages and phases are counted per CTA, not per item), so
// while the element-wise warps finish an item (row sums, accumulators out of TMEM, stores) the producer has fetched
// the next item's [Q; R] tile and first K/V tiles and the score thread has multiplied its first two tiles.  Items
// are drawn, not dealt: the SMs of an HBM-bound grid do not all stream at the same rate, and a fixed share per SM
// (tried first) made the slowest SM's share the step's time.  The producer warp draws (it runs a ring's depth ahead of
// the other roles, which hides the atomic's latency) and hands each item to the other roles through a two-entry ring
// in shared memory (item full / item free barriers); -1 ends the walk.  An item's result does not depend on which CTA
// computes it.
// Barrier discipline: every waiter consumes the phases of a barrier strictly in order, and no barrier can
// complete a second phase before its waiter has seen the first: the S buffers alternate (a full / free pair per
// buffer), the weight tile is single (P full <-> P.V done hand over one tile at a time), the K and V rings
// have a full / free pair per stage, the two [Q; R] tiles a full / free pair each, the accumulators a
// final / free pair per item.
struct RowsItem {
    int b, hkv, split, L, jt0, n_tiles;
    int row_off, rows;  // this item's rows of the KV head: row_off ... row_off + rows - 1
    size_t row0, kv_row0;
};

__device__ __forceinline__ RowsItem rows_item(const RowsParams& p, int item)
{
    RowsItem it;
    const int part = item % p.parts;
    item /= p.parts;
    it.row_off = part * p.rows_per_part;
    it.rows = min(p.rows_per_part, p.rows - it.row_off);
    it.split = item % p.num_splits;
    const int bh = item / p.num_splits;
    it.b = bh / p.Hkv;
    it.hkv = bh - it.b * p.Hkv;
    const int G = p.Hq / p.Hkv;
    int L = p.seqlens ? p.seqlens[it.b] : p.T_max;
    it.L = max(0, min(L, p.T_max));
    it.row0 = (static_cast<size_t>(it.b) * p.Hq + static_cast<size_t>(it.hkv) * G) * p.Lq + it.row_off;  // first row of this item
    it.kv_row0 = (static_cast<size_t>(it.b) * p.Hkv + it.hkv) * p.T_max;
    const int n_all = (it.L + BK - 1) / BK;
    it.jt0 = it.split * p.tiles_per_split;
    it.n_tiles = max(0, min(n_all, it.jt0 + p.tiles_per_split) - it.jt0);
    return it;
}

template <int NR, int HD>
__global__ void __launch_bounds__(RowsCfg<NR, HD>::kThreads, 1)
plx_decode_rows_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmR,
                       const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                       const RowsParams p)
{
    using C = RowsCfg<NR, HD>;
    constexpr int kTileKV = C::kTileKV, kBoxes = C::kBoxes, REC = C::REC;
    constexpr int RPT = C::RPT, kEwWarps = C::kEwWarps, kEwThreads = C::kEwThreads, kMmaWarp = C::kMmaWarp,
                  kPvWarp = C::kPvWarp, kTmaWarp = C::kTmaWarp;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    uint8_t* const smem = smem_raw;
    if ((base & 1023u) != 0) {  // the layout has no room for alignment slack
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, PLX_ERR_ALIGNMENT);
        return;
    }
    // lets the kernel that follows in the stream be scheduled now if it is a programmatic dependent (the merge kernel of
    // a split call); it waits for this grid's completion before it touches memory.  An unsplit grid does not signal (its
    // successor, the next step's kernel, starts when it ends): that kernel's CTAs moving in beside a grid smaller than
    // the device measured 2-3 % slower (16 x 8192 keys: 82 -> 84.5 us).
    if (p.num_splits > 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    ROWS_STAMP(0);  // kernel start
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    auto bar = [&](int slot) { return base + C::kOffBar + 8 * slot; };
    float* const ref = reinterpret_cast<float*>(smem + C::kOffRef);
    float* const alpha = reinterpret_cast<float*>(smem + C::kOffAlpha);
    float* const wmax = reinterpret_cast<float*>(smem + C::kOffWmax);
    volatile int* const items = reinterpret_cast<volatile int*>(smem + C::kOffItems);
    // the q-th item of this CTA as the producer handed it over (-1: no more); `arrive`: this thread counts towards the
    // ring entry's release
    auto take_item = [&](int q, bool arrive) {
        const int ib = q & 1;
        wait_or_flag(bar(kBarItemFull + ib), (q >> 1) & 1, p.status);
        const int item = items[ib];
        if (arrive) mbar_arrive(bar(kBarItemFree + ib));
        return item;
    };
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1);
            mbar_init(bar(kBarKFree + s), 1);
            mbar_init(bar(kBarVFull + s), 1);
            mbar_init(bar(kBarVFree + s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarQRFull + s), 1);
            mbar_init(bar(kBarQRFree + s), 1);
            mbar_init(bar(kBarSFull + s), 1);
            mbar_init(bar(kBarSFree + s), kEwThreads);
        }
        mbar_init(bar(kBarPFull), kEwThreads);
        mbar_init(bar(kBarPvDone), 1);
        mbar_init(bar(kBarFinal), 1);
        mbar_init(bar(kBarOFree), kEwThreads);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarItemFull + s), 1);
            mbar_init(bar(kBarItemFree + s), kEwThreads + 2);  // every element-wise thread and the two issuing threads
        }
        fence_barrier_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(base + C::kOffTmemSlot, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + C::kOffTmemSlot);
    ROWS_STAMP(1);  // barriers, TMEM, CTA-wide sync done
    // The kernel is launched as a programmatic dependent of whatever precedes it in the stream (the previous step's
    // merge or kernel): its launch and the set-up above may overlap that kernel's tail, and nothing that kernel produces
    // or still reads (q, r, the caches, lengths, the workspace, the ticket) is touched before it has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // Every role walks the same items in the same order; `n` counts the items that hold keys (the others only get
    // their empty records or zero rows written), `g` the tiles of all items so far.
    if (warp == kTmaWarp) {
        if (lane == 0) {
            prefetch_tensormap(&tmQ);
            prefetch_tensormap(&tmR);
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
        }
        int n = 0, g = 0, drawn = 0;
        auto draw = [&]() {
            int v = 0;
            if (p.ticket) {
                if (lane == 0) {
                    v = atomicAdd(p.ticket, 1);
                    // every CTA draws exactly one item past the end; the last such draw of the launch resets the word
                    if (v == p.n_items + static_cast<int>(gridDim.x) - 1) atomicExch(p.ticket, 0);
                }
                v = __shfl_sync(0xffffffffu, v, 0);
            } else {
                v = static_cast<int>(blockIdx.x) + drawn * static_cast<int>(gridDim.x);
                ++drawn;
            }
            return v;
        };
        ROWS_T0;
        for (int q = 0;; ++q) {
            // drawn when the previous item's last tile has been issued, which is a ring's depth ahead of the other roles;
            // drawing earlier still would tie uneven items to a CTA long before it can start them
            const int drawn_item = draw();
            const int item = drawn_item < p.n_items ? drawn_item : -1;
            const int ib = q & 1;
            if (q >= 2) wait_or_flag(bar(kBarItemFree + ib), ((q >> 1) - 1) & 1, p.status);
            if (lane == 0) {
                items[ib] = item;
                mbar_arrive(bar(kBarItemFull + ib));
            }
            __syncwarp();
            if (item < 0) break;
            const RowsItem it = rows_item(p, item);
            if (it.n_tiles == 0) continue;
            const int qb = n & 1;
            if (n >= 2) wait_or_flag(bar(kBarQRFree + qb), ((n >> 1) - 1) & 1, p.status);
            if (lane == 0) {
                mbar_expect_tx(bar(kBarQRFull + qb), C::kTileQR);
#pragma unroll
                for (int h = 0; h < kBoxes; ++h) {
                    const uint32_t dst = base + C::kOffQR + qb * C::kTileQR + h * C::kBoxQR;
                    tma_load_2d(dst, &tmQ, bar(kBarQRFull + qb), 64 * h, static_cast<int>(it.row0));
                    tma_load_2d(dst + NR * 128, &tmR, bar(kBarQRFull + qb), 64 * h, static_cast<int>(it.row0));
                }
            }
            ++n;
            if (!p.block_table) {
                if (lane == 0) {
                    for (int j = 0; j < it.n_tiles; ++j, ++g) {
                        const int sk = g % C::kStagesK, sv = g % C::kStagesV;
                        const int krow = static_cast<int>(it.kv_row0) + (it.jt0 + j) * BK;
                        ROWS_T(18);
                        if (g >= C::kStagesK) wait_or_flag(bar(kBarKFree + sk), (g / C::kStagesK - 1) & 1, p.status);
                        ROWS_T(16);
                        mbar_expect_tx(bar(kBarKFull + sk), kTileKV);
#pragma unroll
                        for (int h = 0; h < kBoxes; ++h)
                            tma_load_2d(base + C::kOffK + sk * kTileKV + h * kBoxKV, &tmK, bar(kBarKFull + sk), 64 * h, krow);
                        ROWS_T(18);
                        if (g >= C::kStagesV) wait_or_flag(bar(kBarVFree + sv), (g / C::kStagesV - 1) & 1, p.status);
                        ROWS_T(17);
                        mbar_expect_tx(bar(kBarVFull + sv), kTileKV);
#pragma unroll
                        for (int h = 0; h < kBoxes; ++h)
                            tma_load_2d(base + C::kOffV + sv * kTileKV + h * kBoxKV, &tmV, bar(kBarVFull + sv), 64 * h, krow);
                    }
                }
            } else {
                // Paged: the tile is fetched in boxes of page_box keys, each from its page, one (box, 64-column half)
                // per lane of this warp (a page size of 16 means sixteen copies per tile and tensor).  Boxes that lie
                // wholly past the context are not fetched (their pages need not exist): those rows of the tile keep
                // what an earlier tile left there, their scores are masked and their V rows are cleared before use.
                const int32_t* const table = p.block_table + static_cast<size_t>(it.b) * p.max_pages;
                const int pb = p.page_box;
                const int my_box = lane / kBoxes, my_half = lane % kBoxes;
                for (int j = 0; j < it.n_tiles; ++j, ++g) {
                    const int sk = g % C::kStagesK, sv = g % C::kStagesV;
                    const int key0 = (it.jt0 + j) * BK;
                    const int nbox = min(BK / pb, (it.L - key0 + pb - 1) / pb);
                    const uint32_t bytes = static_cast<uint32_t>(nbox) * pb * 128 * kBoxes;
                    int row = 0;
                    if (my_box < nbox) {
                        const int key = key0 + my_box * pb;
                        const int pg = key / p.page_size;
                        int id = __ldg(table + pg);
#if PLX_DEBUG_CHECKS
                        if (id < 0 || (static_cast<long long>(id) * p.Hkv + it.hkv + 1) * p.page_size > p.pool_rows) {
                            if (p.status) atomicExch(p.status, PLX_ERR_DEVICE_CHECK);  // a page id outside the pool: not followed
                            id = 0;
                        }
#endif
                        row = (id * p.Hkv + it.hkv) * p.page_size + (key - pg * p.page_size);
                    }
                    const uint32_t off = static_cast<uint32_t>(my_half * kBoxKV + my_box * pb * 128);
                    if (g >= C::kStagesK) wait_or_flag(bar(kBarKFree + sk), (g / C::kStagesK - 1) & 1, p.status);
                    if (lane == 0) mbar_expect_tx(bar(kBarKFull + sk), bytes);
                    __syncwarp();
                    if (my_box < nbox) tma_load_2d(base + C::kOffK + sk * kTileKV + off, &tmK, bar(kBarKFull + sk), 64 * my_half, row);
                    if (g >= C::kStagesV) wait_or_flag(bar(kBarVFree + sv), (g / C::kStagesV - 1) & 1, p.status);
                    if (lane == 0) mbar_expect_tx(bar(kBarVFull + sv), bytes);
                    __syncwarp();
                    if (my_box < nbox) tma_load_2d(base + C::kOffV + sv * kTileKV + off, &tmV, bar(kBarVFull + sv), 64 * my_half, row);
                }
            }
            __syncwarp();
        }
        if (lane == 0) ROWS_FLUSH(16);
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ===================== score products =====================
        // One issuing thread; the value products are issued from a warp of their own, so that the waits of one (K and
        // the S buffer / the weights and V) do not delay the other's products.
        constexpr uint32_t idesc_s = make_idesc(BK, 2 * NR, 0, 0);   // K-major A (K tile), K-major B ([Q; R])
        int n = 0, g = 0;
        ROWS_T0;
        for (int q = 0;; ++q) {
            const int item = take_item(q, lane == 0);
            if (item < 0) break;
            const RowsItem it = rows_item(p, item);
            if (it.n_tiles == 0) continue;
            const int qb = n & 1;
            wait_or_flag(bar(kBarQRFull + qb), (n >> 1) & 1, p.status);
            const uint64_t dQR = make_smem_desc(base + C::kOffQR + qb * C::kTileQR, 0, 1024);
            for (int j = 0; j < it.n_tiles; ++j, ++g) {  // runs at most two tiles ahead of the element-wise warps (two S buffers)
                const int s = g & 1, sk = g % C::kStagesK;
                ROWS_T(12);
                wait_or_flag(bar(kBarKFull + sk), (g / C::kStagesK) & 1, p.status);
                ROWS_T(8);
                if (g >= 2) wait_or_flag(bar(kBarSFree + s), ((g >> 1) - 1) & 1, p.status);
                ROWS_T(9);
                if (lane == 0) {
                    tc_fence_after();
                    const uint64_t dK = make_smem_desc(base + C::kOffK + sk * kTileKV, 0, 1024);
#pragma unroll
                    for (int ks = 0; ks < HD / 16; ++ks) {
                        const uint64_t aoff = static_cast<uint64_t>(((ks >> 2) * kBoxKV + (ks & 3) * 32) >> 4);
                        const uint64_t boff = static_cast<uint64_t>(((ks >> 2) * C::kBoxQR + (ks & 3) * 32) >> 4);
                        mma_ss(tmem + C::kColS + s * 2 * NR, dK + aoff, dQR + boff, idesc_s, ks > 0);
                    }
                    tc_commit(bar(kBarSFull + s));
                    tc_commit(bar(kBarKFree + sk));
                    if (j == it.n_tiles - 1) tc_commit(bar(kBarQRFree + qb));  // this item's [Q; R] tile has been read
                }
                __syncwarp();
            }
            ++n;
        }
        if (lane == 0) ROWS_FLUSH(8);
        __syncwarp();
    } else if (warp == kPvWarp) {
        // ===================== value products =====================
        // MN-major A (V tile: head dimension on M), MN-major B (weights).  M is 128 at either head dimension: at 64 the
        // second 64-wide block of A is the first one again (block distance 0), so accumulator lanes 64-127 repeat
        // lanes 0-63 and are ignored
        constexpr uint32_t idesc_pv = make_idesc(128, 4 * NR, 1, 1);
        const uint64_t dP = make_smem_desc(base + C::kOffP, kBlockP, 1024);
        int n = 0, g = 0;
        for (int q = 0;; ++q) {
            const int item = take_item(q, lane == 0);
            if (item < 0) break;
            const RowsItem it = rows_item(p, item);
            if (it.n_tiles == 0) continue;
            for (int j = 0; j < it.n_tiles; ++j, ++g) {
                const int sv = g % C::kStagesV;
                wait_or_flag(bar(kBarPFull), g & 1, p.status);
                wait_or_flag(bar(kBarVFull + sv), (g / C::kStagesV) & 1, p.status);
                // the accumulators of the previous item have been read
                if (j == 0 && n > 0) wait_or_flag(bar(kBarOFree), (n - 1) & 1, p.status);
                if (lane == 0) {
                    tc_fence_after();
                    const uint64_t dV = make_smem_desc(base + C::kOffV + sv * kTileKV, HD == 128 ? kBoxKV : 0, 1024);
#pragma unroll
                    for (int ks = 0; ks < BK / 16; ++ks) {
                        const uint64_t koff = static_cast<uint64_t>((ks * 2048) >> 4);
                        mma_ss(tmem + C::kColO, dV + koff, dP + koff, idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                    }
                    tc_commit(bar(kBarPvDone));
                    tc_commit(bar(kBarVFree + sv));
                    if (j == it.n_tiles - 1) tc_commit(bar(kBarFinal));
                }
                __syncwarp();
            }
            ++n;
        }
    } else {
        // ===================== element-wise warps =====================
        // thread = (key of the tile = TMEM lane, eight of the rows)
        const int quarter = warp & 3, part = warp >> 2;
        const int kr = quarter * 32 + lane;
        const int c0 = RPT * part;  // first row of this thread's columns
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const int swz = kr & 7;
        const float4* const ref4 = reinterpret_cast<const float4*>(ref + c0);
        int n = 0, g = 0;
        ROWS_T0;

        for (int q = 0;; ++q) {
            const int item = take_item(q, true);
            if (item < 0) break;
            const RowsItem it = rows_item(p, item);
            const int L = it.L, jt0 = it.jt0, n_tiles = it.n_tiles;
            const size_t row0 = it.row0;
            // bit c: row c0 + c exists.  With fewer than NR rows the padding rows (whatever the [Q; R] boxes hold past the
            // last row: the next part's or the next head's rows, or the zeros of the tensor map's bounds) are carried like
            // real rows through the fully visible tiles (their columns of the weights and accumulators touch no other
            // row's) and get weights of zero in the masked ones; nothing of them is stored
            const uint32_t row_mask = it.rows - c0 >= RPT ? (1u << RPT) - 1u : (it.rows > c0 ? (1u << (it.rows - c0)) - 1u : 0u);
            if (n_tiles == 0) {  // no key for this split: empty records (only m is ever read), or rows of zeros
                if (p.partials) {
                    for (int i = threadIdx.x; i < it.rows; i += kEwThreads)
                        p.partials[((row0 + i) * p.num_splits + it.split) * REC] = -INFINITY;
                } else {
                    for (int i = threadIdx.x; i < it.rows * HD; i += kEwThreads) store_value(p.out, row0 * HD + i, 0.0f, p.out_dtype);
                }
                continue;
            }
            // the previous item's epilogue has read the references and the row-sum scratch
            ew_barrier<kEwThreads>();
            if (threadIdx.x < NR) ref[threadIdx.x] = -INFINITY;
            ew_barrier<kEwThreads>();
            float d1[RPT], d2[RPT];
#pragma unroll
            for (int c = 0; c < RPT; ++c) d1[c] = d2[c] = 0.0f;

            for (int j = 0; j < n_tiles; ++j, ++g) {
                const int s = g & 1, sv = g % C::kStagesV;
                const int key = (jt0 + j) * BK + kr;
                // some (key, row) pair of this tile may be invisible: the last Lq - 1 keys, the end of the context
                const bool need_mask = (jt0 + j) * BK + BK > L - (p.Lq - 1);
                const uint32_t Sb = lane_base + C::kColS + s * 2 * NR;
                // bit c of vis: row c0 + c sees this thread's key (token i of a head sees the first L - (Lq - 1 - i) keys)
                uint32_t vis = (1u << RPT) - 1u;
                if (need_mask) {
                    vis = 0u;
                    int tok = (it.row_off + c0) % p.Lq;
#pragma unroll
                    for (int c = 0; c < RPT; ++c) {
                        if (key < L - (p.Lq - 1 - tok)) vis |= 1u << c;
                        if (++tok == p.Lq) tok = 0;
                    }
                    vis &= row_mask;
                }
                ROWS_T(7);
                wait_or_flag(bar(kBarSFull + s), (g >> 1) & 1, p.status);
                if (g == 0) ROWS_STAMP(2);  // first scores ready
                if (g == 1) ROWS_STAMP(3);  // second tile's scores ready
                ROWS_T(0);
                tc_fence_after();
                uint32_t a[RPT], gq[RPT];
                ld_cols(Sb + c0, a);
                ld_cols(Sb + NR + c0, gq);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar(kBarSFree + s));  // the score buffer is in registers

                // exponents against the references as they stand; does any visible score need a reference to move?
                // `plain`: every row sees every key of the tile (CTA-uniform): packed arithmetic, no selects; a row
                // without a reference yet gives x = +inf and raises the flag by itself
                const bool plain = !need_mask;
                float x[RPT];
                bool flag = false;
                if (plain) {
                    const uint64_t sc2 = pack_f2(p.scale_log2e, p.scale_log2e);
                    float mx = -INFINITY;
#pragma unroll
                    for (int c4 = 0; c4 < RPT / 4; ++c4) {
                        const float4 r4 = ref4[c4];
                        const int c = 4 * c4;
                        unpack_f2(fma2(pack_f2(__uint_as_float(a[c]), __uint_as_float(a[c + 1])), sc2, pack_f2(-r4.x, -r4.y)), x[c], x[c + 1]);
                        unpack_f2(fma2(pack_f2(__uint_as_float(a[c + 2]), __uint_as_float(a[c + 3])), sc2, pack_f2(-r4.z, -r4.w)), x[c + 2],
                                  x[c + 3]);
                        mx = max3(mx, x[c], x[c + 1]);
                        mx = max3(mx, x[c + 2], x[c + 3]);
                    }
                    flag = mx > kRowsLazyThreshold;
                } else {
#pragma unroll
                    for (int c4 = 0; c4 < RPT / 4; ++c4) {
                        const float4 r4 = ref4[c4];
                        const float rf[4] = {r4.x, r4.y, r4.z, r4.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int c = 4 * c4 + e;
                            const bool seen = rf[e] > -INFINITY;
                            x[c] = fmaf(__uint_as_float(a[c]), p.scale_log2e, -(seen ? rf[e] : 0.0f));
                            flag |= ((vis >> c) & 1u) && (!seen || x[c] > kRowsLazyThreshold);
                        }
                    }
                }
                ROWS_T(1);
                const bool moved = ew_barrier_or<kEwThreads>(flag);
                ROWS_T(2);
                if (moved) {
                    // ---- some reference has to move: the tile's maximum of every row over its visible keys ----
                    float v[RPT];
#pragma unroll
                    for (int c = 0; c < RPT; ++c) v[c] = ((vis >> c) & 1u) ? __uint_as_float(a[c]) * p.scale_log2e : -INFINITY;
                    const float m = warp_transpose_reduce<RPT, true>(v, lane);
                    if (lane < RPT) wmax[warp * RPT + lane] = m;
                    ew_barrier<kEwThreads>();
                    if (threadIdx.x < NR) {
                        const int row = threadIdx.x, pr = row / RPT, c = row % RPT;
                        const float tm = fmaxf(fmaxf(wmax[(4 * pr + 0) * RPT + c], wmax[(4 * pr + 1) * RPT + c]),
                                               fmaxf(wmax[(4 * pr + 2) * RPT + c], wmax[(4 * pr + 3) * RPT + c]));
                        const float old = ref[row];
                        float al = 1.0f;
                        if (tm > old + kRowsLazyThreshold) {  // also the first visible key of a row (old = -inf)
                            al = (old > -INFINITY) ? ex2(old - tm) : 0.0f;
                            ref[row] = tm;
                        }
                        alpha[row] = al;
                    }
                    ew_barrier<kEwThreads>();
                    if (j > 0) {
                        // move the accumulated state to the new references (this thread's TMEM lane is a head dimension here)
                        wait_or_flag(bar(kBarPvDone), (g - 1) & 1, p.status);
                        tc_fence_after();
                        float al[RPT];
#pragma unroll
                        for (int c = 0; c < RPT; ++c) al[c] = alpha[c0 + c];
#pragma unroll
                        for (int which = 0; which < 4; ++which) {
                            uint32_t o[RPT];
                            const uint32_t col = lane_base + C::kColO + which * NR + c0;
                            ld_cols(col, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < RPT; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * al[c]);
                            st_cols(col, o);
                        }
                        tmem_wait_st();
                        tc_fence_before();
#pragma unroll
                        for (int c = 0; c < RPT; ++c) {
                            d1[c] *= al[c];
                            d2[c] *= al[c];
                        }
                    }
#pragma unroll
                    for (int c = 0; c < RPT; ++c) {
                        const float rf = ref[c0 + c];
                        x[c] = fmaf(__uint_as_float(a[c]), p.scale_log2e, -((rf > -INFINITY) ? rf : 0.0f));
                    }
                }

                ROWS_T(6);
                // ---- weights, row sums, bf16 parts and residuals ----
                uint32_t w4[4][RPT / 2];  // P1, P1 residual, P2, P2 residual: two rows per word
                if (plain) {
                    const uint64_t neg1 = pack_f2(-1.0f, -1.0f);
#pragma unroll
                    for (int c = 0; c < RPT; c += 2) {
                        const uint64_t P1 = pack_f2(ex2(x[c]), ex2(x[c + 1]));
                        const uint64_t P2 = mul2(P1, pack_f2(__uint_as_float(gq[c]), __uint_as_float(gq[c + 1])));
                        unpack_f2(add2(pack_f2(d1[c], d1[c + 1]), P1), d1[c], d1[c + 1]);
                        unpack_f2(add2(pack_f2(d2[c], d2[c + 1]), P2), d2[c], d2[c + 1]);
                        float lo, hi;
                        unpack_f2(P1, lo, hi);
                        const uint32_t b1 = pack2(lo, hi);
                        unpack_f2(P2, lo, hi);
                        const uint32_t b2 = pack2(lo, hi);
                        w4[0][c >> 1] = b1;
                        w4[2][c >> 1] = b2;
                        unpack_f2(fma2(bf16x2_to_f2(b1), neg1, P1), lo, hi);  // what the bf16 rounding left over
                        w4[1][c >> 1] = pack2(lo, hi);
                        unpack_f2(fma2(bf16x2_to_f2(b2), neg1, P2), lo, hi);
                        w4[3][c >> 1] = pack2(lo, hi);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < RPT; c += 2) {
                        float p1[2], p2[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const bool ok = (vis >> (c + e)) & 1u;
                            p1[e] = ok ? ex2(x[c + e]) : 0.0f;
                            p2[e] = ok ? p1[e] * __uint_as_float(gq[c + e]) : 0.0f;
                            d1[c + e] += p1[e];
                            d2[c + e] += p2[e];
                        }
                        const __nv_bfloat162 b1 = __floats2bfloat162_rn(p1[0], p1[1]), b2 = __floats2bfloat162_rn(p2[0], p2[1]);
                        w4[0][c >> 1] = *reinterpret_cast<const uint32_t*>(&b1);
                        w4[2][c >> 1] = *reinterpret_cast<const uint32_t*>(&b2);
                        w4[1][c >> 1] = pack2(p1[0] - __low2float(b1), p1[1] - __high2float(b1));
                        w4[3][c >> 1] = pack2(p2[0] - __low2float(b2), p2[1] - __high2float(b2));
                    }
                }

                ROWS_T(3);
                // the previous weight tile (the last one of the previous item, for an item's first) has been consumed
                if (g > 0) wait_or_flag(bar(kBarPvDone), (g - 1) & 1, p.status);
                ROWS_T(4);
                // weight tile: [128 keys][4 NR columns] bf16 in 64-column blocks of 128 bytes per key, 128-byte swizzle
                // (chunk index XOR key mod 8); column which * NR + row
#pragma unroll
                for (int which = 0; which < 4; ++which)
#pragma unroll
                    for (int q8 = 0; q8 < RPT / 8; ++q8) {
                        const int n0 = which * NR + c0 + 8 * q8;  // first of eight columns
                        uint8_t* const dst = smem + C::kOffP + (n0 >> 6) * kBlockP + kr * 128 + ((((n0 & 63) >> 3) ^ swz) << 4);
                        *reinterpret_cast<uint4*>(dst) =
                            make_uint4(w4[which][4 * q8], w4[which][4 * q8 + 1], w4[which][4 * q8 + 2], w4[which][4 * q8 + 3]);
                    }
                if ((jt0 + j) * BK + BK > L && part == 0) {
                    // the context ends inside this tile: rows of V past it may hold anything (NaN included); their
                    // weights are exact zeros, so clear them once the tile has landed
                    wait_or_flag(bar(kBarVFull + sv), (g / C::kStagesV) & 1, p.status);
                    if (key >= L) {
                        uint8_t* const vrow = smem + C::kOffV + sv * kTileKV + kr * 128;
#pragma unroll
                        for (int i = 0; i < 8 * kBoxes; ++i)
                            *reinterpret_cast<uint4*>(vrow + (i >> 3) * kBoxKV + (i & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                fence_proxy_async_smem();
                mbar_arrive(bar(kBarPFull));
                ROWS_T(5);
            }

            // ---- row sums over the keys (while the last value product runs), then the epilogue: this thread's TMEM lane is
            // head dimension kr ----
            ROWS_STAMP(4);  // last weights handed over
            float* const dsum = reinterpret_cast<float*>(smem + C::kOffDsum);
            {
                const float t1 = warp_transpose_reduce<RPT, false>(d1, lane);
                const float t2 = warp_transpose_reduce<RPT, false>(d2, lane);
                if (lane < RPT) {
                    dsum[(warp * RPT + lane) * 2] = t1;
                    dsum[(warp * RPT + lane) * 2 + 1] = t2;
                }
            }
            ew_barrier<kEwThreads>();
            float* const dtot = dsum + kEwWarps * RPT * 2;
            if (threadIdx.x < NR) {
                const int row = threadIdx.x, pr = row / RPT, c = row % RPT;
                float t1 = 0.0f, t2 = 0.0f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    t1 += dsum[((4 * pr + w) * RPT + c) * 2];
                    t2 += dsum[((4 * pr + w) * RPT + c) * 2 + 1];
                }
                dtot[2 * row] = t1;
                dtot[2 * row + 1] = t2;
            }
            ew_barrier<kEwThreads>();
            wait_or_flag(bar(kBarFinal), n & 1, p.status);
            ROWS_STAMP(5);  // last value product done
            tc_fence_after();
            {
                uint32_t u0[RPT], u1[RPT], w0[RPT], w1[RPT];
                ld_cols(lane_base + C::kColO + 0 * NR + c0, u0);
                ld_cols(lane_base + C::kColO + 1 * NR + c0, u1);
                ld_cols(lane_base + C::kColO + 2 * NR + c0, w0);
                ld_cols(lane_base + C::kColO + 3 * NR + c0, w1);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar(kBarOFree));  // the accumulators are in registers: the next item's value products may start
#pragma unroll
                for (int c = 0; c < RPT; ++c) {
                    const int row = c0 + c;
                    if (!((row_mask >> c) & 1u) || kr >= HD) continue;  // (head dimension 64: lanes 64-127 repeat lanes 0-63)
                    const float O1 = __uint_as_float(u0[c]) + __uint_as_float(u1[c]);
                    const float O2 = __uint_as_float(w0[c]) + __uint_as_float(w1[c]);
                    const float D1 = dtot[2 * row], D2 = dtot[2 * row + 1];
                    if (p.partials) {
                        float* rec = p.partials + ((row0 + row) * p.num_splits + it.split) * REC;
                        rec[4 + kr] = O1;
                        rec[4 + HD + kr] = O2;
                        if (kr == 0) {
                            const float rf = ref[row];
                            rec[0] = (rf > -INFINITY) ? rf * kLn2 : -INFINITY;
                            rec[1] = D1;
                            rec[2] = D2;
                            rec[3] = 0.0f;
                        }
                    } else {
                        float o = 0.0f;
                        if (D1 > 0.0f) {
                            const float inv = 1.0f / D1;
                            o = O1 * inv * (1.0f + D2 * inv) - O2 * inv;
                        }
                        store_value(p.out, (row0 + row) * HD + kr, o, p.out_dtype);
                    }
                }
            }
            ++n;
        }
        if (threadIdx.x == 0) ROWS_FLUSH(0);
    }

    ROWS_STAMP(6);  // epilogue stores issued
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, C::kTmemCols);
    }
    ROWS_STAMP(7);  // end
}

template <int NR, int HD>
int launch_rows(const CUtensorMap& tmQ, const CUtensorMap& tmR, const CUtensorMap& tmK, const CUtensorMap& tmV,
                const RowsParams& rp, unsigned grid, int dev, cudaStream_t stream)
{
    static bool configured[64] = {false};
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        if (cudaFuncSetAttribute(plx_decode_rows_kernel<NR, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 RowsCfg<NR, HD>::kSmemBytes) != cudaSuccess)
            return PLX_ERR_CUDA;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(RowsCfg<NR, HD>::kThreads, 1, 1);
    cfg.dynamicSmemBytes = RowsCfg<NR, HD>::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, plx_decode_rows_kernel<NR, HD>, tmQ, tmR, tmK, tmV, rp) == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}

}  // namespace

// ---------------------------------------------------------------------------
// Host side (reached through parallax_decode_fwd_multi and parallax_decode_fwd_rows)
// ---------------------------------------------------------------------------
bool plx_decode_rows_supported(int Hq, int Hkv, int D, int Lq)
{
    return (D == 64 || D == 128) && Hkv > 0 && Hq % Hkv == 0 && Lq > 0 && static_cast<long long>(Hq / Hkv) * Lq <= kMaxRows;
}

// q, r, out [B, Hq, Lq, D]; `records` / `record_bytes`: room for split records (may be null: one split).
// Paged cache: block_table != nullptr, k_cache / v_cache are the page pools of pool_rows rows, T_max = page_size * max_pages.
bool plx_decode_rows_page_size_ok(int page_size) { return page_size > 0 && page_size % 16 == 0 && (BK % page_size == 0 || page_size % BK == 0); }

// Modelled time (us) of a step of `base` (sequence, KV head) pairs, each cut into c splits of a context of `tiles`
// 128-key tiles, on `sms` SMs; used only to choose c.  The items run in generations of `sms`; a 128-key tile takes the
// longer of the SM's own time for it (the element-wise chain: about 0.62 / 0.78 us at sixteen rows and D = 128 / 64,
// 1.15 / 1.10 us at 32 rows) and its share of HBM (tile bytes x active SMs / 7 TB/s), so a last generation of few
// items runs at the SM's pace while full ones run at HBM's; an item costs 1.2 us besides its tiles, a split step its
// merge (5 us and the records written and read).  Fitted to and checked against measured steps of 20...128 sequences
// of 2048...16384 keys (within 5 % on all of them but two, 8 % on those).
static double rows_step_model(long long base, int sms, int tiles, int c, int nr, int D, long long rows, int page_box, int parts)
{
    const long long items = base * c;
    const int tps = (tiles + c - 1) / c;
    double t_sm = nr == 16 ? (D == 128 ? 0.62 : 0.78) : (D == 128 ? 1.15 : 1.10);
    // small pages: the producer warp's copies per tile set the SM's pace (16-key pages: 1.6 us measured)
    if (page_box > 0 && page_box <= 32 && t_sm < 25.6 / page_box) t_sm = 25.6 / page_box;
    // K and V tile, bf16, every SM streaming; the parts of a KV head's rows run side by side and share their tiles in L2
    const double t_hbm = 2.0 * 128 * D * 2 * sms / 7.0e6 / parts;
    const long long full = items / sms, rem = items % sms;
    double t = static_cast<double>(full) * tps * (t_sm > t_hbm ? t_sm : t_hbm);
    if (rem) {
        const double share = t_hbm * static_cast<double>(rem) / sms;
        t += tps * (t_sm > share ? t_sm : share);
    }
    t += 1.2 * static_cast<double>((items + sms - 1) / sms);
    if (c > 1) t += 5.0 + 2.0 * static_cast<double>(rows) * c * (2 * D + 4) * 4 / 7.0e6;
    return t;
}

// The split count the library plans for a call with room for its records (num_splits = 0).
int plx_decode_rows_plan(int B, int Hq, int Hkv, int D, int Lq, int T_max, int page_size, int sms)
{
    const int rows = (Hq / Hkv) * Lq;
    const int parts = rows > 32 ? 2 : 1, rows_per_part = (rows + parts - 1) / parts;
    const long long base_ctas = static_cast<long long>(B) * Hkv * parts;
    const int tiles_max = (T_max + BK - 1) / BK;
    const int nr = rows_per_part <= 16 ? 16 : 32;
    const int page_box = page_size > 0 ? (page_size < BK ? page_size : BK) : 0;
    int ns = 1;
    if (base_ctas < sms) {
        const long long want = sms / base_ctas;
        const long long most = tiles_max / 4 > 1 ? tiles_max / 4 : 1;
        ns = static_cast<int>(want < most ? want : most);
        if (ns > 64) ns = 64;
    } else {
        double best = 1e30;
        for (const int c : {1, 2, 3, 4, 6, 8}) {
            if (c > 1 && tiles_max / c < 8) break;
            const double cost = rows_step_model(base_ctas, sms, tiles_max, c, nr, D, static_cast<long long>(B) * Hq * Lq, page_box, parts);
            if (cost < best * 0.995) {  // a larger count has to pay for its records
                best = cost;
                ns = c;
            }
        }
    }
    const int tps = (tiles_max + ns - 1) / ns;
    return (tiles_max + tps - 1) / tps;  // no split without a tile
}

int plx_decode_rows_fwd(const void* q, const void* r, const void* k_cache, const void* v_cache, const int32_t* seqlens,
                        void* out, int B, int Hq, int Hkv, int D, int Lq, int T_max, float scale, int out_dtype,
                        void* records, size_t record_bytes, int num_splits, int32_t* status, cudaStream_t stream,
                        const int32_t* block_table, int page_size, int max_pages, long long pool_rows, int32_t* ticket)
{
    if (!q || !r || !k_cache || !v_cache || !out) return PLX_ERR_NULL_POINTER;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Lq <= 0 || T_max <= 0 || Hq % Hkv != 0) return PLX_ERR_BAD_SHAPE;
    if (!plx_decode_rows_supported(Hq, Hkv, D, Lq)) return PLX_ERR_UNSUPPORTED;
    if (block_table && (!plx_decode_rows_page_size_ok(page_size) || max_pages <= 0 || pool_rows <= 0)) return PLX_ERR_UNSUPPORTED;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (num_splits < 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    const long long q_rows = static_cast<long long>(B) * Hq * Lq;
    const long long kv_rows = block_table ? pool_rows : static_cast<long long>(B) * Hkv * T_max;
    const int page_box = block_table ? (page_size < BK ? page_size : BK) : BK;
    if (q_rows >= (1LL << 31) - 65536 || kv_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    if (!plx_aligned(q, 16) || !plx_aligned(r, 16) || !plx_aligned(k_cache, 16) || !plx_aligned(v_cache, 16) ||
        !plx_aligned(out, 16) || (records && !plx_aligned(records, 16)))
        return PLX_ERR_ALIGNMENT;
    // more than 32 rows per KV head: two items of half the rows each, neighbours in the item order, so that they run at
    // the same time on two SMs and the second one's K/V tiles come out of L2
    const int rows = (Hq / Hkv) * Lq;
    const int parts = rows > 32 ? 2 : 1, rows_per_part = (rows + parts - 1) / parts;
    const int nr = rows_per_part <= 16 ? 16 : 32;

    CUtensorMap tmQ, tmR, tmK, tmV;
    int rc;
    const CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
    if ((rc = make_tensor_map_2d(&tmQ, q, D, static_cast<uint64_t>(q_rows), nr, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmR, r, D, static_cast<uint64_t>(q_rows), nr, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmK, k_cache, D, static_cast<uint64_t>(kv_rows), page_box, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmV, v_cache, D, static_cast<uint64_t>(kv_rows), page_box, promo)) != PLX_OK) return rc;

    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return PLX_ERR_CUDA;
    // Split plan (one CTA per SM is resident).  Fewer CTAs than SMs: as many splits as keep the grid within one
    // generation, at least four 128-key tiles each.  More: the split count whose modelled time is least
    // (rows_step_model), at least eight tiles each.  Always what the record space holds.
    const long long base_ctas = static_cast<long long>(B) * Hkv * parts;
    const int tiles_max = (T_max + BK - 1) / BK;
    int ns = 1;
    if (records) {
        if (num_splits == 0) {
            ns = plx_decode_rows_plan(B, Hq, Hkv, D, Lq, T_max, block_table ? page_size : 0, sms);
        } else {
            ns = num_splits < tiles_max ? num_splits : tiles_max;
        }
        while (ns > 1 && static_cast<size_t>(q_rows) * ns * (2 * D + 4) * sizeof(float) > record_bytes) --ns;
    } else if (num_splits > 1) {
        return PLX_ERR_WORKSPACE;
    }
    const int tps = (tiles_max + ns - 1) / ns;
    ns = (tiles_max + tps - 1) / tps;  // no split without a tile
    if (base_ctas * ns > 0x7fffffffLL) return PLX_ERR_BAD_SHAPE;
    RowsParams rp{seqlens, out, ns > 1 ? static_cast<float*>(records) : nullptr, status, B, Hq, Hkv, Lq, T_max,
                  rows, parts, rows_per_part, ns, tps, static_cast<int>(base_ctas * ns), ticket,
                  scale * 1.4426950408889634f, out_dtype, block_table,
                  page_size, max_pages, page_box, pool_rows};
    PlxNvtxRange nvtx_range("plx_decode_rows_fwd");
    // With a ticket word and more items than SMs: one CTA per SM, each drawing items until none is left (item i of a CTA
    // overlaps the end of item i - 1).  Otherwise one CTA per item.
    const long long n_items = base_ctas * ns;
    if (!ticket || n_items <= sms) rp.ticket = nullptr;
    const unsigned grid = static_cast<unsigned>(rp.ticket ? sms : n_items);
    if (D == 128)
        rc = nr == 16 ? launch_rows<16, 128>(tmQ, tmR, tmK, tmV, rp, grid, dev, stream)
                      : launch_rows<32, 128>(tmQ, tmR, tmK, tmV, rp, grid, dev, stream);
    else
        rc = nr == 16 ? launch_rows<16, 64>(tmQ, tmR, tmK, tmV, rp, grid, dev, stream)
                      : launch_rows<32, 64>(tmQ, tmR, tmK, tmV, rp, grid, dev, stream);
    if (rc != PLX_OK) return rc;
    if (ns > 1)
        return plx_combine_after_producer(static_cast<const float*>(records), out, static_cast<int>(q_rows), D, ns,
                                          out_dtype, stream);
    return PLX_OK;
}

#if PLX_TRACE
extern "C" int plx_rows_trace_read(long long* host, int n, int reset)
{
    if (cudaMemcpyFromSymbol(host, g_rows_trace, n * sizeof(long long)) != cudaSuccess) return PLX_ERR_CUDA;
    if (reset) {
        long long zeros[32] = {0};
        if (cudaMemcpyToSymbol(g_rows_trace, zeros, sizeof zeros) != cudaSuccess) return PLX_ERR_CUDA;
    }
    return PLX_OK;
}
#endif

extern "C" int parallax_decode_fwd_rows(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                        const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                                        int T_max, float scale, int out_dtype, void* workspace, size_t workspace_bytes,
                                        int num_splits, int32_t* status, void* stream)
{
    return plx_decode_rows_fwd(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, Lq, T_max, scale, out_dtype, workspace,
                               workspace_bytes, num_splits, status, static_cast<cudaStream_t>(stream), nullptr, 0, 0, 0, nullptr);
}
