// Parallax multi-token causal forward (prefill, chunked prefill, multi-token decode) for B200
// (sm_100a): Algorithm 1 with a 128-row query tile per CTA on the 5th-generation tensor cores.
//
// CTA = (sequence, query head, 128 query rows): 8 softmax warps (two threads per query row; the
// row is TMEM lane t, and each of the two threads owns 32 of the tile's 64 keys), two MMA warps
// (lane 0 of one issues the score MMAs, lane 0 of the other the value MMAs: a tcgen05.mma costs its
// issuing thread 80-100 cycles whatever its size, so one thread cannot keep the pipe busy) and one
// TMA producer warp.  Per 64-key tile j:
//
//   TMA      K(j), V(j) -> shared memory (128-byte swizzle), separate three-stage rings for K and V
//   MMA      S1 = Q K^T, S2 = R K^T      tcgen05.mma SS -> TMEM (one buffer: the softmax warps pull a
//                                        tile into registers and release it at once, so S(j+1) is
//                                        computed while they work on tile j)
//   softmax  tcgen05.ld S1, S2; causal mask; row max (each of the row's two threads reads the whole
//            S1 row, so no exchange or barrier is needed; the probe branch never drives the max);
//            lazy rescale of the TMEM accumulators (only when the max grows by more than 2^8);
//            P1 = exp2(S1 s - m), P2 = P1 * S2, row sums d1, d2.
//            The bf16 parts of P1, P2 and their bf16 rounding RESIDUALS go to a P region of TMEM of
//            their own (written once P.V(j-1) has drained).
//   MMA      O1 += P1 V + P1res V, O2 += P2 V + P2res V   (A from TMEM; V MN-major from smem)
//
// The residuals keep about 16 mantissa bits of P: P2 = P1 * S2 is amplified by |S2| ~ sqrt(D)
// before the two branches cancel in the final line, and rows that see only a few keys would
// otherwise lose two digits.
// A product with both operands in shared memory runs at the shared-memory bandwidth (6 KiB per
// K = 16 step of an N = 64 product), so every P operand is kept in TMEM: only Q/R, K and V are read
// from shared memory by the tensor cores.
// TMEM (512 columns): S1 | S2 (64 fp32 columns each), P1 | P2 bf16 and their residuals (4 x 32
// packed columns), O1, O2 (128 each).
// Epilogue: O1/d1 (1 + d2/d1) - O2/d1 straight from TMEM to global memory.
// Every wait is bounded; a wait that runs out sets the status word and control flow continues
// uniformly so that TMEM is always released.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <type_traits>

#include "parallax.h"
#include "plx_common.cuh"
#include "plx_internal.h"
#include "plx_tcgen05.cuh"

namespace {

constexpr int BM = 128;  // query rows per CTA = TMEM lanes
constexpr int BN = 64;   // keys per tile
// head dimension: template parameter HD in {64, 128}; shared-memory and TMEM offsets are sized for 128
constexpr int kSoftmaxWarps = 8;
constexpr int kSplit = kSoftmaxWarps / 4;         // threads per query row
constexpr int kKeysPerThread = BN / kSplit;       // 32
static_assert(kSplit == 2, "the softmax code below is written for two threads per row");
constexpr int kSoftmaxThreads = kSoftmaxWarps * 32;
constexpr int kMmaWarp = kSoftmaxWarps;      // issues the score MMAs, owns the TMEM allocation
constexpr int kPvWarp = kSoftmaxWarps + 1;   // issues the value MMAs
constexpr int kTmaWarp = kSoftmaxWarps + 2;
constexpr int kPrefillThreads = (kSoftmaxWarps + 3) * 32;
constexpr int kQBox = BM * 128;            // [128 rows x 64 columns] bf16 box of Q / R / P residual: 16 KiB
constexpr int kKvBox = BN * 128;           // [64 keys x 64 columns] bf16 box of K / V: 8 KiB
constexpr int kQTile = 2 * kQBox;          // Q or R tile, two column boxes
constexpr int kKvTile = 2 * kKvBox;        // K or V tile, two column boxes
constexpr int kOffQ = 0;
constexpr int kOffR = kQTile;
constexpr int kKStages = 3, kVStages = 3;  // a V tile is held until its value products have drained
constexpr int kOffK = 2 * kQTile;
constexpr int kOffV = kOffK + kKStages * kKvTile;
constexpr int kOffBar = kOffV + kVStages * kKvTile;
constexpr int kNumBars = 24;
constexpr int kOffTmemSlot = kOffBar + kNumBars * 8;
constexpr int kOffSum = kOffTmemSlot + 16;         // float2 [kSplit][128 rows]
constexpr int kOffMax = kOffSum + kSplit * BM * 8;  // float [2 tile parities][kSplit][128 rows]: row-max exchange (D = 64)
constexpr int kSmemBytes = 1024 + kOffMax + 2 * kSplit * BM * 4;
constexpr uint32_t kColS1 = 0, kColS2 = 64;                  // fp32 scores
constexpr uint32_t kColP = 128;  // P region(s): P1 | P2 packed bf16 (32 columns = 64 keys each) [| residuals]
constexpr uint32_t kTmemCols = 512;
// The P region is double-buffered wherever 512 columns allow it (plain weights, or head dimension 64):
// the softmax warps then store tile j while P.V(j-1) is still reading tile j-1.
template <bool kResidual, int HD>
struct TmemMap {
    static constexpr uint32_t kPWidth = kResidual ? 128 : 64;
    static constexpr int kPBuffers = (kColP + 2 * kPWidth + 2 * HD <= kTmemCols) ? 2 : 1;
    static constexpr uint32_t kColO1 = kColP + kPBuffers * kPWidth, kColO2 = kColO1 + HD;
    static_assert(kColO2 + HD <= kTmemCols, "TMEM budget");
};
constexpr float kLazyThreshold = 8.0f;  // log2 units

struct PrefillParams {
    const int32_t* seqlens;
    void* out;
    int32_t* status;
    int B, Hq, Hkv, Lq, T_max, q_tiles;
    float scale_log2e;
    int out_dtype;
    // optional per-row state for the backward (all three or none): lse, tbar fp32 [B,Hq,Lq]; vbar as out
    float* lse;
    float* tbar;
    void* vbar;
    // paged cache: int32 [B, max_pages] page ids (else nullptr); page_size is a multiple of the 64-key tile
    const int32_t* block_table;
    int page_size, max_pages;
    // Query heads whose rows share one 128-row tile: 1, or the whole group Hq / Hkv of a KV head when
    // (Hq / Hkv) * Lq <= 128 (their rows are contiguous in [B, Hq, Lq, D]), which then reads K/V once per
    // KV head and fills the tile with real rows.  Row r of a packed tile is token r mod Lq of head r / Lq.
    int pack;
    // Split-KV (short chunks on few sequences, where one CTA per row tile would leave SMs idle): CTA
    // (tile, split) walks key tiles [split * tiles_per_split, (split + 1) * tiles_per_split) and writes, per
    // row, the unnormalised state (m ln 2, d1, d2, 0, O1[D], O2[D]) as record `split` of the row's num_splits
    // records in `partials` (the decode path's record format; m = -inf marks an empty record); the rows are
    // finished by the decode path's merge kernel.  partials == nullptr: one CTA per tile, final output.
    float* partials;
    int num_splits, tiles_per_split;
    // PLX_P_BF16_ADAPTIVE runs as two launches over the same tiles, the plain build and the residual build; a
    // CTA leaves at once unless its tile is of its launch's kind: tile_filter 1 = only row tiles in which some
    // row sees fewer than residual_min_keys keys, 2 = only the others, 0 = every tile.  qt_hi: one past the last
    // row tile this launch covers (the host narrows the grids when the contexts are uniform).
    int tile_filter, residual_min_keys, qt_hi;
};

// barrier among the softmax warps only (named barrier 1)
__device__ __forceinline__ void softmax_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory"); }

// ---------------------------------------------------------------------------
// Kernel
// ---------------------------------------------------------------------------
// barrier slots
// Every waiter consumes the phases of a barrier strictly in order (a parity wait cannot tell phase
// n from phase n-2).  With two P buffers the softmax warps may finish tile j+1 before the value issuer has
// looked at tile j, so "P ready" and "P.V done" each use two barriers in turn (+ (j & 1)): a barrier then
// never gets more than one phase ahead of its waiter.  The end of
// all tensor work has its own single-phase barrier kBarFinal.
enum : int { kBarQ = 0, kBarSFull = 1, kBarSFree = 2, kBarPFull = 3 /* and 4 */, kBarODone = 18 /* and 19 */, kBarFinal = 5, kBarKFull = 6,
             kBarKFree = 9, kBarVFull = 12, kBarVFree = 15 };

// kResidual: also carry the bf16 rounding residuals of P1, P2 (fp32-class accuracy); without them P is
// plain bf16, the precision class of a bf16 tensor-core attention kernel.
template <bool kResidual, int HD>
__global__ void __launch_bounds__(kPrefillThreads, 1)
plx_prefill_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmR,
                   const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                   const PrefillParams p)
{
    static_assert(HD == 64 || HD == 128, "head dimension");
    using TM = TmemMap<kResidual, HD>;
    constexpr uint32_t kColO1 = TM::kColO1, kColO2 = TM::kColO2;
    constexpr int kPBuffers = TM::kPBuffers;
    constexpr bool kExchangeMax = (HD == 64);  // see the row maximum in the softmax warps
    constexpr int kBoxes = HD / 64;  // 64-column boxes per Q / R / K / V row
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* const smem = smem_raw + (base - raw_addr);

    // lets the merge kernel of a split-KV call (launched as a programmatic dependent) be scheduled now; it waits
    // for this grid's completion before it reads a record
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pack = p.pack;
    const int heads = p.B * (pack > 1 ? p.Hkv : p.Hq);  // tiles' owners: KV heads when packed, else query heads
    const int split = p.partials ? static_cast<int>(blockIdx.x % p.num_splits) : 0;
    const int tile_id = p.partials ? static_cast<int>(blockIdx.x / p.num_splits) : static_cast<int>(blockIdx.x);
    const int qt = p.qt_hi - 1 - tile_id / heads;  // heaviest (latest) tiles first
    const int bh = tile_id % heads;
    int b, hq, hkv;
    if (pack > 1) {
        b = bh / p.Hkv;
        hkv = bh - b * p.Hkv;
        hq = hkv * pack;  // first query head of the group
    } else {
        b = bh / p.Hq;
        hq = bh - b * p.Hq;
        hkv = hq / (p.Hq / p.Hkv);
    }
    const int rows = p.Lq * pack;  // rows owned by this (sequence, head or head group)

    int L = p.seqlens ? p.seqlens[b] : p.T_max;
    L = max(0, min(L, p.T_max));
    const int q0 = qt * BM;
    if (p.tile_filter) {
        // fewest keys a row of this tile sees (a packed tile holds token 0 of every head)
        const bool few = L - p.Lq + (pack > 1 ? 0 : q0) + 1 < p.residual_min_keys;
        if (few != (p.tile_filter == 1)) return;
    }
    const int q_hi = min(q0 + BM, rows);
    const int tok_hi = pack > 1 ? p.Lq : q_hi;                 // one past the latest token in this tile
    const int kv_end = min(L, max(0, L - p.Lq + tok_hi));  // keys visible to the latest token of this tile
    const int n_tiles_all = (kv_end + BN - 1) / BN;
    // this CTA's key tiles: all of them, or its split's share; jt0 is the first one's index in the context
    const int jt0 = p.partials ? split * p.tiles_per_split : 0;
    const int n_tiles = p.partials ? max(0, min(n_tiles_all, jt0 + p.tiles_per_split) - jt0) : n_tiles_all;
    const size_t out_row0 = (static_cast<size_t>(b) * p.Hq + hq) * p.Lq;

    if (n_tiles == 0 && p.partials) {  // no key tile for this split: empty records (only m is ever read)
        constexpr int REC = 2 * HD + 4;
        for (int i = threadIdx.x; i < q_hi - q0; i += kPrefillThreads)
            p.partials[((out_row0 + q0 + i) * p.num_splits + split) * REC] = -INFINITY;
        return;
    }
    if (n_tiles == 0) {  // nothing visible to any row: zeros
        for (int i = threadIdx.x; i < (q_hi - q0) * HD; i += kPrefillThreads) {
            const size_t idx = (out_row0 + q0) * HD + i;
            if (p.out_dtype == PLX_OUT_F32) {
                static_cast<float*>(p.out)[idx] = 0.0f;
                if (p.vbar) static_cast<float*>(p.vbar)[idx] = 0.0f;
            } else {
                static_cast<__nv_bfloat16*>(p.out)[idx] = __float2bfloat16_rn(0.0f);
                if (p.vbar) static_cast<__nv_bfloat16*>(p.vbar)[idx] = __float2bfloat16_rn(0.0f);
            }
        }
        if (p.lse)
            for (int i = threadIdx.x; i < q_hi - q0; i += kPrefillThreads) {
                p.lse[out_row0 + q0 + i] = INFINITY;
                p.tbar[out_row0 + q0 + i] = 0.0f;
            }
        return;
    }

    const uint32_t sQ = base + kOffQ, sR = base + kOffR;
    auto bar = [&](int slot) { return base + kOffBar + 8 * slot; };

    const int kv_row0 = (b * p.Hkv + hkv) * p.T_max;
    // first cache row of key tile j: contiguous slab, or (page id * Hkv + hkv) * page_size + offset in the page
    const int32_t* const table = p.block_table ? p.block_table + static_cast<size_t>(b) * p.max_pages : nullptr;
    auto tile_row = [&](int j) {
        if (!table) return kv_row0 + (jt0 + j) * BN;
        const int key = (jt0 + j) * BN, pg = key / p.page_size;
        return (__ldg(table + pg) * p.Hkv + hkv) * p.page_size + (key - pg * p.page_size);
    };

    // TMA producer's loads (only its lane 0 calls these)
    auto load_k = [&](int j) {
        const int s = j % kKStages;
        if (j >= kKStages) wait_or_flag(bar(kBarKFree + s), ((j - kKStages) / kKStages) & 1, p.status);
        const uint32_t dst = base + kOffK + s * kKvTile;
        const int row = tile_row(j);
        mbar_expect_tx(bar(kBarKFull + s), kBoxes * kKvBox);
#pragma unroll
        for (int h = 0; h < kBoxes; ++h) tma_load_2d(dst + h * kKvBox, &tmK, bar(kBarKFull + s), 64 * h, row);
    };
    auto load_v = [&](int j) {
        const int s = j % kVStages;
        if (j >= kVStages) wait_or_flag(bar(kBarVFree + s), ((j - kVStages) / kVStages) & 1, p.status);
        const uint32_t dst = base + kOffV + s * kKvTile;
        const int row = tile_row(j);
        mbar_expect_tx(bar(kBarVFull + s), kBoxes * kKvBox);
#pragma unroll
        for (int h = 0; h < kBoxes; ++h) tma_load_2d(dst + h * kKvBox, &tmV, bar(kBarVFull + s), 64 * h, row);
    };
    // The producer thread initialises the barriers itself and starts the first loads at once: they fly
    // while the other warps allocate TMEM and meet at the CTA barrier.
    if (warp == kTmaWarp && lane == 0) {
        mbar_init(bar(kBarQ), 1);
        for (int s = 0; s < kKStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1);
            mbar_init(bar(kBarKFree + s), 1);
        }
        for (int s = 0; s < kVStages; ++s) {
            mbar_init(bar(kBarVFull + s), 1);
            mbar_init(bar(kBarVFree + s), 1);
        }
        mbar_init(bar(kBarSFull), 1);
        mbar_init(bar(kBarSFree), kSoftmaxThreads);
        mbar_init(bar(kBarPFull), kSoftmaxThreads);
        mbar_init(bar(kBarPFull + 1), kSoftmaxThreads);
        mbar_init(bar(kBarODone), 1);
        mbar_init(bar(kBarODone + 1), 1);
        mbar_init(bar(kBarFinal), 1);
        fence_barrier_init();
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmR);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
        const int q_row = static_cast<int>(out_row0) + q0;
        mbar_expect_tx(bar(kBarQ), 2 * kBoxes * kQBox);
#pragma unroll
        for (int h = 0; h < kBoxes; ++h) {
            tma_load_2d(sQ + h * kQBox, &tmQ, bar(kBarQ), 64 * h, q_row);
            tma_load_2d(sR + h * kQBox, &tmR, bar(kBarQ), 64 * h, q_row);
        }
        for (int j = 0; j < kKStages && j < n_tiles; ++j) load_k(j);
    }
    if (warp == kMmaWarp) {
        tmem_alloc(base + kOffTmemSlot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + kOffTmemSlot);

    if (warp == kTmaWarp) {
        // ===================== TMA producer =====================
        // K runs kKStages tiles ahead of the score products, V follows the value products.
        if (lane == 0) {
            for (int j = 0; j < n_tiles; ++j) {
                load_v(j);
                if (j + kKStages < n_tiles) load_k(j + kKStages);
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ===================== score-product issuer =====================
        constexpr uint32_t idesc_s = make_idesc(BM, BN, 0, 0);  // Q/R and K both K-major

        // rows of a K tile past the context may hold anything: clear them (all 32 lanes)
        auto clear_tail = [&](uint8_t* tile, int j) {
            const int valid = L - (jt0 + j) * BN;
            if (valid < BN) {
                const int nrows = BN - valid;
                for (int i = lane; i < kBoxes * nrows * 8; i += 32) {
                    const int box = i / (nrows * 8), rem = i - box * nrows * 8;
                    const int rr = valid + (rem >> 3), ch = rem & 7;
                    *reinterpret_cast<uint4*>(tile + box * kKvBox + rr * 128 + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async_smem();
            }
            __syncwarp();
        };
        // Every shared-memory descriptor is built ONCE here; inside the loops a descriptor is a base plus
        // a compile-time constant in its start-address field (units of 16 bytes).  The issuing thread has
        // no other warp to hide latency behind, so anything rebuilt per MMA lands on the critical path.
        const uint64_t dQ = make_smem_desc(sQ, 0, 1024), dR = make_smem_desc(sR, 0, 1024);
        const uint64_t dK0 = make_smem_desc(base + kOffK, 0, 1024);

        // ---- S(j) may overwrite the score buffer as soon as every softmax thread holds tile j-1 in
        //      registers ----
        wait_or_flag(bar(kBarQ), 0, p.status);
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j % kKStages;
            wait_or_flag(bar(kBarKFull + s), (j / kKStages) & 1, p.status);
            clear_tail(smem + kOffK + s * kKvTile, j);
            if (j >= 1) wait_or_flag(bar(kBarSFree), (j - 1) & 1, p.status);
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dK = dK0 + static_cast<uint64_t>((s * kKvTile) >> 4);
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint64_t koff = static_cast<uint64_t>(((ks >> 2) * kKvBox + (ks & 3) * 32) >> 4);
                    const uint64_t qoff = static_cast<uint64_t>(((ks >> 2) * kQBox + (ks & 3) * 32) >> 4);
                    mma_ss(tmem + kColS1, dQ + qoff, dK + koff, idesc_s, ks > 0);
                    mma_ss(tmem + kColS2, dR + qoff, dK + koff, idesc_s, ks > 0);
                }
                tc_commit(bar(kBarSFull));
                tc_commit(bar(kBarKFree + s));
            }
            __syncwarp();
        }
        // all tensor work of this CTA has drained before TMEM is released
        wait_or_flag(bar(kBarFinal), 0, p.status);
    } else if (warp == kPvWarp) {
        // ===================== value-product issuer =====================
        constexpr uint32_t idesc_o = make_idesc(BM, HD, 0, 1);  // P K-major from TMEM, V MN-major
        const uint64_t dV0 = make_smem_desc(base + kOffV, kKvBox, 1024);
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j % kVStages;
            wait_or_flag(bar(kBarVFull + s), (j / kVStages) & 1, p.status);
            {   // rows of the V tile past the context may hold anything: clear them (all 32 lanes)
                const int valid = L - (jt0 + j) * BN;
                if (valid < BN) {
                    uint8_t* tile = smem + kOffV + s * kKvTile;
                    const int nrows = BN - valid;
                    for (int i = lane; i < kBoxes * nrows * 8; i += 32) {
                        const int box = i / (nrows * 8), rem = i - box * nrows * 8;
                        const int rr = valid + (rem >> 3), ch = rem & 7;
                        *reinterpret_cast<uint4*>(tile + box * kKvBox + rr * 128 + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                    fence_proxy_async_smem();
                }
                __syncwarp();
            }
            wait_or_flag(bar(kBarPFull + (j & 1)), (j >> 1) & 1, p.status);
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dV = dV0 + static_cast<uint64_t>((s * kKvTile) >> 4);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks) {
                    // keys 32h..32h+31 of a row were packed by its thread h: k-step ks = 8 packed columns
                    const uint64_t dv = dV + static_cast<uint64_t>((ks * 2048) >> 4);
                    const uint32_t acc = (j > 0 || ks > 0) ? 1u : 0u;
                    const uint32_t pcol = tmem + kColP + (j % kPBuffers) * TM::kPWidth + ks * 8;  // P1 | P2 [| P1res | P2res]
                    mma_ts(tmem + kColO1, pcol, dv, idesc_o, acc);
                    if (kResidual) mma_ts(tmem + kColO1, pcol + 64, dv, idesc_o, 1u);
                    mma_ts(tmem + kColO2, pcol + 32, dv, idesc_o, acc);
                    if (kResidual) mma_ts(tmem + kColO2, pcol + 96, dv, idesc_o, 1u);
                }
                tc_commit(bar(kBarODone + (j & 1)));
                tc_commit(bar(kBarVFree + s));
                if (j == n_tiles - 1) tc_commit(bar(kBarFinal));
            }
            __syncwarp();
        }
    } else {
        // ===================== softmax warps =====================
        // thread = (part, row): row = TMEM lane; part selects keys 32*part .. 32*part+31 of every tile
        const int part = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const int qi = q0 + row;
        const bool row_valid = qi < rows;
        const int limit = row_valid ? (L - p.Lq + (pack > 1 ? qi % p.Lq : qi)) : 0x7fffffff;  // last visible key of this row
        const uint32_t lane_base = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        float2* const s_sum = reinterpret_cast<float2*>(smem + kOffSum);
        const bool scale_neg = p.scale_log2e < 0.0f;
        float m_run = -INFINITY, d1 = 0.0f, d2 = 0.0f;

        // Scores of the current tile: this thread's 32 softmax scores (a) and probe scores (g), plus the
        // other half of the S1 row (v) for the row maximum (read redundantly by both threads of the row:
        // no exchange, no barrier).  Once they sit in registers the score buffer is released.
        uint32_t a[kKeysPerThread], g[kKeysPerThread], v[32];

        for (int j = 0; j < n_tiles; ++j) {
            const int tile0 = (jt0 + j) * BN, key0 = tile0 + kKeysPerThread * part;
            // some row of the tile is cut by the diagonal (a packed tile holds token 0 of every head)
            const bool need_mask = tile0 + BN - 1 > L - p.Lq + (pack > 1 ? 0 : q0);
            wait_or_flag(bar(kBarSFull), j & 1, p.status);
            tc_fence_after();
            tmem_ld32(lane_base + kColS1 + 32 * part, a);
            if constexpr (!kExchangeMax) tmem_ld32(lane_base + kColS1 + 32 * (part ^ 1), v);
            tmem_ld32(lane_base + kColS2 + 32 * part, g);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(kBarSFree));  // S(j+1) may be computed

            // ---- row maximum: extreme raw score in four independent chains, one multiply by the scale
            //      afterwards (min if the scale is negative).  D = 128: each thread also reads the other half
            //      of the row (no exchange, no barrier).  D = 64, where the softmax warps are the bound: each
            //      thread reduces its own half and the two warps of a row group swap the result through
            //      shared memory behind a 64-thread named barrier (one per tile; slots alternate by parity) ----
            float mx;
            {
                const float init = scale_neg ? INFINITY : -INFINITY;
                float ext[4] = {init, init, init, init};
                if constexpr (kExchangeMax) {
                    if (need_mask) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float x0 = (key0 + i <= limit) ? __uint_as_float(a[i]) : init;
                            ext[i & 3] = scale_neg ? fminf(ext[i & 3], x0) : fmaxf(ext[i & 3], x0);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; i += 2)
                            ext[(i >> 1) & 3] = scale_neg ? min3(ext[(i >> 1) & 3], __uint_as_float(a[i]), __uint_as_float(a[i + 1]))
                                                          : max3(ext[(i >> 1) & 3], __uint_as_float(a[i]), __uint_as_float(a[i + 1]));
                    }
                } else {
                    const int other0 = tile0 + 32 * (part ^ 1);
                    if (need_mask) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float x0 = (key0 + i <= limit) ? __uint_as_float(a[i]) : init;
                            const float x1 = (other0 + i <= limit) ? __uint_as_float(v[i]) : init;
                            ext[i & 3] = scale_neg ? min3(ext[i & 3], x0, x1) : max3(ext[i & 3], x0, x1);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float x0 = __uint_as_float(a[i]), x1 = __uint_as_float(v[i]);
                            ext[i & 3] = scale_neg ? min3(ext[i & 3], x0, x1) : max3(ext[i & 3], x0, x1);
                        }
                    }
                }
                float e = scale_neg ? fminf(fminf(ext[0], ext[1]), fminf(ext[2], ext[3]))
                                    : fmaxf(fmaxf(ext[0], ext[1]), fmaxf(ext[2], ext[3]));
                if constexpr (kExchangeMax) {
                    float* const s_max = reinterpret_cast<float*>(smem + kOffMax) + (j & 1) * kSplit * BM;
                    s_max[part * BM + row] = e;
                    asm volatile("bar.sync %0, 64;" ::"r"(2 + (warp & 3)) : "memory");  // the two warps of these 32 rows
                    const float o = s_max[(part ^ 1) * BM + row];
                    e = scale_neg ? fminf(e, o) : fmaxf(e, o);
                }
                mx = (fabsf(e) == INFINITY) ? -INFINITY : e * p.scale_log2e;  // nothing visible: -inf
            }

            // ---- lazy reference update (warp-uniform decision: tcgen05.ld/st are warp-wide; the other
            //      warp of these rows sees the same scores and take the same decision) ----
            const bool grow = mx > m_run + kLazyThreshold;
            // P.V(t) has drained once barrier kBarODone + (t & 1) has completed its phase t >> 1
            auto wait_pv = [&](int t) { wait_or_flag(bar(kBarODone + (t & 1)), (t >> 1) & 1, p.status); };
            if (__any_sync(0xffffffffu, grow)) {
                const float m_new = fmaxf(m_run, mx);
                if (j > 0) {
                    // the previous tile's second product must have drained before O is touched
                    wait_pv(j - 1);
                    tc_fence_after();
                    const float alpha = (m_new > -INFINITY) ? ex2(m_run - m_new) : 1.0f;  // m_run = -inf gives 0
                    d1 *= alpha;
                    d2 *= alpha;
                    const uint32_t colO = part ? kColO2 : kColO1;  // thread 0 of the row rescales O1, thread 1 O2
#pragma unroll 1
                    for (int c = 0; c < HD / 32; ++c) {
                        uint32_t v[32];
                        tmem_ld32(lane_base + colO + c * 32, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                        tmem_st32(lane_base + colO + c * 32, v);
                    }
                }
                m_run = m_new;
            }
            const float m_use = (m_run > -INFINITY) ? m_run : 0.0f;

            // ---- P1, P2: bf16 parts and bf16 residuals, packed two keys per register ----
            uint32_t hi1[kKeysPerThread / 2], hi2[kKeysPerThread / 2];
            uint32_t lo1[kKeysPerThread / 2], lo2[kKeysPerThread / 2];  // unused (and removed) without residuals
            const uint64_t sc2 = pack_f2(p.scale_log2e, p.scale_log2e), nm2 = pack_f2(-m_use, -m_use);
            const uint64_t neg1 = pack_f2(-1.0f, -1.0f);
            uint64_t sum1 = pack_f2(0.0f, 0.0f), sum2 = sum1;  // row sums as (even keys, odd keys) pairs
            auto emit = [&](auto mask_tag) {
                constexpr bool kMask = decltype(mask_tag)::value;
#pragma unroll
                for (int q8 = 0; q8 < kKeysPerThread / 8; ++q8) {
#pragma unroll
                    for (int e2 = 0; e2 < 4; ++e2) {
                        const int i = q8 * 8 + e2 * 2;
                        float e0, e1;
                        unpack_f2(fma2(pack_f2(__uint_as_float(a[i]), __uint_as_float(a[i + 1])), sc2, nm2), e0, e1);
                        float x0 = ex2(e0), x1 = ex2(e1);
                        if (kMask) {  // the probe scores are finite (real keys, or rows cleared to zero), so P2 follows
                            x0 = (key0 + i <= limit) ? x0 : 0.0f;
                            x1 = (key0 + i + 1 <= limit) ? x1 : 0.0f;
                        }
                        const uint64_t x2 = pack_f2(x0, x1);
                        const uint64_t y2 = mul2(x2, pack_f2(__uint_as_float(g[i]), __uint_as_float(g[i + 1])));
                        sum1 = add2(sum1, x2);
                        sum2 = add2(sum2, y2);
                        float y0, y1;
                        unpack_f2(y2, y0, y1);
                        const uint32_t h1 = pack2(x0, x1), h2 = pack2(y0, y1);
                        hi1[q8 * 4 + e2] = h1;
                        hi2[q8 * 4 + e2] = h2;
                        if (kResidual) {
                            float r0, r1;
                            unpack_f2(fma2(bf16x2_to_f2(h1), neg1, x2), r0, r1);
                            lo1[q8 * 4 + e2] = pack2(r0, r1);
                            unpack_f2(fma2(bf16x2_to_f2(h2), neg1, y2), r0, r1);
                            lo2[q8 * 4 + e2] = pack2(r0, r1);
                        }
                    }
                }
            };
            if (need_mask)
                emit(std::true_type{});
            else
                emit(std::false_type{});
            {
                float s0, s1;
                unpack_f2(sum1, s0, s1);
                d1 += s0 + s1;
                unpack_f2(sum2, s0, s1);
                d2 += s0 + s1;
            }
            // This tile's P region was last read by P.V(j - kPBuffers)
            if (j >= kPBuffers) wait_pv(j - kPBuffers);
            tc_fence_after();
            const uint32_t pcol = lane_base + kColP + (j % kPBuffers) * TM::kPWidth + (kKeysPerThread / 2) * part;
            tmem_st16(pcol, hi1);
            tmem_st16(pcol + 32, hi2);
            if constexpr (kResidual) {
                tmem_st16(pcol + 64, lo1);
                tmem_st16(pcol + 96, lo2);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(kBarPFull + (j & 1)));
        }

        // ---- epilogue: each of the row's two threads writes 64 of the 128 output columns ----
        s_sum[part * BM + row] = make_float2(d1, d2);
        softmax_barrier();
        const float2 other = s_sum[(part ^ 1) * BM + row];
        d1 += other.x;
        d2 += other.y;
        wait_or_flag(bar(kBarFinal), 0, p.status);
        tc_fence_after();
        const bool has_keys = d1 > 0.0f;
        const float inv = has_keys ? 1.0f / d1 : 0.0f;
        const float f1 = inv * (1.0f + d2 * inv);
        if (p.partials) {
            // split-KV: this row's unnormalised state as record `split` (see PrefillParams::partials)
            constexpr int REC = 2 * HD + 4;
            float* rec = p.partials + ((out_row0 + qi) * p.num_splits + split) * REC;
            if (row_valid && part == 0) {
                *reinterpret_cast<float4*>(rec) =
                    make_float4(has_keys ? m_run * 0.6931471805599453f : -INFINITY, d1, d2, 0.0f);
            }
#pragma unroll 1
            for (int c = 0; c < HD / 64; ++c) {
                uint32_t u[32], w[32];
                tmem_ld32(lane_base + kColO1 + (HD / 2) * part + c * 32, u);
                tmem_ld32(lane_base + kColO2 + (HD / 2) * part + c * 32, w);
                tmem_wait_ld();
                if (row_valid && has_keys) {
                    float4* d1p = reinterpret_cast<float4*>(rec + 4 + (HD / 2) * part + c * 32);
                    float4* d2p = reinterpret_cast<float4*>(rec + 4 + HD + (HD / 2) * part + c * 32);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        d1p[i] = make_float4(__uint_as_float(u[4 * i]), __uint_as_float(u[4 * i + 1]),
                                             __uint_as_float(u[4 * i + 2]), __uint_as_float(u[4 * i + 3]));
                        d2p[i] = make_float4(__uint_as_float(w[4 * i]), __uint_as_float(w[4 * i + 1]),
                                             __uint_as_float(w[4 * i + 2]), __uint_as_float(w[4 * i + 3]));
                    }
                }
            }
        } else {
        const size_t orow = (out_row0 + qi) * HD + (HD / 2) * part;  // each thread writes HD/2 columns
        if (p.lse && row_valid && part == 0) {
            // m_run is a reference exponent in log2 units (not necessarily the maximum): lse = m + log(omega)
            p.lse[out_row0 + qi] = has_keys ? (m_run + log2f(d1)) * 0.6931471805599453f : INFINITY;
            p.tbar[out_row0 + qi] = has_keys ? d2 * inv : 0.0f;
        }
#pragma unroll 1
        for (int c = 0; c < HD / 64; ++c) {
            uint32_t u[32], w[32];
            tmem_ld32(lane_base + kColO1 + (HD / 2) * part + c * 32, u);
            tmem_ld32(lane_base + kColO2 + (HD / 2) * part + c * 32, w);
            tmem_wait_ld();
            if (row_valid) {
                float o[32];
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    o[i] = has_keys ? (__uint_as_float(u[i]) * f1 - __uint_as_float(w[i]) * inv) : 0.0f;
                if (p.out_dtype == PLX_OUT_F32) {
                    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.out) + orow + c * 32);
#pragma unroll
                    for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                } else {
                    uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out) + orow + c * 32);
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        dst[i] = make_uint4(pack2(o[8 * i], o[8 * i + 1]), pack2(o[8 * i + 2], o[8 * i + 3]),
                                            pack2(o[8 * i + 4], o[8 * i + 5]), pack2(o[8 * i + 6], o[8 * i + 7]));
                }
                if (p.vbar) {  // vbar = O1 / d1, the softmax-weighted value mean
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(u[i]) * inv;
                    if (p.out_dtype == PLX_OUT_F32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.vbar) + orow + c * 32);
#pragma unroll
                        for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.vbar) + orow + c * 32);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            dst[i] = make_uint4(pack2(o[8 * i], o[8 * i + 1]), pack2(o[8 * i + 2], o[8 * i + 3]),
                                                pack2(o[8 * i + 4], o[8 * i + 5]), pack2(o[8 * i + 6], o[8 * i + 7]));
                    }
                }
            }
        }
        }  // final output (no split)
    }

    // release TMEM (same warp that allocated it), after every TMEM access of the CTA
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

static int prefill_impl(const void* q, const void* r, const void* k_cache, const void* v_cache,
                        const int32_t* seqlens, void* out, float* lse, float* tbar, void* vbar, int B, int Hq,
                        int Hkv, int D, int Lq, int T_max, float scale, int out_dtype, int p_precision,
                        int32_t* status, void* stream, const int32_t* block_table = nullptr, int page_size = 0,
                        int max_pages = 0, long long pool_rows = 0, void* workspace = nullptr,
                        size_t workspace_bytes = 0, int num_splits = 1)
{
    if (p_precision != PLX_P_BF16_RESIDUAL && p_precision != PLX_P_BF16 && p_precision != PLX_P_BF16_ADAPTIVE)
        return PLX_ERR_BAD_SHAPE;
    if (!q || !r || !k_cache || !v_cache || !out) return PLX_ERR_NULL_POINTER;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Lq <= 0 || T_max <= 0 || Hq % Hkv != 0) return PLX_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return PLX_ERR_UNSUPPORTED;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    const long long q_rows = static_cast<long long>(B) * Hq * Lq;
    const long long kv_rows = block_table ? pool_rows : static_cast<long long>(B) * Hkv * T_max;
    if (q_rows >= (1LL << 31) - 65536 || kv_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    if (!plx_aligned(q, 16) || !plx_aligned(r, 16) || !plx_aligned(k_cache, 16) || !plx_aligned(v_cache, 16) ||
        !plx_aligned(out, 16) || (vbar && !plx_aligned(vbar, 16)))
        return PLX_ERR_ALIGNMENT;
    if (num_splits < 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    if (workspace && !plx_aligned(workspace, 16)) return PLX_ERR_ALIGNMENT;
    if (num_splits > 1 && (!workspace || lse))  // no room for the records; saved state and splits do not combine
        return workspace ? PLX_ERR_BAD_SHAPE : PLX_ERR_WORKSPACE;
    const int G = Hq / Hkv;
    const int pack = (G > 1 && static_cast<long long>(G) * Lq <= BM) ? G : 1;
    const int q_tiles = pack > 1 ? 1 : (Lq + BM - 1) / BM;
    if (static_cast<long long>(q_tiles) * B * Hq > 0x7fffffffLL) return PLX_ERR_BAD_SHAPE;

    CUtensorMap tmQ, tmR, tmK, tmV;
    int rc;
    const CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
    if ((rc = make_tensor_map_2d(&tmQ, q, D, static_cast<uint64_t>(q_rows), BM, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmR, r, D, static_cast<uint64_t>(q_rows), BM, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmK, k_cache, D, static_cast<uint64_t>(kv_rows), BN, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmV, v_cache, D, static_cast<uint64_t>(kv_rows), BN, promo)) != PLX_OK) return rc;

    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PLX_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        bool ok = true;
        ok &= cudaFuncSetAttribute(plx_prefill_kernel<true, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
        ok &= cudaFuncSetAttribute(plx_prefill_kernel<false, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
        ok &= cudaFuncSetAttribute(plx_prefill_kernel<true, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
        ok &= cudaFuncSetAttribute(plx_prefill_kernel<false, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
        if (!ok) return PLX_ERR_CUDA;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    // Split-KV plan: only when one CTA per row tile leaves SMs idle (short chunks on few sequences) and the
    // caller supplied room for the records; about one CTA per SM, at least eight 64-key tiles per split.
    const long long base_ctas = static_cast<long long>(q_tiles) * B * (pack > 1 ? Hkv : Hq);
    const int tiles_max = (T_max + BN - 1) / BN;
    int ns = 1;
    if (workspace && !lse) {
        if (num_splits == 0) {
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return PLX_ERR_CUDA;
            if (base_ctas < sms) {
                const long long want = sms / base_ctas;  // one CTA per SM at most: a second generation would double the time
                const long long most = tiles_max / 8 > 1 ? tiles_max / 8 : 1;
                ns = static_cast<int>(want < most ? want : most);
                if (ns > 64) ns = 64;
            }
        } else {
            ns = num_splits < tiles_max ? num_splits : tiles_max;
        }
        const size_t rec_bytes = static_cast<size_t>(2 * D + 4) * sizeof(float);
        while (ns > 1 && static_cast<size_t>(q_rows) * ns * rec_bytes > workspace_bytes) --ns;  // what the workspace holds
    }
    int tps = (tiles_max + ns - 1) / ns;
    ns = (tiles_max + tps - 1) / tps;  // no split without a tile
    PrefillParams pp{seqlens, out, status, B, Hq, Hkv, Lq, T_max, q_tiles, scale * 1.4426950408889634f, out_dtype,
                     lse, tbar, vbar, block_table, page_size, max_pages, pack,
                     ns > 1 ? static_cast<float*>(workspace) : nullptr, ns, tps, 0, 0, q_tiles};
    if (base_ctas * ns > 0x7fffffffLL) return PLX_ERR_BAD_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PlxNvtxRange nvtx_range("plx_prefill_fwd");
    const long long ctas_per_qt = static_cast<long long>(B) * (pack > 1 ? Hkv : Hq) * ns;
    auto launch = [&](bool res, const PrefillParams& prm, int qt_lo, int qt_hi) {
        if (qt_hi <= qt_lo) return;
        PrefillParams lp = prm;
        lp.qt_hi = qt_hi;
        const unsigned grid = static_cast<unsigned>((qt_hi - qt_lo) * ctas_per_qt);
        if (D == 128) {
            if (res)
                plx_prefill_kernel<true, 128><<<grid, kPrefillThreads, kSmemBytes, st>>>(tmQ, tmR, tmK, tmV, lp);
            else
                plx_prefill_kernel<false, 128><<<grid, kPrefillThreads, kSmemBytes, st>>>(tmQ, tmR, tmK, tmV, lp);
        } else {
            if (res)
                plx_prefill_kernel<true, 64><<<grid, kPrefillThreads, kSmemBytes, st>>>(tmQ, tmR, tmK, tmV, lp);
            else
                plx_prefill_kernel<false, 64><<<grid, kPrefillThreads, kSmemBytes, st>>>(tmQ, tmR, tmK, tmV, lp);
        }
    };
    if (p_precision == PLX_P_BF16_ADAPTIVE) {
        // Two launches: the plain build for the row tiles all of whose rows see at least PLX_P_ADAPTIVE_MIN_KEYS
        // keys, the residual build for the others.  Uniform contexts: the boundary is known here and each grid
        // covers only its tiles; ragged contexts: both grids cover every tile and a CTA of the wrong kind leaves
        // at once (the boundary depends on seqlens, which lives on the device).
        pp.residual_min_keys = PLX_P_ADAPTIVE_MIN_KEYS;
        int qt_split = 0;  // row tiles below it carry residuals
        if (!seqlens) {
            if (pack > 1) {
                qt_split = (T_max - Lq + 1 < PLX_P_ADAPTIVE_MIN_KEYS) ? 1 : 0;
            } else {
                const long long first_plain_row = static_cast<long long>(PLX_P_ADAPTIVE_MIN_KEYS) - 1 - (T_max - Lq);  // q0 >= this: plain
                qt_split = first_plain_row <= 0 ? 0 : static_cast<int>((first_plain_row + BM - 1) / BM);
                if (qt_split > q_tiles) qt_split = q_tiles;
            }
        }
        PrefillParams plain = pp, resid = pp;
        plain.tile_filter = 2;
        resid.tile_filter = 1;
        launch(false, plain, seqlens ? 0 : qt_split, q_tiles);
        launch(true, resid, 0, seqlens ? q_tiles : qt_split);
    } else {
        launch(p_precision == PLX_P_BF16_RESIDUAL, pp, 0, q_tiles);
    }
    if (cudaGetLastError() != cudaSuccess) return PLX_ERR_CUDA;
    if (ns > 1)  // finish the rows: the decode path's merge over B * Hq * Lq rows of ns records each
        return plx_combine_after_producer(static_cast<const float*>(workspace), out, static_cast<int>(q_rows), D, ns,
                                          out_dtype, st);
    return PLX_OK;
}

extern "C" size_t parallax_prefill_workspace_bytes(int B, int Hq, int D, int Lq, int max_splits)
{
    if (B <= 0 || Hq <= 0 || D <= 0 || Lq <= 0 || max_splits <= 0 || max_splits > PLX_MAX_SPLITS) return 0;
    return static_cast<size_t>(B) * Hq * Lq * max_splits * (2 * D + 4) * sizeof(float);
}

extern "C" int parallax_prefill_fwd_ex(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                       const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                                       int T_max, float scale, int out_dtype, int p_precision, void* workspace,
                                       size_t workspace_bytes, int num_splits, int32_t* status, void* stream)
{
    return prefill_impl(q, r, k_cache, v_cache, seqlens, out, nullptr, nullptr, nullptr, B, Hq, Hkv, D, Lq, T_max, scale,
                        out_dtype, p_precision, status, stream, nullptr, 0, 0, 0, workspace, workspace_bytes, num_splits);
}

extern "C" int parallax_prefill_fwd(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                    const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                                    int T_max, float scale, int out_dtype, int p_precision, int32_t* status,
                                    void* stream)
{
    return prefill_impl(q, r, k_cache, v_cache, seqlens, out, nullptr, nullptr, nullptr, B, Hq, Hkv, D, Lq, T_max, scale,
                        out_dtype, p_precision, status, stream);
}

extern "C" int parallax_prefill_fwd_save(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                         const int32_t* seqlens, void* out, float* lse, float* tbar, void* vbar, int B,
                                         int Hq, int Hkv, int D, int Lq, int T_max, float scale, int out_dtype,
                                         int p_precision, int32_t* status, void* stream)
{
    if (!lse || !tbar || !vbar) return PLX_ERR_NULL_POINTER;
    return prefill_impl(q, r, k_cache, v_cache, seqlens, out, lse, tbar, vbar, B, Hq, Hkv, D, Lq, T_max, scale, out_dtype,
                        p_precision, status, stream);
}

extern "C" int parallax_prefill_fwd_paged(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                          const int32_t* block_table, const int32_t* seqlens, void* out, int B, int Hq,
                                          int Hkv, int D, int Lq, int num_pages, int page_size, int max_pages_per_seq,
                                          float scale, int out_dtype, int p_precision, int32_t* status, void* stream)
{
    if (!block_table) return PLX_ERR_NULL_POINTER;
    if (num_pages <= 0 || page_size <= 0 || page_size % BN != 0 || max_pages_per_seq <= 0) return PLX_ERR_BAD_SHAPE;
    const long long T_max = static_cast<long long>(page_size) * max_pages_per_seq;
    const long long pool_rows = static_cast<long long>(num_pages) * (Hkv > 0 ? Hkv : 1) * page_size;
    if (T_max >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    return prefill_impl(q, r, k_pages, v_pages, seqlens, out, nullptr, nullptr, nullptr, B, Hq, Hkv, D, Lq,
                        static_cast<int>(T_max), scale, out_dtype, p_precision, status, stream, block_table, page_size,
                        max_pages_per_seq, pool_rows);
}

extern "C" int parallax_prefill_fwd_paged_ex(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                             const int32_t* block_table, const int32_t* seqlens, void* out, int B,
                                             int Hq, int Hkv, int D, int Lq, int num_pages, int page_size,
                                             int max_pages_per_seq, float scale, int out_dtype, int p_precision,
                                             void* workspace, size_t workspace_bytes, int num_splits, int32_t* status,
                                             void* stream)
{
    if (!block_table) return PLX_ERR_NULL_POINTER;
    if (num_pages <= 0 || page_size <= 0 || page_size % BN != 0 || max_pages_per_seq <= 0) return PLX_ERR_BAD_SHAPE;
    const long long T_max = static_cast<long long>(page_size) * max_pages_per_seq;
    const long long pool_rows = static_cast<long long>(num_pages) * (Hkv > 0 ? Hkv : 1) * page_size;
    if (T_max >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    return prefill_impl(q, r, k_pages, v_pages, seqlens, out, nullptr, nullptr, nullptr, B, Hq, Hkv, D, Lq,
                        static_cast<int>(T_max), scale, out_dtype, p_precision, status, stream, block_table, page_size,
                        max_pages_per_seq, pool_rows, workspace, workspace_bytes, num_splits);
}
