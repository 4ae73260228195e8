// Parallax backward of the multi-token causal forward for B200 (sm_100a): the closed-form gradients
// of App. "Parallax Backward" (Eq. "bwd_dq", "bwd_dr", "bwd_dk", "bwd_dv"), streamed in the two
// passes the appendix names, both on the 5th-generation tensor cores (tcgen05, accumulators in TMEM).
//
//   prep        tau_i = dO_i . o_i, beta_i = dO_i . vbar_i (Eq. "bwd_projections"); one float4 per row:
//               (lse_i * log2 e, tbar_i, tau_i, beta_i)
//   row pass    CTA = (sequence, query head, 128 query rows); streams 64-key tiles of K (four stages: a
//               K tile is held until its gradient products have drained) and V (two stages):
//                 S1 = Q K^T, S2 = R K^T, A = dO V^T     (tcgen05.mma SS -> TMEM, one issuing warp each)
//                 p = exp2(S1 s - lse), delta = A - beta, c = tbar - S2
//                 G1 = p (A - tau + c delta), G2 = -p delta               (bf16, back into TMEM)
//                 dQ += G1 K, dR += G2 K                                  (A from TMEM, K MN-major)
//               epilogue: dQ * scale, dR.
//   column pass CTA = (sequence, KV head, 128 keys); streams 64-row tiles of Q, R, dO of every query
//               head of the group, with the roles of the operands exchanged (keys are the TMEM lanes):
//                 [S1^T S2^T] = K [Q; R]^T (one N = 128 product: Q and R rows are neighbours in shared
//                 memory), A^T = V dO^T                                   (one issuing warp each)
//                 W = p (1 + c), G1 = p (A - tau + c delta) * scale, G2 = -p delta
//                 dV += W dO, dK += G1 Q + G2 R       (W, G1 from TMEM; G2 from a swizzled smem tile)
//
// The softmax weights come straight from the saved log-sum-exp, so there is no running maximum and
// no rescaling.  TMEM (512 columns): S1 | S2 | A (64 fp32 columns each), two packed-bf16 operand
// regions (32 columns each), two [128 x D] fp32 accumulators.  The score buffer is single: the
// element-wise warps pull a tile into registers and release the buffer at once, so the next tile's
// score products overlap their arithmetic.  Measured on a cycle timeline of one CTA: the MMAs with both
// operands in shared memory run at the shared-memory bandwidth (an M = 128, N = 64, K = 16 step reads
// 6 KiB for 32 cycles of math), not at the tensor pipe's rate; that, not instruction issue, bounds
// both passes.
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
#include "plx_tcgen05.cuh"

namespace {

constexpr int BM = 128;  // stationary rows per CTA = TMEM lanes
constexpr int BN = 64;   // streamed rows per step
#ifndef PLX_BWD_PARTS
#define PLX_BWD_PARTS 2
#endif
// Element-wise warps: kParts threads per TMEM lane, each owning BN / kParts columns of a step (four
// threads per lane measured 5-8 % slower than two).
constexpr int kParts = PLX_BWD_PARTS;
static_assert(kParts == 2 || kParts == 4, "two or four threads per TMEM lane");
constexpr int kEwWarps = 4 * kParts;
constexpr int kEwThreads = kEwWarps * 32;
constexpr int kPerThread = BN / kParts;      // streamed columns per element-wise thread
// Issuing a tcgen05.mma costs its thread 80-100 cycles whatever the tile size, so the score products
// of a step are issued by several warps in parallel (one product each), the gradient products by one more.
constexpr int kScoreWarp = kEwWarps;         // first score-issuing warp; owns the TMEM allocation
constexpr int kRowScoreWarps = 3;            // row pass: S1 | S2 | A
constexpr int kColScoreWarps = 2;            // column pass: [S1^T S2^T] (one N = 128 product) | A^T
constexpr int kRowThreads = (kEwWarps + kRowScoreWarps + 2) * 32;
constexpr int kColThreads = (kEwWarps + kColScoreWarps + 2) * 32;
constexpr int kBigBox = BM * 128;            // [128 rows x 64 columns] bf16: 16 KiB
constexpr int kSmallBox = BN * 128;          // [64 rows x 64 columns] bf16: 8 KiB
constexpr int kBigTile = 2 * kBigBox, kSmallTile = 2 * kSmallBox;
constexpr int kQRBox = 2 * kSmallBox;         // column pass: [64 Q rows | 64 R rows] of one 64-column box
constexpr uint32_t kColS1 = 0, kColS2 = 64, kColA = 128, kColGx = 192, kColGy = 224, kColAcc1 = 256, kColAcc2 = 384;
constexpr uint32_t kTmemCols = 512;
constexpr int kStatsBytes = BN * 16;         // one float4 per streamed row

// row pass: Q | R | dO stationary, K and V two stages each
constexpr int kRowOffQ = 0, kRowOffR = kBigTile, kRowOffDO = 2 * kBigTile;
constexpr int kRowKStages = 4;  // a K tile is held from its score products until its gradient products have drained
constexpr int kRowOffK = 3 * kBigTile, kRowOffV = kRowOffK + kRowKStages * kSmallTile;
constexpr int kRowOffBar = kRowOffV + 2 * kSmallTile;
// column pass: K | V stationary, three stages of (Q, R, dO) (a stage is held until its gradient products
// have drained), two slots of per-row records, the G2 operand tile.  This fills the 227 KiB a CTA may
// have, so the kernel relies on the dynamic shared memory starting on a 1024-byte boundary (checked).
constexpr int kColOffK = 0, kColOffV = kBigTile;
constexpr int kColStages = 3;
constexpr int kColStage = 3 * kSmallTile;
constexpr int kColOffIn = 2 * kBigTile;
constexpr int kColOffStats = kColOffIn + kColStages * kColStage;
constexpr int kColOffG2 = kColOffStats + 2 * kStatsBytes;
constexpr int kColOffBar = kColOffG2 + kBigBox;
constexpr int kNumBars = 24;
constexpr int kRowSmemBytes = 1024 + kRowOffBar + kNumBars * 8 + 16;
constexpr int kColSmemBytes = kColOffBar + kNumBars * 8 + 16;
static_assert(kColSmemBytes <= 232448, "column pass: shared memory budget");
static_assert(kColStage % 1024 == 0 && kColOffG2 % 1024 == 0, "swizzled tiles need 1024-byte alignment");

template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[N])
{
    if constexpr (N == 32) tmem_ld32(taddr, r);
    else tmem_ld16(taddr, r);
}
template <int N>
__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const uint32_t (&r)[N])
{
    if constexpr (N == 16) tmem_st16(taddr, r);
    else tmem_st8(taddr, r);
}

struct BwdParams {
    const int32_t* seqlens;
    const float4* stats;  // [B*Hq*Lq (+ BN padding)]: lse * log2(e), tbar, tau, beta
    void* g0;             // row pass: dq      column pass: dk
    void* g1;             // row pass: dr      column pass: dv
    int32_t* status;
    int B, Hq, Hkv, Lq, T_max, tiles;
    float scale, scale_log2e;
    int grad_dtype;
};

// ---------------------------------------------------------------------------
// prep: tau, beta and the packed per-row record
// ---------------------------------------------------------------------------
template <int HD, typename IoT>
__global__ void __launch_bounds__(256)
plx_bwd_prep_kernel(const __nv_bfloat16* __restrict__ dout, const IoT* __restrict__ out, const IoT* __restrict__ vbar,
                    const float* __restrict__ lse, const float* __restrict__ tbar, float4* __restrict__ stats,
                    long long rows)
{
    const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    float tau = 0.0f, beta = 0.0f;
#pragma unroll
    for (int c = 0; c < HD / 32; ++c) {
        const size_t idx = static_cast<size_t>(row) * HD + c * 32 + lane;
        const float g = __bfloat162float(dout[idx]);
        tau += g * static_cast<float>(out[idx]);
        beta += g * static_cast<float>(vbar[idx]);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        tau += __shfl_xor_sync(0xffffffffu, tau, off);
        beta += __shfl_xor_sync(0xffffffffu, beta, off);
    }
    if (lane == 0) stats[row] = make_float4(lse[row] * 1.4426950408889634f, tbar[row], tau, beta);
}

__device__ __forceinline__ void store_row_chunk(void* base, size_t idx, const float (&o)[32], int dtype)
{
    if (dtype == PLX_OUT_F32) {
        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(base) + idx);
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
    } else {
        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + idx);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(pack2(o[8 * i], o[8 * i + 1]), pack2(o[8 * i + 2], o[8 * i + 3]),
                                pack2(o[8 * i + 4], o[8 * i + 5]), pack2(o[8 * i + 6], o[8 * i + 7]));
    }
}

__device__ __forceinline__ void zero_rows(void* base, size_t first_elem, int count, int dtype)
{
    for (int i = threadIdx.x; i < count; i += blockDim.x) {
        if (dtype == PLX_OUT_F32)
            static_cast<float*>(base)[first_elem + i] = 0.0f;
        else
            static_cast<__nv_bfloat16*>(base)[first_elem + i] = __float2bfloat16_rn(0.0f);
    }
}

// rows `valid` .. `rows`-1 of a swizzled tile (boxes of `box_bytes`) are cleared by one warp
template <int kBoxes>
__device__ __forceinline__ void clear_tile_tail(uint8_t* tile, int box_bytes, int valid, int rows, int lane)
{
    if (valid < rows) {
        const int nrows = rows - max(valid, 0);
        const int first = max(valid, 0);
        for (int i = lane; i < kBoxes * nrows * 8; i += 32) {
            const int box = i / (nrows * 8), rem = i - box * nrows * 8;
            const int rr = first + (rem >> 3), ch = rem & 7;
            *reinterpret_cast<uint4*>(tile + box * box_bytes + rr * 128 + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async_smem();
    }
    __syncwarp();
}

// barrier slots (both passes)
// Every waiter consumes the phases of a barrier strictly in order, once per step.
enum : int { kBarStat = 0, kBarAFull = 1, kBarAFree = 3, kBarBFull = 5, kBarBFree = 7, kBarSFull = 9, kBarSFree = 10,
             kBarGFull = 11, kBarODone = 12, kBarFinal = 13, kBarKFull = 14, kBarKFree = 18 };

// ---------------------------------------------------------------------------
// row pass: dQ, dR
// ---------------------------------------------------------------------------
template <int HD>
__global__ void __launch_bounds__(kRowThreads, 1)
plx_bwd_row_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmR,
                   const __grid_constant__ CUtensorMap tmDO, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const BwdParams p)
{
    constexpr int kBoxes = HD / 64;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* const smem = smem_raw + (base - raw_addr);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kOutWarp = kScoreWarp + kRowScoreWarps, kTmaWarp = kOutWarp + 1;
    const int heads = p.B * p.Hq;
    const int qt = p.tiles - 1 - static_cast<int>(blockIdx.x / heads);  // heaviest (latest) tiles first
    const int bh = blockIdx.x % heads;
    const int b = bh / p.Hq, hq = bh - b * p.Hq;
    const int hkv = hq / (p.Hq / p.Hkv);

    int L = p.seqlens ? p.seqlens[b] : p.T_max;
    L = max(0, min(L, p.T_max));
    const int q0 = qt * BM;
    const int q_hi = min(q0 + BM, p.Lq);
    const int kv_end = min(L, max(0, L - p.Lq + q_hi));  // keys visible to the last row of this tile
    const int n_tiles = (kv_end + BN - 1) / BN;
    const size_t row0 = (static_cast<size_t>(b) * p.Hq + hq) * p.Lq;

    if (n_tiles == 0) {  // no row of the tile sees a key
        zero_rows(p.g0, (row0 + q0) * HD, (q_hi - q0) * HD, p.grad_dtype);
        zero_rows(p.g1, (row0 + q0) * HD, (q_hi - q0) * HD, p.grad_dtype);
        return;
    }

    auto bar = [&](int slot) { return base + kRowOffBar + 8 * slot; };
    const int kTmemSlot = kRowOffBar + kNumBars * 8;
    if (threadIdx.x == 0) {
        mbar_init(bar(kBarStat), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarBFull + s), 1);   // V stage
            mbar_init(bar(kBarBFree + s), 1);
        }
        for (int s = 0; s < kRowKStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1);
            mbar_init(bar(kBarKFree + s), 1);
        }
        mbar_init(bar(kBarSFull), kRowScoreWarps);
        mbar_init(bar(kBarSFree), kEwThreads);
        mbar_init(bar(kBarGFull), kEwThreads);
        mbar_init(bar(kBarODone), 1);
        mbar_init(bar(kBarFinal), 1);
        fence_barrier_init();
    }
    if (warp == kScoreWarp) {
        tmem_alloc(base + kTmemSlot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + kTmemSlot);
    const int kv_row0 = (b * p.Hkv + hkv) * p.T_max;

    if (warp == kTmaWarp) {
        if (lane == 0) {
            prefetch_tensormap(&tmQ);
            prefetch_tensormap(&tmR);
            prefetch_tensormap(&tmDO);
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
            const int q_row = static_cast<int>(row0) + q0;
            mbar_expect_tx(bar(kBarStat), 3 * kBoxes * kBigBox);
#pragma unroll
            for (int h = 0; h < kBoxes; ++h) {
                tma_load_2d(base + kRowOffQ + h * kBigBox, &tmQ, bar(kBarStat), 64 * h, q_row);
                tma_load_2d(base + kRowOffR + h * kBigBox, &tmR, bar(kBarStat), 64 * h, q_row);
                tma_load_2d(base + kRowOffDO + h * kBigBox, &tmDO, bar(kBarStat), 64 * h, q_row);
            }
            for (int j = 0; j < n_tiles; ++j) {
                const int s = j & 1, sk = j % kRowKStages;
                if (j >= kRowKStages) wait_or_flag(bar(kBarKFree + sk), ((j - kRowKStages) / kRowKStages) & 1, p.status);
                mbar_expect_tx(bar(kBarKFull + sk), kBoxes * kSmallBox);
#pragma unroll
                for (int h = 0; h < kBoxes; ++h)
                    tma_load_2d(base + kRowOffK + sk * kSmallTile + h * kSmallBox, &tmK, bar(kBarKFull + sk), 64 * h, kv_row0 + j * BN);
                if (j >= 2) wait_or_flag(bar(kBarBFree + s), ((j - 2) >> 1) & 1, p.status);
                mbar_expect_tx(bar(kBarBFull + s), kBoxes * kSmallBox);
#pragma unroll
                for (int h = 0; h < kBoxes; ++h)
                    tma_load_2d(base + kRowOffV + s * kSmallTile + h * kSmallBox, &tmV, bar(kBarBFull + s), 64 * h, kv_row0 + j * BN);
            }
        }
        __syncwarp();
    } else if (warp >= kScoreWarp && warp < kOutWarp) {
        // ===================== score products, one per warp: S1 = Q K^T | S2 = R K^T | A = dO V^T =====================
        const int which = warp - kScoreWarp;
        constexpr uint32_t idesc_s = make_idesc(BM, BN, 0, 0);
        const uint64_t dA = make_smem_desc(base + (which == 0 ? kRowOffQ : which == 1 ? kRowOffR : kRowOffDO), 0, 1024);
        const uint64_t dB0 = make_smem_desc(base + (which == 2 ? kRowOffV : kRowOffK), 0, 1024);
        const uint32_t dst = tmem + (which == 0 ? kColS1 : which == 1 ? kColS2 : kColA);
        wait_or_flag(bar(kBarStat), 0, p.status);
        for (int j = 0; j < n_tiles; ++j) {
            const int s = which == 2 ? (j & 1) : (j % kRowKStages);  // V: two stages, K: kRowKStages
            if (which == 2)
                wait_or_flag(bar(kBarBFull + s), (j >> 1) & 1, p.status);
            else
                wait_or_flag(bar(kBarKFull + s), (j / kRowKStages) & 1, p.status);
            if (L - j * BN < BN) {
                // Rows past the context may hold anything: clear them (K by the first warp, V by the third) so
                // that masked weights meet finite numbers; the three warps meet before any of them issues.
                if (which == 0) clear_tile_tail<kBoxes>(smem + kRowOffK + s * kSmallTile, kSmallBox, L - j * BN, BN, lane);
                if (which == 2) clear_tile_tail<kBoxes>(smem + kRowOffV + s * kSmallTile, kSmallBox, L - j * BN, BN, lane);
                asm volatile("bar.sync 2, %0;" ::"n"(kRowScoreWarps * 32) : "memory");
            }
            if (j >= 1) wait_or_flag(bar(kBarSFree), (j - 1) & 1, p.status);  // the previous tile sits in registers
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dB = dB0 + static_cast<uint64_t>((s * kSmallTile) >> 4);
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint64_t soff = static_cast<uint64_t>(((ks >> 2) * kSmallBox + (ks & 3) * 32) >> 4);
                    const uint64_t boff = static_cast<uint64_t>(((ks >> 2) * kBigBox + (ks & 3) * 32) >> 4);
                    mma_ss(dst, dA + boff, dB + soff, idesc_s, ks > 0);
                }
                tc_commit(bar(kBarSFull));
                if (which == 2) tc_commit(bar(kBarBFree + s));  // V(j) has no other reader
            }
            __syncwarp();
        }
        if (which == 0) wait_or_flag(bar(kBarFinal), 0, p.status);  // all tensor work has drained before TMEM is released
    } else if (warp == kOutWarp) {
        // ===================== gradient products: dQ += G1 K, dR += G2 K =====================
        constexpr uint32_t idesc_o = make_idesc(BM, HD, 0, 1);  // G K-major from TMEM, K tile MN-major
        const uint64_t dK0 = make_smem_desc(base + kRowOffK, kSmallBox, 1024);
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j % kRowKStages;
            wait_or_flag(bar(kBarKFull + s), (j / kRowKStages) & 1, p.status);
            wait_or_flag(bar(kBarGFull), j & 1, p.status);
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dK = dK0 + static_cast<uint64_t>((s * kSmallTile) >> 4);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks) {
                    const uint64_t dk = dK + static_cast<uint64_t>((ks * 2048) >> 4);
                    const uint32_t acc = (j > 0 || ks > 0) ? 1u : 0u;
                    mma_ts(tmem + kColAcc1, tmem + kColGx + ks * 8, dk, idesc_o, acc);
                    mma_ts(tmem + kColAcc2, tmem + kColGy + ks * 8, dk, idesc_o, acc);
                }
                tc_commit(bar(kBarODone));
                tc_commit(bar(kBarKFree + s));
                if (j == n_tiles - 1) tc_commit(bar(kBarFinal));
            }
            __syncwarp();
        }
    } else {
        // ===================== element-wise warps =====================
        // thread = (part, row): row = TMEM lane; part selects keys 32*part .. 32*part+31 of every tile
        const int part = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const int qi = q0 + row;
        const bool row_valid = qi < p.Lq;
        const int limit = row_valid ? (L - p.Lq + qi) : -1;  // last visible key of this row
        const uint32_t lane_base = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        float4 st = make_float4(INFINITY, 0.0f, 0.0f, 0.0f);  // rows outside the problem: p = 0
        if (row_valid) st = p.stats[row0 + qi];
        const uint64_t sc2 = pack_f2(p.scale_log2e, p.scale_log2e), nl2 = pack_f2(-st.x, -st.x);
        const uint64_t tb2 = pack_f2(st.y, st.y), ntau2 = pack_f2(-st.z, -st.z), nbeta2 = pack_f2(-st.w, -st.w);
        const uint64_t neg1 = pack_f2(-1.0f, -1.0f);

        for (int j = 0; j < n_tiles; ++j) {
            const int tile0 = j * BN, key0 = tile0 + kPerThread * part;
            const bool need_mask = tile0 + BN - 1 > L - p.Lq + q0;  // some row of the tile is cut by the diagonal
            uint32_t a[kPerThread], g[kPerThread], av[kPerThread];
            wait_or_flag(bar(kBarSFull), j & 1, p.status);
            tc_fence_after();
            tmem_ld_cols(lane_base + kColS1 + kPerThread * part, a);
            tmem_ld_cols(lane_base + kColS2 + kPerThread * part, g);
            tmem_ld_cols(lane_base + kColA + kPerThread * part, av);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(kBarSFree));  // the score buffer may be overwritten

            uint32_t h1[kPerThread / 2], h2[kPerThread / 2];
            auto emit = [&](auto mask_tag) {
                constexpr bool kMask = decltype(mask_tag)::value;
#pragma unroll
                for (int i = 0; i < kPerThread; i += 2) {
                    float e0, e1;
                    unpack_f2(fma2(pack_f2(__uint_as_float(a[i]), __uint_as_float(a[i + 1])), sc2, nl2), e0, e1);
                    float x0 = ex2(e0), x1 = ex2(e1);
                    if (kMask) {
                        x0 = (key0 + i <= limit) ? x0 : 0.0f;
                        x1 = (key0 + i + 1 <= limit) ? x1 : 0.0f;
                    }
                    const uint64_t x2 = pack_f2(x0, x1);
                    const uint64_t a2 = pack_f2(__uint_as_float(av[i]), __uint_as_float(av[i + 1]));
                    const uint64_t delta = add2(a2, nbeta2);
                    const uint64_t c2 = fma2(pack_f2(__uint_as_float(g[i]), __uint_as_float(g[i + 1])), neg1, tb2);
                    const uint64_t inner = fma2(c2, delta, add2(a2, ntau2));  // a - tau + (tbar - t) delta
                    float y0, y1, z0, z1;
                    unpack_f2(mul2(x2, inner), y0, y1);
                    unpack_f2(mul2(mul2(x2, neg1), delta), z0, z1);
                    h1[i >> 1] = pack2(y0, y1);
                    h2[i >> 1] = pack2(z0, z1);
                }
            };
            if (need_mask)
                emit(std::true_type{});
            else
                emit(std::false_type{});
            if (j >= 1) wait_or_flag(bar(kBarODone), (j - 1) & 1, p.status);  // G of the previous tile has been consumed
            tc_fence_after();
            tmem_st_cols(lane_base + kColGx + (kPerThread / 2) * part, h1);
            tmem_st_cols(lane_base + kColGy + (kPerThread / 2) * part, h2);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(kBarGFull));
        }

        // ---- epilogue: each of the row's two threads writes HD/2 columns of dQ and dR ----
        wait_or_flag(bar(kBarFinal), 0, p.status);
        tc_fence_after();
        const size_t orow = (row0 + qi) * HD + (HD / 2) * part;
#pragma unroll 1
        for (int c = 0; c < (part < 2 ? HD / 64 : 0); ++c) {  // the first two threads of a row write half of it each
            uint32_t u[32], w[32];
            tmem_ld32(lane_base + kColAcc1 + (HD / 2) * part + c * 32, u);
            tmem_ld32(lane_base + kColAcc2 + (HD / 2) * part + c * 32, w);
            tmem_wait_ld();
            if (row_valid) {
                float o[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(u[i]) * p.scale;
                store_row_chunk(p.g0, orow + c * 32, o, p.grad_dtype);
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(w[i]);
                store_row_chunk(p.g1, orow + c * 32, o, p.grad_dtype);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kScoreWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

// ---------------------------------------------------------------------------
// column pass: dK, dV
// ---------------------------------------------------------------------------
template <int HD>
__global__ void __launch_bounds__(kColThreads, 1)
plx_bwd_col_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                   const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmR,
                   const __grid_constant__ CUtensorMap tmDO, const BwdParams p)
{
    constexpr int kBoxes = HD / 64;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    uint8_t* const smem = smem_raw;
    if ((base & 1023u) != 0) {  // the layout below has no room for alignment slack
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, PLX_ERR_ALIGNMENT);
        return;
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kOutWarp = kScoreWarp + kColScoreWarps, kTmaWarp = kOutWarp + 1;
    const int streams = p.B * p.Hkv;
    const int kt = static_cast<int>(blockIdx.x / streams);  // earliest key tiles (most rows) first
    const int bs = blockIdx.x % streams;
    const int b = bs / p.Hkv, hkv = bs - b * p.Hkv;
    const int G = p.Hq / p.Hkv;

    int L = p.seqlens ? p.seqlens[b] : p.T_max;
    L = max(0, min(L, p.T_max));
    const int k0 = kt * BM;
    const int k_hi = min(k0 + BM, p.T_max);
    const size_t kv_row0 = (static_cast<size_t>(b) * p.Hkv + hkv) * p.T_max;

    // query rows that see a key of this tile: qi >= k0 - (L - Lq)
    const int qi_min = max(0, k0 - (L - p.Lq));
    const int i0 = qi_min / BN;
    const int n_i = (p.Lq + BN - 1) / BN;
    const int per_head = n_i - i0;
    const int steps = (k0 < L && per_head > 0) ? G * per_head : 0;
    if (steps == 0) {  // keys past the context, or seen by no row
        zero_rows(p.g0, (kv_row0 + k0) * HD, (k_hi - k0) * HD, p.grad_dtype);
        zero_rows(p.g1, (kv_row0 + k0) * HD, (k_hi - k0) * HD, p.grad_dtype);
        return;
    }

    auto bar = [&](int slot) { return base + kColOffBar + 8 * slot; };
    const int kTmemSlot = kColOffBar + kNumBars * 8;
    if (threadIdx.x == 0) {
        mbar_init(bar(kBarStat), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(kBarAFull + s), 1);            // slot of per-row records
            mbar_init(bar(kBarAFree + s), kEwThreads);
        }
        for (int s = 0; s < kColStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1);            // stage of (Q, R, dO)
            mbar_init(bar(kBarKFree + s), 1);
        }
        mbar_init(bar(kBarSFull), kColScoreWarps);
        mbar_init(bar(kBarSFree), kEwThreads);
        mbar_init(bar(kBarGFull), kEwThreads);
        mbar_init(bar(kBarODone), 1);
        mbar_init(bar(kBarFinal), 1);
        fence_barrier_init();
    }
    if (warp == kScoreWarp) {
        tmem_alloc(base + kTmemSlot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + kTmemSlot);

    // step t -> (query head of the group, 64-row tile)
    auto step_head = [&](int t) { return hkv * G + t / per_head; };
    auto step_tile = [&](int t) { return i0 + t % per_head; };

    if (warp == kTmaWarp) {
        if (lane == 0) {
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
            prefetch_tensormap(&tmQ);
            prefetch_tensormap(&tmR);
            prefetch_tensormap(&tmDO);
            mbar_expect_tx(bar(kBarStat), 2 * kBoxes * kBigBox);
#pragma unroll
            for (int h = 0; h < kBoxes; ++h) {
                tma_load_2d(base + kColOffK + h * kBigBox, &tmK, bar(kBarStat), 64 * h, static_cast<int>(kv_row0) + k0);
                tma_load_2d(base + kColOffV + h * kBigBox, &tmV, bar(kBarStat), 64 * h, static_cast<int>(kv_row0) + k0);
            }
            for (int t = 0; t < steps; ++t) {
                const int s = t % kColStages, ss = t & 1;
                if (t >= kColStages) wait_or_flag(bar(kBarKFree + s), ((t - kColStages) / kColStages) & 1, p.status);
                const uint32_t dst = base + kColOffIn + s * kColStage;
                const size_t qrow = (static_cast<size_t>(b) * p.Hq + step_head(t)) * p.Lq + static_cast<size_t>(step_tile(t)) * BN;
                mbar_expect_tx(bar(kBarKFull + s), 3 * kBoxes * kSmallBox);
#pragma unroll
                for (int h = 0; h < kBoxes; ++h) {
                    // Q and R rows of one 64-column box are neighbours: one N = 128 operand [Q; R] for the score product
                    tma_load_2d(dst + h * kQRBox, &tmQ, bar(kBarKFull + s), 64 * h, static_cast<int>(qrow));
                    tma_load_2d(dst + h * kQRBox + kSmallBox, &tmR, bar(kBarKFull + s), 64 * h, static_cast<int>(qrow));
                    tma_load_2d(dst + 2 * kSmallTile + h * kSmallBox, &tmDO, bar(kBarKFull + s), 64 * h, static_cast<int>(qrow));
                }
                // the rows' records: their slot is free once the element-wise warps of step t - 2 have read it
                if (t >= 2) wait_or_flag(bar(kBarAFree + ss), ((t - 2) >> 1) & 1, p.status);
                mbar_expect_tx(bar(kBarAFull + ss), kStatsBytes);
                bulk_load(base + kColOffStats + ss * kStatsBytes, p.stats + qrow, kStatsBytes, bar(kBarAFull + ss));
            }
        }
        __syncwarp();
    } else if (warp >= kScoreWarp && warp < kOutWarp) {
        // ===================== score products: [S1^T S2^T] = K [Q; R]^T (one N = 128 product) | A^T = V dO^T =====================
        const int which = warp - kScoreWarp;
        constexpr uint32_t idesc_qr = make_idesc(BM, 2 * BN, 0, 0), idesc_a = make_idesc(BM, BN, 0, 0);
        const uint64_t dA = make_smem_desc(base + (which == 0 ? kColOffK : kColOffV), 0, 1024);
        const uint64_t dB0 = make_smem_desc(base + kColOffIn + (which == 0 ? 0 : 2 * kSmallTile), 0, 1024);
        wait_or_flag(bar(kBarStat), 0, p.status);
        if (L - k0 < BM) {  // keys past the context: clear their rows once (K by the first warp, V by the second)
            clear_tile_tail<kBoxes>(smem + (which == 0 ? kColOffK : kColOffV), kBigBox, L - k0, BM, lane);
            asm volatile("bar.sync 2, %0;" ::"n"(kColScoreWarps * 32) : "memory");
        }
        for (int t = 0; t < steps; ++t) {
            const int s = t % kColStages;
            wait_or_flag(bar(kBarKFull + s), (t / kColStages) & 1, p.status);
            if (t >= 1) wait_or_flag(bar(kBarSFree), (t - 1) & 1, p.status);
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dB = dB0 + static_cast<uint64_t>((s * kColStage) >> 4);
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint64_t aoff = static_cast<uint64_t>(((ks >> 2) * kBigBox + (ks & 3) * 32) >> 4);
                    if (which == 0)
                        mma_ss(tmem + kColS1, dA + aoff, dB + static_cast<uint64_t>(((ks >> 2) * kQRBox + (ks & 3) * 32) >> 4), idesc_qr, ks > 0);
                    else
                        mma_ss(tmem + kColA, dA + aoff, dB + static_cast<uint64_t>(((ks >> 2) * kSmallBox + (ks & 3) * 32) >> 4), idesc_a, ks > 0);
                }
                tc_commit(bar(kBarSFull));
            }
            __syncwarp();
        }
        if (which == 0) wait_or_flag(bar(kBarFinal), 0, p.status);
    } else if (warp == kOutWarp) {
        // ===================== gradient products: dV += W dO, dK += G1 Q + G2 R =====================
        constexpr uint32_t idesc_o = make_idesc(BM, HD, 0, 1);
        // streamed tiles as MN-major B operands: dO in 8 KiB boxes, Q and R interleaved in 16 KiB boxes
        const uint64_t dDO0 = make_smem_desc(base + kColOffIn + 2 * kSmallTile, kSmallBox, 1024);
        const uint64_t dQ0 = make_smem_desc(base + kColOffIn, kQRBox, 1024);
        const uint64_t dG2 = make_smem_desc(base + kColOffG2, 0, 1024);
        for (int t = 0; t < steps; ++t) {
            const int s = t % kColStages;
            wait_or_flag(bar(kBarKFull + s), (t / kColStages) & 1, p.status);
            wait_or_flag(bar(kBarGFull), t & 1, p.status);
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dQ = dQ0 + static_cast<uint64_t>((s * kColStage) >> 4);
                const uint64_t dR = dQ + static_cast<uint64_t>(kSmallBox >> 4);
                const uint64_t dDO = dDO0 + static_cast<uint64_t>((s * kColStage) >> 4);
#pragma unroll
                for (int ks = 0; ks < BN / 16; ++ks) {
                    const uint64_t koff = static_cast<uint64_t>((ks * 2048) >> 4);
                    const uint32_t acc = (t > 0 || ks > 0) ? 1u : 0u;
                    mma_ts(tmem + kColAcc2, tmem + kColGx + ks * 8, dDO + koff, idesc_o, acc);   // dV += W dO
                    mma_ts(tmem + kColAcc1, tmem + kColGy + ks * 8, dQ + koff, idesc_o, acc);    // dK += G1 Q
                    mma_ss(tmem + kColAcc1, dG2 + static_cast<uint64_t>((ks * 32) >> 4), dR + koff, idesc_o, 1u);  // dK += G2 R
                }
                tc_commit(bar(kBarODone));
                tc_commit(bar(kBarKFree + s));
                if (t == steps - 1) tc_commit(bar(kBarFinal));
            }
            __syncwarp();
        }
    } else {
        // ===================== element-wise warps =====================
        // thread = (part, key): key = TMEM lane; part selects query rows 32*part .. 32*part+31 of every step
        const int part = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const int key = k0 + row;
        const bool key_valid = key < L;
        const uint32_t lane_base = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const int swz = row & 7;
        const int diag = L - p.Lq;  // row qi sees keys <= diag + qi
        uint8_t* const g2row = smem + kColOffG2 + row * 128;

        for (int t = 0; t < steps; ++t) {
            const int s = t & 1;
            const int qi0 = step_tile(t) * BN + kPerThread * part;  // first query row of this thread's columns
            // masks are needed where the tile meets the diagonal, the end of the context or the end of the rows
            const bool need_mask = (k0 + BM - 1 > diag + step_tile(t) * BN) || (k0 + BM > L) || (step_tile(t) * BN + BN > p.Lq);
            const float4* const stats = reinterpret_cast<const float4*>(smem + kColOffStats + s * kStatsBytes) + kPerThread * part;
            uint32_t a[kPerThread], g[kPerThread], av[kPerThread];
            wait_or_flag(bar(kBarAFull + s), (t >> 1) & 1, p.status);  // the records of this step have landed
            wait_or_flag(bar(kBarSFull), t & 1, p.status);
            tc_fence_after();
            tmem_ld_cols(lane_base + kColS1 + kPerThread * part, a);
            tmem_ld_cols(lane_base + kColS2 + kPerThread * part, g);
            tmem_ld_cols(lane_base + kColA + kPerThread * part, av);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(kBarSFree));

            uint32_t hw[kPerThread / 2], h1[kPerThread / 2], h2[kPerThread / 2];
            auto emit = [&](auto mask_tag) {
                constexpr bool kMask = decltype(mask_tag)::value;
#pragma unroll
                for (int i = 0; i < kPerThread; i += 2) {
                    const float4 st0 = stats[i], st1 = stats[i + 1];  // (lse2, tbar, tau, beta) of the two query rows
                    float x0 = ex2(fmaf(__uint_as_float(a[i]), p.scale_log2e, -st0.x));
                    float x1 = ex2(fmaf(__uint_as_float(a[i + 1]), p.scale_log2e, -st1.x));
                    const float a0 = __uint_as_float(av[i]), a1 = __uint_as_float(av[i + 1]);
                    const float dl0 = a0 - st0.w, dl1 = a1 - st1.w;
                    const float c0 = st0.y - __uint_as_float(g[i]), c1 = st1.y - __uint_as_float(g[i + 1]);
                    float w0 = x0 * (1.0f + c0), w1 = x1 * (1.0f + c1);
                    float y0 = x0 * p.scale * (a0 - st0.z + c0 * dl0), y1 = x1 * p.scale * (a1 - st1.z + c1 * dl1);
                    float z0 = -x0 * dl0, z1 = -x1 * dl1;
                    if (kMask) {  // select on the results: the records of rows outside the problem hold anything
                        const bool v0 = key_valid && (qi0 + i < p.Lq) && (key <= diag + qi0 + i);
                        const bool v1 = key_valid && (qi0 + i + 1 < p.Lq) && (key <= diag + qi0 + i + 1);
                        w0 = v0 ? w0 : 0.0f;
                        y0 = v0 ? y0 : 0.0f;
                        z0 = v0 ? z0 : 0.0f;
                        w1 = v1 ? w1 : 0.0f;
                        y1 = v1 ? y1 : 0.0f;
                        z1 = v1 ? z1 : 0.0f;
                    }
                    hw[i >> 1] = pack2(w0, w1);
                    h1[i >> 1] = pack2(y0, y1);
                    h2[i >> 1] = pack2(z0, z1);
                }
            };
            if (need_mask)
                emit(std::true_type{});
            else
                emit(std::false_type{});
            mbar_arrive(bar(kBarAFree + s));  // the records have been read
            if (t >= 1) wait_or_flag(bar(kBarODone), (t - 1) & 1, p.status);  // the previous operands have been consumed
            tc_fence_after();
            tmem_st_cols(lane_base + kColGx + (kPerThread / 2) * part, hw);
            tmem_st_cols(lane_base + kColGy + (kPerThread / 2) * part, h1);
#pragma unroll
            for (int q8 = 0; q8 < kPerThread / 8; ++q8) {  // G2: K-major [128 keys x 64 rows] tile, 128-byte swizzle
                const int chunk = (part * (kPerThread / 8) + q8) ^ swz;
                *reinterpret_cast<uint4*>(g2row + chunk * 16) = make_uint4(h2[4 * q8], h2[4 * q8 + 1], h2[4 * q8 + 2], h2[4 * q8 + 3]);
            }
            tmem_wait_st();
            tc_fence_before();
            fence_proxy_async_smem();
            mbar_arrive(bar(kBarGFull));
        }

        // ---- epilogue: each of the key's two threads writes HD/2 columns of dK and dV ----
        wait_or_flag(bar(kBarFinal), 0, p.status);
        tc_fence_after();
        const size_t orow = (kv_row0 + key) * HD + (HD / 2) * part;
#pragma unroll 1
        for (int c = 0; c < (part < 2 ? HD / 64 : 0); ++c) {  // the first two threads of a key write half of it each
            uint32_t u[32], w[32];
            tmem_ld32(lane_base + kColAcc1 + (HD / 2) * part + c * 32, u);
            tmem_ld32(lane_base + kColAcc2 + (HD / 2) * part + c * 32, w);
            tmem_wait_ld();
            if (key < p.T_max) {
                float o[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = key_valid ? __uint_as_float(u[i]) : 0.0f;
                store_row_chunk(p.g0, orow + c * 32, o, p.grad_dtype);
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = key_valid ? __uint_as_float(w[i]) : 0.0f;
                store_row_chunk(p.g1, orow + c * 32, o, p.grad_dtype);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kScoreWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

template <typename K>
bool set_smem(K kernel, int bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

}  // namespace

extern "C" size_t parallax_prefill_bwd_workspace_bytes(int B, int Hq, int Lq)
{
    if (B <= 0 || Hq <= 0 || Lq <= 0) return 0;
    return (static_cast<size_t>(B) * Hq * Lq + BN) * sizeof(float4);
}

extern "C" int parallax_prefill_bwd(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                    const void* dout, const void* out, const float* lse, const float* tbar,
                                    const void* vbar, const int32_t* seqlens, void* dq, void* dr, void* dk, void* dv,
                                    int B, int Hq, int Hkv, int D, int Lq, int T_max, float scale, int io_dtype,
                                    int grad_dtype, void* workspace, size_t workspace_bytes, int32_t* status,
                                    void* stream)
{
    if (!q || !r || !k_cache || !v_cache || !dout || !out || !lse || !tbar || !vbar || !dq || !dr || !dk || !dv ||
        !workspace)
        return PLX_ERR_NULL_POINTER;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || Lq <= 0 || T_max <= 0 || Hq % Hkv != 0) return PLX_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return PLX_ERR_UNSUPPORTED;
    if ((io_dtype != PLX_OUT_BF16 && io_dtype != PLX_OUT_F32) || (grad_dtype != PLX_OUT_BF16 && grad_dtype != PLX_OUT_F32))
        return PLX_ERR_BAD_SHAPE;
    const long long q_rows = static_cast<long long>(B) * Hq * Lq, kv_rows = static_cast<long long>(B) * Hkv * T_max;
    if (q_rows >= (1LL << 31) - 65536 || kv_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    const void* ptrs[] = {q, r, k_cache, v_cache, dout, out, vbar, dq, dr, dk, dv, workspace};
    for (const void* ptr : ptrs)
        if (!plx_aligned(ptr, 16)) return PLX_ERR_ALIGNMENT;
    if (workspace_bytes < parallax_prefill_bwd_workspace_bytes(B, Hq, Lq)) return PLX_ERR_WORKSPACE;
    const int q_tiles = (Lq + BM - 1) / BM, k_tiles = (T_max + BM - 1) / BM;
    if (static_cast<long long>(q_tiles) * B * Hq > 0x7fffffffLL || static_cast<long long>(k_tiles) * B * Hkv > 0x7fffffffLL)
        return PLX_ERR_BAD_SHAPE;

    CUtensorMap tmQb, tmRb, tmDOb, tmKs, tmVs, tmQs, tmRs, tmDOs, tmKb, tmVb;  // b: 128-row boxes, s: 64-row boxes
    int rc;
    const CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
    const uint64_t qr = static_cast<uint64_t>(q_rows), kr = static_cast<uint64_t>(kv_rows);
    if ((rc = make_tensor_map_2d(&tmQb, q, D, qr, BM, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmRb, r, D, qr, BM, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmDOb, dout, D, qr, BM, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmKs, k_cache, D, kr, BN, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmVs, v_cache, D, kr, BN, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmQs, q, D, qr, BN, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmRs, r, D, qr, BN, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmDOs, dout, D, qr, BN, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmKb, k_cache, D, kr, BM, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmVb, v_cache, D, kr, BM, promo)) != PLX_OK) return rc;

    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PLX_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        bool ok = set_smem(plx_bwd_row_kernel<128>, kRowSmemBytes) && set_smem(plx_bwd_row_kernel<64>, kRowSmemBytes) &&
                  set_smem(plx_bwd_col_kernel<128>, kColSmemBytes) && set_smem(plx_bwd_col_kernel<64>, kColSmemBytes);
        if (!ok) return PLX_ERR_CUDA;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float4* stats = static_cast<float4*>(workspace);
    const __nv_bfloat16* g = static_cast<const __nv_bfloat16*>(dout);

    PlxNvtxRange nvtx_range("plx_prefill_bwd(prep, row pass, column pass)");
    // the padding records past the last row are read by the column pass (and masked): keep them finite
    if (cudaMemsetAsync(stats + q_rows, 0, BN * sizeof(float4), st) != cudaSuccess) return PLX_ERR_CUDA;
    const unsigned prep_grid = static_cast<unsigned>((q_rows + 7) / 8);
    if (D == 128) {
        if (io_dtype == PLX_OUT_F32)
            plx_bwd_prep_kernel<128, float><<<prep_grid, 256, 0, st>>>(g, static_cast<const float*>(out), static_cast<const float*>(vbar), lse, tbar, stats, q_rows);
        else
            plx_bwd_prep_kernel<128, __nv_bfloat16><<<prep_grid, 256, 0, st>>>(g, static_cast<const __nv_bfloat16*>(out), static_cast<const __nv_bfloat16*>(vbar), lse, tbar, stats, q_rows);
    } else {
        if (io_dtype == PLX_OUT_F32)
            plx_bwd_prep_kernel<64, float><<<prep_grid, 256, 0, st>>>(g, static_cast<const float*>(out), static_cast<const float*>(vbar), lse, tbar, stats, q_rows);
        else
            plx_bwd_prep_kernel<64, __nv_bfloat16><<<prep_grid, 256, 0, st>>>(g, static_cast<const __nv_bfloat16*>(out), static_cast<const __nv_bfloat16*>(vbar), lse, tbar, stats, q_rows);
    }

    const float sl2e = scale * 1.4426950408889634f;
    BwdParams rp{seqlens, stats, dq, dr, status, B, Hq, Hkv, Lq, T_max, q_tiles, scale, sl2e, grad_dtype};
    BwdParams cp{seqlens, stats, dk, dv, status, B, Hq, Hkv, Lq, T_max, k_tiles, scale, sl2e, grad_dtype};
    const unsigned row_grid = static_cast<unsigned>(q_tiles * B * Hq), col_grid = static_cast<unsigned>(k_tiles * B * Hkv);
    if (D == 128) {
        plx_bwd_row_kernel<128><<<row_grid, kRowThreads, kRowSmemBytes, st>>>(tmQb, tmRb, tmDOb, tmKs, tmVs, rp);
        plx_bwd_col_kernel<128><<<col_grid, kColThreads, kColSmemBytes, st>>>(tmKb, tmVb, tmQs, tmRs, tmDOs, cp);
    } else {
        plx_bwd_row_kernel<64><<<row_grid, kRowThreads, kRowSmemBytes, st>>>(tmQb, tmRb, tmDOb, tmKs, tmVs, rp);
        plx_bwd_col_kernel<64><<<col_grid, kColThreads, kColSmemBytes, st>>>(tmKb, tmVb, tmQs, tmRs, tmDOs, cp);
    }
    return cudaGetLastError() == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}
