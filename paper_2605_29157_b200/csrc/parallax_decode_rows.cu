// Multi-token decode step with up to 64 rows per KV head (a few dozen new tokens per sequence times the
// query heads of a GQA group) on the tcgen05 tensor cores, with the KEYS on the TMEM lanes.
//
// The row-major multi-token kernel computes a 128-row tile whatever the number of rows, and the mma.sync decode
// kernel is bound by its SM work from about ten rows on.  Here the tensor time follows the rows present:
//   S^T [128 keys x 2 NR]  = K_c [Q; R]^T        one N = 2 NR product per 128-key tile (Algorithm 1: S1, S2)
//   O1^T [D x NR]         += V_c^T P1^T          A = the V tile read MN-major (head dimension on M), B = P^T
//   O2^T [D x NR]         += V_c^T P2^T
// so a step of r rows costs what r rows cost, and K/V is read once per KV head for all its rows and both
// branches.  The price is that a row's running maximum lives across the 128 lanes of a tile: the element-wise
// threads reduce it with a register transpose inside each warp and one exchange through shared memory per tile,
// and the reference exponent moves only when a tile exceeds it by 2^8 (then the accumulators are rescaled in
// TMEM).  P1, P2 reach the tensor cores as bf16 plus their bf16 rounding residuals, as everywhere in the library.
//
// Output: rows finished in place (one split), or the decode path's partial records
// (m ln 2, d1, d2, 0, O1[D], O2[D]) per (row, split), merged by the decode path's combine kernel.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "parallax.h"
#include "plx_common.cuh"
#include "plx_tcgen05.cuh"

// Defined in parallax_decode.cu: the split merge launched as a programmatic dependent of the kernel before it.
int plx_combine_after_producer(const float* partials, void* out, int rows, int D, int num_splits, int out_dtype,
                               cudaStream_t stream);

namespace {

constexpr int BK = 128;  // keys per tile = TMEM lanes
constexpr int NR = 64;   // rows of a KV head per CTA (the MMA N extent; fewer rows are padded)
constexpr int HD = 128;  // head dimension
constexpr int kEwWarps = 8;                    // element-wise warps: two threads per key, 32 rows each
constexpr int kEwThreads = kEwWarps * 32;
constexpr int kRowsPerThread = NR / 2;
constexpr int kMmaWarp = kEwWarps, kTmaWarp = kEwWarps + 1;
constexpr int kRowsThreads = (kEwWarps + 2) * 32;
constexpr int kBoxKV = BK * 128;       // [128 keys x 64 columns] bf16 box: 16 KiB
constexpr int kTileKV = 2 * kBoxKV;    // K or V tile
constexpr int kBoxQR = 2 * NR * 128;   // [Q rows; R rows] x 64 columns: the N = 2 NR operand of the score product
constexpr int kTileQR = 2 * kBoxQR;
constexpr int kTileP = BK * NR * 2;    // [128 keys x 64 rows] bf16, rows contiguous: one MN-major B operand
constexpr int kStages = 2;
constexpr int kOffQR = 0;
constexpr int kOffK = kOffQR + kTileQR;
constexpr int kOffV = kOffK + kStages * kTileKV;
constexpr int kOffP = kOffV + kStages * kTileKV;  // P1 bf16, P1 residual, P2 bf16, P2 residual
constexpr int kOffBar = kOffP + 4 * kTileP;
enum : int { kBarQR = 0, kBarKFull = 1, kBarKFree = 3, kBarVFull = 5, kBarVFree = 7, kBarSFull = 9, kBarSFree = 11,
             kBarPFull = 13, kBarPvDone = 14, kBarFinal = 15, kNumBars = 16 };
constexpr int kOffTmemSlot = kOffBar + kNumBars * 8;
constexpr int kOffRef = kOffTmemSlot + 16;       // float [NR]: reference exponent of each row (log2 units)
constexpr int kOffAlpha = kOffRef + NR * 4;      // float [NR]: rescale factor of the current tile
constexpr int kOffWmax = kOffAlpha + NR * 4;     // float [8 warps][32 rows]: per-warp tile maxima
constexpr int kRowsSmemBytes = kOffWmax + kEwWarps * 32 * 4;
static_assert(kRowsSmemBytes <= 232448, "shared-memory budget of one CTA");
constexpr uint32_t kColS = 0;                    // two score buffers of 2 NR fp32 columns: S1^T | S2^T
constexpr uint32_t kColO1 = 2 * 2 * NR, kColO2 = kColO1 + NR;
constexpr uint32_t kTmemColsRows = 512;
constexpr float kRowsLazyThreshold = 8.0f;       // log2 units
constexpr float kLn2 = 0.6931471805599453f;
constexpr int REC = 2 * HD + 4;

struct RowsParams {
    const int32_t* seqlens;
    void* out;
    float* partials;   // nullptr: one split, rows finished here
    int32_t* status;
    int B, Hq, Hkv, Lq, T_max;
    int rows;          // (Hq / Hkv) * Lq <= NR rows of a KV head, contiguous in [B, Hq, Lq, D]
    int num_splits, tiles_per_split;
    float scale_log2e;
    int out_dtype;
};

__device__ __forceinline__ void ew_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEwThreads) : "memory"); }
// barrier among the element-wise warps that also ORs a predicate over them
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

// 32 values per lane in, one out: lane l ends up with the reduction over the warp's 32 lanes of value l.
// Each round sends half of the remaining values to the partner lane and keeps the other half (31 shuffles).
template <bool kMax>
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[32], int lane)
{
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int i = 0; i < off; ++i) {
            const float keep = up ? v[i + off] : v[i];
            const float send = up ? v[i] : v[i + off];
            const float recv = __shfl_xor_sync(0xffffffffu, send, off);
            v[i] = kMax ? fmaxf(keep, recv) : keep + recv;
        }
    }
    return v[0];
}

__device__ __forceinline__ void store_value(void* out, size_t idx, float v, int out_dtype)
{
    if (out_dtype == PLX_OUT_F32)
        static_cast<float*>(out)[idx] = v;
    else
        static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(v);
}

// ---------------------------------------------------------------------------
// Kernel: CTA = (sequence, KV head, key split)
// ---------------------------------------------------------------------------
// Barrier discipline: every waiter consumes the phases of a barrier strictly in order, and no barrier can
// complete a second phase before its waiter has seen the first: S buffers alternate (full / free pairs per
// buffer), the P tiles are single (P full <-> P.V done hand over one tile at a time), the K and V rings have
// a full / free pair per stage.
__global__ void __launch_bounds__(kRowsThreads, 1)
plx_decode_rows_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmR,
                       const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                       const RowsParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    uint8_t* const smem = smem_raw;
    if ((base & 1023u) != 0) {  // the layout has no room for alignment slack
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, PLX_ERR_ALIGNMENT);
        return;
    }
    // lets the merge kernel of a split call (launched as a programmatic dependent) be scheduled now; it waits
    // for this grid's completion before it reads a record
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = static_cast<int>(blockIdx.x % p.num_splits);
    const int bh = static_cast<int>(blockIdx.x / p.num_splits);
    const int b = bh / p.Hkv, hkv = bh - b * p.Hkv;
    const int G = p.Hq / p.Hkv;
    int L = p.seqlens ? p.seqlens[b] : p.T_max;
    L = max(0, min(L, p.T_max));
    const size_t row0 = (static_cast<size_t>(b) * p.Hq + static_cast<size_t>(hkv) * G) * p.Lq;  // first row of this KV head
    const size_t kv_row0 = (static_cast<size_t>(b) * p.Hkv + hkv) * p.T_max;
    const int n_all = (L + BK - 1) / BK;
    const int jt0 = split * p.tiles_per_split;
    const int n_tiles = max(0, min(n_all, jt0 + p.tiles_per_split) - jt0);

    if (n_tiles == 0) {  // no key for this split: empty records (only m is ever read), or rows of zeros
        if (p.partials) {
            for (int i = threadIdx.x; i < p.rows; i += kRowsThreads)
                p.partials[((row0 + i) * p.num_splits + split) * REC] = -INFINITY;
        } else {
            for (int i = threadIdx.x; i < p.rows * HD; i += kRowsThreads) store_value(p.out, row0 * HD + i, 0.0f, p.out_dtype);
        }
        return;
    }

    auto bar = [&](int slot) { return base + kOffBar + 8 * slot; };
    float* const ref = reinterpret_cast<float*>(smem + kOffRef);
    float* const alpha = reinterpret_cast<float*>(smem + kOffAlpha);
    float* const wmax = reinterpret_cast<float*>(smem + kOffWmax);
    if (threadIdx.x == 0) {
        mbar_init(bar(kBarQR), 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1);
            mbar_init(bar(kBarKFree + s), 1);
            mbar_init(bar(kBarVFull + s), 1);
            mbar_init(bar(kBarVFree + s), 1);
            mbar_init(bar(kBarSFull + s), 1);
            mbar_init(bar(kBarSFree + s), kEwThreads);
        }
        mbar_init(bar(kBarPFull), kEwThreads);
        mbar_init(bar(kBarPvDone), 1);
        mbar_init(bar(kBarFinal), 1);
        fence_barrier_init();
    }
    if (threadIdx.x < NR) ref[threadIdx.x] = -INFINITY;
    if (warp == kMmaWarp) {
        tmem_alloc(base + kOffTmemSlot, kTmemColsRows);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + kOffTmemSlot);

    if (warp == kTmaWarp) {
        if (lane == 0) {
            prefetch_tensormap(&tmQ);
            prefetch_tensormap(&tmR);
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
            mbar_expect_tx(bar(kBarQR), kTileQR);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                tma_load_2d(base + kOffQR + h * kBoxQR, &tmQ, bar(kBarQR), 64 * h, static_cast<int>(row0));
                tma_load_2d(base + kOffQR + h * kBoxQR + NR * 128, &tmR, bar(kBarQR), 64 * h, static_cast<int>(row0));
            }
            for (int j = 0; j < n_tiles; ++j) {
                const int s = j & 1;
                const int krow = static_cast<int>(kv_row0) + (jt0 + j) * BK;
                if (j >= kStages) wait_or_flag(bar(kBarKFree + s), ((j >> 1) - 1) & 1, p.status);
                mbar_expect_tx(bar(kBarKFull + s), kTileKV);
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    tma_load_2d(base + kOffK + s * kTileKV + h * kBoxKV, &tmK, bar(kBarKFull + s), 64 * h, krow);
                if (j >= kStages) wait_or_flag(bar(kBarVFree + s), ((j >> 1) - 1) & 1, p.status);
                mbar_expect_tx(bar(kBarVFull + s), kTileKV);
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    tma_load_2d(base + kOffV + s * kTileKV + h * kBoxKV, &tmV, bar(kBarVFull + s), 64 * h, krow);
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ===================== score products and value products, one issuing thread =====================
        constexpr uint32_t idesc_s = make_idesc(BK, 2 * NR, 0, 0);   // K-major A (K tile), K-major B ([Q; R])
        constexpr uint32_t idesc_pv = make_idesc(HD, NR, 1, 1);      // MN-major A (V tile: head dimension on M), MN-major B (P^T)
        const uint64_t dQR = make_smem_desc(base + kOffQR, 0, 1024);
        wait_or_flag(bar(kBarQR), 0, p.status);
        auto score = [&](int j) {
            const int s = j & 1;
            wait_or_flag(bar(kBarKFull + s), (j >> 1) & 1, p.status);
            if (j >= 2) wait_or_flag(bar(kBarSFree + s), ((j >> 1) - 1) & 1, p.status);
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dK = make_smem_desc(base + kOffK + s * kTileKV, 0, 1024);
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint64_t aoff = static_cast<uint64_t>(((ks >> 2) * kBoxKV + (ks & 3) * 32) >> 4);
                    const uint64_t boff = static_cast<uint64_t>(((ks >> 2) * kBoxQR + (ks & 3) * 32) >> 4);
                    mma_ss(tmem + kColS + s * 2 * NR, dK + aoff, dQR + boff, idesc_s, ks > 0);
                }
                tc_commit(bar(kBarSFull + s));
                tc_commit(bar(kBarKFree + s));
            }
            __syncwarp();
        };
        score(0);
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1;
            if (j + 1 < n_tiles) score(j + 1);  // runs while the element-wise warps work on tile j
            wait_or_flag(bar(kBarPFull), j & 1, p.status);
            wait_or_flag(bar(kBarVFull + s), (j >> 1) & 1, p.status);
            if (lane == 0) {
                tc_fence_after();
                const uint64_t dV = make_smem_desc(base + kOffV + s * kTileKV, kBoxKV, 1024);
                const uint64_t dP = make_smem_desc(base + kOffP, 0, 1024);
                constexpr uint64_t kPStep = static_cast<uint64_t>(kTileP >> 4);
#pragma unroll
                for (int ks = 0; ks < BK / 16; ++ks) {
                    const uint64_t koff = static_cast<uint64_t>((ks * 2048) >> 4);
                    const uint32_t acc = (j > 0 || ks > 0) ? 1u : 0u;
                    mma_ss(tmem + kColO1, dV + koff, dP + koff, idesc_pv, acc);
                    mma_ss(tmem + kColO1, dV + koff, dP + kPStep + koff, idesc_pv, 1u);
                    mma_ss(tmem + kColO2, dV + koff, dP + 2 * kPStep + koff, idesc_pv, acc);
                    mma_ss(tmem + kColO2, dV + koff, dP + 3 * kPStep + koff, idesc_pv, 1u);
                }
                tc_commit(bar(kBarPvDone));
                tc_commit(bar(kBarVFree + s));
                if (j == n_tiles - 1) tc_commit(bar(kBarFinal));
            }
            __syncwarp();
        }
    } else {
        // ===================== element-wise warps =====================
        // thread = (key of the tile = TMEM lane, half of the rows)
        const int quarter = warp & 3, part = warp >> 2;
        const int kr = quarter * 32 + lane;
        const int c0 = kRowsPerThread * part;  // first row of this thread's columns
        const uint32_t lane_base = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
        const int swz = kr & 7;
        float d1[kRowsPerThread], d2[kRowsPerThread];
#pragma unroll
        for (int c = 0; c < kRowsPerThread; ++c) d1[c] = d2[c] = 0.0f;
        // bit c: row c0 + c exists (fewer than NR rows: the padding rows take part with weights of zero)
        const uint32_t row_mask = p.rows - c0 >= 32 ? 0xffffffffu : (p.rows > c0 ? (1u << (p.rows - c0)) - 1u : 0u);

        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1;
            const int key = (jt0 + j) * BK + kr;
            // some (key, row) pair of this tile may be invisible: the last Lq - 1 keys, the end of the context
            const bool need_mask = (jt0 + j) * BK + BK > L - (p.Lq - 1);
            const uint32_t Sb = lane_base + kColS + s * 2 * NR;
            // bit c of vis: row c0 + c sees this thread's key (token i of a head sees the first L - (Lq - 1 - i) keys)
            uint32_t vis = row_mask;
            if (need_mask) {
                vis = 0u;
                int tok = c0 % p.Lq;
#pragma unroll
                for (int c = 0; c < kRowsPerThread; ++c) {
                    if (key < L - (p.Lq - 1 - tok)) vis |= 1u << c;
                    if (++tok == p.Lq) tok = 0;
                }
                vis &= row_mask;
            }
            wait_or_flag(bar(kBarSFull + s), (j >> 1) & 1, p.status);
            tc_fence_after();

            // ---- pass 1: the tile's maximum of every row, over the 128 keys ----
            {
                uint32_t a[32];
                tmem_ld32(Sb + c0, a);
                tmem_wait_ld();
                float v[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) v[c] = ((vis >> c) & 1u) ? __uint_as_float(a[c]) * p.scale_log2e : -INFINITY;
                const float m = warp_transpose_reduce<true>(v, lane);
                wmax[warp * 32 + lane] = m;
            }
            ew_barrier();
            bool changed = false;
            if (threadIdx.x < NR) {
                const int row = threadIdx.x, pr = row >> 5, c = row & 31;
                const float tm = fmaxf(fmaxf(wmax[(4 * pr + 0) * 32 + c], wmax[(4 * pr + 1) * 32 + c]),
                                       fmaxf(wmax[(4 * pr + 2) * 32 + c], wmax[(4 * pr + 3) * 32 + c]));
                const float old = ref[row];
                float al = 1.0f;
                if (tm > old + kRowsLazyThreshold) {  // also the first visible key of a row (old = -inf)
                    changed = true;
                    al = (old > -INFINITY) ? ex2(old - tm) : 0.0f;
                    ref[row] = tm;
                }
                alpha[row] = al;
            }
            const bool any_changed = ew_barrier_or(changed);

            if (any_changed && j > 0) {
                // rare: move the reference of the accumulated state (this thread's TMEM lane is a head dimension here)
                wait_or_flag(bar(kBarPvDone), (j - 1) & 1, p.status);
                tc_fence_after();
#pragma unroll 1
                for (int which = 0; which < 2; ++which) {
                    uint32_t o[32];
                    const uint32_t col = lane_base + (which ? kColO2 : kColO1) + c0;
                    tmem_ld32(col, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha[c0 + c]);
                    tmem_st32(col, o);
                }
                tmem_wait_st();
                tc_fence_before();
#pragma unroll
                for (int c = 0; c < kRowsPerThread; ++c) {
                    const float al = alpha[c0 + c];
                    d1[c] *= al;
                    d2[c] *= al;
                }
            }

            // ---- pass 2: weights, row sums, bf16 parts and residuals ----
            uint32_t h1[16], l1[16], h2[16], l2[16];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t a[16], g[16];
                tmem_ld16(Sb + c0 + 16 * h, a);
                tmem_ld16(Sb + NR + c0 + 16 * h, g);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; c += 2) {
                    float p1[2], p2[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int cc = 16 * h + c + e;
                        const float rf = ref[c0 + cc];
                        const float x = fmaf(__uint_as_float(a[c + e]), p.scale_log2e, -((rf > -INFINITY) ? rf : 0.0f));
                        const bool ok = (vis >> cc) & 1u;
                        p1[e] = ok ? ex2(x) : 0.0f;
                        p2[e] = ok ? p1[e] * __uint_as_float(g[c + e]) : 0.0f;
                        d1[cc] += p1[e];
                        d2[cc] += p2[e];
                    }
                    const int o = (16 * h + c) >> 1;
                    const __nv_bfloat162 b1 = __floats2bfloat162_rn(p1[0], p1[1]), b2 = __floats2bfloat162_rn(p2[0], p2[1]);
                    h1[o] = *reinterpret_cast<const uint32_t*>(&b1);
                    h2[o] = *reinterpret_cast<const uint32_t*>(&b2);
                    l1[o] = pack2(p1[0] - __low2float(b1), p1[1] - __high2float(b1));
                    l2[o] = pack2(p2[0] - __low2float(b2), p2[1] - __high2float(b2));
                }
            }
            tc_fence_before();
            mbar_arrive(bar(kBarSFree + s));  // the score buffer is in registers

            if (j > 0) wait_or_flag(bar(kBarPvDone), (j - 1) & 1, p.status);  // the previous P tiles have been consumed
            // P^T tiles: [128 keys][64 rows] bf16, 128 bytes per key, 128-byte swizzle (chunk index XOR key mod 8)
            uint8_t* const prow = smem + kOffP + kr * 128;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const int chunk = ((4 * part + q4) ^ swz) * 16;
                *reinterpret_cast<uint4*>(prow + chunk) = make_uint4(h1[4 * q4], h1[4 * q4 + 1], h1[4 * q4 + 2], h1[4 * q4 + 3]);
                *reinterpret_cast<uint4*>(prow + kTileP + chunk) = make_uint4(l1[4 * q4], l1[4 * q4 + 1], l1[4 * q4 + 2], l1[4 * q4 + 3]);
                *reinterpret_cast<uint4*>(prow + 2 * kTileP + chunk) = make_uint4(h2[4 * q4], h2[4 * q4 + 1], h2[4 * q4 + 2], h2[4 * q4 + 3]);
                *reinterpret_cast<uint4*>(prow + 3 * kTileP + chunk) = make_uint4(l2[4 * q4], l2[4 * q4 + 1], l2[4 * q4 + 2], l2[4 * q4 + 3]);
            }
            if ((jt0 + j) * BK + BK > L && part == 0) {
                // the context ends inside this tile: rows of V past it may hold anything (NaN included); their
                // weights are exact zeros, so clear them once the tile has landed
                wait_or_flag(bar(kBarVFull + s), (j >> 1) & 1, p.status);
                if (key >= L) {
                    uint8_t* const vrow = smem + kOffV + s * kTileKV + kr * 128;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        *reinterpret_cast<uint4*>(vrow + i * 16) = make_uint4(0u, 0u, 0u, 0u);
                        *reinterpret_cast<uint4*>(vrow + kBoxKV + i * 16) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(bar(kBarPFull));
        }

        // ---- row sums over the keys, then the epilogue: this thread's TMEM lane is head dimension kr ----
        wait_or_flag(bar(kBarFinal), 0, p.status);
        tc_fence_after();
        float* const dsum = reinterpret_cast<float*>(smem + kOffP);  // the P tiles are idle now: [8 warps][32 rows][2], then [NR][2]
        {
            const float t1 = warp_transpose_reduce<false>(d1, lane);
            const float t2 = warp_transpose_reduce<false>(d2, lane);
            dsum[(warp * 32 + lane) * 2] = t1;
            dsum[(warp * 32 + lane) * 2 + 1] = t2;
        }
        ew_barrier();
        float* const dtot = dsum + kEwWarps * 32 * 2;
        if (threadIdx.x < NR) {
            const int row = threadIdx.x, pr = row >> 5, c = row & 31;
            float t1 = 0.0f, t2 = 0.0f;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                t1 += dsum[((4 * pr + w) * 32 + c) * 2];
                t2 += dsum[((4 * pr + w) * 32 + c) * 2 + 1];
            }
            dtot[2 * row] = t1;
            dtot[2 * row + 1] = t2;
        }
        ew_barrier();
        {
            uint32_t u[32], w[32];
            tmem_ld32(lane_base + kColO1 + c0, u);
            tmem_ld32(lane_base + kColO2 + c0, w);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < kRowsPerThread; ++c) {
                const int row = c0 + c;
                if (!((row_mask >> c) & 1u)) continue;
                const float O1 = __uint_as_float(u[c]), O2 = __uint_as_float(w[c]);
                const float D1 = dtot[2 * row], D2 = dtot[2 * row + 1];
                if (p.partials) {
                    float* rec = p.partials + ((row0 + row) * p.num_splits + split) * REC;
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
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemColsRows);
    }
}

}  // namespace

// ---------------------------------------------------------------------------
// Host side (internal to the library; reached through parallax_decode_fwd_multi)
// ---------------------------------------------------------------------------
// q, r, out [B, Hq, Lq, D] with (Hq / Hkv) * Lq <= 64 rows per KV head, D = 128, bf16 caches [B, Hkv, T_max, D].
// `records` / `record_bytes`: room for split records (may be null: one split).  num_splits 0 = planned.
bool plx_decode_rows_supported(int Hq, int Hkv, int D, int Lq)
{
    return D == HD && Hkv > 0 && Hq % Hkv == 0 && static_cast<long long>(Hq / Hkv) * Lq <= NR;
}

int plx_decode_rows_fwd(const void* q, const void* r, const void* k_cache, const void* v_cache, const int32_t* seqlens,
                        void* out, int B, int Hq, int Hkv, int D, int Lq, int T_max, float scale, int out_dtype,
                        void* records, size_t record_bytes, int num_splits, int32_t* status, cudaStream_t stream)
{
    if (!q || !r || !k_cache || !v_cache || !out) return PLX_ERR_NULL_POINTER;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Lq <= 0 || T_max <= 0 || Hq % Hkv != 0) return PLX_ERR_BAD_SHAPE;
    if (!plx_decode_rows_supported(Hq, Hkv, D, Lq)) return PLX_ERR_UNSUPPORTED;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (num_splits < 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    const long long q_rows = static_cast<long long>(B) * Hq * Lq, kv_rows = static_cast<long long>(B) * Hkv * T_max;
    if (q_rows >= (1LL << 31) - 65536 || kv_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    if (!plx_aligned(q, 16) || !plx_aligned(r, 16) || !plx_aligned(k_cache, 16) || !plx_aligned(v_cache, 16) ||
        !plx_aligned(out, 16) || (records && !plx_aligned(records, 16)))
        return PLX_ERR_ALIGNMENT;

    CUtensorMap tmQ, tmR, tmK, tmV;
    int rc;
    const CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
    if ((rc = make_tensor_map_2d(&tmQ, q, D, static_cast<uint64_t>(q_rows), NR, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmR, r, D, static_cast<uint64_t>(q_rows), NR, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmK, k_cache, D, static_cast<uint64_t>(kv_rows), BK, promo)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmV, v_cache, D, static_cast<uint64_t>(kv_rows), BK, promo)) != PLX_OK) return rc;

    static bool configured[64] = {false};
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return PLX_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        if (cudaFuncSetAttribute(plx_decode_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRowsSmemBytes) !=
            cudaSuccess)
            return PLX_ERR_CUDA;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    // Split plan: one CTA per SM at most (a second generation of a few CTAs would double the time), at least four
    // 128-key tiles per split, what the record space holds.
    const long long base_ctas = static_cast<long long>(B) * Hkv;
    const int tiles_max = (T_max + BK - 1) / BK;
    int ns = 1;
    if (records) {
        if (num_splits == 0) {
            if (base_ctas < sms) {
                const long long want = sms / base_ctas;
                const long long most = tiles_max / 4 > 1 ? tiles_max / 4 : 1;
                ns = static_cast<int>(want < most ? want : most);
                if (ns > 64) ns = 64;
            }
        } else {
            ns = num_splits < tiles_max ? num_splits : tiles_max;
        }
        while (ns > 1 && static_cast<size_t>(q_rows) * ns * REC * sizeof(float) > record_bytes) --ns;
    } else if (num_splits > 1) {
        return PLX_ERR_WORKSPACE;
    }
    const int tps = (tiles_max + ns - 1) / ns;
    ns = (tiles_max + tps - 1) / tps;  // no split without a tile
    if (base_ctas * ns > 0x7fffffffLL) return PLX_ERR_BAD_SHAPE;
    RowsParams rp{seqlens, out, ns > 1 ? static_cast<float*>(records) : nullptr, status, B, Hq, Hkv, Lq, T_max,
                  (Hq / Hkv) * Lq, ns, tps, scale * 1.4426950408889634f, out_dtype};
    PlxNvtxRange nvtx_range("plx_decode_rows_fwd");
    plx_decode_rows_kernel<<<static_cast<unsigned>(base_ctas * ns), kRowsThreads, kRowsSmemBytes, stream>>>(tmQ, tmR, tmK,
                                                                                                          tmV, rp);
    if (cudaGetLastError() != cudaSuccess) return PLX_ERR_CUDA;
    if (ns > 1)
        return plx_combine_after_producer(static_cast<const float*>(records), out, static_cast<int>(q_rows), D, ns,
                                          out_dtype, stream);
    return PLX_OK;
}

extern "C" int parallax_decode_fwd_rows(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                        const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                                        int T_max, float scale, int out_dtype, void* workspace, size_t workspace_bytes,
                                        int num_splits, int32_t* status, void* stream)
{
    return plx_decode_rows_fwd(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, Lq, T_max, scale, out_dtype, workspace,
                               workspace_bytes, num_splits, status, static_cast<cudaStream_t>(stream));
}
