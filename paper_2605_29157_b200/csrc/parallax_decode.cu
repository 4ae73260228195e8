// Parallax decode forward for B200 (sm_100a): kernels and the C-ABI host layer.
//
// One CTA handles one (sequence, KV head, key chunk).  Its four warps take the
// chunk's 16-key tiles round-robin; every warp owns a private multi-stage ring of
// (K tile, V tile) buffers in shared memory that it fills with TMA tensor loads
// (128-byte swizzle) and drains itself, so the hot loop has no CTA-wide barrier.
//
// Per tile (Algorithm 1, one query row per head, both branches on one K/V tile):
//   S^T[16 keys x 8] = K_c . [q_a q_b r_a r_b 0 0 0 0]    mma.sync m16n8k16, keys on M
//   online max from the softmax rows only, exp2, P2 = P1 * S2
//   O^T[D x 8]      += V_c^T . [P1 P2 | bf16 residuals of P1 P2]
// The eight MMA columns of the second product carry P1 and P2 of the two query
// heads of a GQA pair twice: rounded to bf16 and the rounding residual, so the
// accumulated O1, O2 keep ~16 mantissa bits of P at no extra tensor work.
// The running maximum is refreshed lazily (only when a tile exceeds it by more
// than 2^8), which leaves the result unchanged because every sum is relative to
// the same reference exponent.
//
// A chunk's result is either the final row (one split) or an unnormalised partial
// state that the combine kernel merges (App. "Kernel Optimization Details").
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <math.h>
#include <stdint.h>

#include <mutex>

#include <cstddef>
#include <cstring>

#include "parallax.h"
#include "plx_common.cuh"
#include "plx_internal.h"

namespace {

// Compile-time tuning knobs (defaults are the measured best on B200).
#ifndef PLX_WARPS
#define PLX_WARPS 4
#endif
#ifndef PLX_CTAS_PER_SM
#define PLX_CTAS_PER_SM 2
#endif
#ifndef PLX_STAGES_D128
#define PLX_STAGES_D128 3
#endif
#ifndef PLX_STAGES_D64
#define PLX_STAGES_D64 3
#endif
#ifndef PLX_CTAS_PER_SM_D64
#define PLX_CTAS_PER_SM_D64 4
#endif
#ifndef PLX_CTAS_PER_SM_FP8
#define PLX_CTAS_PER_SM_FP8 4
#endif
#ifndef PLX_STAGES_FP8
#define PLX_STAGES_FP8 3
#endif
#ifndef PLX_TWO_STAGE_MAX_CHUNK
#define PLX_TWO_STAGE_MAX_CHUNK 128  // D = 128: chunks up to this many keys use the two-stage ring (three CTAs per SM)
#endif
#ifndef PLX_SMEM_PAD
#define PLX_SMEM_PAD 0  // experiment knob: extra dynamic shared memory per CTA (limits residency)
#endif
#ifndef PLX_L2_PROMOTION
#define PLX_L2_PROMOTION CU_TENSOR_MAP_L2_PROMOTION_L2_256B
#endif
#ifndef PLX_PDL_CHAIN
#define PLX_PDL_CHAIN 1  // launch every decode kernel as a programmatic dependent of its predecessor in the stream
#endif

constexpr int kTileKeys = 16;          // keys per warp tile (the MMA M extent)
constexpr int kWarps = PLX_WARPS;      // warps per CTA
constexpr int kThreads = kWarps * 32;
constexpr int kCtasPerSm = PLX_CTAS_PER_SM;  // resident CTAs the shared-memory budget is sized for
constexpr int kCtasPerSmFp8 = PLX_CTAS_PER_SM_FP8;  // e4m3 cache variant
constexpr int kChunkGranule = kTileKeys * kWarps;  // 64 keys
constexpr float kRescaleThreshold = 8.0f;          // log2 units
constexpr int kHeaderBytes = 256;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kLog2e = 1.4426950408889634f;

// kModeFused: write partial records, then the last CTA of a (sequence, KV head) to finish merges them.
enum Mode : int { kModeFinal = 0, kModePartial = 1, kModePartialWriteEmpty = 2, kModeFused = 3 };

struct KernelParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* r;
    const int32_t* seqlens;
    void* out;
    float* partials;
    int32_t* status;
    int32_t* counters;  // fused mode: one arrival counter per (sequence, KV head), zero between calls
    const int32_t* block_table;  // paged cache: int32 [B, max_pages] page ids, else nullptr (contiguous cache)
    int page_size, max_pages;
    int B, Hq, Hkv, T_max, chunk_len, num_splits;
    float scale_log2e;
    int out_dtype;
    int mode;
    // fp8 (e4m3) cache: the stored keys are k / k_scale and the stored values v / v_scale
    float probe_scale = 1.0f;  // k_scale: multiplies the probe score (the softmax score takes it through scale_log2e)
    float v_scale = 1.0f;      // multiplies both value accumulators
    // per-KV-head scales (device arrays [real KV heads]) instead of the two scalars; scale_log2e then holds
    // the softmax scale alone
    const float* k_scales = nullptr;
    const float* v_scales = nullptr;
    // Group sizes above 4: Hkv counts VIRTUAL KV heads, kv_div of them share one real KV head (each serves
    // at most four query heads; the second reader of a cache row is mostly served by L2, but the bytes
    // delivered to the SMs double: measured 4.4 TB/s of unique KV bytes at G = 8 against 7.1 at G <= 4).
    int kv_div = 1;
    // Several new tokens per sequence (parallax_decode_fwd_multi): query rows are [B, Hq / lq, lq, D], i.e. row
    // v of a sequence is token v % lq of a query head, and token i sees the first L - (lq - 1 - i) keys.
    int lq = 1;
    // host only: launch as a programmatic dependent of the previous kernel in the stream (the kernel's
    // first instruction waits for that kernel's results; see parallax_decode_step)
    int dependent_launch = 0;
    // let the next kernel of the stream start early from this kernel's first instruction on (grids that fill
    // every CTA slot of the device) instead of from its last
    int signal_early = 0;
    // q and r live in page-locked host memory (host-buffer entry): every CTA fetches its group's rows once with
    // 16-byte loads into shared memory (coalesced requests over the host link) instead of building its fragments
    // from 4-byte global loads
    int qr_staged = 0;
    // What the host knows about the buffers, for the index checks of the debug build (PLX_DEBUG_CHECKS):
    // rows each K/V tensor map covers, and the number of records `partials` has room for.
    long long kv_rows = 0;
    long long partial_records = 0;
};

#ifndef PLX_DEBUG_CHECKS
#define PLX_DEBUG_CHECKS 0
#endif

// Timeline instrumentation for experiments (-DPLX_TRACE=1; never part of the shipped build): per CTA
// the %globaltimer at start, first data, end of the tile loop and exit, plus the SM id.
#ifndef PLX_TRACE
#define PLX_TRACE 0
#endif
#if PLX_TRACE
__device__ unsigned long long g_plx_trace[8192 * 5];
__device__ __forceinline__ unsigned long long plx_now()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define PLX_PHASE_DECL long long ph_t = clock64(), ph_acc[4] = {0, 0, 0, 0}
#define PLX_PHASE(i)                     \
    do {                                 \
        const long long now = clock64(); \
        ph_acc[i] += now - ph_t;         \
        ph_t = now;                      \
    } while (0)
#define PLX_PHASE_STORE                                                                                   \
    do {                                                                                                  \
        if (threadIdx.x == 0 && blockIdx.x < 8)                                                           \
            for (int i = 0; i < 4; ++i) g_plx_trace[8192 * 5 - 64 + blockIdx.x * 4 + i] = ph_acc[i];      \
    } while (0)
#define PLX_STAMP(slot)                                                                  \
    do {                                                                                 \
        if (threadIdx.x == 0 && blockIdx.x < 8192) g_plx_trace[blockIdx.x * 5 + (slot)] = plx_now(); \
    } while (0)
#else
#define PLX_STAMP(slot) \
    do {                \
    } while (0)
#define PLX_PHASE_DECL
#define PLX_PHASE(i) \
    do {             \
    } while (0)
#define PLX_PHASE_STORE \
    do {                \
    } while (0)
#endif

// ---------------------------------------------------------------------------
// Warp-level MMA helpers (the mbarrier / TMA wrappers live in plx_common.cuh)
// ---------------------------------------------------------------------------
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&a)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                 : "r"(addr)
                 : "memory");
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&a)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                 : "r"(addr)
                 : "memory");
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

// D[16x8] += A[16x16] (row) * B[16x8] (col), bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Same with fp16 inputs (the fp8-cache variant: e4m3 converts exactly to fp16).
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// two e4m3 values (low 16 bits of x, or high 16 bits) -> fp16x2, exact
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t x, bool high)
{
    uint32_t y;
    const uint16_t h = static_cast<uint16_t>(high ? (x >> 16) : (x & 0xffffu));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(y) : "h"(h));
    return y;
}

__device__ __forceinline__ uint32_t f16x2_from_bf16x2(uint32_t x)
{
    const __half2 h = __floats2half2_rn(__uint_as_float(x << 16), __uint_as_float(x & 0xffff0000u));
    return *reinterpret_cast<const uint32_t*>(&h);
}

// Packs (lo, hi) to fp16x2; with `residual` packs the rounding residuals instead.
__device__ __forceinline__ uint32_t pack_f16_pair(float lo, float hi, bool residual)
{
    __half2 h = __floats2half2_rn(lo, hi);
    if (residual) h = __floats2half2_rn(lo - __low2float(h), hi - __high2float(h));
    return *reinterpret_cast<uint32_t*>(&h);
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Packs (lo, hi) to bf16x2; with `residual` packs the rounding residuals instead.
__device__ __forceinline__ uint32_t pack_bf16_pair(float lo, float hi, bool residual)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    if (residual) h = __floats2bfloat162_rn(lo - __low2float(h), hi - __high2float(h));
    return *reinterpret_cast<uint32_t*>(&h);
}

__device__ __forceinline__ void store_out(void* out, size_t idx, float v, int out_dtype)
{
    if (out_dtype == PLX_OUT_F32)
        static_cast<float*>(out)[idx] = v;
    else
        static_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16_rn(v);
}

// Algorithm 1's final line.
__device__ __forceinline__ float finalize(float O1, float O2, float d1, float d2)
{
    const float inv = 1.0f / d1;
    return O1 * inv * (1.0f + d2 * inv) - O2 * inv;
}

// ---------------------------------------------------------------------------
// Split merge of one (b, hq) row by a CTA of NW warps (App. "Kernel Optimization Details",
// item 3): M = max m_s, weights exp(m_s - M), weighted sums in fixed split order, final line.
// Used by the combine kernel and by the last-arriving CTA of the fused path.  `scratch` is
// 16-byte aligned shared memory of MergeScratch<D, NW>::kFloats floats; every thread of the CTA
// must call this (it synchronises the CTA).
// ---------------------------------------------------------------------------
template <int D, int NW>
struct MergeScratch {
    static constexpr int kAccStride = 2 * D + 4;
    static constexpr int kFloats = PLX_MAX_SPLITS + NW * kAccStride + 4 * NW;
};

template <int D, int NW>
__device__ __forceinline__ void merge_row(const float* __restrict__ base, int count, float* scratch, void* out,
                                          size_t out_off, int out_dtype, int per_group = 0x7fffffff,
                                          size_t group_stride = 0)
{
    // record i lives at base + (i / per_group) * group_stride + (i % per_group) * REC: one group for a
    // single device's splits, one group per rank for partial states gathered from several devices
    constexpr int REC = 2 * D + 4;
    constexpr int VEC = 2 * D / 4;        // float4 slots of O1|O2 in one record
    constexpr int VPL = (VEC + 31) / 32;  // slots per lane
    constexpr int STRIDE = MergeScratch<D, NW>::kAccStride;
    float* s_w = scratch;                         // [PLX_MAX_SPLITS] weights
    float* s_acc = scratch + PLX_MAX_SPLITS;      // [NW][2D+4] per-warp vector sums
    float* s_red = s_acc + NW * STRIDE;           // [4*NW] scalars
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    auto rec_at = [&](int i) {
        const int grp = i / per_group;
        return base + grp * group_stride + static_cast<size_t>(i - grp * per_group) * REC;
    };

    // reference exponent: the largest m among the records in use
    float M = -INFINITY;
    for (int i = tid; i < count; i += NW * 32) M = fmaxf(M, __ldcg(rec_at(i)));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    if (lane == 0) s_red[warp] = M;
    __syncthreads();
    M = s_red[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) M = fmaxf(M, s_red[w]);
    __syncthreads();

    if (!(M > -INFINITY)) {  // no keys at all: a row of zeros
        for (int d = tid; d < D; d += NW * 32) store_out(out, out_off + d, 0.0f, out_dtype);
        return;
    }

    // weights, and the two scalar sums
    float D1 = 0.0f, D2 = 0.0f;
    for (int i = tid; i < count; i += NW * 32) {
        const float* rec = rec_at(i);
        const float m = __ldcg(rec);
        const float a = (m > -INFINITY) ? __expf(m - M) : 0.0f;
        s_w[i] = a;
        if (a != 0.0f) {
            D1 += a * __ldcg(rec + 1);
            D2 += a * __ldcg(rec + 2);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        D1 += __shfl_xor_sync(0xffffffffu, D1, off);
        D2 += __shfl_xor_sync(0xffffffffu, D2, off);
    }
    if (lane == 0) {
        s_red[warp] = D1;
        s_red[NW + warp] = D2;
    }
    __syncthreads();

    // vector part: warp w accumulates records w, w+NW, ... in that order; loads are independent
    float4 acc[VPL];
#pragma unroll
    for (int j = 0; j < VPL; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int i = warp; i < count; i += NW) {
        const float a = s_w[i];
        if (a == 0.0f) continue;  // empty record: its payload is not read
        const float* rec = rec_at(i);
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int slot = lane + 32 * j;
            if (slot < VEC) {
                const float4 x = __ldcg(reinterpret_cast<const float4*>(rec + 4 + slot * 4));
                acc[j].x += a * x.x;
                acc[j].y += a * x.y;
                acc[j].z += a * x.z;
                acc[j].w += a * x.w;
            }
        }
    }
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        const int slot = lane + 32 * j;
        if (slot < VEC) *reinterpret_cast<float4*>(s_acc + warp * STRIDE + slot * 4) = acc[j];
    }
    __syncthreads();

    for (int d = tid; d < D; d += NW * 32) {
        float O1 = 0.0f, O2 = 0.0f, T1 = 0.0f, T2 = 0.0f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            O1 += s_acc[w * STRIDE + d];
            O2 += s_acc[w * STRIDE + D + d];
            T1 += s_red[w];
            T2 += s_red[NW + w];
        }
        store_out(out, out_off + d, finalize(O1, O2, T1, T2), out_dtype);
    }
    __syncthreads();  // scratch is free for the caller's next row
}

// ---------------------------------------------------------------------------
// Main kernel
// ---------------------------------------------------------------------------
template <int D, int NSTAGES, bool FP8 = false>
struct SmemLayout {
    static constexpr int kRowBytes = FP8 ? D : 2 * D;         // bytes of one cache row
    static constexpr int kBoxBytes = kRowBytes < 128 ? kRowBytes : 128;  // bytes of a row inside one TMA box
    static constexpr int kHalves = kRowBytes / kBoxBytes;     // column blocks (TMA boxes) per row
    static constexpr int kHalfBytes = kTileKeys * kBoxBytes;  // one swizzled [16 keys x 128 (64) bytes] box
    static constexpr int kTensorBytes = kHalves * kHalfBytes; // K (or V) tile
    static constexpr int kStageBytes = 2 * kTensorBytes;      // K tile then V tile
    static constexpr int kRingBytes = kWarps * NSTAGES * kStageBytes;
    static constexpr int kBarrierBytes = ((kWarps * NSTAGES + 1) * 8 + 15) / 16 * 16;  // + one for the split-merge staging
    static constexpr int kQrBytes = 2 * 8 * D * 2;  // q and r rows of up to eight heads (host-resident q, r are staged here)
    static constexpr int kTotalBytes = 1024 + kRingBytes + kBarrierBytes + kQrBytes + PLX_SMEM_PAD;  // 1024: alignment slack
};

// FP8: the caches hold e4m3 bytes ([rows, D] bytes, D = 128); tiles are converted exactly to fp16 in
// registers and both products run as fp16 MMAs.  The ldmatrix fragments then hold four consecutive
// head dimensions (score product) or two (value product) where a 16-bit cache gives two / one: the
// score product absorbs that by loading the q / r fragments in the same permuted order, the value
// product by a permutation of its output rows that the epilogue undoes.
template <int D, int G, int NSTAGES, int CTAS, bool FP8 = false>
__global__ void __launch_bounds__(kThreads, CTAS)
plx_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const KernelParams p)
{
    static_assert(SmemLayout<D, NSTAGES, FP8>::kBoxBytes == 128 || (FP8 && D == 64), "64-byte rows: the e4m3 cache at D = 64");
    using SL = SmemLayout<D, NSTAGES, FP8>;
    // Byte offset of 16-byte chunk `chunk` of row `row` inside a K or V tile.  128-byte boxes use the 128-byte
    // swizzle (chunk index XOR row mod 8); the 64-byte rows of an e4m3 cache at D = 64 use the 64-byte swizzle
    // (chunk index XOR (row / 2) mod 4).  Eight consecutive rows of one chunk fall into eight different
    // 16-byte bank groups either way.
    auto tile_off = [](int row, int chunk) -> uint32_t {
        if constexpr (SL::kBoxBytes == 128)
            return static_cast<uint32_t>((chunk >> 3) * SL::kHalfBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
        else
            return static_cast<uint32_t>(row * 64 + ((chunk ^ ((row >> 1) & 3)) << 4));
    };
    // lazy-rescale threshold in log2 units: the weights reach the value product as fp16 in the FP8
    // variant, so they are kept below 2^4 (P2 = P1 * S2 must stay inside the fp16 range)
    constexpr float kThreshold = FP8 ? 4.0f : kRescaleThreshold;
    constexpr int NP = (G + 1) / 2;   // GQA head pairs per KV head
    // Up to two heads: the eight columns of a value MMA hold the pair's weights and their rounding residuals
    // side by side, and the two halves are folded at the end.  More heads: a "quad" of four heads fills the
    // eight columns ([P1a P1b P2a P2b | P1c P1d P2c P2d]) and the residuals go through a second MMA into the
    // SAME accumulator, so four heads cost 32 accumulator registers per lane and eight heads 64.
    constexpr bool SA = G > 2;
    constexpr int NQ = SA ? (NP + 1) / 2 : 1;  // accumulator sets
    constexpr int KSTEPS = D / 16;    // k-steps of the score product
    constexpr int MTILES = D / 16;    // m-tiles of the value product
    constexpr int REC = 2 * D + 4;    // floats per partial record
    static_assert(kWarps * NP * 2 * REC * 4 <= SL::kRingBytes, "merge scratch must fit in the ring");
    __shared__ int s_is_last;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t base_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t* const smem = smem_raw + (base_addr - raw_addr);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t ring = base_addr + warp * NSTAGES * SL::kStageBytes;
    const uint32_t bars = base_addr + SL::kRingBytes + warp * NSTAGES * 8;

    // The part of the prologue that touches no global memory: barriers and the descriptor prefetch
    // (the tensor maps are kernel parameters).
    if (lane == 0) {
        if (warp == 0) {
            prefetch_tensormap(&tmK);
            prefetch_tensormap(&tmV);
        }
#pragma unroll
        for (int s = 0; s < NSTAGES; ++s) mbar_init(bars + 8 * s, 1);
        if (warp == 0) mbar_init(base_addr + SL::kRingBytes + kWarps * NSTAGES * 8, 1);
        fence_barrier_init();
    }
    __syncwarp();

    // The kernel is launched as a programmatic dependent of whatever precedes it in the stream.  If that
    // is a kernel that lets its dependents start early (the upstream step of parallax_decode_step, the
    // staging kernel of the host entry, the previous decode call) this CTA may be resident while it
    // still runs: nothing it produces (q, r, an appended cache row, the workspace) is touched before
    // it has completed and its writes are visible.  After any other kernel the wait returns at once.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // In turn, let the next kernel of the stream be scheduled before this grid has drained (it waits the
    // same way before it touches memory), so that back-to-back decode calls overlap the next call's launch
    // and prologue with this call's tail.  A grid that fills every CTA slot of the device signals at once:
    // the next grid's CTAs then move in as slots free up.  A smaller grid signals at its very end instead
    // (see the last line of the kernel): CTAs that arrive while it still runs would take the free slots
    // beside it and could leave the next call two to an SM on part of the device with the rest idle.
    if (p.signal_early) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    PLX_STAMP(0);
#if PLX_TRACE
    if (threadIdx.x == 0 && blockIdx.x < 8192) {
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        g_plx_trace[blockIdx.x * 5 + 4] = smid;
    }
#endif

    // stream-major order: the splits of one (sequence, KV head) are neighbours in the grid, so its
    // merge happens while other streams are still being read
    const int stream_id = blockIdx.x / p.num_splits;
    const int split = blockIdx.x - stream_id * p.num_splits;
    const int b = stream_id / p.Hkv;
    const int hkv = stream_id - b * p.Hkv;

    int L = p.seqlens ? p.seqlens[b] : p.T_max;
    L = max(0, min(L, p.T_max));
    const int k0 = split * p.chunk_len;

    if (k0 >= L) {
        // Nothing to read.  An empty context still owes a row of zeros (single split), and the
        // stand-alone partial entry point promises an empty record.
        if (p.mode == kModeFinal || (p.mode == kModeFused && L == 0)) {
            if (split == 0)
                for (int i = threadIdx.x; i < G * D; i += kThreads)
                    store_out(p.out, (static_cast<size_t>(b) * p.Hq + hkv * G) * D + i, 0.0f,
                                    p.out_dtype);
        } else if (p.mode == kModePartialWriteEmpty) {
            for (int hl = 0; hl < G; ++hl) {
                float* rec = p.partials +
                             ((static_cast<size_t>(b) * p.Hq + hkv * G + hl) * p.num_splits + split) * REC;
                for (int i = threadIdx.x; i < REC; i += kThreads) rec[i] = (i == 0) ? -INFINITY : 0.0f;
            }
        }
        return;
    }
    const int k1 = min(k0 + p.chunk_len, L);
    const int ntiles = (k1 - k0 + kTileKeys - 1) / kTileKeys;
#if PLX_DEBUG_CHECKS
    {
        // Debug build: every index this CTA will form is affine in values known here, so the extremes are
        // checked once, CTA-uniformly; a violation is reported through the status word and the CTA leaves
        // without touching the address (page ids, which are data, are checked where they are read).
        const int hkv_r = hkv / p.kv_div, Hkv_r = p.Hkv / p.kv_div;
        bool ok = stream_id < p.B * p.Hkv && p.Hq == p.Hkv * G && p.Hkv % p.kv_div == 0 && p.lq >= 1 &&
                  p.chunk_len % kTileKeys == 0 && static_cast<long long>(p.chunk_len) * p.num_splits >= p.T_max;
        if (!p.block_table)
            ok = ok && (static_cast<long long>(b) * Hkv_r + hkv_r) * p.T_max + k1 <= p.kv_rows;
        else
            ok = ok && p.page_size > 0 && p.page_size % kTileKeys == 0 && (k1 + p.page_size - 1) / p.page_size <= p.max_pages;
        if (p.mode != kModeFinal)
            ok = ok && (static_cast<long long>(b) * p.Hq + hkv * G + (G - 1)) * p.num_splits + split < p.partial_records;
        if (p.mode == kModeFused) ok = ok && p.counters != nullptr;
        if (!ok) {
            if (threadIdx.x == 0 && p.status) atomicExch(p.status, PLX_ERR_DEVICE_CHECK);
            return;
        }
    }
#endif
    const int n_my = (ntiles - warp + kWarps - 1) / kWarps;  // tiles warp, warp+4, ... (may be 0)
    // first key of this warp's tile n
    auto tile_key = [&](int n) { return k0 + (warp + n * kWarps) * kTileKeys; };

    const int hkv_real = hkv / p.kv_div, Hkv_real = p.Hkv / p.kv_div;
    float scale_log2e = p.scale_log2e, probe_scale = p.probe_scale, v_scale = p.v_scale;
    if constexpr (FP8) {
        if (p.k_scales) {
            probe_scale = p.k_scales[hkv_real];
            scale_log2e *= probe_scale;
            v_scale = p.v_scales[hkv_real];
        }
    }
    const int row0 = (b * Hkv_real + hkv_real) * p.T_max;  // first cache row of this stream
    // Paged cache: a 16-key tile never straddles a page (page_size is a multiple of 16), so only the
    // tile's first row changes: (page id * Hkv + hkv) * page_size + offset.  Lane 0 keeps the current
    // page id and fetches the next one a page ahead, so the lookup is off the TMA issue path.
    int pg_cur = -1, pg_id_cur = 0, pg_id_next = 0;
    const int32_t* const table = p.block_table ? p.block_table + static_cast<size_t>(b) * p.max_pages : nullptr;
    auto paged_row = [&](int key) {
        const int pg = key / p.page_size;
        if (pg != pg_cur) {
            pg_id_cur = (pg_cur >= 0 && pg == pg_cur + 1) ? pg_id_next : __ldg(table + pg);
            pg_cur = pg;
#if PLX_DEBUG_CHECKS
            if (pg_id_cur < 0 || (static_cast<long long>(pg_id_cur) * Hkv_real + hkv_real + 1) * p.page_size > p.kv_rows) {
                if (p.status) atomicExch(p.status, PLX_ERR_DEVICE_CHECK);  // a page id outside the pool: not followed
                pg_id_cur = 0;
            }
#endif
            if (pg + 1 < p.max_pages) pg_id_next = __ldg(table + pg + 1);
        }
        return (pg_id_cur * Hkv_real + hkv_real) * p.page_size + (key - pg * p.page_size);
    };
    auto issue = [&](int n, int s) {
        const uint32_t bar = bars + 8 * s;
        const uint32_t dst = ring + s * SL::kStageBytes;
        const int row = table ? paged_row(tile_key(n)) : row0 + tile_key(n);
        mbar_expect_tx(bar, SL::kStageBytes);
#pragma unroll
        for (int h = 0; h < SL::kHalves; ++h) {
            tma_load_2d(dst + h * SL::kHalfBytes, &tmK, bar, h * 64, row);
            tma_load_2d(dst + SL::kTensorBytes + h * SL::kHalfBytes, &tmV, bar, h * 64, row);
        }
    };
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < NSTAGES; ++s)
            if (s < n_my) issue(s, s);
    }

    // B fragments of [q_a q_b r_a r_b | q_c q_d r_c r_d]^T, one set per four heads: column n = lane/4; the
    // second head pair of a quad takes the four columns a single pair leaves empty, so one MMA per k-step
    // scores four heads.
    uint32_t bqr[NQ][KSTEPS][2];
    const __nv_bfloat16* q_rows = p.q + (static_cast<size_t>(b) * p.Hq + hkv * G) * D;  // the group's G rows are contiguous
    const __nv_bfloat16* r_rows = p.r + (static_cast<size_t>(b) * p.Hq + hkv * G) * D;
    if (p.qr_staged) {  // CTA-uniform
        constexpr int kN16 = G * D * 2 / 16;  // 16-byte words per tensor
        uint4* const sq = reinterpret_cast<uint4*>(smem + SL::kRingBytes + SL::kBarrierBytes);
        for (int i = threadIdx.x; i < 2 * kN16; i += kThreads)
            sq[i] = i < kN16 ? reinterpret_cast<const uint4*>(q_rows)[i] : reinterpret_cast<const uint4*>(r_rows)[i - kN16];
        __syncthreads();
        q_rows = reinterpret_cast<const __nv_bfloat16*>(sq);
        r_rows = reinterpret_cast<const __nv_bfloat16*>(sq + kN16);
    }
#pragma unroll
    for (int qd = 0; qd < NQ; ++qd) {
        const int n = lane >> 2;
        const int hl = 4 * qd + 2 * (n >> 2) + (n & 1);
        const __nv_bfloat16* src = nullptr;
        if (hl < G) src = ((n & 2) ? r_rows : q_rows) + hl * D;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            if constexpr (FP8) {
                // k-step ks, lane t: dimensions 16 ks + 4 t .. + 3 (the four bytes one ldmatrix register holds)
                const int d = ks * 16 + (lane & 3) * 4;
                bqr[qd][ks][0] = src ? f16x2_from_bf16x2(*reinterpret_cast<const uint32_t*>(src + d)) : 0u;
                bqr[qd][ks][1] = src ? f16x2_from_bf16x2(*reinterpret_cast<const uint32_t*>(src + d + 2)) : 0u;
            } else {
                const int d = ks * 16 + (lane & 3) * 2;
                bqr[qd][ks][0] = src ? *reinterpret_cast<const uint32_t*>(src + d) : 0u;
                bqr[qd][ks][1] = src ? *reinterpret_cast<const uint32_t*>(src + d + 8) : 0u;
            }
        }
    }

    // Running state (Algorithm 1): m in log2 units, d1, d2 as per-lane partial sums.
    float o[NQ][MTILES][4];
    // Up to two heads every lane carries the one pair's state.  With more heads the four lanes of a lane quad
    // share the pairs out (lane t computes pair t; with three pairs lane 3 repeats pair 0, with two pairs lanes
    // 2, 3 repeat pairs 0, 1) and exchange the weights by shuffles when the P^T fragments are built.
    float m_run[2], d1[2], d2[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        m_run[e] = -INFINITY;
        d1[e] = 0.0f;
        d2[e] = 0.0f;
    }
#pragma unroll
    for (int qd = 0; qd < NQ; ++qd)
#pragma unroll
        for (int mt = 0; mt < MTILES; ++mt)
#pragma unroll
            for (int j = 0; j < 4; ++j) o[qd][mt][j] = 0.0f;

    // Per-lane ldmatrix geometry (byte offsets inside a swizzled [16 x 64] box).
    const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8;  // K: matrices 0/1 = keys 0-7 / 8-15
    const int k_csel = lane >> 4;                          //    matrices 2/3 = next 8 columns
    const int v_row = (lane & 7) + ((lane >> 4) & 1) * 8;  // V (transposed): matrices 0/1 = keys 0-7
    const int v_csel = (lane >> 3) & 1;
    // column pair this lane feeds into P^T.  Up to two heads: 0 P1, 1 P2, 2/3 their residuals.  More heads:
    // 0 P1 and 1 P2 of a quad's first pair, 2 P1 and 3 P2 of its second pair.
    const int role = lane & 3;
    const int quad = lane & ~3;
    const int my_pair = !SA ? 0 : NP == 4 ? role : NP == 3 ? (role == 3 ? 0 : role) : (role & 1);
    const int key_lo = lane >> 2;    // key (row of S^T) held in c[0], c[1]; c[2], c[3] hold key_lo + 8

    bool failed = false;
    int s = 0;
    uint32_t parity = 0;
    PLX_PHASE_DECL;
    for (int n = 0; n < n_my; ++n) {
        const uint32_t bar = bars + 8 * s;
        if (!mbar_wait_bounded(bar, parity)) {
            failed = true;
            break;
        }
        PLX_PHASE(0);
        if (n == 0) PLX_STAMP(1);
        const uint32_t sK = ring + s * SL::kStageBytes;
        const uint32_t sV = sK + SL::kTensorBytes;
        const int key_n = tile_key(n);
        const int valid = k1 - key_n;  // >= 1 keys of this tile in range

        if (valid < kTileKeys) {
            // Rows past the context may hold anything (NaN included): clear them in shared memory
            // so they contribute exact zeros to both products.
            uint8_t* tile = smem + (sK - base_addr);
            constexpr int kChunksPerBoxRow = SL::kBoxBytes / 16, kChunksPerBox = kTileKeys * kChunksPerBoxRow;
            for (int i = lane; i < 2 * SL::kHalves * kChunksPerBox; i += 32) {  // every 16-byte chunk of the K and the V tile
                const int box = i / kChunksPerBox, rr = (i % kChunksPerBox) / kChunksPerBoxRow, ch = i % kChunksPerBoxRow;
                if (rr >= valid)
                    *reinterpret_cast<uint4*>(tile + box * SL::kHalfBytes + rr * SL::kBoxBytes + ch * 16) =
                        make_uint4(0u, 0u, 0u, 0u);
            }
            __syncwarp();
        }

        // ---- S^T = K_c . [q r]^T ------------------------------------------------------------
        // two independent accumulator chains (even / odd k-steps) halve the dependent MMA latency
        float c[NQ][4], c2[NQ][4];
#pragma unroll
        for (int qd = 0; qd < NQ; ++qd)
#pragma unroll
            for (int j = 0; j < 4; ++j) c[qd][j] = c2[qd][j] = 0.0f;
        if constexpr (FP8) {
#pragma unroll
            for (int kq = 0; kq < D / 32; ++kq) {  // one ldmatrix covers 16 keys x 32 dimensions = two k-steps
                const int chunk = kq * 2 + k_csel;
                uint32_t a[4];
                ldmatrix_x4(a, sK + tile_off(k_row, chunk));
                const uint32_t f0[4] = {e4m3x2_to_f16x2(a[0], false), e4m3x2_to_f16x2(a[1], false),
                                        e4m3x2_to_f16x2(a[0], true), e4m3x2_to_f16x2(a[1], true)};
                const uint32_t f1[4] = {e4m3x2_to_f16x2(a[2], false), e4m3x2_to_f16x2(a[3], false),
                                        e4m3x2_to_f16x2(a[2], true), e4m3x2_to_f16x2(a[3], true)};
#pragma unroll
                for (int qd = 0; qd < NQ; ++qd) {
                    mma_f16(c[qd], f0, bqr[qd][2 * kq][0], bqr[qd][2 * kq][1]);
                    mma_f16(c2[qd], f1, bqr[qd][2 * kq + 1][0], bqr[qd][2 * kq + 1][1]);
                }
            }
        } else {
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                const int chunk = ks * 2 + k_csel;
                uint32_t a[4];
                ldmatrix_x4(a, sK + tile_off(k_row, chunk));
#pragma unroll
                for (int qd = 0; qd < NQ; ++qd) mma_bf16((ks & 1) ? c2[qd] : c[qd], a, bqr[qd][ks][0], bqr[qd][ks][1]);
            }
        }
#pragma unroll
        for (int qd = 0; qd < NQ; ++qd)
#pragma unroll
            for (int j = 0; j < 4; ++j) c[qd][j] += c2[qd][j];

        PLX_PHASE(1);
        // ---- online softmax state and P^T fragments -----------------------------------------
        uint32_t pb0[NQ], pb1[NQ];   // P^T fragments (bf16 / fp16 parts; with up to two heads also the residuals)
        uint32_t pr0[NQ], pr1[NQ];   // more than two heads: the rounding residuals, a second MMA into the same accumulator
        // With several tokens per sequence the last lq - 1 keys are visible to the later tokens only: in the
        // few tiles that reach into them (warp-uniform test) each head of a pair gets its own key count.
        const int to_end = L - key_n;  // keys from this tile's first to the context's last
        const bool per_head = to_end < kTileKeys + p.lq - 1;
        {
            int valid_a = valid, valid_b = valid;
            if (per_head) {
                const int v0 = hkv * G + 2 * my_pair;
                valid_a = min(valid, to_end - (p.lq - 1 - v0 % p.lq));
                valid_b = min(valid, to_end - (p.lq - 1 - (v0 + 1) % p.lq));
            }
            const bool oka_lo = key_lo < valid_a, oka_hi = key_lo + 8 < valid_a;
            const bool okb_lo = key_lo < valid_b, okb_hi = key_lo + 8 < valid_b;
            // Of the score MMA of the pair's quad, lane 2 (pair & 1) of a lane quad holds the pair's softmax scores
            // (heads a, b; keys key_lo and key_lo + 8) and the next lane its probe scores.
            const int src = quad + 2 * (my_pair & 1);
            float sc[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                sc[j] = __shfl_sync(0xffffffffu, c[0][j], src);
                sc[4 + j] = __shfl_sync(0xffffffffu, c[0][j], src + 1);
                if constexpr (NQ == 2) {
                    const float u = __shfl_sync(0xffffffffu, c[NQ - 1][j], src);
                    const float w = __shfl_sync(0xffffffffu, c[NQ - 1][j], src + 1);
                    if (my_pair >> 1) {
                        sc[j] = u;
                        sc[4 + j] = w;
                    }
                }
            }
            float s1a_lo = sc[0], s1b_lo = sc[1], s1a_hi = sc[2], s1b_hi = sc[3];
            float s2a_lo = sc[4], s2b_lo = sc[5], s2a_hi = sc[6], s2b_hi = sc[7];
            s1a_lo = oka_lo ? s1a_lo * scale_log2e : -INFINITY;
            s1b_lo = okb_lo ? s1b_lo * scale_log2e : -INFINITY;
            s1a_hi = oka_hi ? s1a_hi * scale_log2e : -INFINITY;
            s1b_hi = okb_hi ? s1b_hi * scale_log2e : -INFINITY;
            if constexpr (FP8) {
                s2a_lo *= probe_scale;
                s2b_lo *= probe_scale;
                s2a_hi *= probe_scale;
                s2b_hi *= probe_scale;
            }
            s2a_lo = oka_lo ? s2a_lo : 0.0f;
            s2b_lo = okb_lo ? s2b_lo : 0.0f;
            s2a_hi = oka_hi ? s2a_hi : 0.0f;
            s2b_hi = okb_hi ? s2b_hi : 0.0f;

            float ta = fmaxf(s1a_lo, s1a_hi), tb = fmaxf(s1b_lo, s1b_hi);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, off));
                tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, off));
            }
            // Lazy reference update.  Up to two heads every lane holds the same ta, tb, m_run; with more heads
            // they are per pair, so the warp takes the branch together as soon as any pair needs it (a pair
            // that did not need it moves its reference to its running maximum too, which changes nothing).
            const bool need = ta > m_run[0] + kThreshold || tb > m_run[1] + kThreshold;
            if (SA ? __any_sync(0xffffffffu, need) : need) {
                const float ma = fmaxf(m_run[0], ta), mb = fmaxf(m_run[1], tb);
                // a head that has seen no key yet (and sees none in this tile) keeps its empty state
                const float alpha_a = (ma > -INFINITY) ? fast_exp2(m_run[0] - ma) : 1.0f;
                const float alpha_b = (mb > -INFINITY) ? fast_exp2(m_run[1] - mb) : 1.0f;
                m_run[0] = ma;
                m_run[1] = mb;
                d1[0] *= alpha_a;
                d2[0] *= alpha_a;
                d1[1] *= alpha_b;
                d2[1] *= alpha_b;
#pragma unroll
                for (int qd = 0; qd < NQ; ++qd) {
                    float fa = alpha_a, fb = alpha_b;
                    if constexpr (SA) {
                        // this lane's accumulator columns of quad qd belong to pair 2 qd + (role >> 1), which lane
                        // (quad + that pair) computes; a pair that does not exist has all-zero columns
                        const int owner = quad + min(2 * qd + (role >> 1), NP - 1);
                        fa = __shfl_sync(0xffffffffu, alpha_a, owner);
                        fb = __shfl_sync(0xffffffffu, alpha_b, owner);
                    }
#pragma unroll
                    for (int mt = 0; mt < MTILES; ++mt) {
                        o[qd][mt][0] *= fa;
                        o[qd][mt][1] *= fb;
                        o[qd][mt][2] *= fa;
                        o[qd][mt][3] *= fb;
                    }
                }
            }
            // reference 0 while a head has seen nothing: its scores are all -inf and its weights exact zeros
            const float ref_a = (m_run[0] > -INFINITY) ? m_run[0] : 0.0f;
            const float ref_b = (m_run[1] > -INFINITY) ? m_run[1] : 0.0f;
            const float p1a_lo = fast_exp2(s1a_lo - ref_a);
            const float p1b_lo = fast_exp2(s1b_lo - ref_b);
            const float p1a_hi = fast_exp2(s1a_hi - ref_a);
            const float p1b_hi = fast_exp2(s1b_hi - ref_b);
            const float p2a_lo = p1a_lo * s2a_lo, p2b_lo = p1b_lo * s2b_lo;
            const float p2a_hi = p1a_hi * s2a_hi, p2b_hi = p1b_hi * s2b_hi;
            d1[0] += p1a_lo + p1a_hi;
            d1[1] += p1b_lo + p1b_hi;
            d2[0] += p2a_lo + p2a_hi;
            d2[1] += p2b_lo + p2b_hi;
            const bool second = role & 1;
            if constexpr (!SA) {
                const bool resid = role & 2;
                const uint32_t f_lo = FP8 ? pack_f16_pair(second ? p2a_lo : p1a_lo, second ? p2b_lo : p1b_lo, resid)
                                          : pack_bf16_pair(second ? p2a_lo : p1a_lo, second ? p2b_lo : p1b_lo, resid);
                const uint32_t f_hi = FP8 ? pack_f16_pair(second ? p2a_hi : p1a_hi, second ? p2b_hi : p1b_hi, resid)
                                          : pack_bf16_pair(second ? p2a_hi : p1a_hi, second ? p2b_hi : p1b_hi, resid);
                pb0[0] = movmatrix_trans(f_lo);   // keys 0-7  -> k rows 0-7 of the B operand
                pb1[0] = movmatrix_trans(f_hi);   // keys 8-15 -> k rows 8-15
            } else {
#pragma unroll
                for (int qd = 0; qd < NQ; ++qd) {
                    // column pair (role) of quad qd: P1 (even role) or P2 (odd role) of pair 2 qd + (role >> 1)
                    const int want = 2 * qd + (role >> 1);
                    const int owner = quad + min(want, NP - 1);
                    const float g1a_lo = __shfl_sync(0xffffffffu, p1a_lo, owner), g2a_lo = __shfl_sync(0xffffffffu, p2a_lo, owner);
                    const float g1b_lo = __shfl_sync(0xffffffffu, p1b_lo, owner), g2b_lo = __shfl_sync(0xffffffffu, p2b_lo, owner);
                    const float g1a_hi = __shfl_sync(0xffffffffu, p1a_hi, owner), g2a_hi = __shfl_sync(0xffffffffu, p2a_hi, owner);
                    const float g1b_hi = __shfl_sync(0xffffffffu, p1b_hi, owner), g2b_hi = __shfl_sync(0xffffffffu, p2b_hi, owner);
                    const bool exists = want < NP;
                    const float ya_lo = exists ? (second ? g2a_lo : g1a_lo) : 0.0f, yb_lo = exists ? (second ? g2b_lo : g1b_lo) : 0.0f;
                    const float ya_hi = exists ? (second ? g2a_hi : g1a_hi) : 0.0f, yb_hi = exists ? (second ? g2b_hi : g1b_hi) : 0.0f;
                    pb0[qd] = movmatrix_trans(FP8 ? pack_f16_pair(ya_lo, yb_lo, false) : pack_bf16_pair(ya_lo, yb_lo, false));
                    pb1[qd] = movmatrix_trans(FP8 ? pack_f16_pair(ya_hi, yb_hi, false) : pack_bf16_pair(ya_hi, yb_hi, false));
                    pr0[qd] = movmatrix_trans(FP8 ? pack_f16_pair(ya_lo, yb_lo, true) : pack_bf16_pair(ya_lo, yb_lo, true));
                    pr1[qd] = movmatrix_trans(FP8 ? pack_f16_pair(ya_hi, yb_hi, true) : pack_bf16_pair(ya_hi, yb_hi, true));
                }
            }
        }

        PLX_PHASE(2);
        // ---- O^T += V_c^T . P^T -------------------------------------------------------------
        if constexpr (FP8) {
#pragma unroll
            for (int mq = 0; mq < D / 32; ++mq) {  // one transposed ldmatrix covers two 16-dimension m-tiles
                const int chunk = mq * 2 + v_csel;
                uint32_t a[4];
                ldmatrix_x4_trans(a, sV + tile_off(v_row, chunk));
                // a register holds (key 2t: dims 2g, 2g+1 | key 2t+1: dims 2g, 2g+1): regroup by dimension
                uint32_t x[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) x[i] = __byte_perm(a[i], 0u, 0x3120);
                // m-tile rows g / g+8 carry dimensions 2g / 2g+1 of the 16-dimension block
                const uint32_t f0[4] = {e4m3x2_to_f16x2(x[0], false), e4m3x2_to_f16x2(x[0], true),
                                        e4m3x2_to_f16x2(x[2], false), e4m3x2_to_f16x2(x[2], true)};
                const uint32_t f1[4] = {e4m3x2_to_f16x2(x[1], false), e4m3x2_to_f16x2(x[1], true),
                                        e4m3x2_to_f16x2(x[3], false), e4m3x2_to_f16x2(x[3], true)};
#pragma unroll
                for (int qd = 0; qd < NQ; ++qd) {
                    mma_f16(o[qd][2 * mq], f0, pb0[qd], pb1[qd]);
                    mma_f16(o[qd][2 * mq + 1], f1, pb0[qd], pb1[qd]);
                }
                if constexpr (SA) {
#pragma unroll
                    for (int qd = 0; qd < NQ; ++qd) {
                        mma_f16(o[qd][2 * mq], f0, pr0[qd], pr1[qd]);
                        mma_f16(o[qd][2 * mq + 1], f1, pr0[qd], pr1[qd]);
                    }
                }
            }
        } else {
#pragma unroll
            for (int mt = 0; mt < MTILES; mt += 2) {  // two m-tiles at a time: the residual MMAs follow two others
                uint32_t a0[4], a1[4];
                const int ch0 = mt * 2 + v_csel, ch1 = ch0 + 2;
                ldmatrix_x4_trans(a0, sV + tile_off(v_row, ch0));
                ldmatrix_x4_trans(a1, sV + tile_off(v_row, ch1));
#pragma unroll
                for (int qd = 0; qd < NQ; ++qd) {
                    mma_bf16(o[qd][mt], a0, pb0[qd], pb1[qd]);
                    mma_bf16(o[qd][mt + 1], a1, pb0[qd], pb1[qd]);
                }
                if constexpr (SA) {
#pragma unroll
                    for (int qd = 0; qd < NQ; ++qd) {
                        mma_bf16(o[qd][mt], a0, pr0[qd], pr1[qd]);
                        mma_bf16(o[qd][mt + 1], a1, pr0[qd], pr1[qd]);
                    }
                }
            }
        }

        // The MMAs above have consumed every fragment of this stage (in-order issue), so the
        // buffer can be refilled by the same warp.
        __syncwarp();
        if (lane == 0 && n + NSTAGES < n_my) issue(n + NSTAGES, s);
        if (++s == NSTAGES) {
            s = 0;
            parity ^= 1u;
        }
        PLX_PHASE(3);
    }

    PLX_STAMP(2);
    PLX_PHASE_STORE;
    if (failed) {
        // A wait ran out: record it, give the copies still in flight one more bounded chance to
        // land before this CTA's shared memory is released, and fall through with what we have.
        if (lane == 0 && p.status) atomicExch(p.status, PLX_ERR_DEVICE_TIMEOUT);
        for (int t = 0; t < NSTAGES; ++t) {
            (void)mbar_wait_bounded(bars + 8 * s, parity);
            if (++s == NSTAGES) {
                s = 0;
                parity ^= 1u;
            }
        }
    }

    // ---- per-warp wrap-up: finish the lane-partial sums, fold residual columns ----------------
#pragma unroll
    for (int e = 0; e < 2; ++e) {
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            d1[e] += __shfl_xor_sync(0xffffffffu, d1[e], off);
            d2[e] += __shfl_xor_sync(0xffffffffu, d2[e], off);
        }
    }
    if constexpr (!SA) {  // up to two heads: columns 4-7 accumulated the residual products
#pragma unroll
        for (int mt = 0; mt < MTILES; ++mt)
#pragma unroll
            for (int j = 0; j < 4; ++j) o[0][mt][j] += __shfl_xor_sync(0xffffffffu, o[0][mt][j], 2);
    }

    __syncthreads();  // every warp has drained its ring: reuse it as merge scratch
    float* const scratch = reinterpret_cast<float*>(smem);
    if (lane < NP) {  // lanes 0 .. NP-1 hold the state of pairs 0 .. NP-1
        float* rec_a = scratch + ((warp * NP + lane) * 2 + 0) * REC;
        float* rec_b = rec_a + REC;
        rec_a[0] = m_run[0];
        rec_a[1] = d1[0];
        rec_a[2] = d2[0];
        rec_b[0] = m_run[1];
        rec_b[1] = d1[1];
        rec_b[2] = d2[1];
    }
#pragma unroll
    for (int qd = 0; qd < NQ; ++qd) {
        // Up to two heads: role 0 holds the pair's O1 columns, role 1 its O2 columns.  More heads: roles 0, 1
        // hold O1, O2 of the quad's first pair, roles 2, 3 those of its second pair.
        const int pp = SA ? 2 * qd + (role >> 1) : 0;
        if (SA ? pp < NP : role < 2) {
            float* rec_a = scratch + ((warp * NP + pp) * 2 + 0) * REC;
            float* rec_b = rec_a + REC;
            // accumulator rows g and g + 8 of an m-tile are dimensions g, g + 8 (2g, 2g + 1 in the FP8 variant)
            const int off = 4 + (role & 1) * D + (FP8 ? 2 * key_lo : key_lo);
            constexpr int kUp = FP8 ? 1 : 8;
#pragma unroll
            for (int mt = 0; mt < MTILES; ++mt) {
                rec_a[off + mt * 16] = o[qd][mt][0];
                rec_b[off + mt * 16] = o[qd][mt][1];
                rec_a[off + mt * 16 + kUp] = o[qd][mt][2];
                rec_b[off + mt * 16 + kUp] = o[qd][mt][3];
            }
        }
    }
    __syncthreads();

    // ---- merge the four warps (log-sum-exp) and write the row or the partial record ----------
    for (int idx = threadIdx.x; idx < NP * 2 * D; idx += kThreads) {
        const int pe = idx / D, d = idx - pe * D;
        if (pe >= G) continue;  // odd group size: the pair's second head does not exist
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, scratch[(w * NP * 2 + pe) * REC]);
        const float M_ref = (M > -INFINITY) ? M : 0.0f;  // a head none of whose keys lie in this chunk
        float D1 = 0.0f, D2 = 0.0f, O1 = 0.0f, O2 = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float* rec = scratch + (w * NP * 2 + pe) * REC;
            const float a = fast_exp2(rec[0] - M_ref);  // 0 for a warp that saw no tile
            D1 += a * rec[1];
            D2 += a * rec[2];
            O1 += a * rec[4 + d];
            O2 += a * rec[4 + D + d];
        }
        if constexpr (FP8) {
            O1 *= v_scale;
            O2 *= v_scale;
        }
        const size_t rowidx = static_cast<size_t>(b) * p.Hq + hkv * G + pe;
        if (p.mode == kModeFinal) {
            store_out(p.out, rowidx * D + d, D1 > 0.0f ? finalize(O1, O2, D1, D2) : 0.0f, p.out_dtype);
        } else {
            float* rec = p.partials + (rowidx * p.num_splits + split) * REC;
            rec[4 + d] = O1;
            rec[4 + D + d] = O2;
            if (d == 0) {
                rec[0] = M * kLn2;
                rec[1] = D1;
                rec[2] = D2;
                rec[3] = 0.0f;
            }
        }
    }

    PLX_STAMP(3);
    if (p.mode == kModeFused) {
        // Publish this CTA's records, count the arrival, and let the CTA that completes the
        // (sequence, KV head) merge all of its splits in split order.
        // The CTA barrier orders every thread's record stores before thread 0's arrival, and the
        // arrival is an acquire-release RMW at device scope: release makes this CTA's records visible
        // to whoever observes the count (cumulativity over the barrier), acquire makes the earlier
        // arrivals' records visible to the CTA that completes it.  No per-thread membar is needed.
        __syncthreads();
        const int expected = (L + p.chunk_len - 1) / p.chunk_len;  // CTAs of this stream that hold keys
        if (threadIdx.x == 0) {
            int old;
            asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(p.counters + stream_id) : "memory");
            s_is_last = (old == expected - 1);
            if (s_is_last) {
                p.counters[stream_id] = 0;  // nobody else touches it any more in this launch
                fence_proxy_async();        // the records are read next through the async proxy (bulk copies)
            }
        }
        __syncthreads();
        if (s_is_last) {
            // Stage every record of this stream's G rows into the idle ring with bulk copies (one per
            // row: a row's records are contiguous), then merge out of shared memory.  Rows that have
            // more records than fit are merged batch by batch with a running reference exponent.
            constexpr int CAP = SL::kRingBytes / (REC * 4) / G;  // records per row per batch
            constexpr int NPAIR = (G * D + kThreads - 1) / kThreads;
            const uint32_t mbar = base_addr + SL::kRingBytes + kWarps * NSTAGES * 8;
            float runM[NPAIR], accD1[NPAIR], accD2[NPAIR], accO1[NPAIR], accO2[NPAIR];
#pragma unroll
            for (int j = 0; j < NPAIR; ++j) {
                runM[j] = -INFINITY;
                accD1[j] = accD2[j] = accO1[j] = accO2[j] = 0.0f;
            }
            uint32_t mpar = 0;
            for (int i0 = 0; i0 < expected; i0 += CAP) {
                const int nb = min(CAP, expected - i0);
                if (i0 > 0) __syncthreads();  // previous batch consumed by every thread
                if (threadIdx.x == 0) {
                    mbar_expect_tx(mbar, static_cast<uint32_t>(G * nb * REC * 4));
                    for (int hl = 0; hl < G; ++hl) {
                        const size_t rowidx = static_cast<size_t>(b) * p.Hq + hkv * G + hl;
                        bulk_load(base_addr + hl * CAP * REC * 4, p.partials + (rowidx * p.num_splits + i0) * REC,
                                  static_cast<uint32_t>(nb * REC * 4), mbar);
                    }
                }
                // On a wait that runs out only the status word is set; control flow stays uniform so
                // that every thread still reaches the barrier of the next batch.
                if (!mbar_wait_bounded(mbar, mpar) && p.status) atomicExch(p.status, PLX_ERR_DEVICE_TIMEOUT);
                mpar ^= 1u;
                // Every record staged here was written by a CTA that held at least one key, so all
                // exponents are finite and the loops can run branch-free (and unrolled) over records.
                const float* rows[NPAIR];
                int dd[NPAIR];
                float mb[NPAIR], alpha[NPAIR];
#pragma unroll
                for (int j = 0; j < NPAIR; ++j) {
                    const int pr = min(threadIdx.x + j * kThreads, G * D - 1);  // surplus threads shadow the last pair
                    const int hl = pr / D;
                    dd[j] = pr - hl * D;
                    rows[j] = scratch + hl * CAP * REC;
                    mb[j] = -INFINITY;
                }
#pragma unroll 8
                for (int i = 0; i < nb; ++i)
#pragma unroll
                    for (int j = 0; j < NPAIR; ++j) mb[j] = fmaxf(mb[j], rows[j][i * REC]);
#pragma unroll
                for (int j = 0; j < NPAIR; ++j) {
                    const float Mn = fmaxf(runM[j], mb[j]);
                    alpha[j] = (runM[j] > -INFINITY) ? __expf(runM[j] - Mn) : 0.0f;
                    runM[j] = Mn;
                    accD1[j] *= alpha[j];
                    accD2[j] *= alpha[j];
                    accO1[j] *= alpha[j];
                    accO2[j] *= alpha[j];
                }
#pragma unroll 4
                for (int i = 0; i < nb; ++i) {
#pragma unroll
                    for (int j = 0; j < NPAIR; ++j) {
                        const float* rec = rows[j] + i * REC;
                        const float w = __expf(rec[0] - runM[j]);
                        accD1[j] += w * rec[1];
                        accD2[j] += w * rec[2];
                        accO1[j] += w * rec[4 + dd[j]];
                        accO2[j] += w * rec[4 + D + dd[j]];
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < NPAIR; ++j) {
                const int pr = threadIdx.x + j * kThreads;
                if (pr >= G * D) continue;
                const int hl = pr / D, d = pr - hl * D;
                const size_t rowidx = static_cast<size_t>(b) * p.Hq + hkv * G + hl;
                const float v = (runM[j] > -INFINITY) ? finalize(accO1[j], accO2[j], accD1[j], accD2[j]) : 0.0f;
                store_out(p.out, rowidx * D + d, v, p.out_dtype);
            }
        }
    }
    // every store of this CTA has been issued: the next kernel of the stream may be scheduled
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---------------------------------------------------------------------------
// Combine kernel: one CTA of 8 warps per (b, hq) row.
// ---------------------------------------------------------------------------
constexpr int kCombineWarps = 8;

template <int D>
__global__ void __launch_bounds__(kCombineWarps * 32)
plx_combine_kernel(const float* __restrict__ partials, const int32_t* __restrict__ split_counts,
                   const int32_t* __restrict__ seqlens, int chunk_len, int T_max, void* out, int Hq,
                   int num_splits, int out_dtype, int num_groups, size_t group_stride)
{
    constexpr int REC = 2 * D + 4;
    __shared__ __align__(16) float scratch[MergeScratch<D, kCombineWarps>::kFloats];
    // Launched as a programmatic dependent of the kernel that writes the records (the split-KV multi-token
    // forward does that): wait for its completion before the first read.  A no-op in an ordinary launch.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int row = blockIdx.x;
    const int b = row / Hq;
    if (num_groups > 1) {  // [group][B*Hq][num_splits] records: merge all of them, empty ones are skipped
        merge_row<D, kCombineWarps>(partials + static_cast<size_t>(row) * num_splits * REC, num_groups * num_splits,
                                    scratch, out, static_cast<size_t>(row) * D, out_dtype, num_splits, group_stride);
        return;
    }
    int count = num_splits;
    if (split_counts) {
        count = max(0, min(split_counts[b], num_splits));
    } else if (seqlens) {
        const int L = max(0, min(seqlens[b], T_max));
        count = min(num_splits, (L + chunk_len - 1) / chunk_len);
    }
    merge_row<D, kCombineWarps>(partials + static_cast<size_t>(row) * num_splits * REC, count, scratch, out,
                                static_cast<size_t>(row) * D, out_dtype);
}

// ---------------------------------------------------------------------------
// Combine kernel for many rows of few records each (the split multi-token steps: thousands of rows, two to a few
// splits): one WARP per row, eight rows per CTA.  A CTA per row, as above, takes 18 us for the 8192 rows of a C3 step
// with eight new tokens and 35 us for sixteen, a tenth of the step; this one runs them in a single generation of CTAs.
// Same arithmetic as merge_row (M = max m_s, weights exp(m_s - M), sums in split order, final line), each lane
// holding 2 D / 32 elements of O1 and O2.
// ---------------------------------------------------------------------------
constexpr int kRowCombineWarps = 8;
constexpr int kRowCombineMaxSplits = 16;

template <int D>
__global__ void __launch_bounds__(kRowCombineWarps * 32)
plx_combine_rows_kernel(const float* __restrict__ partials, void* out, int rows, int num_splits, int out_dtype)
{
    constexpr int REC = 2 * D + 4;
    constexpr int EPL = D / 32;  // elements of O1 (and of O2) per lane: 4 or 2
    // launched as a programmatic dependent of the kernel that writes the records
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * kRowCombineWarps + warp;
    if (row >= rows) return;
    const float* const base = partials + static_cast<size_t>(row) * num_splits * REC;
    float M = -INFINITY;
    for (int s = 0; s < num_splits; ++s) M = fmaxf(M, __ldcg(base + static_cast<size_t>(s) * REC));
    float o1[EPL], o2[EPL], D1 = 0.0f, D2 = 0.0f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) o1[e] = o2[e] = 0.0f;
    if (M > -INFINITY) {
        for (int s = 0; s < num_splits; ++s) {
            const float* const rec = base + static_cast<size_t>(s) * REC;
            const float m = __ldcg(rec);
            if (!(m > -INFINITY)) continue;  // empty record: its payload is not read
            const float a = __expf(m - M);
            D1 += a * __ldcg(rec + 1);
            D2 += a * __ldcg(rec + 2);
            if constexpr (EPL == 4) {
                const float4 x = __ldcg(reinterpret_cast<const float4*>(rec + 4) + lane);
                const float4 y = __ldcg(reinterpret_cast<const float4*>(rec + 4 + D) + lane);
                o1[0] += a * x.x; o1[1] += a * x.y; o1[2] += a * x.z; o1[3] += a * x.w;
                o2[0] += a * y.x; o2[1] += a * y.y; o2[2] += a * y.z; o2[3] += a * y.w;
            } else {
                const float2 x = __ldcg(reinterpret_cast<const float2*>(rec + 4) + lane);
                const float2 y = __ldcg(reinterpret_cast<const float2*>(rec + 4 + D) + lane);
                o1[0] += a * x.x; o1[1] += a * x.y;
                o2[0] += a * y.x; o2[1] += a * y.y;
            }
        }
    }
    const bool any = M > -INFINITY && D1 > 0.0f;
#pragma unroll
    for (int e = 0; e < EPL; ++e)
        store_out(out, static_cast<size_t>(row) * D + lane * EPL + e, any ? finalize(o1[e], o2[e], D1, D2) : 0.0f, out_dtype);
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
int device_sm_count(int* sms)
{
    static int cache[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PLX_ERR_CUDA;
    if (dev >= 0 && dev < 64 && cache[dev] > 0) {
        *sms = cache[dev];
        return PLX_OK;
    }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        return PLX_ERR_CUDA;
    if (dev >= 0 && dev < 64) cache[dev] = n;
    *sms = n;
    return PLX_OK;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// workspace = [header 256][arrival counters][q staging][r staging][out staging][partials]
size_t counter_bytes(int B, int Hq) { return align_up(static_cast<size_t>(B) * Hq * sizeof(int32_t), 256); }
size_t staging_bytes(int B, int Hq, int D)
{
    const size_t n = static_cast<size_t>(B) * Hq * D;
    return 2 * align_up(n * 2, 256) + align_up(n * 4, 256);
}
size_t fixed_bytes(int B, int Hq, int D) { return kHeaderBytes + counter_bytes(B, Hq) + staging_bytes(B, Hq, D); }
size_t partial_bytes(int B, int Hq, int D, int splits)
{
    return align_up(static_cast<size_t>(B) * Hq * splits * (2 * D + 4) * sizeof(float), 256);
}

bool shape_ok(int B, int Hq, int Hkv, int D) { return B > 0 && Hq > 0 && Hkv > 0 && D > 0 && Hq % Hkv == 0; }
// Query heads per CTA (g <= 4) and CTAs ("virtual KV heads") per real KV head for a group of G query heads.
void split_group(int G, int* g, int* kv_div, int max_g = 8)
{
    // the largest group size up to max_g that divides G (the kernel is built for 1 .. 8 heads per CTA)
    int best = 1;
    for (int c = 1; c <= max_g && c <= G; ++c)
        if (G % c == 0) best = c;
    *g = best;
    *kv_div = G / best;
}
bool shape_supported(int Hq, int Hkv, int D)
{
    const int G = Hq / Hkv;
    return (D == 64 || D == 128) && G >= 1 && G <= 64;
}
// Rewrites the launch parameters for group sizes above 4 and returns the per-CTA group size.
int apply_group(KernelParams* kp, int Hq, int Hkv, int max_g = 8)
{
    int g = 1, kv_div = 1;
    split_group(Hq / Hkv, &g, &kv_div, max_g);
    kp->Hkv = Hkv * kv_div;
    kp->kv_div = kv_div;
    return g;
}
int virtual_kv_heads(int Hq, int Hkv, int max_g = 8)
{
    int g = 1, kv_div = 1;
    split_group(Hq / Hkv, &g, &kv_div, max_g);
    return Hkv * kv_div;
}
int heads_per_cta(int Hq, int Hkv)
{
    int g = 1, kv_div = 1;
    split_group(Hq / Hkv, &g, &kv_div);
    return g;
}
bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Split plan.  Cost model in units of "time for one resident CTA to stream one key while the device
// is full", calibrated on B200 measurements:
//   - full waves of `slots` CTAs cost `chunk` each;
//   - a last, partial wave of n CTAs runs min(cap, slots/n) times faster per CTA: a lone CTA is
//     limited by its warps' per-tile latency chain, not by bytes in flight, so it pulls ~54 GB/s at
//     D = 128 (cap 2.2: ~135 of 296 CTAs already saturate HBM); at D = 64 the tiles are half as large,
//     four CTAs share an SM and ~310 of 592 saturate HBM (cap 1.9);
//   - ~60 per CTA generation (launch, barrier setup, pipeline fill; empty CTAs of ragged batches too);
//   - a split plan pays ~300 + 2.3 per split (the fused merge on the tail, the later generations' fill);
//   - with unequal contexts the CTAs that finish last run alone for about one chunk.
// All constants are fitted to sweeps of 100-125 (batch, context) cells x 20-30 forced split counts per
// geometry (mean loss of the plan against the best measured split count about 1 %).  The geometries with
// 4 KiB stages (D = 64, e4m3 cache) have their own: a CTA's fixed cost weighs about four times as much per
// key there (100), and a split plan pays ~220 + 6 per split for the merge and the second generation.
// The e4m3 kernel spends twice the instructions per byte, so it needs nearly all four CTAs of an SM to
// saturate HBM (cap 1.5: 384 resident CTAs reach 6.0 TB/s where 512 reach 6.6) and its fixed cost is 140.
// Five to eight heads per CTA (D = 128, 16-bit cache) have constants of their own: a tile costs such a warp ~1560
// cycles instead of ~1170, so a CTA alone on its SM pulls less and the partial-wave speed-up is capped at 1.4; fixed cost
// 200 per CTA generation, merge 150 + 10 per split.  Fitted on a sweep of 14 (batch, context) cells x the split counts
// that give 74...592 CTAs: the plan then loses 0.2-1 % on average against the best measured split count, where the
// two-head constants lost 11 % (worst cell 30 %: 16 x 8192 keys was not split, 118 against 93 us).
// CTAs of a build that fit on one SM (registers and shared memory; mirrors the launch bounds in dispatch_main)
int resident_ctas(int D, bool fp8, int heads_per_cta)
{
    if (fp8) return D == 128 ? (heads_per_cta <= 2 ? kCtasPerSmFp8 : 2) : (heads_per_cta <= 4 ? kCtasPerSmFp8 : 3);
    if (D == 64) return heads_per_cta <= 4 ? PLX_CTAS_PER_SM_D64 : 3;
    return kCtasPerSm;
}

double plan_cost(int chunk, int ns_eff, long long streams, long long slots, bool ragged, int D, bool fp8 = false,
                 int heads_per_cta = 2)
{
    const long long ctas = streams * ns_eff;
    const long long full = ctas / slots, last = ctas % slots;
    const bool small_stage = D < 128 || fp8;  // 4 KiB stages, four CTAs per SM
    const bool many_heads = !small_stage && heads_per_cta >= 5;
    // D = 64, 16-bit cache, five to eight heads per CTA (three CTAs per SM): cap 1.2, fixed cost 300, 10 per split,
    // uneven-spread factor 0.6 (same sweep at D = 64: plan loss 8 % -> 0.1 % on the measured split counts)
    const bool many_heads_d64 = !fp8 && D < 128 && heads_per_cta >= 5;
    const double fixed = fp8 ? 140.0 : many_heads_d64 ? 300.0 : small_stage ? 100.0 : many_heads ? 200.0 : 60.0;
    double cost = static_cast<double>(full) * chunk + fixed * static_cast<double>(ctas) / static_cast<double>(slots) + fixed;
    if (last > 0) {
        const double cap = fp8 ? 1.5 : many_heads_d64 ? 1.2 : small_stage ? 1.9 : many_heads ? 1.4 : 2.2;
        const double speedup = static_cast<double>(slots) / static_cast<double>(last);
        double tail = chunk / (speedup < cap ? speedup : cap);
        if (small_stage) {
            // With four CTAs per SM a partial wave that does not spread evenly over the SMs (304 CTAs on
            // 148 SMs: eight SMs hold three) finishes with its fullest SMs; measured ~14 % for that case.
            const double per_sm = static_cast<double>(last) * resident_ctas(D, fp8, heads_per_cta) / static_cast<double>(slots);
            tail *= 1.0 + (many_heads_d64 ? 0.6 : 0.3) * (ceil(per_sm) / per_sm - 1.0);
        }
        cost += tail;
    }
    if (ns_eff > 1)
        cost += many_heads_d64 ? 220.0 + 10.0 * ns_eff
                : small_stage  ? 220.0 + 6.0 * ns_eff
                : many_heads   ? 150.0 + 10.0 * ns_eff
                               : 300.0 + 2.3 * ns_eff;
    if (ragged) cost += chunk;
    return cost;
}

void plan_splits(int B, int Hkv, int D, int T_max, int num_sms, bool ragged, int* chunk_len, int* num_splits,
                 bool fp8 = false, int heads_per_cta = 2)
{
    const long long streams = static_cast<long long>(B) * Hkv;
    const long long slots = static_cast<long long>(num_sms) * resident_ctas(D, fp8, heads_per_cta);
    const int granules = (T_max + kChunkGranule - 1) / kChunkGranule;
    const int kMinChunk = 256;
    double best_cost = -1.0;
    int best_chunk = granules * kChunkGranule;
    const int max_ns = granules < PLX_MAX_SPLITS ? granules : PLX_MAX_SPLITS;
    int prev_chunk = -1;
    for (int ns = 1; ns <= max_ns; ++ns) {
        const int chunk = ((granules + ns - 1) / ns) * kChunkGranule;
        if (chunk == prev_chunk) continue;
        prev_chunk = chunk;
        if (ns > 1 && chunk < kMinChunk) break;
        const int ns_eff = (T_max + chunk - 1) / chunk;
        const double cost = plan_cost(chunk, ns_eff, streams, slots, ragged, D, fp8, heads_per_cta);
        if (best_cost < 0.0 || cost < best_cost * 0.995) {  // ties go to fewer splits
            best_cost = cost;
            best_chunk = chunk;
        }
    }
    *chunk_len = best_chunk;
    *num_splits = (T_max + best_chunk - 1) / best_chunk;
}

template <int D, int G, int NSTAGES, int CTAS = kCtasPerSm, bool FP8 = false>
int launch_main(const CUtensorMap& tmK, const CUtensorMap& tmV, const KernelParams& kp, cudaStream_t stream)
{
    using SL = SmemLayout<D, NSTAGES, FP8>;
    auto kernel = plx_decode_kernel<D, G, NSTAGES, CTAS, FP8>;
    PlxNvtxRange nvtx_range(kp.mode == kModeFinal ? "plx_decode_main(final)" : kp.mode == kModeFused ? "plx_decode_main(fused merge)"
                                                                                                    : "plx_decode_main(partial)");
    static bool configured[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PLX_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kTotalBytes) != cudaSuccess)
            return PLX_ERR_CUDA;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    const dim3 grid(static_cast<unsigned>(kp.B * kp.Hkv * kp.num_splits), 1, 1);
    // Programmatic stream serialisation: after a kernel that signals its dependents (the previous decode
    // call does, as do the upstream-step and staging kernels) this grid's CTAs may be scheduled before that
    // kernel has drained (they wait before touching memory); after any other kernel the launch behaves like
    // an ordinary one.
    const bool chain = PLX_PDL_CHAIN || kp.dependent_launch != 0;
    KernelParams kpl = kp;
    {
        int num_sms = 0;
        kpl.signal_early = (device_sm_count(&num_sms) == PLX_OK && grid.x >= static_cast<unsigned>(num_sms) * CTAS) ? 1 : 0;
    }
    if (chain) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = SL::kTotalBytes;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, kernel, tmK, tmV, kpl) == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
    }
    kernel<<<grid, kThreads, SL::kTotalBytes, stream>>>(tmK, tmV, kpl);
    return cudaGetLastError() == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}

int dispatch_main(int D, int G, const CUtensorMap& tmK, const CUtensorMap& tmV, const KernelParams& kp,
                  cudaStream_t stream, bool fp8 = false)
{
    if (fp8) {
        // e4m3 cache, D = 128: 4 KiB stages, the byte geometry of a 16-bit cache at D = 64, and the same
        // measured optimum: four CTAs per SM (128 registers per thread at G <= 2), two stages per warp
        // when the grid fills the device, three otherwise.  G = 3, 4 need ~155 registers: two CTAs per SM.
        // D = 64: 64-byte rows, 2 KiB stages (the compute-matched shape of Sec. 3.3 over an e4m3 cache).
        int num_sms = 0;
        if (int rc = device_sm_count(&num_sms); rc != PLX_OK) return rc;
        const long long n_ctas = static_cast<long long>(kp.B) * kp.Hkv * kp.num_splits;
        const bool two_stage = kp.chunk_len <= 2 * kChunkGranule || n_ctas >= 3LL * num_sms;
        if (D == 128) {
            if (two_stage) {
                if (G == 1) return launch_main<128, 1, 2, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
                if (G == 2) return launch_main<128, 2, 2, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
            }
            if (G == 1) return launch_main<128, 1, PLX_STAGES_FP8, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
            if (G == 2) return launch_main<128, 2, PLX_STAGES_FP8, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
            if (G == 3) return launch_main<128, 3, PLX_STAGES_FP8, 2, true>(tmK, tmV, kp, stream);
            if (G == 4) return launch_main<128, 4, PLX_STAGES_FP8, 2, true>(tmK, tmV, kp, stream);
            if (G == 5) return launch_main<128, 5, PLX_STAGES_FP8, 2, true>(tmK, tmV, kp, stream);
            if (G == 6) return launch_main<128, 6, PLX_STAGES_FP8, 2, true>(tmK, tmV, kp, stream);
            if (G == 7) return launch_main<128, 7, PLX_STAGES_FP8, 2, true>(tmK, tmV, kp, stream);
            if (G == 8) return launch_main<128, 8, PLX_STAGES_FP8, 2, true>(tmK, tmV, kp, stream);
        } else if (D == 64) {
            if (G == 1) return launch_main<64, 1, PLX_STAGES_FP8, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
            if (G == 2) return launch_main<64, 2, PLX_STAGES_FP8, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
            if (G == 3) return launch_main<64, 3, PLX_STAGES_FP8, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
            if (G == 4) return launch_main<64, 4, PLX_STAGES_FP8, kCtasPerSmFp8, true>(tmK, tmV, kp, stream);
            if (G == 5) return launch_main<64, 5, PLX_STAGES_FP8, 3, true>(tmK, tmV, kp, stream);
            if (G == 6) return launch_main<64, 6, PLX_STAGES_FP8, 3, true>(tmK, tmV, kp, stream);
            if (G == 7) return launch_main<64, 7, PLX_STAGES_FP8, 3, true>(tmK, tmV, kp, stream);
            if (G == 8) return launch_main<64, 8, PLX_STAGES_FP8, 3, true>(tmK, tmV, kp, stream);
        }
        return PLX_ERR_UNSUPPORTED;
    }
    // D = 128: 8 KiB stages, three per warp, two CTAs per SM (192 KiB of K/V in flight per SM).  A chunk
    // of at most 128 keys gives every warp at most two tiles: a two-stage ring then holds everything,
    // and at 64 KiB a third CTA fits on the SM, which hides more of the fixed per-CTA latency of
    // huge-batch, short-context calls.
    // D = 64: stages are 4 KiB and a CTA's fixed latency weighs twice as much per byte, so four CTAs
    // share an SM (at most 128 registers per thread).  When the grid fills the device (three or more
    // CTAs per SM) two stages per warp measured fastest (128 KiB in flight per SM: deeper rings only
    // lengthen the memory queues); smaller grids keep three stages, each CTA then needs more in flight.
    const long long ctas = static_cast<long long>(kp.B) * kp.Hkv * kp.num_splits;
    // Five to eight heads per CTA keep two accumulator sets (64 registers per lane at D = 128, 32 at D = 64):
    // about 220 / 152 registers per thread, i.e. two CTAs per SM at D = 128 and three at D = 64.
#define PLX_LAUNCH_G(DD, ST, CT, CT_BIG)                                                     \
    switch (G) {                                                                             \
        case 1: return launch_main<DD, 1, ST, CT>(tmK, tmV, kp, stream);                     \
        case 2: return launch_main<DD, 2, ST, CT>(tmK, tmV, kp, stream);                     \
        case 3: return launch_main<DD, 3, ST, CT>(tmK, tmV, kp, stream);                     \
        case 4: return launch_main<DD, 4, ST, CT>(tmK, tmV, kp, stream);                     \
        case 5: return launch_main<DD, 5, ST, CT_BIG>(tmK, tmV, kp, stream);                 \
        case 6: return launch_main<DD, 6, ST, CT_BIG>(tmK, tmV, kp, stream);                 \
        case 7: return launch_main<DD, 7, ST, CT_BIG>(tmK, tmV, kp, stream);                 \
        case 8: return launch_main<DD, 8, ST, CT_BIG>(tmK, tmV, kp, stream);                 \
        default: return PLX_ERR_UNSUPPORTED;                                                 \
    }
    if (D == 128) {
        const bool two_stage = kp.chunk_len <= PLX_TWO_STAGE_MAX_CHUNK;
        if (two_stage) {
            PLX_LAUNCH_G(128, 2, kCtasPerSm, kCtasPerSm)
        }
        PLX_LAUNCH_G(128, PLX_STAGES_D128, kCtasPerSm, kCtasPerSm)
    } else if (D == 64) {
        int num_sms = 0;
        if (int rc = device_sm_count(&num_sms); rc != PLX_OK) return rc;
        const bool two_stage = kp.chunk_len <= 2 * kChunkGranule || ctas >= 3LL * num_sms;
        if (two_stage) {
            PLX_LAUNCH_G(64, 2, PLX_CTAS_PER_SM_D64, 3)
        }
        PLX_LAUNCH_G(64, PLX_STAGES_D64, PLX_CTAS_PER_SM_D64, 3)
    }
#undef PLX_LAUNCH_G
    return PLX_ERR_UNSUPPORTED;
}

int launch_combine(const float* partials, const int32_t* split_counts, const int32_t* seqlens, int chunk_len,
                   int T_max, void* out, int B, int Hq, int D, int num_splits, int out_dtype, cudaStream_t stream,
                   int num_groups = 1, bool dependent_launch = false)
{
    PlxNvtxRange nvtx_range("plx_decode_combine");
    const size_t group_stride = static_cast<size_t>(B) * Hq * num_splits * (2 * D + 4);
    const unsigned rows = static_cast<unsigned>(B * Hq);
    if (dependent_launch) {
        if (D != 64 && D != 128) return PLX_ERR_UNSUPPORTED;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(rows, 1, 1);
        cfg.blockDim = dim3(kCombineWarps * 32, 1, 1);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t e =
            D == 128 ? cudaLaunchKernelEx(&cfg, plx_combine_kernel<128>, partials, split_counts, seqlens, chunk_len, T_max, out,
                                          Hq, num_splits, out_dtype, num_groups, group_stride)
                     : cudaLaunchKernelEx(&cfg, plx_combine_kernel<64>, partials, split_counts, seqlens, chunk_len, T_max, out,
                                          Hq, num_splits, out_dtype, num_groups, group_stride);
        return e == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
    }
    if (D == 128)
        plx_combine_kernel<128><<<rows, kCombineWarps * 32, 0, stream>>>(partials, split_counts, seqlens, chunk_len, T_max,
                                                               out, Hq, num_splits, out_dtype, num_groups, group_stride);
    else if (D == 64)
        plx_combine_kernel<64><<<rows, kCombineWarps * 32, 0, stream>>>(partials, split_counts, seqlens, chunk_len, T_max,
                                                              out, Hq, num_splits, out_dtype, num_groups, group_stride);
    else
        return PLX_ERR_UNSUPPORTED;
    return cudaGetLastError() == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}

int check_inputs(const void* q, const void* r, const void* k, const void* v, int B, int Hq, int Hkv, int D,
                 int T_max)
{
    if (!q || !r || !k || !v) return PLX_ERR_NULL_POINTER;
    if (!shape_ok(B, Hq, Hkv, D) || T_max <= 0) return PLX_ERR_BAD_SHAPE;
    if (!shape_supported(Hq, Hkv, D)) return PLX_ERR_UNSUPPORTED;
    if (static_cast<long long>(B) * Hkv * T_max >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    if (static_cast<long long>(B) * Hkv > 0x7fffffffLL) return PLX_ERR_BAD_SHAPE;
    if (!aligned(q, 4) || !aligned(r, 4) || !aligned(k, 16) || !aligned(v, 16)) return PLX_ERR_ALIGNMENT;
    return PLX_OK;
}

struct Layout {
    bool set = false;
    int T_max = 0;
    int out_dtype = PLX_OUT_BF16;
    void* workspace = nullptr;
    size_t workspace_bytes = 0;
};
Layout g_layout;
std::mutex g_layout_mutex;

}  // namespace

// ---------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------
// Merge launched as a programmatic dependent of the previous kernel in the stream (the split-KV multi-token
// forward, whose CTAs signal early): its launch latency hides behind that kernel.  Internal to the library.
int plx_combine_after_producer(const float* partials, void* out, int rows, int D, int num_splits, int out_dtype,
                               cudaStream_t stream)
{
    if (!partials || !out || rows <= 0 || num_splits <= 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    if (num_splits <= kRowCombineMaxSplits && rows >= 1024 && (D == 64 || D == 128)) {  // many rows, few records each
        PlxNvtxRange nvtx_range("plx_decode_combine(rows)");
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>((rows + kRowCombineWarps - 1) / kRowCombineWarps), 1, 1);
        cfg.blockDim = dim3(kRowCombineWarps * 32, 1, 1);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t e = D == 128 ? cudaLaunchKernelEx(&cfg, plx_combine_rows_kernel<128>, partials, out, rows, num_splits, out_dtype)
                                       : cudaLaunchKernelEx(&cfg, plx_combine_rows_kernel<64>, partials, out, rows, num_splits, out_dtype);
        return e == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
    }
    return launch_combine(partials, nullptr, nullptr, 0, 0, out, 1, rows, D, num_splits, out_dtype, stream, 1, true);
}

// device view of page-locked, device-mapped host memory (nullptr for pageable memory or device pointers)
static void* mapped_host_view(const void* host)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return (attr.type == cudaMemoryTypeHost) ? attr.devicePointer : nullptr;
}

extern "C" {

int parallax_version(void) { return 110; }

const char* parallax_status_string(int status)
{
    switch (status) {
        case PLX_OK: return "ok";
        case PLX_ERR_NULL_POINTER: return "null pointer argument";
        case PLX_ERR_BAD_SHAPE: return "invalid shape or size";
        case PLX_ERR_UNSUPPORTED: return "unsupported head dimension or GQA group size";
        case PLX_ERR_ALIGNMENT: return "misaligned pointer";
        case PLX_ERR_WORKSPACE: return "workspace missing or too small";
        case PLX_ERR_NEED_LAYOUT: return "parallax_set_layout has not been called";
        case PLX_ERR_CUDA: return "CUDA runtime or driver call failed";
        case PLX_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        case PLX_ERR_STATIC_SCRATCH: return "requested splits need more scratch than the built-in static array holds";
        case PLX_ERR_DEVICE_CHECK: return "debug build: a kernel refused an out-of-range index";
        default: return "unknown status";
    }
}

int parallax_partial_stride(int D) { return D > 0 ? 2 * D + 4 : 0; }

size_t parallax_decode_workspace_bytes(int B, int Hq, int D, int max_splits)
{
    if (B <= 0 || Hq <= 0 || D <= 0 || max_splits <= 0 || max_splits > PLX_MAX_SPLITS) return 0;
    return fixed_bytes(B, Hq, D) + partial_bytes(B, Hq, D, max_splits);
}

int parallax_decode_plan(int B, int Hq, int Hkv, int D, int T_max, int num_sms, int has_seqlens, int* chunk_len,
                         int* num_splits)
{
    if (!chunk_len || !num_splits) return PLX_ERR_NULL_POINTER;
    if (!shape_ok(B, Hq, Hkv, D) || T_max <= 0 || num_sms <= 0) return PLX_ERR_BAD_SHAPE;
    plan_splits(B, virtual_kv_heads(Hq, Hkv), D, T_max, num_sms, has_seqlens != 0, chunk_len, num_splits, false,
                heads_per_cta(Hq, Hkv));
    return PLX_OK;
}

int parallax_decode_splitkv_partial(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                    const int32_t* seqlens, float* partials, int B, int Hq, int Hkv, int D,
                                    int T_max, float scale, int chunk_len, int num_splits, int32_t* status,
                                    void* stream)
{
    int rc = check_inputs(q, r, k_cache, v_cache, B, Hq, Hkv, D, T_max);
    if (rc != PLX_OK) return rc;
    if (!partials) return PLX_ERR_NULL_POINTER;
    if (!aligned(partials, 16)) return PLX_ERR_ALIGNMENT;
    if (chunk_len <= 0 || chunk_len % kTileKeys != 0 || num_splits <= 0 || num_splits > PLX_MAX_SPLITS ||
        static_cast<long long>(chunk_len) * num_splits < T_max)
        return PLX_ERR_BAD_SHAPE;
    CUtensorMap tmK, tmV;
    const uint64_t rows = static_cast<uint64_t>(B) * Hkv * T_max;
    if ((rc = make_tensor_map_2d(&tmK, k_cache, D, rows, kTileKeys, PLX_L2_PROMOTION)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmV, v_cache, D, rows, kTileKeys, PLX_L2_PROMOTION)) != PLX_OK) return rc;
    KernelParams kp{static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(r), seqlens, nullptr,
                    partials, status, nullptr, nullptr, 0, 0, B, Hq, Hkv, T_max, chunk_len, num_splits, scale * kLog2e, PLX_OUT_F32,
                    kModePartialWriteEmpty};
    kp.kv_rows = static_cast<long long>(rows);
    kp.partial_records = static_cast<long long>(B) * Hq * num_splits;
    const int g = apply_group(&kp, Hq, Hkv);
    return dispatch_main(D, g, tmK, tmV, kp, static_cast<cudaStream_t>(stream));
}

int parallax_decode_combine(const float* partials, const int32_t* split_counts, void* out, int B, int Hq, int D,
                            int num_splits, int out_dtype, void* stream)
{
    if (!partials || !out) return PLX_ERR_NULL_POINTER;
    if (B <= 0 || Hq <= 0 || num_splits <= 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return PLX_ERR_UNSUPPORTED;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (!aligned(partials, 16) || !aligned(out, 4)) return PLX_ERR_ALIGNMENT;
    return launch_combine(partials, split_counts, nullptr, 0, 0, out, B, Hq, D, num_splits, out_dtype,
                          static_cast<cudaStream_t>(stream));
}

// Shared body of the contiguous and the paged forward.  For a paged cache T_max = max_pages * page_size
// and `kv_rows` = num_pages * Hkv * page_size rows in each pool.
static int decode_fwd_impl(const void* q, const void* r, const void* k_cache, const void* v_cache,
                           const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int T_max,
                           float scale, int out_dtype, void* workspace, size_t workspace_bytes, int num_splits,
                           void* stream, const int32_t* block_table, int page_size, int max_pages, uint64_t kv_rows,
                           bool fp8 = false, float k_scale = 1.0f, float v_scale = 1.0f, bool dependent_launch = false,
                           const float* k_scales = nullptr, const float* v_scales = nullptr, int lq = 1,
                           bool qr_staged = false)
{
    int rc = check_inputs(q, r, k_cache, v_cache, B, Hq, Hkv, D, T_max);
    if (rc != PLX_OK) return rc;
    if (!out) return PLX_ERR_NULL_POINTER;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (num_splits < 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    if (!aligned(out, 4) || (workspace && !aligned(workspace, 16))) return PLX_ERR_ALIGNMENT;

    int chunk_len = 0, ns = 0;
    if (num_splits == 0) {
        int sms = 0;
        if ((rc = device_sm_count(&sms)) != PLX_OK) return rc;
        plan_splits(B, virtual_kv_heads(Hq, Hkv), D, T_max, sms, seqlens != nullptr, &chunk_len, &ns, fp8, heads_per_cta(Hq, Hkv));
        // never plan beyond what the caller's workspace can hold
        if (ns > 1) {
            const size_t fixed = fixed_bytes(B, Hq, D);
            while (ns > 1 && (!workspace || workspace_bytes < fixed + partial_bytes(B, Hq, D, ns))) {
                --ns;
                chunk_len = static_cast<int>(align_up((T_max + ns - 1) / ns, kChunkGranule));
                ns = (T_max + chunk_len - 1) / chunk_len;
            }
        }
    } else {
        chunk_len = static_cast<int>(align_up((T_max + num_splits - 1) / num_splits, kChunkGranule));
        ns = (T_max + chunk_len - 1) / chunk_len;
    }

    float* partials = nullptr;
    if (ns > 1) {
        const size_t fixed = fixed_bytes(B, Hq, D);
        if (!workspace || workspace_bytes < fixed + partial_bytes(B, Hq, D, ns)) return PLX_ERR_WORKSPACE;
        partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + fixed);
    }
    int32_t* status = (workspace && workspace_bytes >= kHeaderBytes) ? static_cast<int32_t*>(workspace) : nullptr;

    CUtensorMap tmK, tmV;
    const uint64_t rows = block_table ? kv_rows : static_cast<uint64_t>(B) * Hkv * T_max;
    // an e4m3 row of D bytes is described as D/2 16-bit elements: same bytes, same swizzle
    const int map_cols = fp8 ? D / 2 : D;
    if ((rc = make_tensor_map_2d(&tmK, k_cache, map_cols, rows, kTileKeys, PLX_L2_PROMOTION)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmV, v_cache, map_cols, rows, kTileKeys, PLX_L2_PROMOTION)) != PLX_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* counters = ns > 1 ? reinterpret_cast<int32_t*>(static_cast<uint8_t*>(workspace) + kHeaderBytes) : nullptr;
    KernelParams kp{static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(r), seqlens, out,
                    partials, status, counters, block_table, page_size, max_pages, B, Hq, Hkv, T_max, chunk_len, ns, scale * kLog2e, out_dtype,
                    ns > 1 ? kModeFused : kModeFinal};
    if (fp8 && k_scales) {
        kp.k_scales = k_scales;
        kp.v_scales = v_scales;
    } else if (fp8) {
        kp.scale_log2e *= k_scale;
        kp.probe_scale = k_scale;
        kp.v_scale = v_scale;
    }
    kp.dependent_launch = dependent_launch ? 1 : 0;
    kp.lq = lq;
    kp.qr_staged = qr_staged ? 1 : 0;
    const int max_g = 8;
    kp.kv_rows = static_cast<long long>(rows);
    if (partials)
        kp.partial_records = static_cast<long long>((workspace_bytes - fixed_bytes(B, Hq, D)) / ((2 * D + 4) * sizeof(float)));
    const int g = apply_group(&kp, Hq, Hkv, max_g);
    return dispatch_main(D, g, tmK, tmV, kp, st, fp8);
}

constexpr int kMaxGroupOneCta = 8;  // query heads per KV head one CTA of the decode kernel serves (= PLX_MULTI_TOKEN_DECODE_ROWS)

int parallax_decode_step(const void* q_raw, const void* r_raw, const void* k_raw, const void* v_raw,
                         const void* q_weight, const void* r_weight, const void* k_weight, const int32_t* seqlens,
                         void* q_out, void* r_out, void* k_cache, void* v_cache, void* out, int B, int Hq, int Hkv,
                         int D, int T_max, float eps, float rope_theta, int rope_on_r, float scale, int out_dtype,
                         void* workspace, size_t workspace_bytes, int num_splits, void* stream)
{
    // validate the attention call before anything is launched: the upstream step writes into the cache
    int rc = check_inputs(q_out, r_out, k_cache, v_cache, B, Hq, Hkv, D, T_max);
    if (rc != PLX_OK) return rc;
    if (!out) return PLX_ERR_NULL_POINTER;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (num_splits < 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    if (!aligned(out, 4) || (workspace && !aligned(workspace, 16))) return PLX_ERR_ALIGNMENT;
    if (num_splits > 1) {  // a forced split count needs its records' room (a planned one adapts to the workspace)
        const int chunk = static_cast<int>(align_up((T_max + num_splits - 1) / num_splits, kChunkGranule));
        const int ns_eff = (T_max + chunk - 1) / chunk;
        if (ns_eff > 1 && (!workspace || workspace_bytes < fixed_bytes(B, Hq, D) + partial_bytes(B, Hq, D, ns_eff)))
            return PLX_ERR_WORKSPACE;
    }
    rc = parallax_decode_prepare(q_raw, r_raw, k_raw, v_raw, q_weight, r_weight, k_weight, seqlens, q_out, r_out, k_cache,
                                 v_cache, B, Hq, Hkv, D, T_max, eps, rope_theta, rope_on_r, stream);
    if (rc != PLX_OK) return rc;
    // groups that parallax_decode_fwd_ex hands to the multi-token entry (more than eight heads per KV head, more than four
    // at D = 128) take that route here too, as an ordinary launch behind the upstream kernel
    if (Hq / Hkv > (D == 128 ? 4 : kMaxGroupOneCta))
        return parallax_decode_fwd_ex(q_out, r_out, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, T_max, scale, out_dtype,
                                      workspace, workspace_bytes, num_splits, stream);
    return decode_fwd_impl(q_out, r_out, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, T_max, scale, out_dtype, workspace,
                           workspace_bytes, num_splits, stream, nullptr, 0, 0, 0, false, 1.0f, 1.0f, true);
}

int parallax_decode_fwd_fp8(const void* q, const void* r, const void* k_cache, const void* v_cache,
                            const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int T_max,
                            float scale, float k_scale, float v_scale, int out_dtype, void* workspace,
                            size_t workspace_bytes, int num_splits, void* stream)
{
    if (!(k_scale > 0.0f) || !(v_scale > 0.0f) || isinf(k_scale) || isinf(v_scale)) return PLX_ERR_BAD_SHAPE;
    return decode_fwd_impl(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, T_max, scale, out_dtype, workspace,
                           workspace_bytes, num_splits, stream, nullptr, 0, 0, 0, true, k_scale, v_scale);
}

// Which kernel takes a step of `rows` = (query heads per KV head) x (new tokens) rows per KV head.  Up to eight
// rows one CTA of the decode kernel can serve a KV head.  Five (at D = 64 nine) to 64 rows go to the keys-on-lanes
// tensor-core kernel (rows_kernel_takes below; parallax_decode_fwd_multi decides that before it asks here).
// For what that kernel does not serve (other page sizes, unaligned rows): nine to sixteen rows that split into two CTAs of at
// most eight (10 = 2 x 5, 12, 14, 16) stay on the decode kernel, the rest goes to the row-major tensor-core kernel: measured
// at 10 / 12 / 16 rows, 8 KV heads, decode kernel against the split-KV tensor-core kernel: 64 x 8192 keys 505 / 525 /
// 533 us against 728 / 754 / 795; 12 x 8192 100 / 101 / 108 against 170 / 173 / 173; 8 x 8192 72 / 72 / 78 against
// 103 / 103 / 95; 4 x 16384 72 / 72 / 79 against 93 / 93 / 103; 2 x 131072 291 / 298 / 332 against 322 / 376 / 366;
// 1 x 32768 47 / 48 / 54 against 50 / 50 / 50 (the one cell it loses, by 7 %).  From 24 rows on the tensor-core kernel
// is faster or equal everywhere.
#ifndef PLX_MULTI_TOKEN_DECODE_ROWS
#define PLX_MULTI_TOKEN_DECODE_ROWS 8
#endif
constexpr int kMultiTokenDecodeRows = PLX_MULTI_TOKEN_DECODE_ROWS;
constexpr int kTwoCtaDecodeRows = 16;
// rows per KV head above which a multi-token step goes to the keys-on-lanes tensor-core kernel
static_assert(kMaxGroupOneCta == kMultiTokenDecodeRows, "parallax_decode_step mirrors the routing of parallax_decode_fwd_ex");
static int rows_kernel_from(int D) { return D == 128 ? 4 : kMultiTokenDecodeRows; }
// Does a step of this shape go to the keys-on-lanes kernel (given that it supports the shape)?  page_size 0: contiguous.
// 33 to 64 rows per KV head run there as two parts that share their K/V through L2: at D = 128 that beats the row-major
// kernel everywhere measured (64 x 8192 keys 676-694 -> 539 us, 128 x 2048 333 -> 292, 16 x 8192 169 -> 146-156,
// 2 x 131072 316-323 -> 280, 1 x 32768 56 -> 46); at D = 64 only long contexts on many sequences (64 x 8192 500 -> 422 us;
// 128 x 2048, 16 x 8192 and 2 x 131072 lose 3-5 %).
static bool rows_kernel_takes(int B, int Hq, int Hkv, int D, int Lq, int T_max, int page_size)
{
    const long long rows = static_cast<long long>(Hq / Hkv) * Lq;
    const int from = (page_size == 0 || page_size >= 64) ? rows_kernel_from(D) : kMultiTokenDecodeRows;
    if (rows <= from || !plx_decode_rows_supported(Hq, Hkv, D, Lq)) return false;
    if (page_size != 0 && !plx_decode_rows_page_size_ok(page_size)) return false;
    if (rows <= 32 || D == 128) return true;
    int sms = 0;
    if (device_sm_count(&sms) != PLX_OK) return false;
    return T_max >= 32 * 128 && 2LL * B * Hkv >= 3LL * sms;
}
// The word of a decode workspace's header from which the CTAs of the multi-token tensor-core kernel draw their items
// (zero between calls, like the status word in front of it).
static int32_t* rows_ticket(void* workspace, size_t workspace_bytes)
{
    return (workspace && workspace_bytes >= kHeaderBytes) ? static_cast<int32_t*>(workspace) + 4 : nullptr;
}

// The part of a decode workspace that holds split records (after the status word, counters and staging).
static void records_region(void* workspace, size_t workspace_bytes, int B, int rows, int D, void** rec, size_t* rec_bytes)
{
    const size_t fixed = fixed_bytes(B, rows, D);
    *rec = (workspace && workspace_bytes > fixed) ? static_cast<uint8_t*>(workspace) + fixed : nullptr;
    *rec_bytes = *rec ? workspace_bytes - fixed : 0;
}
static bool use_tensor_core_kernel(const void* q, const void* r, const void* out, int B, int Hq, int Hkv, int Lq, int D)
{
    const long long rows = static_cast<long long>(Hq / Hkv) * Lq;
    const bool can = aligned(q, 16) && aligned(r, 16) && aligned(out, 16) && (D == 64 || D == 128);
    if (rows > 64) return true;
    if (!can || rows <= kMultiTokenDecodeRows) return false;
    (void)B;
    if (rows <= kTwoCtaDecodeRows) {
        int g = 1, kv_div = 1;
        split_group(static_cast<int>(rows), &g, &kv_div);
        if (kv_div <= 2) return false;
    }
    return true;
}

int parallax_decode_fwd_multi(const void* q, const void* r, const void* k_cache, const void* v_cache,
                              const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq, int T_max,
                              float scale, int out_dtype, void* workspace, size_t workspace_bytes, int num_splits,
                              void* stream)
{
    if (Lq <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || B <= 0) return PLX_ERR_BAD_SHAPE;
    if (workspace && !aligned(workspace, 16)) return PLX_ERR_ALIGNMENT;
    // Up to 64 rows per KV head: the tensor-core kernel with the keys on the accumulator lanes, whose work
    // follows the rows present.  Measured against the routes below (D = 128, 8 KV heads, 10 / 16 / 24 / 32 rows, us per step):
    // 64 x 8192 keys 342 / 350 / 375 / 388 against 474 / 506 / 722 / 766; 16 x 8192 90 / 87 / 91 / 91 against 146 / 154 /
    // 182 / 182; 8 x 8192 53 / 53 / 57 / 58 against 80 / 87 / 116 / 107; 2 x 131072 167 / 169 / 172 / 172 against 323 / 334 /
    // 339 / 339; 1 x 32768 37 / 37 / 39 / 39 against 52 / 59 / 57 / 58.  (Up to eight rows the decode kernel stays ahead
    // or level at large batches: 64 x 8192, 2 / 4 / 8 rows: 298 / 300 / 314 against 324 / 329 / 340.)  At D = 64, same
    // shapes, 16 / 32 rows: 64 x 8192 222 / 308 against 309 / 570; 2 x 131072 98 / 132 against 152 / 267.
    // Since that kernel walks its items, merges with a warp per row and plans its splits by a step model, it is also
    // ahead from five rows on at D = 128 (6 / 8 rows, decode kernel against it: 128 x 2048 167 / 168 against 159 / 159;
    // 32 x 8192 164 / 166 against 154 / 155; 16 x 8192 90 / 92 against 82 / 82; 64 x 8192 and 2 x 131072 level; at four
    // rows the decode kernel leads by 1-10 %); at D = 64 the decode kernel keeps everything up to eight rows (8 rows:
    // 128 x 512 35 against 46, 8 x 8192 30 against 33, 64 x 8192 183 against 178).
    if (rows_kernel_takes(B, Hq, Hkv, D, Lq, T_max, 0) &&
        aligned(q, 16) && aligned(r, 16) && aligned(out, 16) && aligned(k_cache, 16) && aligned(v_cache, 16)) {
        void* rec = nullptr;
        size_t rec_bytes = 0;
        records_region(workspace, workspace_bytes, B, Hq * Lq, D, &rec, &rec_bytes);
        int32_t* status = (workspace && workspace_bytes >= kHeaderBytes) ? static_cast<int32_t*>(workspace) : nullptr;
        return plx_decode_rows_fwd(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, Lq, T_max, scale, out_dtype, rec,
                                   rec_bytes, rec ? num_splits : (num_splits > 1 ? 1 : num_splits), status,
                                   static_cast<cudaStream_t>(stream), nullptr, 0, 0, 0, rows_ticket(workspace, workspace_bytes));
    }
    if (use_tensor_core_kernel(q, r, out, B, Hq, Hkv, Lq, D)) {
        void* rec = nullptr;
        size_t rec_bytes = 0;
        records_region(workspace, workspace_bytes, B, Hq * Lq, D, &rec, &rec_bytes);
        int32_t* status = (workspace && workspace_bytes >= kHeaderBytes) ? static_cast<int32_t*>(workspace) : nullptr;
        return parallax_prefill_fwd_ex(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, Lq, T_max, scale, out_dtype,
                                       PLX_P_BF16_RESIDUAL, rec, rec_bytes, rec ? num_splits : (num_splits > 1 ? 1 : num_splits),
                                       status, stream);
    }
    // token i of query head h is row h * Lq + i of a sequence: a decode call with Hq * Lq query heads whose
    // rows differ only in how many of the last Lq - 1 keys they see
    return decode_fwd_impl(q, r, k_cache, v_cache, seqlens, out, B, Hq * Lq, Hkv, D, T_max, scale, out_dtype, workspace,
                           workspace_bytes, num_splits, stream, nullptr, 0, 0, 0, false, 1.0f, 1.0f, false, nullptr,
                           nullptr, Lq);
}

int parallax_decode_fwd_fp8_per_head(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                     const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int T_max,
                                     float scale, const float* k_scales, const float* v_scales, int out_dtype,
                                     void* workspace, size_t workspace_bytes, int num_splits, void* stream)
{
    if (!k_scales || !v_scales) return PLX_ERR_NULL_POINTER;
    if (!aligned(k_scales, 4) || !aligned(v_scales, 4)) return PLX_ERR_ALIGNMENT;
    return decode_fwd_impl(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, T_max, scale, out_dtype, workspace,
                           workspace_bytes, num_splits, stream, nullptr, 0, 0, 0, true, 1.0f, 1.0f, false, k_scales,
                           v_scales);
}

int parallax_decode_combine_gathered(const float* partials, void* out, int B, int Hq, int D, int num_ranks,
                                     int num_splits, int out_dtype, void* stream)
{
    if (!partials || !out) return PLX_ERR_NULL_POINTER;
    if (B <= 0 || Hq <= 0 || num_ranks <= 0 || num_splits <= 0 ||
        static_cast<long long>(num_ranks) * num_splits > PLX_MAX_SPLITS)
        return PLX_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return PLX_ERR_UNSUPPORTED;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (!aligned(partials, 16) || !aligned(out, 4)) return PLX_ERR_ALIGNMENT;
    if (num_ranks == 1)
        return launch_combine(partials, nullptr, nullptr, 0, 0, out, B, Hq, D, num_splits, out_dtype,
                              static_cast<cudaStream_t>(stream));
    return launch_combine(partials, nullptr, nullptr, 0, 0, out, B, Hq, D, num_splits, out_dtype,
                          static_cast<cudaStream_t>(stream), num_ranks);
}

int parallax_decode_fwd_ex(const void* q, const void* r, const void* k_cache, const void* v_cache,
                           const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int T_max,
                           float scale, int out_dtype, void* workspace, size_t workspace_bytes, int num_splits,
                           void* stream)
{
    // more than eight query heads per KV head (multi-query models; more than four at D = 128, where the keys-on-lanes
    // kernel is ahead from five rows on): the one-token step of the multi-token entry
    if (Hq > 0 && Hkv > 0 && Hq % Hkv == 0 && Hq / Hkv > rows_kernel_from(D))
        return parallax_decode_fwd_multi(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, 1, T_max, scale, out_dtype,
                                         workspace, workspace_bytes, num_splits, stream);
    return decode_fwd_impl(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, T_max, scale, out_dtype, workspace,
                           workspace_bytes, num_splits, stream, nullptr, 0, 0, 0);
}

int parallax_decode_fwd_paged(const void* q, const void* r, const void* k_pages, const void* v_pages,
                              const int32_t* block_table, const int32_t* seqlens, void* out, int B, int Hq, int Hkv,
                              int D, int num_pages, int page_size, int max_pages_per_seq, float scale, int out_dtype,
                              void* workspace, size_t workspace_bytes, int num_splits, void* stream)
{
    if (!block_table) return PLX_ERR_NULL_POINTER;
    if (Hq > 0 && Hkv > 0 && Hq % Hkv == 0 && Hq / Hkv > (page_size >= 64 ? rows_kernel_from(D) : kMultiTokenDecodeRows))  // as in parallax_decode_fwd_ex
        return parallax_decode_fwd_multi_paged(q, r, k_pages, v_pages, block_table, seqlens, out, B, Hq, Hkv, D, 1,
                                               num_pages, page_size, max_pages_per_seq, scale, out_dtype, workspace,
                                               workspace_bytes, num_splits, stream);
    if (num_pages <= 0 || page_size <= 0 || page_size % kTileKeys != 0 || max_pages_per_seq <= 0)
        return PLX_ERR_BAD_SHAPE;
    const long long T_max = static_cast<long long>(page_size) * max_pages_per_seq;
    const long long pool_rows = static_cast<long long>(num_pages) * (Hkv > 0 ? Hkv : 1) * page_size;
    if (T_max >= (1LL << 31) - 65536 || pool_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    return decode_fwd_impl(q, r, k_pages, v_pages, seqlens, out, B, Hq, Hkv, D, static_cast<int>(T_max), scale,
                           out_dtype, workspace, workspace_bytes, num_splits, stream, block_table, page_size,
                           max_pages_per_seq, static_cast<uint64_t>(pool_rows));
}

int parallax_decode_multi_plan(int B, int Hq, int Hkv, int D, int Lq, int T_max, int page_size, int* kernel,
                               int* num_splits)
{
    if (!kernel || !num_splits) return PLX_ERR_NULL_POINTER;
    if (Lq <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || B <= 0 || T_max <= 0 || page_size < 0) return PLX_ERR_BAD_SHAPE;
    const void* const aligned_ptr = reinterpret_cast<const void*>(static_cast<uintptr_t>(256));
    *kernel = PLX_MULTI_KERNEL_DECODE;
    *num_splits = 0;
    if (rows_kernel_takes(B, Hq, Hkv, D, Lq, T_max, page_size)) {
        int sms = 0;
        if (int rc = device_sm_count(&sms); rc != PLX_OK) return rc;
        *kernel = PLX_MULTI_KERNEL_ROWS;
        *num_splits = plx_decode_rows_plan(B, Hq, Hkv, D, Lq, T_max, page_size, sms);
    } else if ((page_size == 0 || page_size % 64 == 0) && use_tensor_core_kernel(aligned_ptr, aligned_ptr, aligned_ptr, B, Hq, Hkv, Lq, D)) {
        *kernel = PLX_MULTI_KERNEL_ROW_MAJOR;
    }
    return PLX_OK;
}

int parallax_decode_fwd_multi_paged(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                    const int32_t* block_table, const int32_t* seqlens, void* out, int B, int Hq,
                                    int Hkv, int D, int Lq, int num_pages, int page_size, int max_pages_per_seq,
                                    float scale, int out_dtype, void* workspace, size_t workspace_bytes, int num_splits,
                                    void* stream)
{
    if (!block_table) return PLX_ERR_NULL_POINTER;
    if (Lq <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || B <= 0) return PLX_ERR_BAD_SHAPE;
    if (workspace && !aligned(workspace, 16)) return PLX_ERR_ALIGNMENT;
    if (num_pages <= 0 || page_size <= 0 || page_size % kTileKeys != 0 || max_pages_per_seq <= 0)
        return PLX_ERR_BAD_SHAPE;
    // (small pages cost that kernel's producer sixteen or eight copies per tile: the earlier start only from 64-key pages on)
    if (rows_kernel_takes(B, Hq, Hkv, D, Lq,
                          static_cast<int>(std::min<long long>(static_cast<long long>(page_size) * max_pages_per_seq, 0x7fffffff)),
                          page_size) &&
        aligned(q, 16) && aligned(r, 16) && aligned(out, 16) && aligned(k_pages, 16) &&
        aligned(v_pages, 16)) {  // as in parallax_decode_fwd_multi
        const long long T_cap = static_cast<long long>(page_size) * max_pages_per_seq;
        const long long pool = static_cast<long long>(num_pages) * Hkv * page_size;
        if (T_cap >= (1LL << 31) - 65536 || pool >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
        void* rec = nullptr;
        size_t rec_bytes = 0;
        records_region(workspace, workspace_bytes, B, Hq * Lq, D, &rec, &rec_bytes);
        int32_t* status = (workspace && workspace_bytes >= kHeaderBytes) ? static_cast<int32_t*>(workspace) : nullptr;
        return plx_decode_rows_fwd(q, r, k_pages, v_pages, seqlens, out, B, Hq, Hkv, D, Lq, static_cast<int>(T_cap), scale,
                                   out_dtype, rec, rec_bytes, rec ? num_splits : (num_splits > 1 ? 1 : num_splits), status,
                                   static_cast<cudaStream_t>(stream), block_table, page_size, max_pages_per_seq, pool,
                                   rows_ticket(workspace, workspace_bytes));
    }
    if (page_size % 64 == 0 && use_tensor_core_kernel(q, r, out, B, Hq, Hkv, Lq, D)) {  // that kernel walks 64-key tiles
        void* rec = nullptr;
        size_t rec_bytes = 0;
        records_region(workspace, workspace_bytes, B, Hq * Lq, D, &rec, &rec_bytes);
        int32_t* status = (workspace && workspace_bytes >= kHeaderBytes) ? static_cast<int32_t*>(workspace) : nullptr;
        return parallax_prefill_fwd_paged_ex(q, r, k_pages, v_pages, block_table, seqlens, out, B, Hq, Hkv, D, Lq, num_pages,
                                             page_size, max_pages_per_seq, scale, out_dtype, PLX_P_BF16_RESIDUAL, rec,
                                             rec_bytes, rec ? num_splits : (num_splits > 1 ? 1 : num_splits), status,
                                             stream);
    }
    if (static_cast<long long>(Hq) * Lq > 64LL * Hkv) return PLX_ERR_UNSUPPORTED;
    const long long T_max = static_cast<long long>(page_size) * max_pages_per_seq;
    const long long pool_rows = static_cast<long long>(num_pages) * Hkv * page_size;
    if (T_max >= (1LL << 31) - 65536 || pool_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    return decode_fwd_impl(q, r, k_pages, v_pages, seqlens, out, B, Hq * Lq, Hkv, D, static_cast<int>(T_max), scale,
                           out_dtype, workspace, workspace_bytes, num_splits, stream, block_table, page_size,
                           max_pages_per_seq, static_cast<uint64_t>(pool_rows), false, 1.0f, 1.0f, false, nullptr, nullptr,
                           Lq);
}

int parallax_decode_fwd_paged_fp8(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                  const int32_t* block_table, const int32_t* seqlens, void* out, int B, int Hq,
                                  int Hkv, int D, int num_pages, int page_size, int max_pages_per_seq, float scale,
                                  float k_scale, float v_scale, int out_dtype, void* workspace,
                                  size_t workspace_bytes, int num_splits, void* stream)
{
    if (!block_table) return PLX_ERR_NULL_POINTER;
    if (!(k_scale > 0.0f) || !(v_scale > 0.0f) || isinf(k_scale) || isinf(v_scale)) return PLX_ERR_BAD_SHAPE;
    if (num_pages <= 0 || page_size <= 0 || page_size % kTileKeys != 0 || max_pages_per_seq <= 0)
        return PLX_ERR_BAD_SHAPE;
    const long long T_max = static_cast<long long>(page_size) * max_pages_per_seq;
    const long long pool_rows = static_cast<long long>(num_pages) * (Hkv > 0 ? Hkv : 1) * page_size;
    if (T_max >= (1LL << 31) - 65536 || pool_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    return decode_fwd_impl(q, r, k_pages, v_pages, seqlens, out, B, Hq, Hkv, D, static_cast<int>(T_max), scale,
                           out_dtype, workspace, workspace_bytes, num_splits, stream, block_table, page_size,
                           max_pages_per_seq, static_cast<uint64_t>(pool_rows), true, k_scale, v_scale);
}

int parallax_decode_fwd_paged_fp8_per_head(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                           const int32_t* block_table, const int32_t* seqlens, void* out, int B,
                                           int Hq, int Hkv, int D, int num_pages, int page_size,
                                           int max_pages_per_seq, float scale, const float* k_scales,
                                           const float* v_scales, int out_dtype, void* workspace,
                                           size_t workspace_bytes, int num_splits, void* stream)
{
    if (!block_table || !k_scales || !v_scales) return PLX_ERR_NULL_POINTER;
    if (!aligned(k_scales, 4) || !aligned(v_scales, 4)) return PLX_ERR_ALIGNMENT;
    if (num_pages <= 0 || page_size <= 0 || page_size % kTileKeys != 0 || max_pages_per_seq <= 0)
        return PLX_ERR_BAD_SHAPE;
    const long long T_max = static_cast<long long>(page_size) * max_pages_per_seq;
    const long long pool_rows = static_cast<long long>(num_pages) * (Hkv > 0 ? Hkv : 1) * page_size;
    if (T_max >= (1LL << 31) - 65536 || pool_rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
    return decode_fwd_impl(q, r, k_pages, v_pages, seqlens, out, B, Hq, Hkv, D, static_cast<int>(T_max), scale,
                           out_dtype, workspace, workspace_bytes, num_splits, stream, block_table, page_size,
                           max_pages_per_seq, static_cast<uint64_t>(pool_rows), true, 1.0f, 1.0f, false, k_scales,
                           v_scales);
}

int parallax_decode_fwd_args(const parallax_decode_args* args)
{
    if (!args) return PLX_ERR_NULL_POINTER;
    // a caller built against an earlier header passes a shorter struct: the missing tail reads as zeros
    if (args->struct_bytes < offsetof(parallax_decode_args, k_scale) || args->struct_bytes > sizeof(parallax_decode_args))
        return PLX_ERR_BAD_SHAPE;
    parallax_decode_args a;
    memset(&a, 0, sizeof a);
    memcpy(&a, args, args->struct_bytes);
    const int Lq = a.Lq > 0 ? a.Lq : 1;
    if (a.Hq <= 0 || a.Hkv <= 0 || a.Hq % a.Hkv != 0) return PLX_ERR_BAD_SHAPE;
    if (Lq > 1 && static_cast<long long>(a.Hq) * Lq > 64LL * a.Hkv) return PLX_ERR_UNSUPPORTED;
    if (a.kv_dtype != PLX_KV_BF16 && a.kv_dtype != PLX_KV_E4M3) return PLX_ERR_BAD_SHAPE;
    const bool fp8 = a.kv_dtype == PLX_KV_E4M3;
    float ks = 1.0f, vs = 1.0f;
    if (fp8) {
        if ((a.k_scales != nullptr) != (a.v_scales != nullptr)) return PLX_ERR_NULL_POINTER;
        if (a.k_scales) {
            if (!aligned(a.k_scales, 4) || !aligned(a.v_scales, 4)) return PLX_ERR_ALIGNMENT;
        } else {
            ks = a.k_scale;
            vs = a.v_scale;
            if (!(ks > 0.0f) || !(vs > 0.0f) || isinf(ks) || isinf(vs)) return PLX_ERR_BAD_SHAPE;
        }
    }
    long long T_max = a.T_max;
    uint64_t pool_rows = 0;
    if (a.block_table) {
        if (a.num_pages <= 0 || a.page_size <= 0 || a.page_size % kTileKeys != 0 || a.max_pages_per_seq <= 0)
            return PLX_ERR_BAD_SHAPE;
        T_max = static_cast<long long>(a.page_size) * a.max_pages_per_seq;
        const long long rows = static_cast<long long>(a.num_pages) * a.Hkv * a.page_size;
        if (T_max >= (1LL << 31) - 65536 || rows >= (1LL << 31) - 65536) return PLX_ERR_BAD_SHAPE;
        pool_rows = static_cast<uint64_t>(rows);
    }
    return decode_fwd_impl(a.q, a.r, a.k_cache, a.v_cache, a.seqlens, a.out, a.B, a.Hq * Lq, a.Hkv, a.D,
                           static_cast<int>(T_max), a.scale, a.out_dtype, a.workspace, a.workspace_bytes, a.num_splits,
                           a.stream, a.block_table, a.page_size, a.max_pages_per_seq, pool_rows, fp8, ks, vs, false,
                           fp8 ? a.k_scales : nullptr, fp8 ? a.v_scales : nullptr, Lq);
}

int parallax_set_layout(int T_max, int out_dtype, void* workspace, size_t workspace_bytes)
{
    if (T_max <= 0 || (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32)) return PLX_ERR_BAD_SHAPE;
    if (workspace && !aligned(workspace, 16)) return PLX_ERR_ALIGNMENT;
    std::lock_guard<std::mutex> lock(g_layout_mutex);
    g_layout.set = true;
    g_layout.T_max = T_max;
    g_layout.out_dtype = out_dtype;
    g_layout.workspace = workspace;
    g_layout.workspace_bytes = workspace ? workspace_bytes : 0;
    return PLX_OK;
}

int parallax_decode_fwd(const void* q, const void* r, const void* k_cache, const void* v_cache,
                        const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, float scale, void* stream)
{
    Layout lay;
    {
        std::lock_guard<std::mutex> lock(g_layout_mutex);
        lay = g_layout;
    }
    if (!lay.set) return PLX_ERR_NEED_LAYOUT;
    return parallax_decode_fwd_ex(q, r, k_cache, v_cache, seqlens, out, B, Hq, Hkv, D, lay.T_max, scale,
                                  lay.out_dtype, lay.workspace, lay.workspace_bytes, 0, stream);
}

int parallax_decode_fwd_host(const void* q_host, const void* r_host, const void* k_cache, const void* v_cache,
                             const int32_t* seqlens, void* out_host, int B, int Hq, int Hkv, int D, int T_max,
                             float scale, int out_dtype, void* workspace, size_t workspace_bytes, int num_splits,
                             void* stream)
{
    if (!q_host || !r_host || !out_host) return PLX_ERR_NULL_POINTER;
    if (!workspace) return PLX_ERR_WORKSPACE;
    if (!shape_ok(B, Hq, Hkv, D)) return PLX_ERR_BAD_SHAPE;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (!aligned(workspace, 16)) return PLX_ERR_ALIGNMENT;
    const size_t n = static_cast<size_t>(B) * Hq * D;
    if (workspace_bytes < fixed_bytes(B, Hq, D)) return PLX_ERR_WORKSPACE;
    uint8_t* ws = static_cast<uint8_t*>(workspace) + kHeaderBytes + counter_bytes(B, Hq);
    void* q_dev = ws;
    void* r_dev = ws + align_up(n * 2, 256);
    void* out_dev = ws + 2 * align_up(n * 2, 256);
    // Page-locked, device-mapped output memory is written by the kernel itself (posted writes over the host
    // link, complete when the stream has synchronised): no device-to-host copy command, one dependency less
    // on the step's critical path.  Pageable memory goes through the workspace and a copy as before.
    // groups above eight heads per KV head go through parallax_decode_fwd_ex (tensor-core kernel) with staged buffers
    const bool big_group = Hq / Hkv > kMultiTokenDecodeRows;
    bool out_direct = false;
    if (void* view = mapped_host_view(out_host); !big_group && view && aligned(view, 4)) {
        out_dev = view;
        out_direct = true;
    }
    const void* q_view = mapped_host_view(q_host);
    const void* r_view = mapped_host_view(r_host);
    const bool in_direct = !big_group && q_view && r_view && aligned(q_view, 16) && aligned(r_view, 16) && (n * 2) % 16 == 0;
    // validate everything before the first copy is enqueued
    int rc = PLX_OK;
    if (big_group) {  // no limit on the group size on that route
        if (!k_cache || !v_cache) return PLX_ERR_NULL_POINTER;
        if (T_max <= 0) return PLX_ERR_BAD_SHAPE;
        if (D != 64 && D != 128) return PLX_ERR_UNSUPPORTED;
        if (!aligned(k_cache, 16) || !aligned(v_cache, 16)) return PLX_ERR_ALIGNMENT;
    } else if ((rc = check_inputs(q_dev, r_dev, k_cache, v_cache, B, Hq, Hkv, D, T_max)) != PLX_OK) {
        return rc;
    }
    if (num_splits < 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    if (num_splits > 1 && !big_group) {  // a forced split count needs its records' room (a planned one adapts)
        const int chunk = static_cast<int>(align_up((T_max + num_splits - 1) / num_splits, kChunkGranule));
        const int ns_eff = (T_max + chunk - 1) / chunk;
        if (ns_eff > 1 && workspace_bytes < fixed_bytes(B, Hq, D) + partial_bytes(B, Hq, D, ns_eff)) return PLX_ERR_WORKSPACE;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Page-locked, device-mapped q and r are not copied at all: the attention kernel's CTAs fetch their own rows over
    // the host link (16-byte loads into shared memory, once per CTA), so the transfer of a later CTA's rows
    // overlaps the K/V streaming of the earlier ones instead of standing in front of the whole kernel.
    if (!in_direct) {
        if (cudaMemcpyAsync(q_dev, q_host, n * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) return PLX_ERR_CUDA;
        if (cudaMemcpyAsync(r_dev, r_host, n * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) return PLX_ERR_CUDA;
    }
    rc = big_group ? parallax_decode_fwd_ex(q_dev, r_dev, k_cache, v_cache, seqlens, out_dev, B, Hq, Hkv, D, T_max, scale,
                                            out_dtype, workspace, workspace_bytes, num_splits, stream)
                   : decode_fwd_impl(in_direct ? q_view : q_dev, in_direct ? r_view : r_dev, k_cache, v_cache, seqlens, out_dev,
                                     B, Hq, Hkv, D, T_max, scale, out_dtype, workspace, workspace_bytes, num_splits, stream,
                                     nullptr, 0, 0, 0, false, 1.0f, 1.0f, false, nullptr, nullptr, 1, in_direct);
    if (rc != PLX_OK) return rc;
    const size_t out_bytes = n * (out_dtype == PLX_OUT_F32 ? 4 : 2);
    if (!out_direct &&
        cudaMemcpyAsync(out_host, out_dev, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return PLX_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PLX_ERR_CUDA;
    return PLX_OK;
}

#if PLX_TRACE
int plx_trace_read(unsigned long long* host, size_t n)
{
    return cudaMemcpyFromSymbol(host, g_plx_trace, n * sizeof(unsigned long long)) == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}
#endif

int parallax_workspace_status(const void* workspace, int32_t* status_host, void* stream)
{
    if (!workspace || !status_host) return PLX_ERR_NULL_POINTER;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(status_host, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return PLX_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return PLX_ERR_CUDA;
    return PLX_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Allocation-free variant of the decode forward.
//
// Some callers cannot hand the library a workspace because they cannot allocate
// device memory at the point where they decode: code running in a region where
// cudaMalloc is not allowed, plug-ins that live inside a host framework's memory
// pool and are forbidden to allocate behind its back, and real-time loops that
// must not hit the allocator's locks.  For them the split-KV partial records live
// in the fixed array below, which every device that loads this library carries
// until the process exits.  The first call on a device looks the array's address
// up, and the first call of a shape (head dimension, group size) on a device sets
// that kernel's shared-memory attribute: make those calls before any stream capture.
// ---------------------------------------------------------------------------
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[PLX_STATIC_SCRATCH_BYTES];

// The array's name is only a host-side handle here; the device address has to be asked for, once
// per device, with that device current.
int static_scratch_address(float** ptr)
{
    static float* cache[64] = {nullptr};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PLX_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (dev >= 0 && dev < 64 && cache[dev]) {
        *ptr = cache[dev];
        return PLX_OK;
    }
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return PLX_ERR_CUDA;
    if (dev >= 0 && dev < 64) cache[dev] = static_cast<float*>(p);
    *ptr = static_cast<float*>(p);
    return PLX_OK;
}

}  // namespace

extern "C" int parallax_decode_fwd_static(const void* q, const void* r, const void* k_cache, const void* v_cache,
                                          const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D,
                                          int T_max, float scale, int out_dtype, int num_splits, void* stream)
{
    int rc = check_inputs(q, r, k_cache, v_cache, B, Hq, Hkv, D, T_max);
    if (rc != PLX_OK) return rc;
    if (!out) return PLX_ERR_NULL_POINTER;
    if (out_dtype != PLX_OUT_BF16 && out_dtype != PLX_OUT_F32) return PLX_ERR_BAD_SHAPE;
    if (num_splits < 0 || num_splits > PLX_MAX_SPLITS) return PLX_ERR_BAD_SHAPE;
    if (!aligned(out, 4)) return PLX_ERR_ALIGNMENT;

    int chunk_len = 0, ns = 0;
    if (num_splits == 0) {
        int sms = 0;
        if ((rc = device_sm_count(&sms)) != PLX_OK) return rc;
        plan_splits(B, virtual_kv_heads(Hq, Hkv), D, T_max, sms, seqlens != nullptr, &chunk_len, &ns, false, heads_per_cta(Hq, Hkv));
        // the planner may only use as many splits as the fixed array can hold
        while (ns > 1 && partial_bytes(B, Hq, D, ns) > PLX_STATIC_SCRATCH_BYTES) {
            --ns;
            chunk_len = static_cast<int>(align_up((T_max + ns - 1) / ns, kChunkGranule));
            ns = (T_max + chunk_len - 1) / chunk_len;
        }
    } else {
        chunk_len = static_cast<int>(align_up((T_max + num_splits - 1) / num_splits, kChunkGranule));
        ns = (T_max + chunk_len - 1) / chunk_len;
        if (ns > 1 && partial_bytes(B, Hq, D, ns) > PLX_STATIC_SCRATCH_BYTES) return PLX_ERR_STATIC_SCRATCH;
    }

    float* partials = nullptr;
    if (ns > 1 && (rc = static_scratch_address(&partials)) != PLX_OK) return rc;

    CUtensorMap tmK, tmV;
    const uint64_t rows = static_cast<uint64_t>(B) * Hkv * T_max;
    if ((rc = make_tensor_map_2d(&tmK, k_cache, D, rows, kTileKeys, PLX_L2_PROMOTION)) != PLX_OK) return rc;
    if ((rc = make_tensor_map_2d(&tmV, v_cache, D, rows, kTileKeys, PLX_L2_PROMOTION)) != PLX_OK) return rc;

    // Nothing in the array has to start at zero: every record the combine reads was written by
    // this call's split kernel first (records of splits past a context are neither written nor read).
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    KernelParams kp{static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(r), seqlens, out,
                    partials, nullptr, nullptr, nullptr, 0, 0, B, Hq, Hkv, T_max, chunk_len, ns, scale * kLog2e, out_dtype,
                    ns > 1 ? kModePartial : kModeFinal};
    kp.kv_rows = static_cast<long long>(rows);
    kp.partial_records = PLX_STATIC_SCRATCH_BYTES / ((2 * D + 4) * sizeof(float));
    const int g = apply_group(&kp, Hq, Hkv);
    if ((rc = dispatch_main(D, g, tmK, tmV, kp, st)) != PLX_OK) return rc;
    if (ns > 1) rc = launch_combine(partials, nullptr, seqlens, chunk_len, T_max, out, B, Hq, D, ns, out_dtype, st);
    return rc;
}
