// Upstream step of a decode call for B200 (sm_100a): RMSNorm and rotary embedding of the new
// token's q, rho and k, and the append of k, v to the cache (Sec. 4.2 and App. "Backbone
// Architecture": RMSNorm on q, k and rho; RoPE with base theta on q and k, optionally on rho).
// Conventions the paper leaves to its Qwen-3 backbone: x / sqrt(mean(x^2) + eps) * weight over the head
// dimension, then the "rotate half" pairing (element i with i + D/2) at position seqlens[b] - 1.
//
// One CTA per sequence; a warp per head row.  A lane holds elements lane + 32 t, so both members of
// a rotation pair sit in the same thread.  Arithmetic in fp32, the rotation angle reduced in fp64
// (positions reach 10^5, where an fp32 angle is off by ~1e-2 rad); one rounding to bf16 at the end.
// The step moves a few hundred KB: it is launch-bound, not a roofline kernel.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "parallax.h"
#include "plx_common.cuh"

namespace {

constexpr int kPrepWarps = 8;

struct PrepareParams {
    const __nv_bfloat16 *q_raw, *r_raw, *k_raw, *v_raw, *wq, *wr, *wk;
    const int32_t* seqlens;
    __nv_bfloat16 *q_out, *r_out, *k_cache, *v_cache;
    int B, Hq, Hkv, T_max;
    float eps;
    double log2_theta;
    int rope_on_r;
};

template <int D>
__global__ void __launch_bounds__(kPrepWarps * 32) plx_prepare_kernel(const PrepareParams p)
{
    constexpr int NT = D / 32;       // elements per lane
    constexpr int HALF_T = NT / 2;   // element t pairs with t + HALF_T
    __shared__ float s_cos[D / 2], s_sin[D / 2];
    // lets a kernel launched as a programmatic dependent (parallax_decode_step) be scheduled on the idle SMs
    // now; it waits for this grid's completion before it reads anything written here
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int L = p.seqlens ? p.seqlens[b] : p.T_max;
    L = min(L, p.T_max);
    if (L <= 0) return;  // the new token is not in this context: nothing to prepare
    const int pos = L - 1;

    for (int i = threadIdx.x; i < D / 2; i += kPrepWarps * 32) {
        const double inv_freq = exp2(-(2.0 * i / D) * p.log2_theta);
        double s, c;
        sincos(static_cast<double>(pos) * inv_freq, &s, &c);
        s_cos[i] = static_cast<float>(c);
        s_sin[i] = static_cast<float>(s);
    }
    __syncthreads();

    const int rows = 2 * p.Hq + 2 * p.Hkv;  // q rows, rho rows, k rows, v rows
    for (int row = warp; row < rows; row += kPrepWarps) {
        const __nv_bfloat16 *src, *w = nullptr;
        __nv_bfloat16* dst;
        bool rotate = true;
        if (row < p.Hq) {
            const size_t off = (static_cast<size_t>(b) * p.Hq + row) * D;
            src = p.q_raw + off;
            dst = p.q_out + off;
            w = p.wq;
        } else if (row < 2 * p.Hq) {
            const size_t off = (static_cast<size_t>(b) * p.Hq + (row - p.Hq)) * D;
            src = p.r_raw + off;
            dst = p.r_out + off;
            w = p.wr;
            rotate = p.rope_on_r != 0;
        } else {
            const bool is_v = row >= 2 * p.Hq + p.Hkv;
            const int h = row - 2 * p.Hq - (is_v ? p.Hkv : 0);
            src = (is_v ? p.v_raw : p.k_raw) + (static_cast<size_t>(b) * p.Hkv + h) * D;
            dst = (is_v ? p.v_cache : p.k_cache) + ((static_cast<size_t>(b) * p.Hkv + h) * p.T_max + pos) * D;
            w = p.wk;
            if (is_v) {  // values are appended unchanged
#pragma unroll
                for (int t = 0; t < NT; ++t) dst[lane + 32 * t] = src[lane + 32 * t];
                continue;
            }
        }
        float x[NT];
        float ss = 0.0f;
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            x[t] = __bfloat162float(src[lane + 32 * t]);
            ss += x[t] * x[t];
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        const float rinv = 1.0f / sqrtf(ss / D + p.eps);
#pragma unroll
        for (int t = 0; t < NT; ++t) x[t] = x[t] * rinv * (w ? __bfloat162float(w[lane + 32 * t]) : 1.0f);
        if (rotate) {
#pragma unroll
            for (int t = 0; t < HALF_T; ++t) {
                const int i = lane + 32 * t;  // pair (i, i + D/2)
                const float c = s_cos[i], s = s_sin[i];
                const float x1 = x[t], x2 = x[t + HALF_T];
                x[t] = x1 * c - x2 * s;
                x[t + HALF_T] = x2 * c + x1 * s;
            }
        }
#pragma unroll
        for (int t = 0; t < NT; ++t) dst[lane + 32 * t] = __float2bfloat16_rn(x[t]);
    }
}

}  // namespace

extern "C" int parallax_decode_prepare(const void* q_raw, const void* r_raw, const void* k_raw, const void* v_raw,
                                       const void* q_weight, const void* r_weight, const void* k_weight,
                                       const int32_t* seqlens, void* q_out, void* r_out, void* k_cache, void* v_cache,
                                       int B, int Hq, int Hkv, int D, int T_max, float eps, float rope_theta,
                                       int rope_on_r, void* stream)
{
    if (!q_raw || !r_raw || !k_raw || !v_raw || !q_out || !r_out || !k_cache || !v_cache) return PLX_ERR_NULL_POINTER;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || T_max <= 0 || Hq % Hkv != 0 || !(eps >= 0.0f) || !(rope_theta > 0.0f))
        return PLX_ERR_BAD_SHAPE;
    if (D != 64 && D != 128) return PLX_ERR_UNSUPPORTED;
    PrepareParams pp{static_cast<const __nv_bfloat16*>(q_raw), static_cast<const __nv_bfloat16*>(r_raw),
                     static_cast<const __nv_bfloat16*>(k_raw), static_cast<const __nv_bfloat16*>(v_raw),
                     static_cast<const __nv_bfloat16*>(q_weight), static_cast<const __nv_bfloat16*>(r_weight),
                     static_cast<const __nv_bfloat16*>(k_weight), seqlens, static_cast<__nv_bfloat16*>(q_out),
                     static_cast<__nv_bfloat16*>(r_out), static_cast<__nv_bfloat16*>(k_cache),
                     static_cast<__nv_bfloat16*>(v_cache), B, Hq, Hkv, T_max, eps,
                     log2(static_cast<double>(rope_theta)), rope_on_r};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PlxNvtxRange nvtx_range("plx_decode_prepare");
    if (D == 128)
        plx_prepare_kernel<128><<<B, kPrepWarps * 32, 0, st>>>(pp);
    else
        plx_prepare_kernel<64><<<B, kPrepWarps * 32, 0, st>>>(pp);
    return cudaGetLastError() == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}
