// Measurement and test aids of the Parallax library (no attention arithmetic here).
//
// 1. A read-only streaming probe: reads a device buffer once and keeps nothing, in the two ways a
//    kernel can pull bytes out of HBM on sm_100a.  The decode kernel is a pure reader, so the copy
//    bandwidth (read + write) is not its ceiling; this probe is.
//      mode PLX_PROBE_VECTOR_LOADS  16-byte loads that bypass L1, eight independent loads per thread
//      mode PLX_PROBE_BULK_COPIES   bulk asynchronous copies into warp-private shared-memory rings
//                                   (the decode kernel's staging geometry with the arithmetic removed)
// 2. A test hook that makes a bounded mbarrier wait run out, so the way every kernel of the library
//    reports a wait that gave up (status word, orderly return) can be exercised without a fault.
#include <cuda_runtime.h>
#include <stdint.h>

#include "parallax.h"
#include "parallax_test_hooks.h"
#include "plx_common.cuh"

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeUnroll = 8;
constexpr int kProbeWarps = 4;            // bulk mode: warps per CTA, each with a ring of its own
constexpr int kProbeStages = 3;
constexpr uint32_t kProbeChunk = 8192;    // bytes per bulk copy (one K + V stage of the decode kernel at D = 128)
constexpr int kSinkSlots = PLX_PROBE_SINK_BYTES / 16;

__device__ __forceinline__ uint4 ld_stream16(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Each CTA reads one contiguous range of `per_cta` 16-byte words; a thread's eight loads are independent.
__global__ void __launch_bounds__(kProbeThreads) plx_read_probe_vec_kernel(const uint4* __restrict__ src, size_t n16,
                                                                            size_t per_cta, uint4* __restrict__ sink)
{
    const size_t begin = static_cast<size_t>(blockIdx.x) * per_cta;
    const size_t end = begin + per_cta < n16 ? begin + per_cta : n16;
    uint4 acc = make_uint4(0u, 0u, 0u, 0u);
    size_t i = begin + threadIdx.x;
    for (; i + static_cast<size_t>(kProbeUnroll - 1) * kProbeThreads < end; i += static_cast<size_t>(kProbeUnroll) * kProbeThreads) {
        uint4 v[kProbeUnroll];
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) v[u] = ld_stream16(src + i + static_cast<size_t>(u) * kProbeThreads);
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) {
            acc.x ^= v[u].x;
            acc.y ^= v[u].y;
            acc.z ^= v[u].z;
            acc.w ^= v[u].w;
        }
    }
    for (; i < end; i += kProbeThreads) {
        const uint4 v = ld_stream16(src + i);
        acc.x ^= v.x;
        acc.y ^= v.y;
        acc.z ^= v.z;
        acc.w ^= v.w;
    }
    // fold the CTA's value into one word per lane group and store once per CTA
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        acc.x ^= __shfl_xor_sync(0xffffffffu, acc.x, off);
        acc.y ^= __shfl_xor_sync(0xffffffffu, acc.y, off);
        acc.z ^= __shfl_xor_sync(0xffffffffu, acc.z, off);
        acc.w ^= __shfl_xor_sync(0xffffffffu, acc.w, off);
    }
    __shared__ uint4 part[kProbeThreads / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint4 t = part[0];
#pragma unroll
        for (int w = 1; w < kProbeThreads / 32; ++w) {
            t.x ^= part[w].x;
            t.y ^= part[w].y;
            t.z ^= part[w].z;
            t.w ^= part[w].w;
        }
        sink[blockIdx.x % kSinkSlots] = t;
    }
}

// Each CTA walks a contiguous range of 8 KiB chunks; warp w takes chunks w, w + 4, ... through a ring of
// three shared-memory slots that lane 0 refills as soon as a slot has landed.  Nothing is computed: one
// word of every landed chunk is read so that the data counts as used.
__global__ void __launch_bounds__(kProbeWarps * 32, 2) plx_read_probe_bulk_kernel(const uint8_t* __restrict__ src,
                                                                                   size_t nchunks, size_t per_cta,
                                                                                   uint4* __restrict__ sink,
                                                                                   int32_t* status)
{
    extern __shared__ uint8_t probe_smem_raw[];
    const uint32_t raw = smem_u32(probe_smem_raw);
    const uint32_t base = (raw + 127u) & ~127u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = base + warp * kProbeStages * kProbeChunk;
    const uint32_t bars = base + kProbeWarps * kProbeStages * kProbeChunk + warp * kProbeStages * 8;
    const size_t begin = static_cast<size_t>(blockIdx.x) * per_cta;
    const size_t end = begin + per_cta < nchunks ? begin + per_cta : nchunks;
    const long long total = begin < end ? static_cast<long long>(end - begin) : 0;
    const int n_my = static_cast<int>((total - warp + kProbeWarps - 1) / kProbeWarps);

    if (lane == 0) {
        for (int s = 0; s < kProbeStages; ++s) mbar_init(bars + 8 * s, 1);
        fence_barrier_init();
    }
    __syncwarp();
    auto issue = [&](int n, int s) {
        mbar_expect_tx(bars + 8 * s, kProbeChunk);
        bulk_load(ring + s * kProbeChunk, src + (begin + warp + static_cast<size_t>(n) * kProbeWarps) * kProbeChunk,
                  kProbeChunk, bars + 8 * s);
    };
    if (lane == 0)
        for (int s = 0; s < kProbeStages; ++s)
            if (s < n_my) issue(s, s);

    uint32_t acc = 0, parity = 0;
    int s = 0;
    bool failed = false;
    for (int n = 0; n < n_my; ++n) {
        if (!mbar_wait_bounded(bars + 8 * s, parity)) {
            failed = true;
            break;
        }
        uint32_t w;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(ring + s * kProbeChunk + lane * 4));
        acc ^= w;
        __syncwarp();
        if (lane == 0 && n + kProbeStages < n_my) issue(n + kProbeStages, s);
        if (++s == kProbeStages) {
            s = 0;
            parity ^= 1u;
        }
    }
    if (failed) {
        // same discipline as the attention kernels: report, give copies in flight a bounded chance to land
        if (lane == 0 && status) atomicExch(status, PLX_ERR_DEVICE_TIMEOUT);
        for (int t = 0; t < kProbeStages; ++t) {
            (void)mbar_wait_bounded(bars + 8 * s, parity);
            if (++s == kProbeStages) {
                s = 0;
                parity ^= 1u;
            }
        }
    }
    if (lane == 0) sink[(blockIdx.x * kProbeWarps + warp) % kSinkSlots] = make_uint4(acc, 0u, 0u, 0u);
}

// One warp arms nothing and waits on a barrier nobody will ever complete, for at most `attempts` polls.
__global__ void plx_test_bounded_wait_kernel(int32_t* status, uint32_t attempts, int32_t* polls_done)
{
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        fence_barrier_init();
    }
    __syncthreads();
    const bool done = mbar_wait_bounded(b, 0u, attempts);
    if (!done && threadIdx.x == 0) {
        atomicExch(status, PLX_ERR_DEVICE_TIMEOUT);
        if (polls_done) *polls_done = static_cast<int32_t>(attempts);
    }
}

}  // namespace

extern "C" {

int parallax_read_probe(const void* src, size_t bytes, void* sink, int mode, int ctas, int32_t* status, void* stream)
{
    if (!src || !sink) return PLX_ERR_NULL_POINTER;
    if (bytes == 0 || bytes % kProbeChunk != 0 || ctas < 0) return PLX_ERR_BAD_SHAPE;
    if (!plx_aligned(src, 16) || !plx_aligned(sink, 16)) return PLX_ERR_ALIGNMENT;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return PLX_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mode == PLX_PROBE_VECTOR_LOADS) {
        const size_t n16 = bytes / 16;
        const size_t grid = ctas ? static_cast<size_t>(ctas) : static_cast<size_t>(sms) * 8;
        const size_t granule = static_cast<size_t>(kProbeThreads) * kProbeUnroll;
        const size_t per_cta = ((n16 + grid - 1) / grid + granule - 1) / granule * granule;
        const size_t used = (n16 + per_cta - 1) / per_cta;
        plx_read_probe_vec_kernel<<<static_cast<unsigned>(used), kProbeThreads, 0, st>>>(
            static_cast<const uint4*>(src), n16, per_cta, static_cast<uint4*>(sink));
    } else if (mode == PLX_PROBE_BULK_COPIES) {
        const size_t nchunks = bytes / kProbeChunk;
        const size_t grid = ctas ? static_cast<size_t>(ctas) : static_cast<size_t>(sms) * 2;
        const size_t per_cta = (nchunks + grid - 1) / grid;
        const size_t used = (nchunks + per_cta - 1) / per_cta;
        constexpr int kSmem = 128 + kProbeWarps * kProbeStages * static_cast<int>(kProbeChunk) + kProbeWarps * kProbeStages * 8;
        static bool configured[64] = {false};
        if (dev < 0 || dev >= 64 || !configured[dev]) {
            if (cudaFuncSetAttribute(plx_read_probe_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) !=
                cudaSuccess)
                return PLX_ERR_CUDA;
            if (dev >= 0 && dev < 64) configured[dev] = true;
        }
        plx_read_probe_bulk_kernel<<<static_cast<unsigned>(used), kProbeWarps * 32, kSmem, st>>>(
            static_cast<const uint8_t*>(src), nchunks, per_cta, static_cast<uint4*>(sink), status);
    } else {
        return PLX_ERR_BAD_SHAPE;
    }
    return cudaGetLastError() == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}

int plx_test_bounded_wait(int32_t* status, uint32_t attempts, int32_t* polls_done, void* stream)
{
    if (!status) return PLX_ERR_NULL_POINTER;
    if (attempts == 0 || attempts > (1u << 16)) return PLX_ERR_BAD_SHAPE;  // a test hook: short waits only
    plx_test_bounded_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, attempts, polls_done);
    return cudaGetLastError() == cudaSuccess ? PLX_OK : PLX_ERR_CUDA;
}

}  // extern "C"
