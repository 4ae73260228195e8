// Shared device-side PTX wrappers (mbarrier, TMA, proxy fences) and host helpers of the Parallax
// kernels.  Internal to the library; everything here has internal linkage.
#ifndef PLX_COMMON_CUH_
#define PLX_COMMON_CUH_

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "parallax.h"

// NVTX ranges around the library's launches (header-only NVTX v3: no link dependency; without a profiler
// attached a push/pop pair is two calls through a no-op function pointer).  -DPLX_NVTX=0 removes them.
#ifndef PLX_NVTX
#define PLX_NVTX 1
#endif
#if PLX_NVTX
#include <nvtx3/nvToolsExt.h>
#endif

namespace {

struct PlxNvtxRange {
#if PLX_NVTX
    explicit PlxNvtxRange(const char* name) { nvtxRangePushA(name); }
    ~PlxNvtxRange() { nvtxRangePop(); }
#else
    explicit PlxNvtxRange(const char*) {}
#endif
    PlxNvtxRange(const PlxNvtxRange&) = delete;
    PlxNvtxRange& operator=(const PlxNvtxRange&) = delete;
};

constexpr uint32_t kWaitLimit = 1u << 22;  // mbarrier try_wait attempts before a wait gives up

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// The retry loop of a bounded wait, kept out of line: with the loop inlined at every wait of a pipelined kernel a
// wait on a phase that had long completed still cost about 200 cycles (measured with clock stamps in the multi-token
// decode kernel); one attempt in line and the loop behind a call took 2-8 % off that kernel's steps and 2-5 % off the
// prefill and backward kernels.
__device__ __noinline__ bool mbar_wait_retry(uint32_t bar, uint32_t parity, uint32_t limit)
{
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// Bounded wait: false if the phase did not complete within `limit` attempts.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = kWaitLimit)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_retry(bar, parity, limit);
}

// 2-D tiled TMA load into this CTA's shared memory (one destination CTA).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x,
                                            int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
        "l"(tm), "r"(bar), "r"(x), "r"(y)
        : "memory");
}

// Plain (untiled) bulk copy global -> this CTA's shared memory; 16-byte aligned, size multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Orders earlier generic-proxy accesses before later async-proxy (TMA, tensor core) accesses.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
// Same, restricted to this CTA's shared memory: much cheaper (no global traffic to drain).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}


// ---------------------------------------------------------------------------
// Host helpers
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link-time libcuda dependency).
inline EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// bf16 [rows, D] row-major viewed in boxes of [box_rows rows, 64 columns] with the 128-byte swizzle (rows of
// 32 columns = 64 bytes: boxes of [box_rows rows, 32 columns] with the 64-byte swizzle); rows past the end read as zero.  Encoding costs about a microsecond of host time and the result is
// a pure function of the arguments, so the last encodings are kept in a small direct-mapped cache
// (decode calls are launch-bound on small batches and reuse the same caches step after step).
inline int make_tensor_map_2d(CUtensorMap* tm, const void* base, int D, uint64_t rows, uint32_t box_rows,
                              CUtensorMapL2promotion promotion)
{
    struct Entry {
        const void* base = nullptr;
        uint64_t rows = 0;
        int D = 0;
        uint32_t box_rows = 0;
        int promotion = -1;
        CUtensorMap map;
    };
    constexpr int kSlots = 128;
    static Entry cache[kSlots];
    static std::mutex mu;
    const size_t h = (reinterpret_cast<uintptr_t>(base) >> 8) * 0x9E3779B97F4A7C15ull + rows * 31 + box_rows;
    Entry& e = cache[(h >> 17) % kSlots];
    {
        std::lock_guard<std::mutex> lock(mu);
        if (e.base == base && e.rows == rows && e.D == D && e.box_rows == box_rows &&
            e.promotion == static_cast<int>(promotion)) {
            *tm = e.map;
            return PLX_OK;
        }
    }
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return PLX_ERR_CUDA;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(D), rows};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(D) * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(D < 64 ? D : 64), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle swizzle = D < 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;
    CUresult rc = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, promotion,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc == CUDA_ERROR_INVALID_CONTEXT || rc == CUDA_ERROR_NOT_INITIALIZED) {
        // The encoder is a driver call and needs a current context; a host thread that has made no runtime
        // call that binds one yet (a framework's worker thread) gets the primary context bound here.  Only
        // then: cudaFree is not allowed while a stream capture is in progress, and a thread that captures
        // has a context already.
        if (cudaFree(nullptr) != cudaSuccess) return PLX_ERR_CUDA;
        rc = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                 CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, promotion,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (rc != CUDA_SUCCESS) return PLX_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    e.base = base;
    e.rows = rows;
    e.D = D;
    e.box_rows = box_rows;
    e.promotion = static_cast<int>(promotion);
    e.map = *tm;
    return PLX_OK;
}

inline bool plx_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace

#endif  // PLX_COMMON_CUH_
