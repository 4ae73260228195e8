"""ctypes binding of the Parallax decode C-ABI library (argument marshalling only).

Function names and argument order follow include/parallax.h.  Tensors are torch
CUDA tensors (device memory and streams are torch's; every step of the path
runs in the library's kernels).  Importing this module loads the in-tree shared
library and raises if it has not been built: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from pathlib import Path
from typing import Optional

import torch

PLX_OK = 0
PLX_ERR_NULL_POINTER = -1
PLX_ERR_BAD_SHAPE = -2
PLX_ERR_UNSUPPORTED = -3
PLX_ERR_ALIGNMENT = -4
PLX_ERR_WORKSPACE = -5
PLX_ERR_NEED_LAYOUT = -6
PLX_ERR_CUDA = -7
PLX_ERR_DEVICE_TIMEOUT = -8
PLX_ERR_STATIC_SCRATCH = -9
PLX_ERR_DEVICE_CHECK = -10
PLX_PROBE_VECTOR_LOADS = 0
PLX_PROBE_BULK_COPIES = 1
PLX_PROBE_SINK_BYTES = 65536
PLX_STATIC_SCRATCH_BYTES = 8 * 1024 * 1024
PLX_OUT_BF16 = 0
PLX_OUT_F32 = 1
PLX_P_BF16_RESIDUAL = 0
PLX_P_BF16 = 1
PLX_P_BF16_ADAPTIVE = 2
PLX_P_ADAPTIVE_MIN_KEYS = 1024
PLX_MAX_SPLITS = 1024

# PARALLAX_LIBRARY selects another build of the same library (the index-checking debug build,
# `python -m paper_2605_29157_b200.build --debug-checks`); the default is the optimised in-tree build.
LIB_PATH = Path(os.environ.get("PARALLAX_LIBRARY") or Path(__file__).resolve().parent / "libparallax.so")

EXPORTS = (
    "parallax_version", "parallax_status_string", "parallax_partial_stride",
    "parallax_decode_workspace_bytes", "parallax_decode_plan", "parallax_decode_fwd_ex",
    "parallax_set_layout", "parallax_decode_fwd", "parallax_decode_splitkv_partial",
    "parallax_decode_combine", "parallax_decode_fwd_host", "parallax_workspace_status",
    "parallax_decode_fwd_static", "parallax_prefill_fwd", "parallax_decode_fwd_paged",
    "parallax_decode_combine_gathered", "parallax_decode_prepare",
    "parallax_prefill_fwd_save", "parallax_prefill_bwd_workspace_bytes", "parallax_prefill_bwd",
    "parallax_decode_fwd_fp8", "parallax_prefill_fwd_paged", "parallax_decode_fwd_paged_fp8",
    "parallax_decode_step", "parallax_decode_fwd_fp8_per_head", "parallax_decode_fwd_paged_fp8_per_head",
    "parallax_decode_fwd_multi", "parallax_prefill_workspace_bytes", "parallax_prefill_fwd_ex",
    "parallax_prefill_fwd_paged_ex", "parallax_decode_fwd_multi_paged", "parallax_decode_fwd_args",
    "parallax_read_probe", "parallax_decode_fwd_rows", "parallax_decode_multi_plan",
)
TEST_HOOK_EXPORTS = ("plx_test_bounded_wait",)


class ParallaxError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"parallax: {status_string(status)} ({status})")


def _load() -> ctypes.CDLL:
    if not LIB_PATH.exists():
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2605_29157_b200.build` "
            "(the CUDA library is the only implementation; there is no fallback)")
    lib = ctypes.CDLL(str(LIB_PATH))
    i32, f32, vp, sz = ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
    ip = ctypes.POINTER(ctypes.c_int)
    sig = {
        "parallax_version": (i32, []),
        "parallax_status_string": (ctypes.c_char_p, [i32]),
        "parallax_partial_stride": (i32, [i32]),
        "parallax_decode_workspace_bytes": (sz, [i32, i32, i32, i32]),
        "parallax_decode_plan": (i32, [i32, i32, i32, i32, i32, i32, i32, ip, ip]),
        "parallax_decode_fwd_ex": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, i32, vp, sz, i32, vp]),
        "parallax_set_layout": (i32, [i32, i32, vp, sz]),
        "parallax_decode_fwd": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, f32, vp]),
        "parallax_decode_splitkv_partial": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, i32, i32, vp, vp]),
        "parallax_decode_combine": (i32, [vp, vp, vp, i32, i32, i32, i32, i32, vp]),
        "parallax_decode_fwd_host": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, i32, vp, sz, i32, vp]),
        "parallax_workspace_status": (i32, [vp, ip, vp]),
        "parallax_decode_fwd_static": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, i32, i32, vp]),
        "parallax_prefill_fwd": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, i32, i32, vp, vp]),
        "parallax_decode_fwd_fp8": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, f32, f32, i32, vp, sz, i32, vp]),
        "parallax_decode_fwd_paged_fp8": (i32, [vp] * 7 + [i32] * 7 + [f32, f32, f32, i32, vp, sz, i32, vp]),
        "parallax_prefill_workspace_bytes": (sz, [i32, i32, i32, i32, i32]),
        "parallax_prefill_fwd_paged_ex": (i32, [vp] * 7 + [i32] * 8 + [f32, i32, i32, vp, sz, i32, vp, vp]),
        "parallax_prefill_fwd_ex": (i32, [vp] * 6 + [i32] * 6 + [f32, i32, i32, vp, sz, i32, vp, vp]),
        "parallax_decode_fwd_multi_paged": (i32, [vp] * 7 + [i32] * 8 + [f32, i32, vp, sz, i32, vp]),
        "parallax_decode_fwd_multi": (i32, [vp] * 6 + [i32] * 6 + [f32, i32, vp, sz, i32, vp]),
        "parallax_decode_fwd_fp8_per_head": (i32, [vp] * 6 + [i32] * 5 + [f32, vp, vp, i32, vp, sz, i32, vp]),
        "parallax_decode_fwd_paged_fp8_per_head": (i32, [vp] * 7 + [i32] * 7 + [f32, vp, vp, i32, vp, sz, i32, vp]),
        "parallax_prefill_fwd_paged": (i32, [vp] * 7 + [i32] * 8 + [f32, i32, i32, vp, vp]),
        "parallax_prefill_fwd_save": (i32, [vp] * 9 + [i32, i32, i32, i32, i32, i32, f32, i32, i32, vp, vp]),
        "parallax_prefill_bwd_workspace_bytes": (sz, [i32, i32, i32]),
        "parallax_prefill_bwd": (i32, [vp] * 14 + [i32, i32, i32, i32, i32, i32, f32, i32, i32, vp, sz, vp, vp]),
        "parallax_decode_prepare": (i32, [vp] * 12 + [i32, i32, i32, i32, i32, f32, f32, i32, vp]),
        "parallax_decode_combine_gathered": (i32, [vp, vp, i32, i32, i32, i32, i32, i32, vp]),
        "parallax_decode_step": (i32, [vp] * 13 + [i32, i32, i32, i32, i32, f32, f32, i32, f32, i32, vp, sz, i32, vp]),
        "parallax_decode_fwd_paged": (i32, [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, f32, i32,
                                            vp, sz, i32, vp]),
        "parallax_read_probe": (i32, [vp, sz, vp, i32, i32, vp, vp]),
        "parallax_decode_fwd_rows": (i32, [vp] * 6 + [i32] * 6 + [f32, i32, vp, sz, i32, vp, vp]),
        "parallax_decode_multi_plan": (i32, [i32] * 7 + [vp, vp]),
        "plx_test_bounded_wait": (i32, [vp, ctypes.c_uint32, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


_lib = _load()


def _check(rc: int) -> None:
    if rc != PLX_OK:
        raise ParallaxError(rc)


def _ptr(t: Optional[torch.Tensor]):
    # a plain int: the argument types are declared, so ctypes converts it without an intermediate object
    return None if t is None else t.data_ptr()


_raw_current_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream):
    """cudaStream_t as an int (0 = the legacy default stream).  Without an argument: torch's current stream of the
    current device, through torch's raw-handle accessor where it exists (building a Stream object costs about 4 us,
    which a launch-bound decode call notices)."""
    if stream is None:
        if _raw_current_stream is not None:
            return _raw_current_stream(torch.cuda.current_device()) or None
        stream = torch.cuda.current_stream()
    return (stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)) or None


def _out_dtype_code(dtype: torch.dtype) -> int:
    if dtype == torch.bfloat16:
        return PLX_OUT_BF16
    if dtype == torch.float32:
        return PLX_OUT_F32
    raise ParallaxError(PLX_ERR_BAD_SHAPE)


def _shapes(q, k):
    B, Hq, D = q.shape
    Bk, Hkv, T_max, Dk = k.shape
    if Bk != B or Dk != D:
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    return B, Hq, Hkv, D, T_max


def _require(*tensors):
    for t in tensors:
        if t is not None and not (t.is_cuda and t.is_contiguous()):
            raise ValueError("parallax: tensors must be contiguous CUDA tensors")


def parallax_version() -> int:
    return int(_lib.parallax_version())


def status_string(status: int) -> str:
    return _lib.parallax_status_string(int(status)).decode()


def parallax_partial_stride(D: int) -> int:
    return int(_lib.parallax_partial_stride(D))


def parallax_decode_workspace_bytes(B: int, Hq: int, D: int, max_splits: int) -> int:
    return int(_lib.parallax_decode_workspace_bytes(B, Hq, D, max_splits))


def parallax_decode_plan(B, Hq, Hkv, D, T_max, num_sms, has_seqlens=False):
    """Returns (chunk_len, num_splits) the library would use on a device with num_sms SMs."""
    c, n = ctypes.c_int(0), ctypes.c_int(0)
    _check(_lib.parallax_decode_plan(B, Hq, Hkv, D, T_max, num_sms, int(bool(has_seqlens)),
                                     ctypes.byref(c), ctypes.byref(n)))
    return c.value, n.value


def alloc_workspace(B: int, Hq: int, D: int, max_splits: int, device) -> torch.Tensor:
    """A zeroed uint8 workspace tensor of the size the library asks for."""
    n = parallax_decode_workspace_bytes(B, Hq, D, max_splits)
    if n == 0:
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    return torch.zeros(n, dtype=torch.uint8, device=device)


def parallax_decode_fwd_ex(q, r, k_cache, v_cache, seqlens, out, scale, workspace=None, num_splits=0, stream=None):
    _require(q, r, k_cache, v_cache, seqlens, out, workspace)
    B, Hq, Hkv, D, T_max = _shapes(q, k_cache)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_ex(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                       B, Hq, Hkv, D, T_max, float(scale), _out_dtype_code(out.dtype),
                                       _ptr(workspace), ws_bytes, int(num_splits), _stream(stream)))
    return out


def parallax_set_layout(T_max: int, out_dtype: torch.dtype, workspace: Optional[torch.Tensor]) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_set_layout(int(T_max), _out_dtype_code(out_dtype), _ptr(workspace), ws_bytes))


def parallax_decode_fwd(q, r, k_cache, v_cache, seqlens, out, scale, stream=None):
    _require(q, r, k_cache, v_cache, seqlens, out)
    B, Hq, Hkv, D, _ = _shapes(q, k_cache)
    _check(_lib.parallax_decode_fwd(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                    B, Hq, Hkv, D, float(scale), _stream(stream)))
    return out


def parallax_decode_splitkv_partial(q, r, k_cache, v_cache, seqlens, partials, scale, chunk_len, num_splits,
                                    status=None, stream=None):
    _require(q, r, k_cache, v_cache, seqlens, partials, status)
    B, Hq, Hkv, D, T_max = _shapes(q, k_cache)
    _check(_lib.parallax_decode_splitkv_partial(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens),
                                                _ptr(partials), B, Hq, Hkv, D, T_max, float(scale),
                                                int(chunk_len), int(num_splits), _ptr(status), _stream(stream)))
    return partials


def parallax_decode_combine(partials, split_counts, out, num_splits, stream=None):
    _require(partials, split_counts, out)
    B, Hq, D = out.shape
    _check(_lib.parallax_decode_combine(_ptr(partials), _ptr(split_counts), _ptr(out), B, Hq, D, int(num_splits),
                                        _out_dtype_code(out.dtype), _stream(stream)))
    return out


def parallax_decode_fwd_host(q_host, r_host, k_cache, v_cache, seqlens, out_host, scale, workspace, num_splits=0,
                             stream=None):
    """q_host, r_host, out_host are CPU tensors (pinned for real overlap); synchronises the stream."""
    _require(k_cache, v_cache, seqlens, workspace)
    for t in (q_host, r_host, out_host):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("parallax: host tensors must be contiguous CPU tensors")
    B, Hq, Hkv, D, T_max = _shapes(q_host, k_cache)
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_host(_ptr(q_host), _ptr(r_host), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens),
                                         _ptr(out_host), B, Hq, Hkv, D, T_max, float(scale),
                                         _out_dtype_code(out_host.dtype), _ptr(workspace), ws_bytes,
                                         int(num_splits), _stream(stream)))
    return out_host


def parallax_workspace_status(workspace, stream=None) -> int:
    s = ctypes.c_int(0)
    _check(_lib.parallax_workspace_status(_ptr(workspace), ctypes.byref(s), _stream(stream)))
    return s.value


def parallax_decode_fwd_static(q, r, k_cache, v_cache, seqlens, out, scale, num_splits=0, stream=None):
    """Decode forward for callers that cannot allocate device memory (no workspace argument): the
    split scratch is a fixed array inside the library, shared by every call on the device, so
    calls must not overlap on the GPU.  Make the first call on a device outside stream capture."""
    _require(q, r, k_cache, v_cache, seqlens, out)
    B, Hq, Hkv, D, T_max = _shapes(q, k_cache)
    _check(_lib.parallax_decode_fwd_static(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                           B, Hq, Hkv, D, T_max, float(scale), _out_dtype_code(out.dtype),
                                           int(num_splits), _stream(stream)))
    return out


def parallax_prefill_fwd(q, r, k_cache, v_cache, seqlens, out, scale, status=None, stream=None,
                         p_precision=PLX_P_BF16_RESIDUAL):
    """Multi-token causal forward: q, r, out [B, Hq, Lq, D]; the Lq tokens are the last Lq positions
    of each context."""
    _require(q, r, k_cache, v_cache, seqlens, out, status)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k_cache.shape
    if Bk != B or Dk != D or tuple(out.shape) != (B, Hq, Lq, D) or tuple(r.shape) != tuple(q.shape):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    _check(_lib.parallax_prefill_fwd(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                     B, Hq, Hkv, D, Lq, T_max, float(scale), _out_dtype_code(out.dtype),
                                     int(p_precision), _ptr(status), _stream(stream)))
    return out


def parallax_prefill_workspace_bytes(B: int, Hq: int, D: int, Lq: int, max_splits: int) -> int:
    return int(_lib.parallax_prefill_workspace_bytes(B, Hq, D, Lq, max_splits))


def parallax_prefill_fwd_ex(q, r, k_cache, v_cache, seqlens, out, scale, workspace=None, num_splits=0, status=None,
                            stream=None, p_precision=PLX_P_BF16_RESIDUAL):
    """parallax_prefill_fwd with split-KV (short chunks on few sequences); workspace: uint8 CUDA tensor of
    parallax_prefill_workspace_bytes(...) bytes, or None for one split."""
    _require(q, r, k_cache, v_cache, seqlens, out, workspace, status)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k_cache.shape
    if Bk != B or Dk != D or tuple(out.shape) != (B, Hq, Lq, D) or tuple(r.shape) != tuple(q.shape):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_prefill_fwd_ex(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                        B, Hq, Hkv, D, Lq, T_max, float(scale), _out_dtype_code(out.dtype),
                                        int(p_precision), _ptr(workspace), ws_bytes, int(num_splits), _ptr(status),
                                        _stream(stream)))
    return out


PLX_MULTI_KERNEL_DECODE, PLX_MULTI_KERNEL_ROWS, PLX_MULTI_KERNEL_ROW_MAJOR = 0, 1, 2


def parallax_decode_multi_plan(B, Hq, Hkv, D, Lq, T_max, page_size=0):
    """(kernel, num_splits) the multi-token entries would use for this shape: kernel is one of PLX_MULTI_KERNEL_*,
    num_splits the planned split count of the keys-on-lanes kernel (0 for the other kernels)."""
    kernel, ns = ctypes.c_int(0), ctypes.c_int(0)
    _check(_lib.parallax_decode_multi_plan(int(B), int(Hq), int(Hkv), int(D), int(Lq), int(T_max), int(page_size),
                                           ctypes.byref(kernel), ctypes.byref(ns)))
    return kernel.value, ns.value


def parallax_decode_fwd_rows(q, r, k_cache, v_cache, seqlens, out, scale, workspace=None, num_splits=0, status=None,
                             stream=None):
    """The keys-on-lanes tensor-core kernel for a step of up to 64 rows per KV head ((Hq / Hkv) * Lq <= 64, D = 64 or 128);
    q, r, out [B, Hq, Lq, D]; workspace: uint8 CUDA tensor of parallax_prefill_workspace_bytes(...) bytes for split
    records, or None for one split.  parallax_decode_fwd_multi picks this kernel by itself."""
    _require(q, r, k_cache, v_cache, seqlens, out, workspace, status)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k_cache.shape
    if Bk != B or Dk != D or tuple(out.shape) != (B, Hq, Lq, D) or tuple(r.shape) != tuple(q.shape):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_rows(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                         B, Hq, Hkv, D, Lq, T_max, float(scale), _out_dtype_code(out.dtype),
                                         _ptr(workspace), ws_bytes, int(num_splits), _ptr(status), _stream(stream)))
    return out


def parallax_decode_fwd_fp8(q, r, k_cache, v_cache, seqlens, out, scale, k_scale, v_scale, workspace=None, num_splits=0,
                            stream=None):
    """Decode forward over an e4m3 cache: k_cache, v_cache [B, Hkv, T_max, D] (torch.float8_e4m3fn or the
    same bytes as uint8) holding k / k_scale and v / v_scale."""
    _require(q, r, k_cache, v_cache, seqlens, out, workspace)
    if k_cache.element_size() != 1 or v_cache.element_size() != 1:
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    B, Hq, Hkv, D, T_max = _shapes(q, k_cache)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_fp8(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                        B, Hq, Hkv, D, T_max, float(scale), float(k_scale), float(v_scale),
                                        _out_dtype_code(out.dtype), _ptr(workspace), ws_bytes, int(num_splits),
                                        _stream(stream)))
    return out


def parallax_decode_fwd_paged_fp8(q, r, k_pages, v_pages, block_table, seqlens, out, scale, k_scale, v_scale,
                                  workspace=None, num_splits=0, stream=None):
    """Decode forward over a paged e4m3 cache: k_pages, v_pages [num_pages, Hkv, page_size, D] (one byte per
    element), block_table int32 [B, max_pages_per_seq]."""
    _require(q, r, k_pages, v_pages, block_table, seqlens, out, workspace)
    B, Hq, D = q.shape
    num_pages, Hkv, page_size, Dk = k_pages.shape
    if (Dk != D or tuple(v_pages.shape) != tuple(k_pages.shape) or k_pages.element_size() != 1 or
            v_pages.element_size() != 1 or block_table.dim() != 2 or block_table.shape[0] != B or
            block_table.dtype != torch.int32):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_paged_fp8(_ptr(q), _ptr(r), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                              _ptr(seqlens), _ptr(out), B, Hq, Hkv, D, num_pages, page_size,
                                              block_table.shape[1], float(scale), float(k_scale), float(v_scale),
                                              _out_dtype_code(out.dtype), _ptr(workspace), ws_bytes,
                                              int(num_splits), _stream(stream)))
    return out


def parallax_decode_fwd_multi(q, r, k_cache, v_cache, seqlens, out, scale, workspace=None, num_splits=0, stream=None):
    """Several new tokens per sequence on the decode kernel: q, r, out [B, Hq, Lq, D]."""
    _require(q, r, k_cache, v_cache, seqlens, out, workspace)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k_cache.shape
    if Bk != B or Dk != D or tuple(out.shape) != tuple(q.shape) or tuple(r.shape) != tuple(q.shape):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_multi(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                          B, Hq, Hkv, D, Lq, T_max, float(scale), _out_dtype_code(out.dtype),
                                          _ptr(workspace), ws_bytes, int(num_splits), _stream(stream)))
    return out


def parallax_decode_fwd_multi_paged(q, r, k_pages, v_pages, block_table, seqlens, out, scale, workspace=None,
                                    num_splits=0, stream=None):
    """parallax_decode_fwd_multi over a paged cache: k_pages, v_pages [num_pages, Hkv, page_size, D]."""
    _require(q, r, k_pages, v_pages, block_table, seqlens, out, workspace)
    B, Hq, Lq, D = q.shape
    num_pages, Hkv, page_size, Dk = k_pages.shape
    if (Dk != D or tuple(out.shape) != tuple(q.shape) or tuple(r.shape) != tuple(q.shape) or block_table.dim() != 2 or
            block_table.shape[0] != B or block_table.dtype != torch.int32 or tuple(v_pages.shape) != tuple(k_pages.shape)):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_multi_paged(_ptr(q), _ptr(r), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                                _ptr(seqlens), _ptr(out), B, Hq, Hkv, D, Lq, num_pages, page_size,
                                                block_table.shape[1], float(scale), _out_dtype_code(out.dtype),
                                                _ptr(workspace), ws_bytes, int(num_splits), _stream(stream)))
    return out


PLX_KV_BF16 = 0
PLX_KV_E4M3 = 1


class ParallaxDecodeArgs(ctypes.Structure):
    """Mirror of parallax_decode_args (include/parallax.h)."""
    _fields_ = [("struct_bytes", ctypes.c_size_t), ("q", ctypes.c_void_p), ("r", ctypes.c_void_p),
                ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p), ("seqlens", ctypes.c_void_p),
                ("out", ctypes.c_void_p), ("B", ctypes.c_int), ("Hq", ctypes.c_int), ("Hkv", ctypes.c_int),
                ("D", ctypes.c_int), ("Lq", ctypes.c_int), ("T_max", ctypes.c_int), ("scale", ctypes.c_float),
                ("out_dtype", ctypes.c_int), ("kv_dtype", ctypes.c_int), ("k_scale", ctypes.c_float),
                ("v_scale", ctypes.c_float), ("k_scales", ctypes.c_void_p), ("v_scales", ctypes.c_void_p),
                ("block_table", ctypes.c_void_p), ("num_pages", ctypes.c_int), ("page_size", ctypes.c_int),
                ("max_pages_per_seq", ctypes.c_int), ("num_splits", ctypes.c_int), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t), ("stream", ctypes.c_void_p)]


_lib.parallax_decode_fwd_args.restype = ctypes.c_int
_lib.parallax_decode_fwd_args.argtypes = [ctypes.POINTER(ParallaxDecodeArgs)]


def parallax_decode_fwd_args(q, r, k_cache, v_cache, seqlens, out, scale, block_table=None, k_scale=None, v_scale=None,
                             workspace=None, num_splits=0, stream=None):
    """Every option of the decode forward in one call.  q, r, out: [B, Hq, D] or [B, Hq, Lq, D]; caches
    contiguous [B, Hkv, T, D] or, with block_table, page pools [num_pages, Hkv, page_size, D]; a one-byte
    cache dtype selects the e4m3 variant, whose scales are two floats or two fp32 CUDA tensors [Hkv]."""
    _require(q, r, k_cache, v_cache, seqlens, out, block_table, workspace)
    a = ParallaxDecodeArgs()
    a.struct_bytes = ctypes.sizeof(ParallaxDecodeArgs)
    if q.dim() == 4:
        B, Hq, Lq, D = q.shape
    else:
        (B, Hq, D), Lq = q.shape, 1
    if tuple(out.shape) != tuple(q.shape) or tuple(r.shape) != tuple(q.shape) or k_cache.shape[-1] != D:
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    a.q, a.r, a.k_cache, a.v_cache = q.data_ptr(), r.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr()
    a.seqlens = None if seqlens is None else seqlens.data_ptr()
    a.out, a.B, a.Hq, a.D, a.Lq = out.data_ptr(), B, Hq, D, Lq
    a.scale, a.out_dtype = float(scale), _out_dtype_code(out.dtype)
    if block_table is not None:
        if block_table.dtype != torch.int32 or block_table.dim() != 2 or block_table.shape[0] != B:
            raise ParallaxError(PLX_ERR_BAD_SHAPE)
        a.num_pages, a.Hkv, a.page_size, _ = k_cache.shape
        a.block_table, a.max_pages_per_seq = block_table.data_ptr(), block_table.shape[1]
    else:
        _, a.Hkv, a.T_max, _ = k_cache.shape
    if k_cache.element_size() == 1:
        a.kv_dtype = PLX_KV_E4M3
        if isinstance(k_scale, torch.Tensor):
            _head_scales(k_scale, v_scale, a.Hkv)
            a.k_scales, a.v_scales = k_scale.data_ptr(), v_scale.data_ptr()
        else:
            a.k_scale, a.v_scale = float(k_scale), float(v_scale)
    if workspace is not None:
        a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    a.num_splits = int(num_splits)
    a.stream = _stream(stream)
    _check(_lib.parallax_decode_fwd_args(ctypes.byref(a)))
    return out


def _head_scales(k_scales, v_scales, Hkv):
    _require(k_scales, v_scales)
    for t in (k_scales, v_scales):
        if t.dtype != torch.float32 or t.numel() != Hkv:
            raise ParallaxError(PLX_ERR_BAD_SHAPE)


def parallax_decode_fwd_fp8_per_head(q, r, k_cache, v_cache, seqlens, out, scale, k_scales, v_scales, workspace=None,
                                     num_splits=0, stream=None):
    """parallax_decode_fwd_fp8 with one scale per KV head: k_scales, v_scales fp32 CUDA tensors [Hkv]."""
    _require(q, r, k_cache, v_cache, seqlens, out, workspace)
    if k_cache.element_size() != 1 or v_cache.element_size() != 1:
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    B, Hq, Hkv, D, T_max = _shapes(q, k_cache)
    _head_scales(k_scales, v_scales, Hkv)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_fp8_per_head(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens),
                                                 _ptr(out), B, Hq, Hkv, D, T_max, float(scale), _ptr(k_scales),
                                                 _ptr(v_scales), _out_dtype_code(out.dtype), _ptr(workspace),
                                                 ws_bytes, int(num_splits), _stream(stream)))
    return out


def parallax_decode_fwd_paged_fp8_per_head(q, r, k_pages, v_pages, block_table, seqlens, out, scale, k_scales,
                                           v_scales, workspace=None, num_splits=0, stream=None):
    """parallax_decode_fwd_paged_fp8 with one scale per KV head: k_scales, v_scales fp32 CUDA tensors [Hkv]."""
    _require(q, r, k_pages, v_pages, block_table, seqlens, out, workspace)
    B, Hq, D = q.shape
    num_pages, Hkv, page_size, Dk = k_pages.shape
    if (Dk != D or tuple(v_pages.shape) != tuple(k_pages.shape) or k_pages.element_size() != 1 or
            v_pages.element_size() != 1 or block_table.dim() != 2 or block_table.shape[0] != B or
            block_table.dtype != torch.int32):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    _head_scales(k_scales, v_scales, Hkv)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_paged_fp8_per_head(_ptr(q), _ptr(r), _ptr(k_pages), _ptr(v_pages),
                                                       _ptr(block_table), _ptr(seqlens), _ptr(out), B, Hq, Hkv, D,
                                                       num_pages, page_size, block_table.shape[1], float(scale),
                                                       _ptr(k_scales), _ptr(v_scales), _out_dtype_code(out.dtype),
                                                       _ptr(workspace), ws_bytes, int(num_splits), _stream(stream)))
    return out


def parallax_prefill_fwd_paged(q, r, k_pages, v_pages, block_table, seqlens, out, scale, status=None, stream=None,
                               p_precision=PLX_P_BF16_RESIDUAL):
    """Multi-token causal forward over a paged cache: k_pages, v_pages [num_pages, Hkv, page_size, D],
    block_table int32 [B, max_pages_per_seq]; page_size a multiple of 64."""
    _require(q, r, k_pages, v_pages, block_table, seqlens, out, status)
    B, Hq, Lq, D = q.shape
    num_pages, Hkv, page_size, Dk = k_pages.shape
    if (Dk != D or tuple(out.shape) != (B, Hq, Lq, D) or tuple(r.shape) != tuple(q.shape) or block_table.dim() != 2 or
            block_table.shape[0] != B or block_table.dtype != torch.int32 or tuple(v_pages.shape) != tuple(k_pages.shape)):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    _check(_lib.parallax_prefill_fwd_paged(_ptr(q), _ptr(r), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                           _ptr(seqlens), _ptr(out), B, Hq, Hkv, D, Lq, num_pages, page_size,
                                           block_table.shape[1], float(scale), _out_dtype_code(out.dtype),
                                           int(p_precision), _ptr(status), _stream(stream)))
    return out


def parallax_prefill_fwd_paged_ex(q, r, k_pages, v_pages, block_table, seqlens, out, scale, workspace=None, num_splits=0,
                                  status=None, stream=None, p_precision=PLX_P_BF16_RESIDUAL):
    """parallax_prefill_fwd_paged with split-KV (workspace as for parallax_prefill_fwd_ex)."""
    _require(q, r, k_pages, v_pages, block_table, seqlens, out, workspace, status)
    B, Hq, Lq, D = q.shape
    num_pages, Hkv, page_size, Dk = k_pages.shape
    if (Dk != D or tuple(out.shape) != (B, Hq, Lq, D) or tuple(r.shape) != tuple(q.shape) or block_table.dim() != 2 or
            block_table.shape[0] != B or block_table.dtype != torch.int32 or tuple(v_pages.shape) != tuple(k_pages.shape)):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_prefill_fwd_paged_ex(_ptr(q), _ptr(r), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                              _ptr(seqlens), _ptr(out), B, Hq, Hkv, D, Lq, num_pages, page_size,
                                              block_table.shape[1], float(scale), _out_dtype_code(out.dtype),
                                              int(p_precision), _ptr(workspace), ws_bytes, int(num_splits),
                                              _ptr(status), _stream(stream)))
    return out


def parallax_prefill_fwd_save(q, r, k_cache, v_cache, seqlens, out, lse, tbar, vbar, scale, status=None, stream=None,
                              p_precision=PLX_P_BF16_RESIDUAL):
    """Training forward: parallax_prefill_fwd that also writes lse, tbar (fp32 [B, Hq, Lq]) and vbar
    (as out) for parallax_prefill_bwd."""
    _require(q, r, k_cache, v_cache, seqlens, out, lse, tbar, vbar, status)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k_cache.shape
    if (Bk != B or Dk != D or tuple(out.shape) != (B, Hq, Lq, D) or tuple(r.shape) != tuple(q.shape) or
            tuple(vbar.shape) != tuple(out.shape) or vbar.dtype != out.dtype or tuple(lse.shape) != (B, Hq, Lq) or
            tuple(tbar.shape) != (B, Hq, Lq) or lse.dtype != torch.float32 or tbar.dtype != torch.float32):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    _check(_lib.parallax_prefill_fwd_save(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(seqlens), _ptr(out),
                                          _ptr(lse), _ptr(tbar), _ptr(vbar), B, Hq, Hkv, D, Lq, T_max, float(scale),
                                          _out_dtype_code(out.dtype), int(p_precision), _ptr(status), _stream(stream)))
    return out


def parallax_prefill_bwd_workspace_bytes(B: int, Hq: int, Lq: int) -> int:
    return int(_lib.parallax_prefill_bwd_workspace_bytes(B, Hq, Lq))


def parallax_prefill_bwd(q, r, k_cache, v_cache, dout, out, lse, tbar, vbar, seqlens, dq, dr, dk, dv, scale,
                         workspace, status=None, stream=None):
    """Backward of parallax_prefill_fwd_save: writes dq, dr [B, Hq, Lq, D] and dk, dv [B, Hkv, T_max, D]
    (all four of one dtype, fp32 or bf16); `workspace` is a uint8 tensor of
    parallax_prefill_bwd_workspace_bytes(B, Hq, Lq) bytes."""
    _require(q, r, k_cache, v_cache, dout, out, lse, tbar, vbar, seqlens, dq, dr, dk, dv, workspace, status)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k_cache.shape
    same_q = all(tuple(t.shape) == (B, Hq, Lq, D) for t in (r, dout, out, vbar, dq, dr))
    same_k = all(tuple(t.shape) == (B, Hkv, T_max, D) for t in (v_cache, dk, dv))
    if (Bk != B or Dk != D or not same_q or not same_k or vbar.dtype != out.dtype or
            any(t.dtype != dq.dtype for t in (dr, dk, dv)) or dout.dtype != torch.bfloat16):
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    _check(_lib.parallax_prefill_bwd(_ptr(q), _ptr(r), _ptr(k_cache), _ptr(v_cache), _ptr(dout), _ptr(out), _ptr(lse),
                                     _ptr(tbar), _ptr(vbar), _ptr(seqlens), _ptr(dq), _ptr(dr), _ptr(dk), _ptr(dv),
                                     B, Hq, Hkv, D, Lq, T_max, float(scale), _out_dtype_code(out.dtype),
                                     _out_dtype_code(dq.dtype), _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _ptr(status), _stream(stream)))
    return dq, dr, dk, dv


def parallax_decode_fwd_paged(q, r, k_pages, v_pages, block_table, seqlens, out, scale, workspace=None, num_splits=0,
                              stream=None):
    """Decode forward over a paged cache: k_pages, v_pages [num_pages, Hkv, page_size, D],
    block_table int32 [B, max_pages_per_seq]."""
    _require(q, r, k_pages, v_pages, block_table, seqlens, out, workspace)
    B, Hq, D = q.shape
    num_pages, Hkv, page_size, Dk = k_pages.shape
    if Dk != D or block_table.shape[0] != B or block_table.dtype != torch.int32:
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_fwd_paged(_ptr(q), _ptr(r), _ptr(k_pages), _ptr(v_pages), _ptr(block_table),
                                          _ptr(seqlens), _ptr(out), B, Hq, Hkv, D, num_pages, page_size,
                                          int(block_table.shape[1]), float(scale), _out_dtype_code(out.dtype),
                                          _ptr(workspace), ws_bytes, int(num_splits), _stream(stream)))
    return out


def parallax_decode_combine_gathered(partials, out, num_ranks, num_splits, stream=None):
    """Merge partial states gathered from `num_ranks` GPUs: partials [num_ranks, B, Hq, num_splits, stride]."""
    _require(partials, out)
    B, Hq, D = out.shape
    _check(_lib.parallax_decode_combine_gathered(_ptr(partials), _ptr(out), B, Hq, D, int(num_ranks), int(num_splits),
                                                 _out_dtype_code(out.dtype), _stream(stream)))
    return out


def parallax_decode_step(q_raw, r_raw, k_raw, v_raw, q_weight, r_weight, k_weight, seqlens, q_out, r_out, k_cache,
                         v_cache, out, scale, workspace=None, num_splits=0, eps=1e-6, rope_theta=1e6, rope_on_r=False,
                         stream=None):
    """parallax_decode_prepare + parallax_decode_fwd_ex in one call, the second launch overlapped with the first."""
    _require(q_raw, r_raw, k_raw, v_raw, q_weight, r_weight, k_weight, seqlens, q_out, r_out, k_cache, v_cache, out,
             workspace)
    B, Hq, D = q_raw.shape
    _, Hkv, T_max, _ = k_cache.shape
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.parallax_decode_step(_ptr(q_raw), _ptr(r_raw), _ptr(k_raw), _ptr(v_raw), _ptr(q_weight),
                                     _ptr(r_weight), _ptr(k_weight), _ptr(seqlens), _ptr(q_out), _ptr(r_out),
                                     _ptr(k_cache), _ptr(v_cache), _ptr(out), B, Hq, Hkv, D, T_max, float(eps),
                                     float(rope_theta), int(bool(rope_on_r)), float(scale),
                                     _out_dtype_code(out.dtype), _ptr(workspace), ws_bytes, int(num_splits),
                                     _stream(stream)))
    return out


def parallax_decode_prepare(q_raw, r_raw, k_raw, v_raw, q_weight, r_weight, k_weight, seqlens, q_out, r_out, k_cache,
                            v_cache, eps=1e-6, rope_theta=1e6, rope_on_r=False, stream=None):
    """RMSNorm + rotary embedding of the new token's q, rho, k and append of k, v to the caches."""
    _require(q_raw, r_raw, k_raw, v_raw, q_weight, r_weight, k_weight, seqlens, q_out, r_out, k_cache, v_cache)
    B, Hq, D = q_raw.shape
    _, Hkv, T_max, _ = k_cache.shape
    _check(_lib.parallax_decode_prepare(_ptr(q_raw), _ptr(r_raw), _ptr(k_raw), _ptr(v_raw), _ptr(q_weight),
                                        _ptr(r_weight), _ptr(k_weight), _ptr(seqlens), _ptr(q_out), _ptr(r_out),
                                        _ptr(k_cache), _ptr(v_cache), B, Hq, Hkv, D, T_max, float(eps),
                                        float(rope_theta), int(bool(rope_on_r)), _stream(stream)))


def parallax_read_probe(src, sink, mode=PLX_PROBE_VECTOR_LOADS, ctas=0, status=None, stream=None, nbytes=None):
    """Reads `nbytes` (default: all) of the device tensor `src` once; `sink` is a device tensor of at
    least PLX_PROBE_SINK_BYTES bytes."""
    _require(src, sink)
    total = src.numel() * src.element_size() if nbytes is None else int(nbytes)
    if sink.numel() * sink.element_size() < PLX_PROBE_SINK_BYTES:
        raise ParallaxError(PLX_ERR_BAD_SHAPE)
    _check(_lib.parallax_read_probe(_ptr(src), total, _ptr(sink), mode, ctas, _ptr(status), _stream(stream)))


def plx_test_bounded_wait(status, attempts, polls_done=None, stream=None):
    """Test hook: one warp polls a barrier nothing arrives on `attempts` times, then sets `status`."""
    _check(_lib.plx_test_bounded_wait(_ptr(status), attempts, _ptr(polls_done), _stream(stream)))
