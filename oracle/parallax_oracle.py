"""Parallax ORACLE, Python side (test infrastructure, not the product).

Only the tests, the smoke check and the bench's CPU-baseline leg may import this
module; the CUDA path never does, and this module imports nothing from it.

Contents
--------
* ``decode_bf16`` / ``decode_f64``: ctypes wrappers around the plain-C fp64
  two-pass implementation in ``parallax_oracle.c`` (the oracle proper:
  Sec. 3.1, Eq. "parallax_forward", scoring form).
* ``prefill_bf16`` / ``prefill_f64``: the same rows for Lq query tokens per
  sequence with the causal limit j <= i of Eq. "parallax_forward".
* ``backward_bf16`` / ``backward_f64`` / ``saved_state_bf16``: the closed-form gradients of
  App. "Parallax Backward" and the per-row state the forward saves for them.
* NumPy fp64 restatements of the *other* forms the paper gives for the same
  output; the CPU tests use them to pin the C oracle and they in turn serve as
  the expected values for the split-KV partial state and the combine step:
    - ``covariance_form``   o_SA - Sigma_KV rho with the explicit D x D
                            weighted covariance (Sec. 3.1, Eq. "parallax_forward",
                            right-hand side; Sigma_KV as defined under
                            Eq. "parameterized_lla")
    - ``expanded_form``     Eq. "parallax_expand" (Sec. 3.3)
    - ``streaming_fold``    the one-pass tile walk of Sec. 3.3 (Algorithm 1) as a running fold of
                            per-tile states, with its final line
    - ``partial_state`` / ``merge_partials``  the unnormalised per-split state
                            (m, d1, d2, O1, O2) and the log-sum-exp merge of
                            App. "Kernel Optimization Details", item 3

Parity status: pinned (see tests/test_oracle_pins.py).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "parallax_oracle.c"
_LIB = _HERE / "libparallax_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (OpenMP, -O2, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        i32, f64, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        for name in ("parallax_oracle_decode_bf16", "parallax_oracle_decode_f64"):
            fn = getattr(lib, name)
            fn.restype = i32
            fn.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f64, i32]
        for name in ("parallax_oracle_prefill_bf16", "parallax_oracle_prefill_f64"):
            fn = getattr(lib, name)
            fn.restype = i32
            fn.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f64, i32]
        for name in ("parallax_oracle_backward_bf16", "parallax_oracle_backward_f64"):
            fn = getattr(lib, name)
            fn.restype = i32
            fn.argtypes = [vp] * 10 + [i32] * 6 + [f64, i32]
        lib.parallax_oracle_saved_state_bf16.restype = i32
        lib.parallax_oracle_saved_state_bf16.argtypes = [vp] * 8 + [i32] * 6 + [f64, i32]
        lib.parallax_oracle_max_threads.restype = i32
        lib.parallax_oracle_max_threads.argtypes = []
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().parallax_oracle_max_threads())


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact conversion of bf16 bit patterns (uint16) to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _call(fn, q, r, k, v, seqlens, scale, threads, dtype):
    q = np.ascontiguousarray(q, dtype=dtype)
    r = np.ascontiguousarray(r, dtype=dtype)
    k = np.ascontiguousarray(k, dtype=dtype)
    v = np.ascontiguousarray(v, dtype=dtype)
    B, Hq, D = q.shape
    Bk, Hkv, T_max, Dk = k.shape
    assert r.shape == q.shape and v.shape == k.shape and Bk == B and Dk == D
    sl_ptr = None
    if seqlens is not None:
        seqlens = np.ascontiguousarray(seqlens, dtype=np.int32)
        assert seqlens.shape == (B,)
        sl_ptr = seqlens.ctypes.data
    out = np.empty((B, Hq, D), dtype=np.float64)
    rc = fn(q.ctypes.data, r.ctypes.data, k.ctypes.data, v.ctypes.data, sl_ptr, out.ctypes.data,
            B, Hq, Hkv, D, T_max, float(scale), int(threads))
    if rc <= 0:
        raise RuntimeError(f"oracle returned {rc}")
    return out, rc


def decode_bf16(q, r, k, v, seqlens, scale, threads: int = 0):
    """Oracle on bf16 bit patterns (uint16 arrays). Returns (out float64 [B,Hq,D], threads used)."""
    return _call(_load().parallax_oracle_decode_bf16, q, r, k, v, seqlens, scale, threads, np.uint16)


def decode_f64(q, r, k, v, seqlens, scale, threads: int = 0):
    """Oracle on float64 arrays. Returns (out float64 [B,Hq,D], threads used)."""
    return _call(_load().parallax_oracle_decode_f64, q, r, k, v, seqlens, scale, threads, np.float64)


def _call_prefill(fn, q, r, k, v, seqlens, scale, threads, dtype):
    q = np.ascontiguousarray(q, dtype=dtype)
    r = np.ascontiguousarray(r, dtype=dtype)
    k = np.ascontiguousarray(k, dtype=dtype)
    v = np.ascontiguousarray(v, dtype=dtype)
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k.shape
    assert r.shape == q.shape and v.shape == k.shape and Bk == B and Dk == D
    sl_ptr = None
    if seqlens is not None:
        seqlens = np.ascontiguousarray(seqlens, dtype=np.int32)
        assert seqlens.shape == (B,)
        sl_ptr = seqlens.ctypes.data
    out = np.empty((B, Hq, Lq, D), dtype=np.float64)
    rc = fn(q.ctypes.data, r.ctypes.data, k.ctypes.data, v.ctypes.data, sl_ptr, out.ctypes.data,
            B, Hq, Hkv, D, Lq, T_max, float(scale), int(threads))
    if rc <= 0:
        raise RuntimeError(f"oracle returned {rc}")
    return out, rc


def prefill_bf16(q, r, k, v, seqlens, scale, threads: int = 0):
    """Multi-token causal forward on bf16 bit patterns: q, r [B,Hq,Lq,D]; the Lq tokens are the last
    Lq positions of each context and token i sees keys 0..L-Lq+i.  Returns (out [B,Hq,Lq,D], threads)."""
    return _call_prefill(_load().parallax_oracle_prefill_bf16, q, r, k, v, seqlens, scale, threads, np.uint16)


def prefill_f64(q, r, k, v, seqlens, scale, threads: int = 0):
    return _call_prefill(_load().parallax_oracle_prefill_f64, q, r, k, v, seqlens, scale, threads, np.float64)


def _call_backward(fn, q, r, k, v, dout, seqlens, scale, threads, dtype):
    q, r, k, v, dout = (np.ascontiguousarray(x, dtype=dtype) for x in (q, r, k, v, dout))
    B, Hq, Lq, D = q.shape
    Bk, Hkv, T_max, Dk = k.shape
    assert r.shape == q.shape and dout.shape == q.shape and v.shape == k.shape and Bk == B and Dk == D
    sl_ptr = None
    if seqlens is not None:
        seqlens = np.ascontiguousarray(seqlens, dtype=np.int32)
        assert seqlens.shape == (B,)
        sl_ptr = seqlens.ctypes.data
    dq, dr = np.empty(q.shape, dtype=np.float64), np.empty(q.shape, dtype=np.float64)
    dk, dv = np.empty(k.shape, dtype=np.float64), np.empty(k.shape, dtype=np.float64)
    rc = fn(q.ctypes.data, r.ctypes.data, k.ctypes.data, v.ctypes.data, dout.ctypes.data, sl_ptr,
            dq.ctypes.data, dr.ctypes.data, dk.ctypes.data, dv.ctypes.data, B, Hq, Hkv, D, Lq, T_max,
            float(scale), int(threads))
    if rc <= 0:
        raise RuntimeError(f"oracle returned {rc}")
    return dq, dr, dk, dv


def backward_bf16(q, r, k, v, dout, seqlens, scale, threads: int = 0):
    """Closed-form gradients (App. "Parallax Backward", Eq. "bwd_dq" .. "bwd_dv") on bf16 bit patterns.
    q, r, dout [B,Hq,Lq,D]; k, v [B,Hkv,T_max,D].  Returns (dq, dr, dk, dv) in float64."""
    return _call_backward(_load().parallax_oracle_backward_bf16, q, r, k, v, dout, seqlens, scale, threads, np.uint16)


def backward_f64(q, r, k, v, dout, seqlens, scale, threads: int = 0):
    return _call_backward(_load().parallax_oracle_backward_f64, q, r, k, v, dout, seqlens, scale, threads, np.float64)


def saved_state_bf16(q, r, k, v, seqlens, scale, threads: int = 0):
    """Per-row state a training forward saves for the backward: (lse [B,Hq,Lq], tbar [B,Hq,Lq],
    vbar [B,Hq,Lq,D]); lse = m + log(omega) in natural-log units, +inf for rows that see no key."""
    q, r, k, v = (np.ascontiguousarray(x, dtype=np.uint16) for x in (q, r, k, v))
    B, Hq, Lq, D = q.shape
    _, Hkv, T_max, _ = k.shape
    sl_ptr = None
    if seqlens is not None:
        seqlens = np.ascontiguousarray(seqlens, dtype=np.int32)
        sl_ptr = seqlens.ctypes.data
    lse, tbar = np.empty((B, Hq, Lq)), np.empty((B, Hq, Lq))
    vbar = np.empty((B, Hq, Lq, D))
    rc = _load().parallax_oracle_saved_state_bf16(q.ctypes.data, r.ctypes.data, k.ctypes.data, v.ctypes.data, sl_ptr,
                                                  lse.ctypes.data, tbar.ctypes.data, vbar.ctypes.data, B, Hq, Hkv, D,
                                                  Lq, T_max, float(scale), int(threads))
    if rc <= 0:
        raise RuntimeError(f"oracle returned {rc}")
    return lse, tbar, vbar


# ---------------------------------------------------------------------------
# Other forms of the same output, one (query head, context) at a time.
# q, r: [D]; K, V: [L, D]; all float64.
# ---------------------------------------------------------------------------

def _softmax_weights(q, K, scale):
    s = scale * (K @ q)
    w = np.exp(s - s.max())
    return w / w.sum()


def covariance_form(q, r, K, V, scale):
    """o_SA - Sigma_KV rho with Sigma_KV = E_p[(v - vbar)(k - kbar)^T] built explicitly
    (Sec. 3.1, Eq. "parallax_forward", right-hand side)."""
    p = _softmax_weights(q, K, scale)
    vbar = p @ V
    kbar = p @ K
    D = K.shape[1]
    sigma = np.zeros((V.shape[1], D))
    for j in range(K.shape[0]):
        sigma += p[j] * np.outer(V[j] - vbar, K[j] - kbar)
    return vbar - sigma @ r


def expanded_form(q, r, K, V, scale):
    """(sum p v)(1 + sum p k.rho) - sum (p k.rho) v   (Sec. 3.3, Eq. "parallax_expand")."""
    p = _softmax_weights(q, K, scale)
    t = K @ r
    return (p @ V) * (1.0 + p @ t) - (p * t) @ V


def partial_state(q, r, K, V, scale, k0, k1):
    """Unnormalised state (m, d1, d2, O1, O2) of the key range [k0, k1), relative to its own
    maximum logit m (natural-log units); an empty range gives (-inf, 0, 0, 0, 0)
    (App. "Kernel Optimization Details", item 3)."""
    Dv = V.shape[1]
    if k1 <= k0:
        return -np.inf, 0.0, 0.0, np.zeros(Dv), np.zeros(Dv)
    Kc, Vc = K[k0:k1], V[k0:k1]
    S1 = (Kc @ q) * scale
    m = S1.max()
    P1 = np.exp(S1 - m)
    P2 = P1 * (Kc @ r)
    return m, P1.sum(), P2.sum(), P1 @ Vc, P2 @ Vc


def merge_partials(states):
    """Log-sum-exp merge of per-split states followed by Algorithm 1's final line
    (App. "Kernel Optimization Details", item 3).  All-empty input gives zeros."""
    Dv = states[0][3].shape[0]
    M = max(s[0] for s in states)
    if not np.isfinite(M):
        return np.zeros(Dv)
    d1 = d2 = 0.0
    O1, O2 = np.zeros(Dv), np.zeros(Dv)
    for (m, a1, a2, B1, B2) in states:
        if not np.isfinite(m):
            continue
        a = np.exp(m - M)
        d1 += a * a1
        d2 += a * a2
        O1 += a * B1
        O2 += a * B2
    return O1 / d1 * (1.0 + d2 / d1) - O2 / d1


def streaming_fold(q, r, K, V, scale, Bc):
    """The single-pass computation of Sec. 3.3 (Algorithm 1) for one query row, stated as a running
    fold: the context is walked once in tiles of Bc keys; each tile's unnormalised state is taken
    relative to the tile's own maximum logit and absorbed into the running state, whichever of the two
    has the smaller reference being rescaled to the larger one.  Both branches (softmax sums and
    probe-weighted sums) share the one reference exponent, which only the softmax logits determine.
    Natural exp with the plain scale; the paper's exp2 with log2(e) folded into s is the same quantity."""
    run = (-np.inf, 0.0, 0.0, np.zeros(V.shape[1]), np.zeros(V.shape[1]))
    for lo in range(0, K.shape[0], Bc):
        tile = partial_state(q, r, K, V, scale, lo, min(lo + Bc, K.shape[0]))
        ref = max(run[0], tile[0])
        keep, take = np.exp(run[0] - ref), np.exp(tile[0] - ref)
        run = (ref,) + tuple(keep * a + take * b for a, b in zip(run[1:], tile[1:]))
    _, d1, d2, O1, O2 = run
    return O1 / d1 * (1.0 + d2 / d1) - O2 / d1


# ---------------------------------------------------------------------------
# Upstream step of a decode call: RMSNorm and rotary embedding of the new token's q, rho, k and the
# append of k, v to the cache (Sec. 4.2 and App. "Backbone Architecture": RMSNorm on q, k and rho;
# RoPE with base theta on q and k, optionally on rho with the same base).
# Readings where the paper is silent (conventions of the Qwen-3 backbone it names): the norm is
# x / sqrt(mean(x^2) + eps) * weight over the head dimension; RoPE pairs element i with i + D/2
# ("rotate half") and rotates the pair by pos * theta^(-2i/D); the norm comes before the rotation.
# ---------------------------------------------------------------------------

def rmsnorm(x, weight, eps):
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * np.asarray(weight, dtype=np.float64)


def rope(x, pos, theta):
    """Rotate-half rotary embedding of the last axis (even length D) at integer position(s) `pos`
    (broadcast against x's leading axes)."""
    x = np.asarray(x, dtype=np.float64)
    D = x.shape[-1]
    half = D // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / D)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def prepare_step(q_raw, r_raw, k_raw, v_raw, wq, wr, wk, seqlens, eps, theta, rope_on_r):
    """q_raw, r_raw [B,Hq,D], k_raw, v_raw [B,Hkv,D] (float64).  Returns q, r [B,Hq,D] and the rows
    k_new, v_new [B,Hkv,D] that belong at cache position seqlens[b] - 1 (the new token is counted)."""
    pos = (np.asarray(seqlens, dtype=np.int64) - 1)[:, None]
    q = rope(rmsnorm(q_raw, wq, eps), pos, theta)
    r = rmsnorm(r_raw, wr, eps)
    if rope_on_r:
        r = rope(r, pos, theta)
    k = rope(rmsnorm(k_raw, wk, eps), pos, theta)
    return q, r, k, np.asarray(v_raw, dtype=np.float64)
