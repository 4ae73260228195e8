"""The index-checking debug build (-DPLX_DEBUG_CHECKS): compiles from the same sources, exports the same
symbols, gives the same results, and reports an out-of-range index through the status word instead of
following it.  This is the library's stand-in for a memory checker on machines where none can be run."""
import ctypes
import importlib.util
import os

import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import assert_parity, oracle_full


@pytest.fixture(scope="module")
def debug_lib_path():
    from paper_2605_29157_b200 import build
    return build.build(debug_checks=True)


def test_debug_build_exports_the_same_symbols(debug_lib_path):
    from paper_2605_29157_b200 import binding
    lib = ctypes.CDLL(str(debug_lib_path))
    for name in binding.EXPORTS + binding.TEST_HOOK_EXPORTS:
        assert hasattr(lib, name), name
    lib.parallax_status_string.restype = ctypes.c_char_p
    assert b"debug build" in lib.parallax_status_string(binding.PLX_ERR_DEVICE_CHECK)


@pytest.fixture(scope="module")
def dbg(debug_lib_path, cuda_device):
    """A second instance of the binding module bound to the debug library (PARALLAX_LIBRARY)."""
    from paper_2605_29157_b200 import binding
    old = os.environ.get("PARALLAX_LIBRARY")
    os.environ["PARALLAX_LIBRARY"] = str(debug_lib_path)
    try:
        spec = importlib.util.spec_from_file_location("paper_2605_29157_b200._binding_debug", binding.__file__)
        mod = importlib.util.module_from_spec(spec)
        spec.loader.exec_module(mod)
    finally:
        if old is None:
            del os.environ["PARALLAX_LIBRARY"]
        else:
            os.environ["PARALLAX_LIBRARY"] = old
    assert str(mod.LIB_PATH) == str(debug_lib_path)
    return mod


@pytest.mark.gpu
@pytest.mark.parametrize("D,G,T,ns,ragged", [(128, 2, 1000, 1, False), (128, 2, 5000, 7, True), (64, 4, 3000, 0, True),
                                             (128, 3, 777, 4, False), (128, 8, 1500, 5, True), (64, 1, 17, 1, False)])
def test_small_parity_cases_through_the_checking_build(dbg, oracle, D, G, T, ns, ragged):
    cfg = wl.DecodeConfig("dbg", B=3, Hq=2 * G, Hkv=2, D=D, T_max=T, ragged=(1, T) if ragged else None, seed=31 + T)
    x = wl.make_inputs(cfg, "cuda", poison_padding=True)
    want = oracle_full(oracle, x, cfg.scale, x["seqlens_host"])
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = dbg.alloc_workspace(cfg.B, cfg.Hq, cfg.D, dbg.PLX_MAX_SPLITS, "cuda")
    dbg.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, ns)
    torch.cuda.synchronize()
    assert dbg.parallax_workspace_status(ws) == 0
    assert_parity(out.cpu().numpy(), want, torch.float32, "checking build, contiguous")
    # paged cache, the stand-alone split + combine pair and the scratch-free entry on the same inputs
    kp, vp, table = wl.to_paged(x["k"], x["v"], 64, seed=5)
    out.fill_(float("nan"))
    lens = x["seqlens"] if x["seqlens"] is not None else torch.full((cfg.B,), T, dtype=torch.int32, device="cuda")
    dbg.parallax_decode_fwd_paged(x["q"], x["r"], kp, vp, table, lens, out, cfg.scale, ws, ns)
    torch.cuda.synchronize()
    assert dbg.parallax_workspace_status(ws) == 0
    assert_parity(out.cpu().numpy(), want, torch.float32, "checking build, paged")
    out.fill_(float("nan"))
    dbg.parallax_decode_fwd_static(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ns)
    torch.cuda.synchronize()
    assert_parity(out.cpu().numpy(), want, torch.float32, "checking build, static scratch")


@pytest.mark.gpu
def test_a_page_id_outside_the_pool_is_reported_not_followed(dbg):
    """A block table that names a page the pool does not have: the checking build sets the status word
    to PLX_ERR_DEVICE_CHECK and reads page 0 instead; nothing faults and the next call is clean."""
    cfg = wl.DecodeConfig("dbg-page", B=2, Hq=4, Hkv=2, D=128, T_max=512, seed=77)
    x = wl.make_inputs(cfg, "cuda")
    kp, vp, table = wl.to_paged(x["k"], x["v"], 64, seed=6)
    good = table.clone()
    table[1, 3] = kp.shape[0] + 40
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = dbg.alloc_workspace(cfg.B, cfg.Hq, cfg.D, 8, "cuda")
    dbg.parallax_decode_fwd_paged(x["q"], x["r"], kp, vp, table, None, out, cfg.scale, ws, 1)
    torch.cuda.synchronize()
    assert dbg.parallax_workspace_status(ws) == dbg.PLX_ERR_DEVICE_CHECK
    assert torch.isfinite(out).all()
    ws.zero_()
    dbg.parallax_decode_fwd_paged(x["q"], x["r"], kp, vp, good, None, out, cfg.scale, ws, 1)
    torch.cuda.synchronize()
    assert dbg.parallax_workspace_status(ws) == 0


@pytest.mark.gpu
def test_multi_token_step_through_the_checking_build(dbg, oracle):
    """Twelve and 24 rows per KV head (the keys-on-lanes kernel) through the checking build: same results over a
    contiguous and a paged cache; a page id outside the pool is reported through the status word, not followed."""
    Lq = 6
    for G in (2, 4):
        cfg = wl.DecodeConfig("dbg-rows", B=3, Hq=2 * G, Hkv=2, D=128, T_max=900, ragged=(Lq, 900), seed=91 + G)
        x = wl.make_prefill_inputs(cfg, Lq, "cuda")
        bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
        want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], x["seqlens_host"], cfg.scale)
        out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
        ws = dbg.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, 8, "cuda")
        dbg.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, 0)
        torch.cuda.synchronize()
        assert dbg.parallax_workspace_status(ws) == 0
        assert_parity(out.cpu().numpy(), want, torch.float32, f"checking build, {G * Lq} rows")
        kp, vp, table = wl.to_paged(x["k"], x["v"], 32, seed=4)
        out.fill_(float("nan"))
        dbg.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, 3)
        torch.cuda.synchronize()
        assert dbg.parallax_workspace_status(ws) == 0
        assert_parity(out.cpu().numpy(), want, torch.float32, f"checking build, paged, {G * Lq} rows")
    bad = table.clone()
    bad[0, 0] = kp.shape[0] + 17
    dbg.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, bad, x["seqlens"], out, cfg.scale, ws, 1)
    torch.cuda.synchronize()
    assert dbg.parallax_workspace_status(ws) == dbg.PLX_ERR_DEVICE_CHECK
    assert torch.isfinite(out).all()
    ws.zero_()
    dbg.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, 1)
    torch.cuda.synchronize()
    assert dbg.parallax_workspace_status(ws) == 0
