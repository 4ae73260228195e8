"""The options-struct entry point (parallax_decode_fwd_args): bit-identical to the specific entry points
where one exists, and parity against the oracle for combinations none of them names."""
import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import assert_parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def plx(cuda_device):
    from paper_2605_29157_b200 import binding
    return binding


def test_args_entry_equals_the_specific_entries(plx):
    cfg = wl.DecodeConfig("args", B=3, Hq=8, Hkv=2, D=128, T_max=1500, ragged=(1, 1500), seed=2300)
    x = wl.make_inputs(cfg, "cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * 4, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device="cuda")
    a, b = new(cfg.B, cfg.Hq, cfg.D), new(cfg.B, cfg.Hq, cfg.D)
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], a, cfg.scale, ws, 0)
    plx.parallax_decode_fwd_args(x["q"], x["r"], x["k"], x["v"], x["seqlens"], b, cfg.scale, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    # paged
    kp, vp, table = wl.to_paged(x["k"], x["v"], 64, seed=1)
    plx.parallax_decode_fwd_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], a, cfg.scale, ws, 3)
    plx.parallax_decode_fwd_args(x["q"], x["r"], kp, vp, x["seqlens"], b, cfg.scale, block_table=table, workspace=ws,
                                 num_splits=3)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    # e4m3, per-tensor and per-head scales
    k8, ks = wl.quantize_e4m3(x["k"])
    v8, vs = wl.quantize_e4m3(x["v"])
    plx.parallax_decode_fwd_fp8(x["q"], x["r"], k8, v8, x["seqlens"], a, cfg.scale, ks, vs, ws, 0)
    plx.parallax_decode_fwd_args(x["q"], x["r"], k8, v8, x["seqlens"], b, cfg.scale, k_scale=ks, v_scale=vs, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    k8h, ksh = wl.quantize_e4m3_per_head(x["k"])
    v8h, vsh = wl.quantize_e4m3_per_head(x["v"])
    plx.parallax_decode_fwd_fp8_per_head(x["q"], x["r"], k8h, v8h, x["seqlens"], a, cfg.scale, ksh, vsh, ws, 2)
    plx.parallax_decode_fwd_args(x["q"], x["r"], k8h, v8h, x["seqlens"], b, cfg.scale, k_scale=ksh, v_scale=vsh,
                                 workspace=ws, num_splits=2)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    # several tokens (four rows per KV head: both entries use the decode kernel; from five rows on at this head dimension
    # the routed entry hands the step to the keys-on-lanes kernel, which rounds differently)
    cfg2 = wl.DecodeConfig("args multi", B=3, Hq=4, Hkv=2, D=128, T_max=1500, ragged=(2, 1500), seed=2301)
    y = wl.make_prefill_inputs(cfg2, 2, "cuda")
    assert plx.parallax_decode_multi_plan(cfg2.B, cfg2.Hq, cfg2.Hkv, cfg2.D, 2, cfg2.T_max)[0] == plx.PLX_MULTI_KERNEL_DECODE
    a4, b4 = new(cfg2.B, cfg2.Hq, 2, cfg2.D), new(cfg2.B, cfg2.Hq, 2, cfg2.D)
    plx.parallax_decode_fwd_multi(y["q"], y["r"], y["k"], y["v"], y["seqlens"], a4, cfg2.scale, ws, 0)
    plx.parallax_decode_fwd_args(y["q"], y["r"], y["k"], y["v"], y["seqlens"], b4, cfg2.scale, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(a4, b4)


@pytest.mark.parametrize("Lq,page_size,per_head,ns", [(3, 64, True, 0), (4, 128, False, 5), (2, 16, True, 1)])
def test_several_tokens_over_a_paged_e4m3_cache(plx, oracle, Lq, page_size, per_head, ns):
    """A combination only the options struct reaches: multi-token step + paged pools + e4m3 bytes (+ per-head
    scales).  Oracle: the multi-token causal forward on the dequantised cache."""
    cfg = wl.DecodeConfig("args combo", B=3, Hq=4, Hkv=2, D=128, T_max=1200, ragged=(Lq, 1200), seed=2400 + Lq)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    if per_head:
        k8, ks = wl.quantize_e4m3_per_head(x["k"])
        v8, vs = wl.quantize_e4m3_per_head(x["v"])
        ksn, vsn = ks.cpu().numpy().astype(np.float64)[None, :, None, None], vs.cpu().numpy().astype(np.float64)[None, :, None, None]
    else:
        k8, ks = wl.quantize_e4m3(x["k"])
        v8, vs = wl.quantize_e4m3(x["v"])
        ks, vs = float(np.float32(ks)), float(np.float32(vs))
        ksn, vsn = ks, vs
    kp, vp, table = wl.to_paged(k8.to(torch.float16), v8.to(torch.float16), page_size, seed=9)
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, plx.PLX_MAX_SPLITS if ns == 0 else ns, "cuda")
    plx.parallax_decode_fwd_args(x["q"], x["r"], kp.to(torch.float8_e4m3fn), vp.to(torch.float8_e4m3fn), x["seqlens"], out,
                                 cfg.scale, block_table=table, k_scale=ks, v_scale=vs, workspace=ws, num_splits=ns)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    kd = k8.float().cpu().numpy().astype(np.float64) * ksn
    vd = v8.float().cpu().numpy().astype(np.float64) * vsn
    want, _ = oracle.prefill_f64(x["q"].double().cpu().numpy(), x["r"].double().cpu().numpy(), kd, vd,
                                 x["seqlens_host"], cfg.scale)
    assert_parity(out.cpu().numpy(), want, torch.float32, "multi + paged + e4m3")


def test_args_entry_rejects_bad_structs(plx):
    import ctypes
    a = plx.ParallaxDecodeArgs()
    assert plx._lib.parallax_decode_fwd_args(None) == plx.PLX_ERR_NULL_POINTER
    a.struct_bytes = 8
    assert plx._lib.parallax_decode_fwd_args(ctypes.byref(a)) == plx.PLX_ERR_BAD_SHAPE
    a.struct_bytes = ctypes.sizeof(plx.ParallaxDecodeArgs) + 8
    assert plx._lib.parallax_decode_fwd_args(ctypes.byref(a)) == plx.PLX_ERR_BAD_SHAPE
    a.struct_bytes = ctypes.sizeof(plx.ParallaxDecodeArgs)
    a.Hq, a.Hkv, a.kv_dtype = 4, 2, 7
    assert plx._lib.parallax_decode_fwd_args(ctypes.byref(a)) == plx.PLX_ERR_BAD_SHAPE
