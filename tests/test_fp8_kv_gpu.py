"""GPU parity of the decode forward over an e4m3 KV cache.  The cache values the kernel sees are
exactly k8 * k_scale and v8 * v_scale, so the oracle is the unchanged fp64 decode oracle on those
dequantised values, and the bars are those of the 16-bit path."""
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


def run_case(plx, oracle, cfg, out_dtype=torch.float32, num_splits=0, poison=False):
    x = wl.make_inputs(cfg, "cuda", poison_padding=poison)
    k8, ks = wl.quantize_e4m3(x["k"])
    v8, vs = wl.quantize_e4m3(x["v"])
    ks32, vs32 = float(np.float32(ks)), float(np.float32(vs))   # what the C ABI receives
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=out_dtype, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS if num_splits == 0 else num_splits, "cuda")
    plx.parallax_decode_fwd_fp8(x["q"], x["r"], k8, v8, x["seqlens"], out, cfg.scale, ks32, vs32, ws, num_splits)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    kd = k8.float().cpu().numpy().astype(np.float64) * ks32
    vd = v8.float().cpu().numpy().astype(np.float64) * vs32
    sl = x["seqlens_host"]
    if sl is not None:  # the oracle never reads past a context; keep NaN padding out of its inputs anyway
        for b in range(cfg.B):
            kd[b, :, int(sl[b]):] = 0.0
            vd[b, :, int(sl[b]):] = 0.0
    qd, rd = x["q"].double().cpu().numpy(), x["r"].double().cpu().numpy()
    want, _ = oracle.decode_f64(qd, rd, kd, vd, sl, cfg.scale)
    return assert_parity(out.float().cpu().numpy(), want, out_dtype, cfg.name)


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("T", [1, 2, 15, 16, 17, 63, 64, 65, 127, 300, 1000])
def test_fp8_shape_sweep_single_split(plx, oracle, D, G, T):
    """D = 64: 64-byte cache rows, staged in boxes with the 64-byte swizzle."""
    cfg = wl.DecodeConfig(f"fp8 D={D} G={G} T={T}", B=2, Hq=2 * G, Hkv=2, D=D, T_max=T, seed=900 + T)
    run_case(plx, oracle, cfg, num_splits=1)


@pytest.mark.parametrize("D,G", [(128, 1), (128, 2), (128, 4), (64, 2), (64, 3), (128, 7), (64, 8)])
@pytest.mark.parametrize("T,ns", [(130, 2), (1000, 3), (4096, 0), (5000, 7), (12800, 120)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_fp8_split_kv(plx, oracle, D, G, T, ns, out_dtype):
    cfg = wl.DecodeConfig(f"fp8 split D={D} G={G} T={T} ns={ns}", B=3, Hq=2 * G, Hkv=2, D=D, T_max=T, seed=11 * T + ns)
    run_case(plx, oracle, cfg, out_dtype=out_dtype, num_splits=ns)


def test_fp8_head_dim_64_ragged_paged_and_groups_above_four(plx, oracle):
    """The compute-matched shape over an e4m3 cache: ragged lengths with NaN padding, a paged cache, and a
    group of eight query heads (one CTA per KV head, two accumulator sets)."""
    cfg = wl.DecodeConfig("fp8 d64 ragged", B=5, Hq=16, Hkv=2, D=64, T_max=2500, ragged=(1, 2500), seed=955)
    run_case(plx, oracle, cfg, poison=True)
    x = wl.make_inputs(cfg, "cuda", poison_padding=True)
    k8, ks = wl.quantize_e4m3(x["k"])
    v8, vs = wl.quantize_e4m3(x["v"])
    ks32, vs32 = float(np.float32(ks)), float(np.float32(vs))
    kp, vp, table = wl.to_paged(k8.to(torch.float16), v8.to(torch.float16), 64, seed=3)   # fp16 holds every e4m3 value and NaN
    kp, vp = kp.to(torch.float8_e4m3fn), vp.to(torch.float8_e4m3fn)
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    ref = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    got = torch.full_like(ref, float("nan"))
    plx.parallax_decode_fwd_fp8(x["q"], x["r"], k8, v8, x["seqlens"], ref, cfg.scale, ks32, vs32, ws, 3)
    plx.parallax_decode_fwd_paged_fp8(x["q"], x["r"], kp, vp, table, x["seqlens"], got, cfg.scale, ks32, vs32, ws, 3)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    # same arithmetic, but the padded paged context is cut into other chunks: equal up to fp32 summation order
    assert torch.isfinite(got).all() and (got - ref).abs().max().item() <= 1e-4 * ref.abs().max().item()


def test_fp8_ragged_batch_with_poisoned_padding(plx, oracle):
    cfg = wl.DecodeConfig("fp8 ragged", B=6, Hq=8, Hkv=4, D=128, T_max=3000, ragged=(1, 3000), seed=931)
    run_case(plx, oracle, cfg, poison=True)


def test_fp8_large_probe(plx, oracle):
    """Probe scores of a few hundred: P2 = P1 * S2 has to stay inside the fp16 range on its way to the
    value product (the lazy-rescale threshold of this variant is chosen for that)."""
    cfg = wl.DecodeConfig("fp8 probe", B=2, Hq=4, Hkv=2, D=128, T_max=777, seed=932)
    x = wl.make_inputs(cfg, "cuda")
    x["r"] = (x["r"].float() * 12.0).to(torch.bfloat16)
    k8, ks = wl.quantize_e4m3(x["k"])
    v8, vs = wl.quantize_e4m3(x["v"])
    ks32, vs32 = float(np.float32(ks)), float(np.float32(vs))
    out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_fp8(x["q"], x["r"], k8, v8, None, out, cfg.scale, ks32, vs32, None, 1)
    torch.cuda.synchronize()
    want, _ = oracle.decode_f64(x["q"].double().cpu().numpy(), x["r"].double().cpu().numpy(),
                                k8.float().cpu().numpy().astype(np.float64) * ks32,
                                v8.float().cpu().numpy().astype(np.float64) * vs32, None, cfg.scale)
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # outputs reach |o| ~ 1e2 here: the bar is relative
    assert np.sqrt(np.mean((got - want) ** 2)) <= 2e-4 * np.sqrt(np.mean(want ** 2))


def test_fp8_rejects_other_head_dims_and_bad_scales(plx):
    cfg = wl.DecodeConfig("fp8 d32", B=1, Hq=2, Hkv=1, D=32, T_max=64, seed=1)
    x = wl.make_inputs(cfg, "cuda")
    k8, _ = wl.quantize_e4m3(x["k"])
    out = torch.empty(1, 2, 32, dtype=torch.float32, device="cuda")
    with pytest.raises(plx.ParallaxError) as e:
        plx.parallax_decode_fwd_fp8(x["q"], x["r"], k8, k8, None, out, 0.1, 1.0, 1.0, None, 1)
    assert e.value.status == plx.PLX_ERR_UNSUPPORTED
    with pytest.raises(plx.ParallaxError) as e:
        plx.parallax_decode_fwd_fp8(x["q"], x["r"], k8, k8, None, out, 0.1, 0.0, 1.0, None, 1)
    assert e.value.status == plx.PLX_ERR_BAD_SHAPE


@pytest.mark.parametrize("page_size,T,ns", [(16, 300, 1), (64, 1000, 0), (128, 2500, 7)])
def test_fp8_paged_cache(plx, oracle, page_size, T, ns):
    """Paged e4m3 cache: quantise, scatter into page pools under a random page order (unused pages and
    page tails hold NaN bytes), decode through the block table."""
    cfg = wl.DecodeConfig("fp8 paged", B=3, Hq=4, Hkv=2, D=128, T_max=T, ragged=(1, T), seed=940 + page_size)
    x = wl.make_inputs(cfg, "cuda")
    k8, ks = wl.quantize_e4m3(x["k"])
    v8, vs = wl.quantize_e4m3(x["v"])
    ks32, vs32 = float(np.float32(ks)), float(np.float32(vs))
    # to_paged works on any dtype that can hold NaN: scatter the fp16 images, then requantise exactly
    kp, vp, table = wl.to_paged(k8.to(torch.float16), v8.to(torch.float16), page_size, seed=3)
    kp8, vp8 = kp.to(torch.float8_e4m3fn), vp.to(torch.float8_e4m3fn)
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS if ns == 0 else ns, "cuda")
    plx.parallax_decode_fwd_paged_fp8(x["q"], x["r"], kp8, vp8, table, x["seqlens"], out, cfg.scale, ks32, vs32, ws, ns)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    sl = x["seqlens_host"]
    kd = k8.float().cpu().numpy().astype(np.float64) * ks32
    vd = v8.float().cpu().numpy().astype(np.float64) * vs32
    want, _ = oracle.decode_f64(x["q"].double().cpu().numpy(), x["r"].double().cpu().numpy(), kd, vd, sl, cfg.scale)
    assert_parity(out.cpu().numpy(), want, torch.float32, f"fp8 paged ps={page_size}")


def _per_head_case(cfg, seed_gain):
    """Inputs whose KV heads have very different magnitudes (a per-tensor scale would waste most of the
    e4m3 range on the small heads), quantised per head."""
    x = wl.make_inputs(cfg, "cuda")
    gains = torch.tensor([4.0 ** ((h * seed_gain) % 5 - 2) for h in range(cfg.Hkv)], device="cuda")
    x["k"] = (x["k"].float() * gains[None, :, None, None]).to(torch.bfloat16)
    x["v"] = (x["v"].float() * gains.flip(0)[None, :, None, None]).to(torch.bfloat16)
    k8, ks = wl.quantize_e4m3_per_head(x["k"])
    v8, vs = wl.quantize_e4m3_per_head(x["v"])
    kd = k8.float().cpu().numpy().astype(np.float64) * ks.cpu().numpy().astype(np.float64)[None, :, None, None]
    vd = v8.float().cpu().numpy().astype(np.float64) * vs.cpu().numpy().astype(np.float64)[None, :, None, None]
    return x, k8, v8, ks, vs, kd, vd


@pytest.mark.parametrize("Hq,Hkv,T,ns", [(4, 2, 300, 1), (16, 8, 4096, 0), (12, 4, 2500, 5), (16, 2, 1000, 0)])
def test_fp8_per_head_scales(plx, oracle, Hq, Hkv, T, ns):
    cfg = wl.DecodeConfig("fp8 per head", B=3, Hq=Hq, Hkv=Hkv, D=128, T_max=T, ragged=(1, T), seed=960 + T)
    x, k8, v8, ks, vs, kd, vd = _per_head_case(cfg, 3)
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS if ns == 0 else ns, "cuda")
    plx.parallax_decode_fwd_fp8_per_head(x["q"], x["r"], k8, v8, x["seqlens"], out, cfg.scale, ks, vs, ws, ns)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    want, _ = oracle.decode_f64(x["q"].double().cpu().numpy(), x["r"].double().cpu().numpy(), kd, vd,
                                x["seqlens_host"], cfg.scale)
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # head magnitudes span 4^-2 .. 4^2: the bar is relative to each KV head's output scale
    G = Hq // Hkv
    for h in range(Hkv):
        w, g = want[:, h * G:(h + 1) * G], got[:, h * G:(h + 1) * G]
        assert np.sqrt(np.mean((g - w) ** 2)) <= 2e-4 * max(np.sqrt(np.mean(w ** 2)), 1e-30), h
    # equal scales reproduce the per-tensor entry point bit for bit
    one_k, one_v = float(ks.max()), float(vs.max())
    k8u, v8u = (x["k"].float() / one_k).to(torch.float8_e4m3fn), (x["v"].float() / one_v).to(torch.float8_e4m3fn)
    a, b = torch.empty_like(out), torch.empty_like(out)
    plx.parallax_decode_fwd_fp8(x["q"], x["r"], k8u, v8u, x["seqlens"], a, cfg.scale, one_k, one_v, ws, ns)
    plx.parallax_decode_fwd_fp8_per_head(x["q"], x["r"], k8u, v8u, x["seqlens"], b, cfg.scale,
                                         torch.full_like(ks, one_k), torch.full_like(vs, one_v), ws, ns)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_fp8_per_head_scales_paged(plx, oracle):
    cfg = wl.DecodeConfig("fp8 per head paged", B=3, Hq=8, Hkv=4, D=128, T_max=1500, ragged=(1, 1500), seed=977)
    x, k8, v8, ks, vs, kd, vd = _per_head_case(cfg, 2)
    kp, vp, table = wl.to_paged(k8.to(torch.float16), v8.to(torch.float16), 64, seed=5)
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    plx.parallax_decode_fwd_paged_fp8_per_head(x["q"], x["r"], kp.to(torch.float8_e4m3fn), vp.to(torch.float8_e4m3fn),
                                               table, x["seqlens"], out, cfg.scale, ks, vs, ws, 0)
    ref = torch.empty_like(out)
    plx.parallax_decode_fwd_fp8_per_head(x["q"], x["r"], k8, v8, x["seqlens"], ref, cfg.scale, ks, vs, ws, 0)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    want, _ = oracle.decode_f64(x["q"].double().cpu().numpy(), x["r"].double().cpu().numpy(), kd, vd,
                                x["seqlens_host"], cfg.scale)
    got = out.cpu().numpy().astype(np.float64)
    assert np.sqrt(np.mean((got - want) ** 2)) <= 2e-4 * np.sqrt(np.mean(want ** 2))
    assert np.abs(got - ref.cpu().numpy()).max() <= 1e-5 * np.abs(want).max()
