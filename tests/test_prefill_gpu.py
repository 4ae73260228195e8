"""GPU parity of the multi-token causal forward (tcgen05 kernel) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import MAX_ABS_TOL, MEAN_ABS_TOL, errors

pytestmark = pytest.mark.gpu

# Same bars as the decode path: the stated absolute ones, plus the internal relative-RMS bars
# (P reaches the second product as bf16 plus its bf16 residual, so accuracy is fp32-class).
from parity_util import REL_RMS_TOL_BF16, REL_RMS_TOL_F32


@pytest.fixture(scope="module")
def plx(cuda_device):
    from paper_2605_29157_b200 import binding
    return binding


def run_case(plx, oracle, cfg, Lq, out_dtype=torch.float32, poison=False, seqlens=None):
    x = wl.make_prefill_inputs(cfg, Lq, "cuda", poison_padding=poison)
    sl_host = x["seqlens_host"]
    if seqlens is not None:
        sl_host = np.asarray(seqlens, dtype=np.int32)
        x["seqlens"] = torch.from_numpy(sl_host).cuda()
        for b in range(cfg.B):
            x["k"][b, :, int(sl_host[b]):] = float("nan")
            x["v"][b, :, int(sl_host[b]):] = float("nan")
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=out_dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_prefill_fwd(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], sl_host, cfg.scale)
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    e = errors(got, want)
    if out_dtype == torch.float32:
        assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= REL_RMS_TOL_F32, e
    else:
        # Early causal rows reach |o| ~ 10-30, where half a bf16 ulp (2^-9 |o|) alone exceeds 2e-2:
        # the element bound is the stated bar or the output format's own rounding, whichever is larger.
        bound = np.maximum(MAX_ABS_TOL, 2.0 ** -8 * np.abs(want))
        assert (np.abs(got - want) <= bound).all(), e
        assert e["mean_abs"] <= max(MEAN_ABS_TOL, 2.0 ** -9 * float(np.abs(want).mean())), e
        assert e["rel_rms"] <= REL_RMS_TOL_BF16, e
    return e


@pytest.mark.parametrize("Lq,T", [(128, 128), (1, 128), (1, 300), (37, 37), (100, 500), (256, 256), (300, 1000), (512, 512)])
def test_prefill_shapes(plx, oracle, Lq, T):
    """Full prefill (Lq = context), chunked prefill (Lq < context), single-token, ragged tiles."""
    cfg = wl.DecodeConfig("pf", B=2, Hq=4, Hkv=2, D=128, T_max=T, seed=300 + Lq + T)
    print(run_case(plx, oracle, cfg, Lq))


@pytest.mark.parametrize("G", [1, 2, 4])
def test_prefill_gqa_and_bf16_out(plx, oracle, G):
    cfg = wl.DecodeConfig("pfg", B=1, Hq=2 * G, Hkv=2, D=128, T_max=640, seed=310 + G)
    run_case(plx, oracle, cfg, 384, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("Lq,T,out_dtype", [(1, 200, torch.float32), (130, 130, torch.float32), (200, 777, torch.bfloat16),
                                            (512, 512, torch.float32)])
def test_prefill_head_dim_64(plx, oracle, Lq, T, out_dtype):
    """The compute-matched head dimension (64): one 64-column box per row, four k-steps per score product."""
    cfg = wl.DecodeConfig("pf64", B=2, Hq=4, Hkv=2, D=64, T_max=T, ragged=(max(1, T // 2), T), seed=350 + Lq)
    run_case(plx, oracle, cfg, Lq, out_dtype=out_dtype, poison=True)


def test_prefill_ragged_poisoned_and_short_contexts(plx, oracle):
    """Per-sequence context lengths with NaN padding; one context shorter than Lq (its first tokens
    see no key and give zeros), one of exactly Lq, one empty."""
    cfg = wl.DecodeConfig("pfr", B=5, Hq=4, Hkv=2, D=128, T_max=700, seed=320)
    run_case(plx, oracle, cfg, 200, seqlens=[700, 333, 200, 150, 0])


def test_prefill_matches_decode_entry_for_one_token(plx, oracle):
    """Lq = 1 is the decode step: both entry points against each other on the same inputs."""
    cfg = wl.DecodeConfig("pf1", B=3, Hq=8, Hkv=4, D=128, T_max=2000, seed=330)
    x = wl.make_inputs(cfg, "cuda")
    dec = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, dec, cfg.scale, None, 1)
    pre = torch.empty(cfg.B, cfg.Hq, 1, cfg.D, dtype=torch.float32, device="cuda")
    plx.parallax_prefill_fwd(x["q"].unsqueeze(2).contiguous(), x["r"].unsqueeze(2).contiguous(), x["k"], x["v"], None, pre, cfg.scale)
    torch.cuda.synchronize()
    e = errors(pre[:, :, 0].cpu().numpy(), dec.cpu().numpy())
    assert e["rel_rms"] <= REL_RMS_TOL_F32 and e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL, e


def test_prefill_plain_bf16_weights(plx, oracle):
    """PLX_P_BF16: the weights reach the value product as plain bf16.  On a chunked-prefill shape (every
    row sees >= 2000 keys) the rounding averages out and the stated bars hold; the relative RMS error is
    of the order 2^-9 * sqrt(D) / sqrt(effective keys)."""
    cfg = wl.DecodeConfig("pfb", B=2, Hq=4, Hkv=2, D=128, T_max=2304, seed=340)
    Lq = 256
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    out = torch.empty(cfg.B, cfg.Hq, Lq, cfg.D, dtype=torch.float32, device="cuda")
    plx.parallax_prefill_fwd(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, p_precision=plx.PLX_P_BF16)
    torch.cuda.synchronize()
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    e = errors(out.cpu().numpy(), want)
    assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= 1e-2, e


@pytest.mark.parametrize("D,G,Lq,T", [(128, 2, 2500, 2500), (64, 2, 2400, 2400), (128, 1, 700, 1900), (128, 4, 16, 3000),
                                      (128, 4, 20, 600)])
def test_prefill_adaptive_residuals(plx, oracle, D, G, Lq, T):
    """PLX_P_BF16_ADAPTIVE: row tiles in which some row sees fewer than PLX_P_ADAPTIVE_MIN_KEYS keys carry the
    residual products and keep the fp32-class result; the other tiles send plain bf16 weights, whose rounding
    then averages over at least that many keys: the stated bars hold with room, the relative RMS error is at
    the level of a bf16 output's own rounding.  Covers both tile kinds in one call, a chunk whose rows all see
    more than the limit (every tile plain, incl. the two-buffer use of the P region), and a packed tile."""
    cfg = wl.DecodeConfig("adaptive", B=2, Hq=2 * G, Hkv=2, D=D, T_max=T, seed=350 + Lq)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_prefill_fwd(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, status, p_precision=plx.PLX_P_BF16_ADAPTIVE)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    packed = G > 1 and G * Lq <= 128
    first_visible = (T - Lq + 1) + (np.zeros(Lq, dtype=np.int64) if packed else 128 * (np.arange(Lq) // 128))   # fewest keys seen in the row's tile
    with_res = first_visible < plx.PLX_P_ADAPTIVE_MIN_KEYS
    if with_res.any():
        e = errors(got[:, :, with_res], want[:, :, with_res])
        assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= REL_RMS_TOL_F32, ("residual tiles", e)
    if (~with_res).any():
        e = errors(got[:, :, ~with_res], want[:, :, ~with_res])
        assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= REL_RMS_TOL_BF16, ("plain tiles", e)
        assert e["rel_rms"] > REL_RMS_TOL_F32, "these tiles were expected to run without residual products"


@pytest.mark.parametrize("name", ["P1", "P2", "P3", "P4"])
def test_prefill_full_size_in_the_bench_configuration(plx, oracle, name):
    """Full-size prefill workloads with the entry point, workspace and dtypes the bench times (bf16 output;
    P4's few row tiles make the library divide the keys among CTAs and finish with its merge kernel),
    checked on sampled rows: each row is a one-token problem for the oracle."""
    cfg, Lq = wl.PREFILL_CONFIGS[name]
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(min(plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, 64), 1 << 30), dtype=torch.uint8,
                     device="cuda")
    plx.parallax_prefill_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.isfinite(out.float()).all()
    g = np.random.default_rng(11)
    rows = [(int(g.integers(cfg.B)), int(g.integers(cfg.Hq)), int(i)) for i in
            list(g.integers(0, Lq, size=300)) + [i for i in (0, 1, 63, 64, 127, 128, Lq - 1) if i < Lq]]
    for (b, h, i) in rows:
        n = cfg.T_max - Lq + i + 1
        hkv = h // cfg.G
        want, _ = oracle.decode_bf16(wl.bf16_bits(x["q"][b:b + 1, h:h + 1, i]), wl.bf16_bits(x["r"][b:b + 1, h:h + 1, i]),
                                     wl.bf16_bits(x["k"][b:b + 1, hkv:hkv + 1, :n]), wl.bf16_bits(x["v"][b:b + 1, hkv:hkv + 1, :n]),
                                     None, cfg.scale)
        got = out[b, h, i].float().cpu().numpy()
        bound = np.maximum(MAX_ABS_TOL, 2.0 ** -8 * np.abs(want[0, 0]))
        assert (np.abs(got - want[0, 0]) <= bound).all(), (b, h, i)


@pytest.mark.parametrize("page_size,Lq,T", [(64, 200, 700), (128, 64, 1000), (256, 300, 300)])
def test_prefill_paged_cache(plx, oracle, page_size, Lq, T):
    """Chunked prefill over a paged cache (random page order, NaN in unused pages and page tails) gives
    what the contiguous entry point's oracle gives."""
    cfg = wl.DecodeConfig("pfp", B=3, Hq=4, Hkv=2, D=128, T_max=T, ragged=(max(Lq, T // 2), T), seed=370 + page_size)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    kp, vp, table = wl.to_paged(x["k"], x["v"], page_size, seed=5)
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_prefill_fwd_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], x["seqlens_host"], cfg.scale)
    e = errors(out.cpu().numpy(), want)
    assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= REL_RMS_TOL_F32, e


@pytest.mark.parametrize("prec", ["residual", "plain"])
def test_prefill_head_dim_64_at_scale(plx, oracle, prec):
    """Head dimension 64 on a grid of several thousand CTAs with 64 tiles each, both weight precisions
    (with two P buffers the softmax warps can run a tile ahead of the value issuer: every hand-off barrier
    has to tolerate that).  Sampled rows against the oracle; the plain-bf16 mode gets its own, wider bar."""
    cfg = wl.DecodeConfig("pf64-scale", B=8, Hq=16, Hkv=8, D=64, T_max=4096, seed=391)
    Lq = 4096
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_prefill_fwd(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, status,
                             p_precision=plx.PLX_P_BF16_RESIDUAL if prec == "residual" else plx.PLX_P_BF16)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.isfinite(out).all()
    g = np.random.default_rng(13)
    rows = [(int(g.integers(cfg.B)), int(g.integers(cfg.Hq)), int(i)) for i in list(g.integers(512, Lq, size=24)) + [Lq - 1]]
    for (b, h, i) in rows:
        hkv = h // cfg.G
        want, _ = oracle.decode_bf16(wl.bf16_bits(x["q"][b:b + 1, h:h + 1, i]), wl.bf16_bits(x["r"][b:b + 1, h:h + 1, i]),
                                     wl.bf16_bits(x["k"][b:b + 1, hkv:hkv + 1, :i + 1]), wl.bf16_bits(x["v"][b:b + 1, hkv:hkv + 1, :i + 1]),
                                     None, cfg.scale)
        err = np.abs(out[b, h, i].cpu().numpy() - want[0, 0])
        assert err.max() <= (MAX_ABS_TOL if prec == "residual" else 5e-2), (b, h, i, err.max())


@pytest.mark.parametrize("G,Lq", [(2, 64), (2, 65), (4, 32), (4, 33), (8, 16), (8, 5), (16, 8), (3, 42), (3, 43)])
def test_prefill_packed_tiles(plx, oracle, G, Lq):
    """When a KV head's query heads fit one 128-row tile together (G * Lq <= 128) they share it: row r is
    token r mod Lq of head r / Lq.  Both sides of that boundary, contexts shorter than Lq (the first tokens
    of every head see nothing), an empty context, NaN padding."""
    cfg = wl.DecodeConfig("pack", B=4, Hq=2 * G, Hkv=2, D=128, T_max=300, seed=700 + 10 * G + Lq)
    run_case(plx, oracle, cfg, Lq, seqlens=[300, max(Lq - 3, 1), 0, 131])
    cfg64 = wl.DecodeConfig("pack64", B=2, Hq=2 * G, Hkv=2, D=64, T_max=200, seed=800 + 10 * G + Lq)
    run_case(plx, oracle, cfg64, Lq, out_dtype=torch.bfloat16)


def run_split(plx, oracle, cfg, Lq, ns, seqlens=None, out_dtype=torch.float32, prec=None, max_splits=None):
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    sl_host = None
    if seqlens is not None:
        sl_host = np.asarray(seqlens, dtype=np.int32)
        x["seqlens"] = torch.from_numpy(sl_host).cuda()
        for b in range(cfg.B):
            x["k"][b, :, int(sl_host[b]):] = float("nan")
            x["v"][b, :, int(sl_host[b]):] = float("nan")
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=out_dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    nbytes = plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, max_splits or max(ns, 64))
    ws = torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda")      # NaN bit patterns
    plx.parallax_prefill_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, ns, status,
                                p_precision=plx.PLX_P_BF16_RESIDUAL if prec is None else prec)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], sl_host, cfg.scale)
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    e = errors(got, want)
    if out_dtype == torch.float32:
        assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= REL_RMS_TOL_F32, e
    else:   # as in run_case: the output format's own half-ulp on rows with large |o|
        assert (np.abs(got - want) <= np.maximum(MAX_ABS_TOL, 2.0 ** -8 * np.abs(want))).all(), e
        assert e["mean_abs"] <= max(MEAN_ABS_TOL, 2.0 ** -9 * float(np.abs(want).mean())), e
        assert e["rel_rms"] <= REL_RMS_TOL_BF16, e
    return x, out


@pytest.mark.parametrize("Lq,T,ns", [(16, 1000, 3), (64, 4096, 0), (128, 5000, 7), (200, 2048, 4), (37, 700, 11),
                                     (300, 300, 2), (8, 32768, 0)])
@pytest.mark.parametrize("D", [64, 128])
def test_prefill_split_kv(plx, oracle, Lq, T, ns, D):
    """Key tiles of a row tile divided among several CTAs, rows finished by the merge kernel: forced and
    planned split counts, splits that the causal diagonal leaves without a tile for the early row tiles,
    packed (G * Lq <= 128) and plain tiles."""
    cfg = wl.DecodeConfig("pf split", B=2, Hq=4, Hkv=2, D=D, T_max=T, seed=2100 + Lq + T)
    run_split(plx, oracle, cfg, Lq, ns)


def test_prefill_split_kv_ragged_bf16_and_small_workspace(plx, oracle):
    """Ragged contexts (splits past a context's end write empty records), contexts shorter than the chunk,
    an empty context, bf16 output, plain-bf16 weights, and a workspace that holds fewer splits than asked."""
    cfg = wl.DecodeConfig("pf split ragged", B=5, Hq=8, Hkv=2, D=128, T_max=3000, seed=2201)
    sl = [3000, 1234, 40, 0, 64]
    run_split(plx, oracle, cfg, 48, 6, seqlens=sl)
    run_split(plx, oracle, cfg, 48, 0, seqlens=sl, out_dtype=torch.bfloat16)
    run_split(plx, oracle, cfg, 48, 16, seqlens=sl, max_splits=3)
    x = wl.make_prefill_inputs(cfg, 48, "cuda")
    a = torch.empty(cfg.B, cfg.Hq, 48, cfg.D, dtype=torch.float32, device="cuda")
    b = torch.empty_like(a)
    ws = torch.empty(plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, 48, 8), dtype=torch.uint8, device="cuda")
    plx.parallax_prefill_fwd(x["q"], x["r"], x["k"], x["v"], None, a, cfg.scale, p_precision=plx.PLX_P_BF16)
    plx.parallax_prefill_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, b, cfg.scale, ws, 8, p_precision=plx.PLX_P_BF16)
    torch.cuda.synchronize()
    e = errors(b.cpu().numpy(), a.cpu().numpy())
    assert e["rel_rms"] <= 3e-3, e          # plain-bf16 weights round differently per split: same class, not same bits
    # one split (or no workspace) is the unsplit kernel, bit for bit
    c = torch.empty_like(a)
    plx.parallax_prefill_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, c, cfg.scale, None, 0, p_precision=plx.PLX_P_BF16)
    torch.cuda.synchronize()
    assert torch.equal(a, c)


@pytest.mark.parametrize("page_size,Lq,T,ns", [(64, 40, 3000, 5), (128, 128, 2500, 0), (256, 16, 4096, 3)])
def test_prefill_paged_cache_split_kv(plx, oracle, page_size, Lq, T, ns):
    """Split-KV over a paged cache: a split's first key tile is looked up through the block table."""
    cfg = wl.DecodeConfig("pfp split", B=2, Hq=4, Hkv=2, D=128, T_max=T, ragged=(max(Lq, T // 2), T), seed=390 + page_size)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    kp, vp, table = wl.to_paged(x["k"], x["v"], page_size, seed=6)
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.full((plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, 64),), 0xFF, dtype=torch.uint8, device="cuda")
    plx.parallax_prefill_fwd_paged_ex(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, ns, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], x["seqlens_host"], cfg.scale)
    e = errors(out.cpu().numpy(), want)
    assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= REL_RMS_TOL_F32, e


def test_prefill_adaptive_residuals_ragged_contexts(plx, oracle):
    """Ragged contexts: which tiles carry residuals depends on seqlens (device data), so both launches of the
    adaptive mode cover every tile and each CTA decides for itself.  Every row is written exactly once: the
    output starts as NaN and must come back finite and within the bars of its tile's kind; split-KV too."""
    cfg = wl.DecodeConfig("adaptive ragged", B=4, Hq=4, Hkv=2, D=128, T_max=2600, seed=377)
    Lq = 300
    lens = np.array([2600, 1200, 310, 0], dtype=np.int32)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    x["seqlens"] = torch.from_numpy(lens).cuda()
    for b in range(cfg.B):
        x["k"][b, :, int(lens[b]):] = float("nan")
        x["v"][b, :, int(lens[b]):] = float("nan")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], lens, cfg.scale)
    ws = torch.empty(plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, 8), dtype=torch.uint8, device="cuda")
    for ns in (1, 5):
        out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        plx.parallax_prefill_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, ns, status,
                                    p_precision=plx.PLX_P_BF16_ADAPTIVE)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = out.cpu().numpy()
        assert np.isfinite(got).all()
        for b in range(cfg.B):
            first_visible = (int(lens[b]) - Lq + 1) + 128 * (np.arange(Lq) // 128)
            with_res = first_visible < plx.PLX_P_ADAPTIVE_MIN_KEYS
            for sel, tol in ((with_res, REL_RMS_TOL_F32), (~with_res, REL_RMS_TOL_BF16)):
                if sel.any() and np.abs(want[b][:, sel]).max() > 0:
                    e = errors(got[b][:, sel], want[b][:, sel])
                    assert e["max_abs"] <= MAX_ABS_TOL and e["mean_abs"] <= MEAN_ABS_TOL and e["rel_rms"] <= tol, (ns, b, e)
        assert np.all(got[3] == 0.0)      # the empty context
