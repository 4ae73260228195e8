"""GPU parity of the keys-on-lanes tensor-core kernel for multi-token decode steps (parallax_decode_fwd_rows:
up to 32 rows per KV head) against the fp64 oracle of the multi-token causal forward."""
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


def run_rows(plx, oracle, cfg, Lq, ns=1, seqlens=None, out_dtype=torch.float32, poison=True, label=""):
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    sl_host = None
    if seqlens is not None:
        sl_host = np.asarray(seqlens, dtype=np.int32)
        x["seqlens"] = torch.from_numpy(sl_host).cuda()
        if poison:
            for b in range(cfg.B):
                x["k"][b, :, max(int(sl_host[b]), 0):] = float("nan")
                x["v"][b, :, max(int(sl_host[b]), 0):] = float("nan")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"],
                                  None if sl_host is None else np.clip(sl_host, 0, cfg.T_max), cfg.scale)
    ws = None
    if ns != 1:
        nbytes = plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, plx.PLX_MAX_SPLITS if ns == 0 else ns)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=out_dtype, device="cuda")
    plx.parallax_decode_fwd_rows(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, ns, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all(), "non-finite output"
    if out_dtype == torch.float32:
        assert_parity(got, want, out_dtype, f"{cfg.name} Lq={Lq} ns={ns} {label}")
    else:   # rows with few keys reach |o| ~ 10: the output format's own half-ulp is part of the bound
        assert (np.abs(got - want) <= np.maximum(2e-2, 2.0 ** -8 * np.abs(want))).all()
    return x, out


@pytest.mark.parametrize("G,Lq", [(2, 8), (2, 16), (4, 8), (1, 32), (2, 5), (4, 3), (8, 4), (1, 1), (2, 12), (3, 7), (1, 16), (8, 2),
                                  (2, 9), (5, 5)])
@pytest.mark.parametrize("T", [128, 129, 200, 256, 1000])
def test_rows_single_split(plx, oracle, G, Lq, T):
    """One CTA per KV head: full and ragged last tiles, the last Lq - 1 keys straddling a tile boundary."""
    cfg = wl.DecodeConfig("rows", B=2, Hq=2 * G, Hkv=2, D=128, T_max=T, seed=2100 + T + Lq)
    run_rows(plx, oracle, cfg, Lq, ns=1)


@pytest.mark.parametrize("Lq,T,ns", [(8, 1000, 3), (16, 4096, 0), (8, 5000, 7), (12, 2048, 16), (16, 1030, 4), (10, 3000, 0),
                                     (5, 8192, 64), (16, 640, 5)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_rows_split_kv(plx, oracle, Lq, T, ns, out_dtype):
    """Split contexts (forced and planned): the split that holds the last keys gives some tokens an empty record."""
    cfg = wl.DecodeConfig("rows split", B=3, Hq=4, Hkv=2, D=128, T_max=T, seed=2200 + T)
    run_rows(plx, oracle, cfg, Lq, ns=ns, out_dtype=out_dtype)


@pytest.mark.parametrize("ns", [1, 0, 6])
def test_rows_ragged_contexts_with_poisoned_padding(plx, oracle, ns):
    """Per-sequence lengths incl. empty, shorter than Lq, one key, tile-aligned and ragged; NaN behind every context."""
    Lq = 12
    cfg = wl.DecodeConfig("rows ragged", B=8, Hq=4, Hkv=2, D=128, T_max=1500, seed=2300)
    run_rows(plx, oracle, cfg, Lq, ns=ns, seqlens=[0, 1, 5, 12, 128, 129, 1024, 1500])


def test_rows_split_boundary_inside_the_new_tokens(plx, oracle):
    """A split boundary that falls inside the last Lq keys: the last split holds only keys the first tokens must not see."""
    Lq = 16
    for T in (256 + 1, 256 + 9, 384 + 15, 512 + 3):
        cfg = wl.DecodeConfig("rows boundary", B=2, Hq=4, Hkv=2, D=128, T_max=T, seed=2400 + T)
        run_rows(plx, oracle, cfg, Lq, ns=(T + 127) // 128)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G,Lq", [(2, 5), (2, 12), (1, 9), (3, 7)])
@pytest.mark.parametrize("ns", [1, 3])
def test_rows_padding_rows_read_hostile_neighbours(plx, oracle, D, G, Lq, ns):
    """Fewer rows than the tile holds: the padding rows of a CTA are whatever follows its rows in q and r (the next KV
    head's, or nothing after the last one).  With NaN, infinities and huge values there, the rows of the head in front
    must come out as if the neighbours were not there."""
    T = 900
    cfg = wl.DecodeConfig("rows hostile", B=2, Hq=3 * G, Hkv=3, D=D, T_max=T, seed=2450 + D + Lq)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    hostile = torch.tensor([float("nan"), float("inf"), -float("inf"), 3.0e38, -3.0e38, 1.0e4], device="cuda")
    for name in ("q", "r"):   # the middle KV head's rows of both sequences
        mid = x[name][:, G:2 * G]
        mid.copy_(hostile[torch.arange(mid.numel(), device="cuda") % hostile.numel()].view(mid.shape).to(mid.dtype))
    ws = torch.empty(plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, 8), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((cfg.B, cfg.Hq, Lq, D), float("nan"), dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_rows(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, ns, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = out.cpu().numpy()
    keep = [h for h in range(cfg.Hq) if not G <= h < 2 * G]
    assert np.isfinite(got[:, keep]).all()
    assert_parity(got[:, keep], want[:, keep], torch.float32, f"hostile neighbours D={D} G={G} Lq={Lq} ns={ns}")


@pytest.mark.parametrize("Lq", [8, 14])
@pytest.mark.parametrize("kind", ["peaked", "growing"])
def test_rows_reference_moves_late(plx, oracle, kind, Lq):
    """Scores that keep growing along the context (the reference exponent moves in many tiles, the accumulators are
    rescaled in TMEM each time) and one dominant key late in the context; at 16 and 28 rows per KV head."""
    T = 2048
    cfg = wl.DecodeConfig("rows " + kind, B=2, Hq=4, Hkv=2, D=128, T_max=T, seed=2500)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    if kind == "peaked":
        x["k"][:, :, 1777] = x["q"][:, ::2, 0].to(x["k"].dtype) * 3.0    # one key aligned with a query
    else:
        ramp = torch.linspace(0.2, 3.0, T, device="cuda").view(1, 1, T, 1)
        x["k"] = (x["k"].float() * ramp).to(torch.bfloat16)
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    for ns in (1, 4):
        ws = torch.empty(plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, 8), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
        plx.parallax_decode_fwd_rows(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, ns, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert_parity(out.cpu().numpy(), want, torch.float32, f"{kind} ns={ns}")


@pytest.mark.parametrize("G,Lq", [(2, 8), (2, 16), (4, 3), (8, 4), (1, 1), (2, 5), (3, 7), (1, 32)])
@pytest.mark.parametrize("T", [128, 200, 1000])
def test_rows_head_dimension_64(plx, oracle, G, Lq, T):
    """The same kernel at head dimension 64 (one 64-column box per row; the value product keeps M = 128 with its
    second block repeating the first): single split, planned splits, ragged with NaN padding."""
    cfg = wl.DecodeConfig("rows d64", B=2, Hq=2 * G, Hkv=2, D=64, T_max=T, seed=2800 + T + Lq)
    run_rows(plx, oracle, cfg, Lq, ns=1)
    if T == 1000:
        run_rows(plx, oracle, cfg, Lq, ns=0, label="planned")
        run_rows(plx, oracle, cfg, Lq, ns=3, seqlens=[max(1, Lq - 1), 777], label="ragged")


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G,Lq", [(2, 17), (2, 24), (2, 32), (4, 12), (1, 33), (8, 8), (3, 11), (1, 64)])
@pytest.mark.parametrize("T,ns", [(128, 1), (300, 1), (1000, 3)])
def test_rows_thirty_three_to_sixty_four_rows_in_two_parts(plx, oracle, D, G, Lq, T, ns):
    """More than 32 rows per KV head: two items of half the rows each (the second part's tokens start in the middle of
    a head's tokens, or with another head), one split and three, full and ragged last tiles."""
    cfg = wl.DecodeConfig("rows parts", B=2, Hq=2 * G, Hkv=2, D=D, T_max=T, seed=3300 + G * Lq + T)
    run_rows(plx, oracle, cfg, Lq, ns=ns)


def test_rows_two_parts_ragged_paged_and_walked(plx, oracle):
    """48 rows per KV head over contexts of their own lengths (empty, shorter than the new tokens, one key), through the
    routed entry: contiguous with more items than SMs (the ticket walk over parts) and over 64-key pages."""
    Lq, T, Hkv = 24, 700, 8
    B = torch.cuda.get_device_properties(0).multi_processor_count // (2 * Hkv) + 2
    cfg = wl.DecodeConfig("rows parts walk", B=B, Hq=2 * Hkv, Hkv=Hkv, D=128, T_max=T, seed=3400)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    rng = np.random.default_rng(5)
    sl = rng.integers(0, T + 1, size=B).astype(np.int32)
    sl[:4] = (0, Lq - 1, 1, T)
    x["seqlens"] = torch.from_numpy(sl).cuda()
    for b in range(B):
        x["k"][b, :, int(sl[b]):] = float("nan")
        x["v"][b, :, int(sl[b]):] = float("nan")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], sl, cfg.scale)
    assert plx.parallax_decode_multi_plan(B, cfg.Hq, Hkv, 128, Lq, T)[0] == plx.PLX_MULTI_KERNEL_ROWS
    ws = plx.alloc_workspace(B, cfg.Hq * Lq, cfg.D, 4, "cuda")
    for ns in (1, 2):
        out = torch.full((B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
        plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, ns)
        torch.cuda.synchronize()
        assert plx.parallax_workspace_status(ws) == 0
        assert int(ws[:256].view(torch.int32).abs().sum().item()) == 0
        assert_parity(out.cpu().numpy(), want, torch.float32, f"two parts walked ns={ns}")
    x["k"].nan_to_num_(0.0)
    x["v"].nan_to_num_(0.0)
    kp, vp, table = wl.to_paged(x["k"], x["v"], 64, seed=3)
    out = torch.full((B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, 0)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    assert_parity(out.cpu().numpy(), want, torch.float32, "two parts paged")


def test_rows_rejects_what_it_does_not_serve(plx):
    q = torch.zeros(1, 4, 40, 128, dtype=torch.bfloat16, device="cuda")      # 80 rows per KV head
    k = torch.zeros(1, 2, 256, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, 4, 40, 128, dtype=torch.float32, device="cuda")
    with pytest.raises(plx.ParallaxError) as e:
        plx.parallax_decode_fwd_rows(q, q, k, k, None, out, 0.1)
    assert e.value.status == plx.PLX_ERR_UNSUPPORTED
    q = torch.zeros(1, 4, 4, 32, dtype=torch.bfloat16, device="cuda")        # head dimension 32
    k = torch.zeros(1, 2, 256, 32, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, 4, 4, 32, dtype=torch.float32, device="cuda")
    with pytest.raises(plx.ParallaxError) as e:
        plx.parallax_decode_fwd_rows(q, q, k, k, None, out, 0.1)
    assert e.value.status == plx.PLX_ERR_UNSUPPORTED
    q = torch.zeros(1, 4, 4, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 2, 256, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, 4, 4, 128, dtype=torch.float32, device="cuda")
    with pytest.raises(plx.ParallaxError) as e:                                # splits without room for records
        plx.parallax_decode_fwd_rows(q, q, k, k, None, out, 0.1, None, 3)
    assert e.value.status == plx.PLX_ERR_WORKSPACE


@pytest.mark.parametrize("page_size", [16, 32, 64, 128, 256, 48])
@pytest.mark.parametrize("Lq,ns", [(6, 1), (12, 0), (16, 5)])
def test_rows_over_a_paged_cache(plx, oracle, page_size, Lq, ns):
    """parallax_decode_fwd_multi_paged at 12 to 32 rows per KV head: page sizes that divide the 128-key tile or are a
    multiple of it go to the keys-on-lanes kernel (a tile fetched page by page), 48 takes the older routes; random page
    order, NaN in unused pages and page tails, ragged contexts incl. one shorter than Lq + a page."""
    T = 1536
    cfg = wl.DecodeConfig("rows paged", B=4, Hq=4, Hkv=2, D=128, T_max=T, ragged=(Lq, T), seed=2600 + page_size)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    kp, vp, table = wl.to_paged(x["k"], x["v"], page_size, seed=9)
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, plx.PLX_MAX_SPLITS if ns == 0 else ns, "cuda")
    plx.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, ns)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], x["seqlens_host"], cfg.scale)
    assert_parity(out.cpu().numpy(), want, torch.float32, f"rows paged ps={page_size} Lq={Lq}")


def test_multi_query_group_of_sixteen_in_one_token_steps(plx, oracle):
    """One token, sixteen and 24 query heads per KV head: parallax_decode_fwd_ex hands the step to the keys-on-lanes kernel."""
    for G in (16, 24):
        cfg = wl.DecodeConfig("mqa rows", B=3, Hq=2 * G, Hkv=2, D=128, T_max=2100, ragged=(1, 2100), seed=2700 + G)
        x = wl.make_inputs(cfg, "cuda", poison_padding=True)
        from parity_util import oracle_full
        want = oracle_full(oracle, x, cfg.scale, x["seqlens_host"])
        out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
        ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
        plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, 0)
        torch.cuda.synchronize()
        assert plx.parallax_workspace_status(ws) == 0
        assert_parity(out.cpu().numpy(), want, torch.float32, f"G={G}")


def test_rows_step_replayed_from_a_cuda_graph(plx, oracle):
    """A sixteen-row step with planned splits (kernel + merge) captured into a CUDA graph and replayed over new
    inputs in the same buffers: bit-identical to the eager call, two replays in a row."""
    Lq = 8
    cfg = wl.DecodeConfig("rows graph", B=4, Hq=4, Hkv=2, D=128, T_max=3000, seed=2900)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    out = torch.zeros(cfg.B, cfg.Hq, Lq, cfg.D, dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, 16, "cuda")
    plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0)   # warm up outside capture
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0, stream)
    for seed in (1, 2):
        y = wl.make_prefill_inputs(wl.scaled(cfg, seed=cfg.seed + seed), Lq, "cuda")
        for n in ("q", "r", "k", "v"):
            x[n].copy_(y[n])
        eager = torch.empty_like(out)
        plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], None, eager, cfg.scale, ws, 0)
        torch.cuda.synchronize()
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert plx.parallax_workspace_status(ws) == 0
        assert torch.equal(out, eager)
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    assert_parity(out.cpu().numpy(), want, torch.float32, "graph replay")


def _sm_count():
    return torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("D,Lq,T,ns", [(128, 8, 600, 1), (128, 16, 900, 3), (64, 8, 700, 2), (64, 12, 400, 1)])
def test_rows_more_items_than_sms_drawn_from_the_ticket(plx, oracle, D, Lq, T, ns):
    """More (sequence, KV head, split) items than SMs through the routed entry with a zeroed workspace: one CTA per SM
    draws items from the workspace's ticket word and carries its rings and barrier phases from item to item.  Equal
    contexts and contexts of their own lengths (empty ones and ones shorter than the new tokens among them: items
    without keys inside the walk); three calls in a row on the same workspace (the word is back at zero each time)
    must agree bit for bit."""
    Hkv = 8
    B = (_sm_count() + Hkv * ns - 1) // (Hkv * ns) + 3          # a few items more than SMs, not a multiple of them
    assert B * Hkv * ns > _sm_count()
    cfg = wl.DecodeConfig("rows ticket", B=B, Hq=2 * Hkv, Hkv=Hkv, D=D, T_max=T, seed=3100 + D + Lq)
    rng = np.random.default_rng(cfg.seed)
    ragged = rng.integers(0, T + 1, size=B).astype(np.int32)
    ragged[:4] = (0, Lq - 1, T, 1)
    for seqlens in (None, ragged):
        x = wl.make_prefill_inputs(cfg, Lq, "cuda")
        if seqlens is not None:
            x["seqlens"] = torch.from_numpy(seqlens).cuda()
            for b in range(B):
                x["k"][b, :, int(seqlens[b]):] = float("nan")
                x["v"][b, :, int(seqlens[b]):] = float("nan")
        bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
        want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], seqlens, cfg.scale)
        ws = plx.alloc_workspace(B, cfg.Hq * Lq, D, max(ns, 1), "cuda")
        outs = []
        for _ in range(3):
            out = torch.full((B, cfg.Hq, Lq, D), float("nan"), dtype=torch.float32, device="cuda")
            plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, ns)
            torch.cuda.synchronize()
            assert plx.parallax_workspace_status(ws) == 0
            outs.append(out)
        assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
        assert int(ws[:256].view(torch.int32).abs().sum().item()) == 0      # status and ticket are zero again
        assert_parity(outs[0].cpu().numpy(), want, torch.float32, f"ticket D={D} Lq={Lq} ns={ns} ragged={seqlens is not None}")
        if ns == 1:     # without a workspace: one CTA per item, the same items, the same bits
            out = torch.full((B, cfg.Hq, Lq, D), float("nan"), dtype=torch.float32, device="cuda")
            plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, None, 1)
            torch.cuda.synchronize()
            assert torch.equal(out, outs[0])


def test_rows_ticket_walk_over_a_paged_cache_and_from_a_cuda_graph(plx, oracle):
    """The item walk over a paged cache (16-key pages), eager and replayed twice from a CUDA graph."""
    Lq, T, page_size, Hkv = 8, 500, 16, 8
    B = _sm_count() // Hkv + 5
    cfg = wl.DecodeConfig("rows ticket paged", B=B, Hq=2 * Hkv, Hkv=Hkv, D=128, T_max=T, ragged=(Lq, T), seed=3200)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    kp, vp, table = wl.to_paged(x["k"], x["v"], page_size, seed=11)
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], x["seqlens_host"], cfg.scale)
    ws = plx.alloc_workspace(B, cfg.Hq * Lq, cfg.D, 1, "cuda")
    out = torch.full((B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, 1)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    assert_parity(out.cpu().numpy(), want, torch.float32, "ticket paged")
    eager = out.clone()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            plx.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, 1, stream)
    for _ in range(2):
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert plx.parallax_workspace_status(ws) == 0
        assert torch.equal(out, eager)


@pytest.mark.parametrize("kind", ["peaked", "ascending", "probe_offset", "scale0", "negative_scale"])
def test_rows_robustness_distributions(plx, oracle, kind):
    """Inputs that stress the lazily moving references and the cancellation in the covariance branch, at sixteen rows
    per KV head, one and eight splits: sharp distributions, scores that grow with every tile, a large common probe
    component, a zero and a negative softmax scale."""
    from parity_util import errors
    Lq = 8
    cfg = wl.DecodeConfig("rows rob", B=2, Hq=4, Hkv=2, D=128, T_max=2048, seed=3100)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    scale = cfg.scale
    if kind == "peaked":
        x["q"] = (x["q"].float() * 4).to(torch.bfloat16)
    elif kind == "ascending":
        for b in range(cfg.B):
            for h in range(cfg.Hkv):
                order = torch.argsort(x["k"][b, h].float() @ x["q"][b, h * cfg.G, 0].float())
                x["k"][b, h] = x["k"][b, h][order]
                x["v"][b, h] = x["v"][b, h][order]
    elif kind == "probe_offset":
        for b in range(cfg.B):
            for h in range(cfg.Hkv):
                rdir = x["r"][b, h * cfg.G, 0].float()
                x["k"][b, h] = (x["k"][b, h].float() + 0.5 * rdir[None, :]).to(torch.bfloat16)
    elif kind == "scale0":
        scale = 0.0
    elif kind == "negative_scale":
        scale = -cfg.scale
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, scale)
    ws = torch.empty(plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, 8), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for ns in (1, 8):
        out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
        plx.parallax_decode_fwd_rows(x["q"], x["r"], x["k"], x["v"], None, out, scale, ws, ns, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        e = errors(out.cpu().numpy(), want)
        assert e["rel_rms"] <= 1e-3 and e["max_abs"] <= 2e-2 * max(1.0, e["rms"]), (kind, ns, e)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("T", [1, 5, 17, 100])
def test_rows_tiny_contexts(plx, oracle, D, T):
    """Caches smaller than one 128-key tile (and than the tile's copy box), contexts shorter than the number of new
    tokens: the tokens that see no key give rows of zeros."""
    for Lq in (5, 16):
        cfg = wl.DecodeConfig("rows tiny", B=1, Hq=2, Hkv=1, D=D, T_max=T, seed=3200 + T)
        x, out = run_rows(plx, oracle, cfg, Lq, ns=1)
        if T < Lq:   # token i sees T - (Lq - 1 - i) keys: the first Lq - T tokens see none
            assert (out[:, :, :Lq - T] == 0).all()
