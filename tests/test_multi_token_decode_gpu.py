"""GPU parity of the multi-token decode step against the fp64 oracle of the multi-token causal forward.
parallax_decode_fwd_multi runs up to eight rows per KV head on the decode kernel and hands larger steps to
the tensor-core kernels (keys on the lanes up to 32 rows, row-major above); parallax_decode_fwd_args
always stays on the decode kernel.  Every case runs through
both entries, so the decode kernel's per-head key counts are covered at every row count."""
import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import assert_parity, errors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def plx(cuda_device):
    from paper_2605_29157_b200 import binding
    return binding


def run_case(plx, oracle, cfg, Lq, ns=0, seqlens=None, out_dtype=torch.float32, poison=True):
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
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, plx.PLX_MAX_SPLITS if ns == 0 else ns, "cuda")
    for entry in ("args", "multi"):     # decode kernel always / routed by row count
        out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=out_dtype, device="cuda")
        if entry == "multi":
            plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, ns)
        else:
            plx.parallax_decode_fwd_args(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, workspace=ws,
                                         num_splits=ns)
        torch.cuda.synchronize()
        assert plx.parallax_workspace_status(ws) == 0
        got = out.float().cpu().numpy()
        assert np.isfinite(got).all(), "non-finite output"
        if out_dtype == torch.float32:
            e = assert_parity(got, want, out_dtype, f"{cfg.name} Lq={Lq} ns={ns} {entry}")
        else:   # rows with few keys reach |o| ~ 10: the output format's own half-ulp is part of the bound
            assert (np.abs(got - want) <= np.maximum(2e-2, 2.0 ** -8 * np.abs(want))).all(), entry
            e = None
    return x, out, e


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 2, 4])
@pytest.mark.parametrize("Lq", [1, 2, 3, 4, 5, 8, 16])
def test_multi_token_single_split(plx, oracle, D, G, Lq):
    """Every tail shape of the per-head key counts: the last Lq - 1 keys straddle tiles and warps."""
    for T in (Lq, 17, 64 + Lq, 333):
        if T < Lq:
            continue
        cfg = wl.DecodeConfig("multi", B=2, Hq=2 * G, Hkv=2, D=D, T_max=T, seed=1300 + T + Lq)
        run_case(plx, oracle, cfg, Lq, ns=1)


@pytest.mark.parametrize("Lq,T,ns", [(2, 1000, 3), (4, 4096, 0), (8, 5000, 7), (3, 2048, 16), (16, 1030, 4), (32, 3000, 0)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_multi_token_split_kv(plx, oracle, Lq, T, ns, out_dtype):
    """Split contexts: the chunk that holds the last keys gives some tokens an empty record (none of its
    keys is visible to them), which the merge has to skip."""
    cfg = wl.DecodeConfig("multi split", B=3, Hq=4, Hkv=2, D=128, T_max=T, seed=1400 + T)
    run_case(plx, oracle, cfg, Lq, ns=ns, out_dtype=out_dtype)


def test_multi_token_chunk_boundary_inside_the_new_tokens(plx, oracle):
    """A split boundary that falls inside the last Lq keys: the last chunk then holds only keys that the
    first tokens must not see (their record of that chunk is empty), for every token offset."""
    Lq = 8
    for T in (256 + 1, 256 + 4, 256 + 7, 512 + 3):
        cfg = wl.DecodeConfig("multi boundary", B=2, Hq=4, Hkv=2, D=128, T_max=T, seed=1500 + T)
        run_case(plx, oracle, cfg, Lq, ns=(T + 255) // 256)


def test_multi_token_ragged_and_short_contexts(plx, oracle):
    """Contexts shorter than the number of new tokens (the first tokens see nothing: rows of zeros), empty
    contexts, NaN padding."""
    Lq = 6
    cfg = wl.DecodeConfig("multi ragged", B=8, Hq=4, Hkv=2, D=128, T_max=700, seed=1601)
    sl = [0, 1, 3, 6, 7, 100, 699, 700]
    for ns in (1, 0, 5):
        x, out, _ = run_case(plx, oracle, cfg, Lq, ns=ns, seqlens=sl)
        got = out.cpu().numpy()
        assert (got[0] == 0).all()
        assert (got[1, :, :Lq - 1] == 0).all() and np.abs(got[1, :, Lq - 1]).max() > 0
        assert (got[2, :, :Lq - 3] == 0).all()


def test_multi_token_equals_the_tensor_core_kernel_and_single_token_calls(plx, oracle):
    """Same numbers as parallax_prefill_fwd (fp32-class on both sides), and token i equals a one-token
    decode call over the first L - Lq + 1 + i keys."""
    Lq = 4
    cfg = wl.DecodeConfig("multi eq", B=2, Hq=8, Hkv=2, D=128, T_max=1500, seed=1700)
    x, out, _ = run_case(plx, oracle, cfg, Lq, ns=0, seqlens=[1500, 911], poison=False)
    ref = torch.empty_like(out)
    plx.parallax_prefill_fwd(x["q"], x["r"], x["k"], x["v"], x["seqlens"], ref, cfg.scale)
    torch.cuda.synchronize()
    e = errors(out.cpu().numpy(), ref.cpu().numpy())
    assert e["rel_rms"] <= 5e-5, e
    one = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    for i in range(Lq):
        sl = (x["seqlens"] - (Lq - 1 - i)).to(torch.int32)
        plx.parallax_decode_fwd_ex(x["q"][:, :, i].contiguous(), x["r"][:, :, i].contiguous(), x["k"], x["v"], sl, one,
                                   cfg.scale, None, 1)
        torch.cuda.synchronize()
        e = errors(out[:, :, i].cpu().numpy(), one.cpu().numpy())
        assert e["rel_rms"] <= 5e-5, (i, e)


def test_row_counts_beyond_the_decode_kernel(plx, oracle):
    """More than 64 rows per KV head: the decode kernel refuses (options-struct entry), the multi-token entry
    hands the step to the tensor-core kernel, with or without a workspace."""
    cfg = wl.DecodeConfig("multi big", B=2, Hq=4, Hkv=2, D=128, T_max=700, seed=1900)
    Lq = 40
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    out = torch.empty(cfg.B, cfg.Hq, Lq, cfg.D, dtype=torch.float32, device="cuda")
    with pytest.raises(plx.ParallaxError) as e:
        plx.parallax_decode_fwd_args(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale)
    assert e.value.status == plx.PLX_ERR_UNSUPPORTED
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    for ws in (None, plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, 16, "cuda")):
        out.fill_(float("nan"))
        plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0)
        torch.cuda.synchronize()
        assert_parity(out.cpu().numpy(), want, torch.float32, "routed")


@pytest.mark.parametrize("page_size,Lq,T,ns", [(16, 3, 300, 1), (64, 4, 2500, 0), (128, 8, 1000, 5)])
def test_multi_token_paged_cache(plx, oracle, page_size, Lq, T, ns):
    """The same step over a paged cache (random page order, NaN in unused pages and page tails)."""
    cfg = wl.DecodeConfig("multi paged", B=3, Hq=4, Hkv=2, D=128, T_max=T, ragged=(Lq, T), seed=1800 + page_size)
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    kp, vp, table = wl.to_paged(x["k"], x["v"], page_size, seed=7)
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, plx.PLX_MAX_SPLITS if ns == 0 else ns, "cuda")
    plx.parallax_decode_fwd_multi_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, ns)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], x["seqlens_host"], cfg.scale)
    assert_parity(out.cpu().numpy(), want, torch.float32, f"multi paged ps={page_size}")


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G,Lq", [(2, 5), (2, 6), (2, 8), (4, 4), (2, 7)])
def test_ten_to_sixteen_rows(plx, oracle, D, G, Lq):
    """10 / 12 / 14 / 16 rows per KV head: the keys-on-lanes tensor-core kernel through the multi-token entry, two
    CTAs of the decode kernel (five to eight rows each) through the options-struct entry, at both head dimensions.
    Ragged contexts, NaN padding, planned splits."""
    B, Hkv = 16, 8
    cfg = wl.DecodeConfig("ten to sixteen rows", B=B, Hq=Hkv * G, Hkv=Hkv, D=D, T_max=700, seed=1700 + G * Lq)
    g = np.random.default_rng(G * 100 + Lq)
    lens = g.integers(Lq, 701, size=B)
    lens[0], lens[1] = 700, Lq
    run_case(plx, oracle, cfg, Lq, ns=0, seqlens=lens)


def test_the_plan_query_names_the_kernel_that_runs(plx):
    """parallax_decode_multi_plan: the decode kernel up to four rows per KV head at D = 128 and up to eight at D = 64,
    the keys-on-lanes kernel up to 64 rows (over pages only for page sizes it can tile; from five rows only over pages
    of at least 64 keys; 33 to 64 rows at D = 64 only for long contexts on many sequences), the row-major kernel above; a split count only for the keys-on-lanes kernel."""
    K = plx
    plan = lambda **kw: plx.parallax_decode_multi_plan(kw.get("B", 4), kw.get("Hq", 4), 2, kw.get("D", 128), kw["Lq"],
                                                       kw.get("T", 4096), kw.get("ps", 0))
    assert plan(Lq=1) == (K.PLX_MULTI_KERNEL_DECODE, 0) and plan(Lq=2)[0] == K.PLX_MULTI_KERNEL_DECODE
    assert plan(Lq=3)[0] == K.PLX_MULTI_KERNEL_ROWS and plan(Lq=16)[0] == K.PLX_MULTI_KERNEL_ROWS
    assert plan(Lq=17)[0] == K.PLX_MULTI_KERNEL_ROWS and plan(Lq=32)[0] == K.PLX_MULTI_KERNEL_ROWS    # two parts of 17 / 32 rows
    assert plan(Lq=33)[0] == K.PLX_MULTI_KERNEL_ROW_MAJOR and plan(Lq=200) == (K.PLX_MULTI_KERNEL_ROW_MAJOR, 0)
    assert plan(Lq=20, D=64)[0] == K.PLX_MULTI_KERNEL_ROW_MAJOR           # at D = 64 only long contexts on many sequences
    assert plan(Lq=20, D=64, B=128, T=8192)[0] == K.PLX_MULTI_KERNEL_ROWS
    assert plan(Lq=4, D=64)[0] == K.PLX_MULTI_KERNEL_DECODE and plan(Lq=5, D=64)[0] == K.PLX_MULTI_KERNEL_ROWS
    assert plan(Lq=3, ps=16)[0] == K.PLX_MULTI_KERNEL_DECODE and plan(Lq=3, ps=64)[0] == K.PLX_MULTI_KERNEL_ROWS
    assert plan(Lq=8, ps=16)[0] == K.PLX_MULTI_KERNEL_ROWS and plan(Lq=8, ps=48)[0] != K.PLX_MULTI_KERNEL_ROWS
    kernel, ns = plan(Lq=8, B=1, T=32768)         # two items on a whole GPU: split as far as four tiles per split allow
    assert kernel == K.PLX_MULTI_KERNEL_ROWS and 2 <= ns <= 64
    assert plan(Lq=8, B=256, T=2048) == (K.PLX_MULTI_KERNEL_ROWS, 1)
    with pytest.raises(plx.ParallaxError):
        plx.parallax_decode_multi_plan(4, 5, 2, 128, 1, 4096, 0)


@pytest.mark.parametrize("name,Lq,nrows", [("C3", 4, 512), ("C3", 8, 768), ("C3", 24, 512), ("C5", 8, 768), ("C6", 16, 512),
                                            ("C4", 16, 256), ("C2", 8, 512)])
def test_multi_token_full_size_in_the_bench_configuration(plx, oracle, name, Lq, nrows):
    """The decode configurations at full size with several new tokens per sequence, in the launch configuration the
    bench times (routed entry, planned splits, bf16 output): sampled (sequence, head, token) rows against the fp64
    oracle of the ONE-token path on the context that token sees (token i sees the first L - (Lq - 1 - i) keys), which is
    what the multi-token causal rule says.  Covers the item walk (C3, C5, C6), two parts of the rows (C3 with 24
    tokens), few long streams (C4) and a grid smaller than the device (C2)."""
    cfg = wl.CONFIGS[name]
    x = wl.make_prefill_inputs(cfg, Lq, "cuda", poison_padding=(name == "C5"))
    out = torch.full((cfg.B, cfg.Hq, Lq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, 0)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    assert torch.isfinite(out.float()).all()
    rng = np.random.default_rng(11)
    picks = {(0, 0, 0), (cfg.B - 1, cfg.Hq - 1, Lq - 1), (0, cfg.Hq - 1, 0)}
    while len(picks) < nrows:
        picks.add((int(rng.integers(cfg.B)), int(rng.integers(cfg.Hq)), int(rng.integers(Lq))))
    picks = sorted(picks)
    sl = x["seqlens_host"]
    G = cfg.Hq // cfg.Hkv
    got, want = [], []
    for (b, h, i) in picks:
        L = cfg.T_max if sl is None else int(sl[b])
        Li = max(L - (Lq - 1 - i), 0)
        got.append(out[b, h, i].float().cpu().numpy())
        if Li == 0:
            want.append(np.zeros(cfg.D))
            continue
        hkv = h // G
        q = wl.bf16_bits(x["q"][b:b + 1, h:h + 1, i])
        r = wl.bf16_bits(x["r"][b:b + 1, h:h + 1, i])
        k = wl.bf16_bits(x["k"][b:b + 1, hkv:hkv + 1, :Li])
        v = wl.bf16_bits(x["v"][b:b + 1, hkv:hkv + 1, :Li])
        o, _ = oracle.decode_bf16(q, r, k, v, np.array([Li], dtype=np.int32), cfg.scale)
        want.append(o[0, 0])
    e = assert_parity(np.stack(got), np.stack(want), torch.bfloat16, f"{name} Lq={Lq}")
    print(name, Lq, e)
