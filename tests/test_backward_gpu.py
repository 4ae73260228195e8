"""GPU parity of the training forward's saved state and of the backward (tcgen05 row and column
passes) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import errors

pytestmark = pytest.mark.gpu

# The weights and gradient coefficients reach the tensor cores as bf16 (relative rounding 2^-9 per
# element, independent from element to element); a gradient entry is a sum of such terms with random
# signs, so its error is about 2^-9 of the RMS of the gradient tensor, sqrt(terms) times below the
# worst case.  Bars: relative RMS error <= 1e-2 (measured: about 2e-3).  Element by element the bound
# has to allow for an entry that is the difference of a few large products (with one query row,
# dk_j = scale g1_j q + g2_j rho is two products, each carrying its coefficient's rounding undiluted):
# 2^-7 of the entry's own magnitude plus one bf16 ulp (2^-8) of the tensor's largest entry.
REL_RMS_TOL = 1e-2
ELEM_REL_TOL = 2.0 ** -7
ELEM_MAX_TOL = 2.0 ** -8


@pytest.fixture(scope="module")
def plx(cuda_device):
    from paper_2605_29157_b200 import binding
    return binding


def check_grad(name, got, want):
    got = np.asarray(got, dtype=np.float64)
    assert np.isfinite(got).all(), name
    rms = float(np.sqrt(np.mean(want ** 2)))
    if rms == 0.0:
        assert np.all(got == 0.0), name
        return 0.0
    err = got - want
    rel = float(np.sqrt(np.mean(err ** 2))) / rms
    worst = float((np.abs(err) - ELEM_REL_TOL * np.abs(want)).max()) / float(np.abs(want).max())
    assert rel <= REL_RMS_TOL and worst <= ELEM_MAX_TOL, (name, rel, worst)
    return rel


def run_case(plx, oracle, cfg, Lq, io_dtype=torch.float32, grad_dtype=torch.float32, seqlens=None, poison=False):
    x = wl.make_prefill_inputs(cfg, Lq, "cuda", poison_padding=poison)
    sl_host = x["seqlens_host"]
    if seqlens is not None:
        sl_host = np.asarray(seqlens, dtype=np.int32)
        x["seqlens"] = torch.from_numpy(sl_host).cuda()
        for b in range(cfg.B):
            x["k"][b, :, int(sl_host[b]):] = float("nan")
            x["v"][b, :, int(sl_host[b]):] = float("nan")
    B, Hq, Hkv, D, T = cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T_max
    g = torch.Generator(device="cuda").manual_seed(cfg.seed + 77)
    dout = torch.randn(B, Hq, Lq, D, device="cuda", generator=g).to(torch.bfloat16)
    out = torch.full((B, Hq, Lq, D), float("nan"), dtype=io_dtype, device="cuda")
    vbar = torch.full_like(out, float("nan"))
    lse = torch.full((B, Hq, Lq), float("nan"), dtype=torch.float32, device="cuda")
    tbar = torch.full_like(lse, float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_prefill_fwd_save(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, lse, tbar, vbar, cfg.scale, status)
    dq = torch.full((B, Hq, Lq, D), float("nan"), dtype=grad_dtype, device="cuda")
    dr = torch.full_like(dq, float("nan"))
    dk = torch.full((B, Hkv, T, D), float("nan"), dtype=grad_dtype, device="cuda")
    dv = torch.full_like(dk, float("nan"))
    ws = torch.empty(plx.parallax_prefill_bwd_workspace_bytes(B, Hq, Lq), dtype=torch.uint8, device="cuda")
    plx.parallax_prefill_bwd(x["q"], x["r"], x["k"], x["v"], dout, out, lse, tbar, vbar, x["seqlens"], dq, dr, dk, dv,
                             cfg.scale, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    # saved state
    w_lse, w_tbar, w_vbar = oracle.saved_state_bf16(bits["q"], bits["r"], bits["k"], bits["v"], sl_host, cfg.scale)
    g_lse = lse.cpu().numpy().astype(np.float64)
    empty = np.isinf(w_lse)
    assert np.array_equal(np.isinf(g_lse) & (g_lse > 0), empty)
    assert np.abs(g_lse[~empty] - w_lse[~empty]).max(initial=0.0) <= 2e-4
    assert np.abs(tbar.cpu().numpy() - w_tbar).max() <= 2e-3 * max(1.0, np.abs(w_tbar).max())
    e = errors(vbar.float().cpu().numpy(), w_vbar)
    assert e["rel_rms"] <= (2e-4 if io_dtype == torch.float32 else 4e-3), e
    # gradients
    want = oracle.backward_bf16(bits["q"], bits["r"], bits["k"], bits["v"], wl.bf16_bits(dout), sl_host, cfg.scale)
    got = [t.float().cpu().numpy() for t in (dq, dr, dk, dv)]
    return {n: check_grad(n, a, b) for n, a, b in zip(("dq", "dr", "dk", "dv"), got, want)}


@pytest.mark.parametrize("Lq,T", [(128, 128), (64, 64), (1, 100), (37, 37), (100, 500), (256, 256), (300, 1000), (512, 512)])
def test_backward_shapes(plx, oracle, Lq, T):
    """Training shape (Lq = context), rows against a longer cached prefix, one token, ragged tiles."""
    cfg = wl.DecodeConfig("bw", B=2, Hq=4, Hkv=2, D=128, T_max=T, seed=500 + Lq + T)
    print(run_case(plx, oracle, cfg, Lq))


@pytest.mark.parametrize("G", [1, 2, 4])
def test_backward_gqa_and_bf16_io(plx, oracle, G):
    """The key and value gradients sum over the query heads of a group; bf16 forward output / saved mean
    and bf16 gradients."""
    cfg = wl.DecodeConfig("bwg", B=1, Hq=2 * G, Hkv=2, D=128, T_max=448, seed=510 + G)
    run_case(plx, oracle, cfg, 320, io_dtype=torch.bfloat16, grad_dtype=torch.bfloat16)


@pytest.mark.parametrize("Lq,T", [(1, 200), (130, 130), (200, 777), (512, 512)])
def test_backward_head_dim_64(plx, oracle, Lq, T):
    cfg = wl.DecodeConfig("bw64", B=2, Hq=4, Hkv=2, D=64, T_max=T, ragged=(max(1, T // 2), T), seed=550 + Lq)
    run_case(plx, oracle, cfg, Lq, poison=True)


def test_backward_ragged_poisoned_and_short_contexts(plx, oracle):
    """Per-sequence context lengths with NaN padding; one context shorter than Lq (rows without keys),
    one of exactly Lq, one empty: padded key rows and key-less query rows get exact zeros."""
    cfg = wl.DecodeConfig("bwr", B=5, Hq=4, Hkv=2, D=128, T_max=700, seed=520)
    run_case(plx, oracle, cfg, 200, seqlens=[700, 333, 200, 150, 0])


def test_backward_is_repeatable(plx, oracle):
    """No atomics anywhere: two runs give the same bits."""
    cfg = wl.DecodeConfig("bwd", B=2, Hq=4, Hkv=2, D=128, T_max=384, seed=530)
    Lq = 384
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    dout = torch.randn(2, 4, Lq, 128, device="cuda").to(torch.bfloat16)
    out = torch.empty(2, 4, Lq, 128, dtype=torch.float32, device="cuda")
    vbar, lse = torch.empty_like(out), torch.empty(2, 4, Lq, dtype=torch.float32, device="cuda")
    tbar = torch.empty_like(lse)
    plx.parallax_prefill_fwd_save(x["q"], x["r"], x["k"], x["v"], None, out, lse, tbar, vbar, cfg.scale)
    ws = torch.empty(plx.parallax_prefill_bwd_workspace_bytes(2, 4, Lq), dtype=torch.uint8, device="cuda")
    runs = []
    for _ in range(2):
        grads = [torch.empty(2, 4, Lq, 128, device="cuda") for _ in range(2)] + [torch.empty(2, 2, 384, 128, device="cuda") for _ in range(2)]
        plx.parallax_prefill_bwd(x["q"], x["r"], x["k"], x["v"], dout, out, lse, tbar, vbar, None, *grads, cfg.scale, ws)
        torch.cuda.synchronize()
        runs.append(grads)
    for a, b in zip(*runs):
        assert torch.equal(a, b)


def test_backward_full_size_in_the_bench_configuration(plx, oracle):
    """T1 at full size with the dtypes the bench times (bf16 output / saved mean / gradients): dq, dr on
    sampled rows (each row is a one-token problem for the oracle), dk, dv for one whole (sequence, KV head)
    group (the oracle needs every row of the group for them)."""
    cfg, Lq = wl.BACKWARD_CONFIGS["T1"]
    B, Hq, Hkv, D, T, G = cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T_max, cfg.G
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    gen = torch.Generator(device="cuda").manual_seed(cfg.seed + 5)
    dout = torch.randn(B, Hq, Lq, D, device="cuda", generator=gen).to(torch.bfloat16)
    out = torch.empty(B, Hq, Lq, D, dtype=torch.bfloat16, device="cuda")
    vbar = torch.empty_like(out)
    lse = torch.empty(B, Hq, Lq, dtype=torch.float32, device="cuda")
    tbar = torch.empty_like(lse)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_prefill_fwd_save(x["q"], x["r"], x["k"], x["v"], None, out, lse, tbar, vbar, cfg.scale, status)
    dq, dr = torch.empty_like(out), torch.empty_like(out)
    dk = torch.empty(B, Hkv, T, D, dtype=torch.bfloat16, device="cuda")
    dv = torch.empty_like(dk)
    ws = torch.empty(plx.parallax_prefill_bwd_workspace_bytes(B, Hq, Lq), dtype=torch.uint8, device="cuda")
    plx.parallax_prefill_bwd(x["q"], x["r"], x["k"], x["v"], dout, out, lse, tbar, vbar, None, dq, dr, dk, dv,
                             cfg.scale, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    # The forward output the backward reads is bf16 here: tau = dO . o inherits its rounding (2^-9 of |o|
    # per element), which adds about 2^-9 |o| |dO| sqrt(D) / |g| to the relative error of dq: the relative
    # RMS bar stays 1e-2, the element bound is taken against the sampled rows' largest entry.
    g = np.random.default_rng(7)
    rows = [(int(g.integers(B)), int(g.integers(Hq)), int(i)) for i in
            list(g.integers(0, Lq, size=120)) + [0, 1, 63, 64, 127, 128, Lq - 1]]
    got_q, got_r, want_q, want_r = [], [], [], []
    for (b, h, i) in rows:
        hkv = h // G
        sl = slice(0, i + 1)
        one = lambda t: wl.bf16_bits(t[b:b + 1, h:h + 1, i:i + 1])
        kb, vb = wl.bf16_bits(x["k"][b:b + 1, hkv:hkv + 1, sl]), wl.bf16_bits(x["v"][b:b + 1, hkv:hkv + 1, sl])
        wq, wr, _, _ = oracle.backward_bf16(one(x["q"]), one(x["r"]), kb, vb, one(dout), None, cfg.scale)
        want_q.append(wq[0, 0, 0])
        want_r.append(wr[0, 0, 0])
        got_q.append(dq[b, h, i].float().cpu().numpy())
        got_r.append(dr[b, h, i].float().cpu().numpy())
    check_grad("dq (sampled rows)", np.stack(got_q), np.stack(want_q))
    check_grad("dr (sampled rows)", np.stack(got_r), np.stack(want_r))

    b, hkv = 3, 5
    hs = slice(hkv * G, (hkv + 1) * G)
    grp = lambda t: wl.bf16_bits(t[b:b + 1, hs])
    kb, vb = wl.bf16_bits(x["k"][b:b + 1, hkv:hkv + 1]), wl.bf16_bits(x["v"][b:b + 1, hkv:hkv + 1])
    _, _, wk, wv = oracle.backward_bf16(grp(x["q"]), grp(x["r"]), kb, vb, grp(dout), None, cfg.scale)
    check_grad("dk (one group)", dk[b, hkv].float().cpu().numpy(), wk[0, 0])
    check_grad("dv (one group)", dv[b, hkv].float().cpu().numpy(), wv[0, 0])

    # Every (sequence, KV head) group by two invariances of the forward: one vector added to all keys
    # changes nothing, so the key gradients of a group sum to zero; one vector added to all values is added
    # to every output row, so the value gradients sum to the group's summed upstream gradient.  A lost
    # tile or a wrong mask leaves a relative defect of the order of 1 / (number of tiles) ~ 1e-2.
    dkf, dvf = dk.float(), dv.float()
    assert (dkf.sum(dim=2).abs() <= 2e-3 * dkf.abs().sum(dim=2)).all()
    want_sum = dout.float().reshape(B, Hkv, G, Lq, D).sum(dim=(2, 3))
    assert ((dvf.sum(dim=2) - want_sum).abs() <= 2e-3 * dvf.abs().sum(dim=2)).all()


def test_backward_full_size_long_sequence(plx, oracle):
    """T2 (two sequences of 16384 tokens) at full size with the bench's dtypes.  dq, dr on sampled rows.  dk, dv
    of the LAST 256 keys of one (sequence, KV head) group: only the last 256 rows see those keys, so the oracle's
    backward of those rows alone (a 256-token problem on the full context) gives their complete gradients.
    Every group by the two shift invariances."""
    cfg, Lq = wl.BACKWARD_CONFIGS["T2"]
    B, Hq, Hkv, D, T, G = cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T_max, cfg.G
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    gen = torch.Generator(device="cuda").manual_seed(cfg.seed + 5)
    dout = torch.randn(B, Hq, Lq, D, device="cuda", generator=gen).to(torch.bfloat16)
    out = torch.empty(B, Hq, Lq, D, dtype=torch.bfloat16, device="cuda")
    vbar = torch.empty_like(out)
    lse = torch.empty(B, Hq, Lq, dtype=torch.float32, device="cuda")
    tbar = torch.empty_like(lse)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_prefill_fwd_save(x["q"], x["r"], x["k"], x["v"], None, out, lse, tbar, vbar, cfg.scale, status)
    dq, dr = torch.empty_like(out), torch.empty_like(out)
    dk = torch.empty(B, Hkv, T, D, dtype=torch.bfloat16, device="cuda")
    dv = torch.empty_like(dk)
    ws = torch.empty(plx.parallax_prefill_bwd_workspace_bytes(B, Hq, Lq), dtype=torch.uint8, device="cuda")
    plx.parallax_prefill_bwd(x["q"], x["r"], x["k"], x["v"], dout, out, lse, tbar, vbar, None, dq, dr, dk, dv,
                             cfg.scale, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    g = np.random.default_rng(17)
    rows = [(int(g.integers(B)), int(g.integers(Hq)), int(i)) for i in
            list(g.integers(0, Lq, size=60)) + [0, 127, 128, Lq - 1]]
    got_q, got_r, want_q, want_r = [], [], [], []
    for (b, h, i) in rows:
        hkv = h // G
        one = lambda t: wl.bf16_bits(t[b:b + 1, h:h + 1, i:i + 1])
        kb, vb = wl.bf16_bits(x["k"][b:b + 1, hkv:hkv + 1, :i + 1]), wl.bf16_bits(x["v"][b:b + 1, hkv:hkv + 1, :i + 1])
        wq, wr, _, _ = oracle.backward_bf16(one(x["q"]), one(x["r"]), kb, vb, one(dout), None, cfg.scale)
        want_q.append(wq[0, 0, 0])
        want_r.append(wr[0, 0, 0])
        got_q.append(dq[b, h, i].float().cpu().numpy())
        got_r.append(dr[b, h, i].float().cpu().numpy())
    check_grad("dq (sampled rows)", np.stack(got_q), np.stack(want_q))
    check_grad("dr (sampled rows)", np.stack(got_r), np.stack(want_r))

    b, hkv, tail = 1, 6, 256
    hs = slice(hkv * G, (hkv + 1) * G)
    last = lambda t: wl.bf16_bits(t[b:b + 1, hs, Lq - tail:])
    kb, vb = wl.bf16_bits(x["k"][b:b + 1, hkv:hkv + 1]), wl.bf16_bits(x["v"][b:b + 1, hkv:hkv + 1])
    _, _, wk, wv = oracle.backward_bf16(last(x["q"]), last(x["r"]), kb, vb, last(dout), None, cfg.scale)
    check_grad("dk (last keys of one group)", dk[b, hkv, T - tail:].float().cpu().numpy(), wk[0, 0, T - tail:])
    check_grad("dv (last keys of one group)", dv[b, hkv, T - tail:].float().cpu().numpy(), wv[0, 0, T - tail:])

    dkf, dvf = dk.float(), dv.float()
    assert (dkf.sum(dim=2).abs() <= 2e-3 * dkf.abs().sum(dim=2)).all()
    want_sum = dout.float().reshape(B, Hkv, G, Lq, D).sum(dim=(2, 3))
    assert ((dvf.sum(dim=2) - want_sum).abs() <= 2e-3 * dvf.abs().sum(dim=2)).all()


def test_autograd_front_end(plx, oracle):
    """torch.autograd wrapper: out.backward() routes to the library's backward; gradients against the oracle."""
    from paper_2605_29157_b200.autograd import parallax_attention
    cfg = wl.DecodeConfig("ag", B=2, Hq=4, Hkv=2, D=128, T_max=320, seed=560)
    Lq = 320
    x = wl.make_prefill_inputs(cfg, Lq, "cuda")
    leaves = {n: x[n].clone().requires_grad_(True) for n in ("q", "r", "k", "v")}
    out = parallax_attention(leaves["q"], leaves["r"], leaves["k"], leaves["v"], cfg.scale)
    gen = torch.Generator(device="cuda").manual_seed(561)
    dout = torch.randn(out.shape, device="cuda", generator=gen).to(torch.bfloat16)
    out.backward(dout)
    torch.cuda.synchronize()
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    want_out, _ = oracle.prefill_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale)
    assert np.abs(out.detach().float().cpu().numpy() - want_out).max() <= np.maximum(2e-2, 2.0 ** -8 * np.abs(want_out)).max()
    want = oracle.backward_bf16(bits["q"], bits["r"], bits["k"], bits["v"], wl.bf16_bits(dout), None, cfg.scale)
    for name, w in zip(("q", "r", "k", "v"), want):
        check_grad("d" + name, leaves[name].grad.float().cpu().numpy(), w)
