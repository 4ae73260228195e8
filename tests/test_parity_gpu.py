"""GPU parity: the CUDA path through the C ABI against the fp64 oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import assert_parity, errors, oracle_full, oracle_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def plx(cuda_device):
    from paper_2605_29157_b200 import binding
    return binding


def run_fwd(plx, x, cfg, out_dtype, num_splits=0, dev="cuda"):
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=out_dtype, device=dev)
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS if num_splits == 0 else num_splits, dev)
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, num_splits)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    return out.float().cpu().numpy()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("T", [1, 2, 15, 16, 17, 63, 64, 65, 127, 300, 1000])
def test_shape_sweep_single_split(plx, oracle, D, G, T):
    """One CTA per stream, every tail shape of the 16-key tile and the 4-warp round robin."""
    cfg = wl.DecodeConfig("sweep", B=2, Hq=2 * G, Hkv=2, D=D, T_max=T, seed=100 + T)
    x = wl.make_inputs(cfg, "cuda")
    want = oracle_full(oracle, x, cfg.scale)
    got = run_fwd(plx, x, cfg, torch.float32, num_splits=1)
    assert_parity(got, want, torch.float32, f"D={D} G={G} T={T}")


@pytest.mark.parametrize("D,G", [(64, 2), (64, 3), (128, 1), (128, 2), (128, 3), (128, 4), (128, 5), (128, 7), (128, 8),
                                 (64, 6), (64, 8)])
@pytest.mark.parametrize("T,ns", [(130, 2), (1000, 3), (1000, 16), (4096, 0), (5000, 7)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_split_kv(plx, oracle, D, G, T, ns, out_dtype):
    """Several key chunks merged by the combine kernel, ragged last chunk, planned and forced splits."""
    cfg = wl.DecodeConfig("split", B=3, Hq=2 * G, Hkv=2, D=D, T_max=T, seed=7 * T + ns)
    x = wl.make_inputs(cfg, "cuda")
    want = oracle_full(oracle, x, cfg.scale)
    got = run_fwd(plx, x, cfg, out_dtype, num_splits=ns)
    assert_parity(got, want, out_dtype, f"D={D} G={G} T={T} ns={ns}")


@pytest.mark.parametrize("D,G", [(128, 2), (128, 4), (128, 1), (64, 2), (64, 4), (128, 6), (128, 8), (64, 7)])
def test_many_splits_batched_merge(plx, oracle, D, G):
    """More splits per row than the merging CTA can stage at once (47 records per row at D=128,
    G=2; 23 at G=4): the merge runs in several batches with a running reference exponent.  Ragged
    lengths make the number of live splits differ per sequence."""
    cfg = wl.DecodeConfig("many", B=3, Hq=2 * G, Hkv=2, D=D, T_max=12800, ragged=(6000, 12800), seed=77 + D + G)
    x = wl.make_inputs(cfg, "cuda", poison_padding=True)
    want = oracle_full(oracle, x, cfg.scale, x["seqlens_host"])
    got = run_fwd(plx, x, cfg, torch.float32, num_splits=200)
    assert_parity(got, want, torch.float32, f"many splits D={D} G={G}")


def test_maximum_split_count(plx, oracle):
    """PLX_MAX_SPLITS chunks of 64 keys (the finest granularity): 22 merge batches per row."""
    cfg = wl.DecodeConfig("maxsplit", B=1, Hq=4, Hkv=2, D=128, T_max=64 * 1024, seed=88)
    x = wl.make_inputs(cfg, "cuda")
    want = oracle_full(oracle, x, cfg.scale)
    got = run_fwd(plx, x, cfg, torch.float32, num_splits=plx.PLX_MAX_SPLITS)
    assert_parity(got, want, torch.float32, "1024 splits")


@pytest.mark.parametrize("ns", [1, 0, 5])
def test_ragged_poisoned_padding_and_empty_rows(plx, oracle, ns):
    """Per-sequence lengths over a padded cache whose padding is NaN; lengths 0 and 1 included."""
    cfg = wl.DecodeConfig("ragged", B=9, Hq=4, Hkv=2, D=128, T_max=700, ragged=(1, 700), seed=5)
    x = wl.make_inputs(cfg, "cuda", poison_padding=True)
    sl = x["seqlens_host"].copy()
    sl[0], sl[1], sl[2], sl[3] = 0, 1, 16, 17
    for b in range(4):
        x["k"][b, :, sl[b]:] = float("nan")
        x["v"][b, :, sl[b]:] = float("nan")
    x["seqlens"] = torch.from_numpy(sl).cuda()
    want = oracle_full(oracle, x, cfg.scale, sl)
    got = run_fwd(plx, x, cfg, torch.float32, num_splits=ns)
    assert (got[0] == 0).all()
    assert_parity(got, want, torch.float32, f"ragged ns={ns}")


def test_context_lengths_outside_the_cache_are_clamped(plx, oracle):
    """A length below zero reads as an empty context (a row of zeros), a length beyond the cache's
    capacity as a full cache: no entry point reads outside the buffers it was given."""
    cfg = wl.DecodeConfig("clamp", B=4, Hq=4, Hkv=2, D=128, T_max=500, seed=71)
    x = wl.make_inputs(cfg, "cuda")
    given = np.array([-7, 500 + 1000, 2 ** 31 - 1, 123], dtype=np.int32)
    meant = np.array([0, 500, 500, 123], dtype=np.int32)
    x["seqlens"] = torch.from_numpy(given).cuda()
    want = oracle_full(oracle, x, cfg.scale, meant)
    for ns in (1, 0, 4):
        got = run_fwd(plx, x, cfg, torch.float32, num_splits=ns)
        assert (got[0] == 0).all()
        assert_parity(got, want, torch.float32, f"clamped ns={ns}")


def test_special_cases_on_gpu(plx, oracle):
    """rho = 0 gives softmax attention; one key returns its value (same pins as the oracle's)."""
    cfg = wl.DecodeConfig("sp", B=2, Hq=4, Hkv=2, D=128, T_max=333, seed=11)
    x = wl.make_inputs(cfg, "cuda")
    x["r"].zero_()
    got = run_fwd(plx, x, cfg, torch.float32, num_splits=1)
    G = cfg.G
    kf, vf, qf = x["k"].double(), x["v"].double(), x["q"].double()
    for b in range(cfg.B):
        for hq in range(cfg.Hq):
            p = torch.softmax(kf[b, hq // G] @ qf[b, hq] * cfg.scale, dim=0)
            want = (p[None] @ vf[b, hq // G])[0].cpu().numpy()
            np.testing.assert_allclose(got[b, hq], want, rtol=0, atol=2e-4)
    cfg1 = wl.DecodeConfig("one", B=2, Hq=4, Hkv=2, D=64, T_max=40, seed=12)
    x = wl.make_inputs(cfg1, "cuda")
    x["seqlens"] = torch.ones(2, dtype=torch.int32, device="cuda")
    got = run_fwd(plx, x, cfg1, torch.float32, num_splits=1)
    for hq in range(4):
        # O1/d1 (1 + t) - t O1/d1 with |t| ~ sqrt(D): the two probe terms cancel, each good to ~2^-17
        np.testing.assert_allclose(got[:, hq], x["v"][:, hq // 2, 0].float().cpu().numpy(), rtol=0, atol=5e-5)


@pytest.mark.parametrize("kind", ["peaked", "ascending", "probe_offset", "scale0", "negative_scale"])
def test_robustness_distributions(plx, oracle, kind):
    """Inputs that stress the online maximum and the cancellation in the covariance branch."""
    cfg = wl.DecodeConfig("rob", B=2, Hq=4, Hkv=2, D=128, T_max=2048, seed=21)
    x = wl.make_inputs(cfg, "cuda")
    scale = cfg.scale
    if kind == "peaked":
        x["q"] = (x["q"].float() * 4).to(torch.bfloat16)
    elif kind == "ascending":
        # keys ordered by ascending logit of head 0: the running maximum grows at every tile
        for b in range(cfg.B):
            for h in range(cfg.Hkv):
                order = torch.argsort(x["k"][b, h].float() @ x["q"][b, h * cfg.G].float())
                x["k"][b, h] = x["k"][b, h][order]
                x["v"][b, h] = x["v"][b, h][order]
    elif kind == "probe_offset":
        # every key shares a large component along the probe: t_j = c + small
        for b in range(cfg.B):
            for h in range(cfg.Hkv):
                rdir = x["r"][b, h * cfg.G].float()
                x["k"][b, h] = (x["k"][b, h].float() + 0.5 * rdir[None, :]).to(torch.bfloat16)
    elif kind == "scale0":
        scale = 0.0
    elif kind == "negative_scale":
        scale = -cfg.scale
    want = oracle_full(oracle, x, scale)
    out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, 8, "cuda")
    for ns in (1, 8):
        plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, out, scale, ws, ns)
        torch.cuda.synchronize()
        e = errors(out.cpu().numpy(), want)
        assert e["rel_rms"] <= 1e-3 and e["max_abs"] <= 2e-2 * max(1.0, e["rms"]), (kind, ns, e)


def test_partial_entry_point_matches_oracle_state(plx, oracle):
    """The stand-alone split kernel: every record against the oracle's per-split state (compared
    after moving both to the oracle's reference exponent), empty records where the split is past
    the context."""
    cfg = wl.DecodeConfig("part", B=3, Hq=4, Hkv=2, D=128, T_max=400, seed=31)
    x = wl.make_inputs(cfg, "cuda")
    sl = np.array([400, 130, 0], dtype=np.int32)
    x["seqlens"] = torch.from_numpy(sl).cuda()
    chunk, ns = 96, 5
    stride = plx.parallax_partial_stride(cfg.D)
    assert stride == 2 * cfg.D + 4
    partials = torch.full((cfg.B, cfg.Hq, ns, stride), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_decode_splitkv_partial(x["q"], x["r"], x["k"], x["v"], x["seqlens"], partials, cfg.scale, chunk, ns, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    P = partials.cpu().numpy().astype(np.float64)
    f = {n: x[n].double().cpu().numpy() for n in ("q", "r", "k", "v")}
    D = cfg.D
    for b in range(cfg.B):
        for hq in range(cfg.Hq):
            K, V = f["k"][b, hq // 2, :sl[b]], f["v"][b, hq // 2, :sl[b]]
            for s in range(ns):
                k0, k1 = min(s * chunk, sl[b]), min((s + 1) * chunk, sl[b])
                m, d1, d2, O1, O2 = oracle.partial_state(f["q"][b, hq], f["r"][b, hq], K, V, cfg.scale, k0, k1)
                rec = P[b, hq, s]
                if k1 <= k0:
                    assert rec[0] == -np.inf and (rec[1:] == 0).all()
                    continue
                assert rec[0] <= m + 1e-4 and rec[0] >= m - 8 * np.log(2) - 1e-4
                a = np.exp(rec[0] - m)
                np.testing.assert_allclose(a * rec[1], d1, rtol=2e-5, atol=1e-6)
                np.testing.assert_allclose(a * rec[2], d2, rtol=0, atol=2e-4 * max(1.0, abs(d1)) )
                np.testing.assert_allclose(a * rec[4:4 + D], O1, rtol=0, atol=1e-4 * max(1.0, np.sqrt(d1)))
                np.testing.assert_allclose(a * rec[4 + D:4 + 2 * D], O2, rtol=0, atol=1e-3 * max(1.0, np.sqrt(d1)))
    # and the exported combine turns those records into the oracle's output
    out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    plx.parallax_decode_combine(partials, None, out, ns)
    torch.cuda.synchronize()
    want = oracle_full(oracle, x, cfg.scale, sl)
    assert_parity(out.cpu().numpy(), want, torch.float32, "partial+combine")


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_combine_entry_point_alone(plx, oracle, D, out_dtype):
    """Combine kernel on synthetic records (not produced by the main kernel): exponents spread over
    a wide range, empty records, per-sequence split counts; against the oracle's merge."""
    g = np.random.default_rng(41)
    B, Hq, ns = 3, 4, 37
    stride = 2 * D + 4
    P = np.zeros((B, Hq, ns, stride), dtype=np.float32)
    P[..., 0] = g.uniform(-30, 30, (B, Hq, ns))
    P[..., 1] = g.uniform(0.5, 50, (B, Hq, ns))
    P[..., 2] = g.standard_normal((B, Hq, ns)) * 20
    P[..., 4:] = g.standard_normal((B, Hq, ns, 2 * D)) * 5
    empty = g.random((B, Hq, ns)) < 0.2
    P[empty, 0] = -np.inf
    P[empty, 1:] = 0
    P[1, 2, :, 0] = -np.inf          # a row with nothing at all
    P[1, 2, :, 1:] = 0
    counts = np.array([ns, 5, ns], dtype=np.int32)
    P[1, :, 5:] = np.nan             # records past the count must not be read into the result
    out = torch.empty(B, Hq, D, dtype=out_dtype, device="cuda")
    plx.parallax_decode_combine(torch.from_numpy(P).cuda(), torch.from_numpy(counts).cuda(), out, ns)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    P64 = P.astype(np.float64)
    for b in range(B):
        for h in range(Hq):
            states = [(P64[b, h, s, 0], P64[b, h, s, 1], P64[b, h, s, 2], P64[b, h, s, 4:4 + D], P64[b, h, s, 4 + D:])
                      for s in range(counts[b])]
            want = oracle.merge_partials(states)
            tol = 1e-4 if out_dtype == torch.float32 else 1e-2
            np.testing.assert_allclose(got[b, h], want, rtol=tol, atol=tol * max(1.0, np.abs(want).max()))
    assert (got[1, 2] == 0).all()


def test_bitwise_repeatable(plx):
    """Fixed merge order: two runs give identical bits (also a smoke test for races)."""
    cfg = wl.DecodeConfig("rep", B=4, Hq=16, Hkv=8, D=128, T_max=3000, seed=51)
    x = wl.make_inputs(cfg, "cuda")
    outs = []
    for _ in range(3):
        out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
        ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
        plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0)
        torch.cuda.synchronize()
        outs.append(out.clone())
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_short_form_and_host_entry(plx, oracle):
    """parallax_decode_fwd after parallax_set_layout, and the host-buffer entry point, give the
    same bits as the explicit form."""
    cfg = wl.DecodeConfig("short", B=4, Hq=16, Hkv=8, D=128, T_max=1500, seed=61)
    x = wl.make_inputs(cfg, "cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    ref = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.bfloat16, device="cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, ref, cfg.scale, ws, 0)
    out = torch.empty_like(ref)
    plx.parallax_set_layout(cfg.T_max, torch.bfloat16, ws)
    plx.parallax_decode_fwd(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale)
    torch.cuda.synchronize()
    assert torch.equal(out, ref)
    qh, rh = x["q"].cpu().pin_memory(), x["r"].cpu().pin_memory()
    oh = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.bfloat16).pin_memory()
    plx.parallax_decode_fwd_host(qh, rh, x["k"], x["v"], None, oh, cfg.scale, ws, 0)
    assert torch.equal(oh, ref.cpu())
    # pageable host memory takes the staged route (copies through the workspace); page-locked memory is
    # written by the kernel directly: same bits either way, and with fp32 output and several forced splits
    for pinned in (False, True):
        for dtype, ns in ((torch.bfloat16, 0), (torch.float32, 5)):
            want_dev = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=dtype, device="cuda")
            plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, want_dev, cfg.scale, ws, ns)
            torch.cuda.synchronize()
            q2, r2 = x["q"].cpu(), x["r"].cpu()
            o2 = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=dtype)
            if pinned:
                q2, r2, o2 = q2.pin_memory(), r2.pin_memory(), o2.pin_memory()
            plx.parallax_decode_fwd_host(q2, r2, x["k"], x["v"], None, o2, cfg.scale, ws, ns)
            assert torch.equal(o2, want_dev.cpu()), (pinned, dtype)
    want = oracle_full(oracle, x, cfg.scale)
    assert_parity(ref.float().cpu().numpy(), want, torch.bfloat16, "short form")


def test_host_entry_sees_host_writes_between_steps(plx, oracle):
    """The same page-locked q, r, out buffers reused step after step with new contents written by the
    host in between (the kernel reads them over the host link): every step uses that step's values."""
    cfg = wl.DecodeConfig("host steps", B=4, Hq=16, Hkv=8, D=128, T_max=900, seed=62)
    x = wl.make_inputs(cfg, "cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    qh = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.bfloat16).pin_memory()
    rh = torch.empty_like(qh).pin_memory()
    oh = torch.empty_like(qh).pin_memory()
    g = torch.Generator().manual_seed(63)
    ref = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.bfloat16, device="cuda")
    for step in range(6):
        qh.copy_(torch.randn(cfg.B, cfg.Hq, cfg.D, generator=g).to(torch.bfloat16))
        rh.copy_(torch.randn(cfg.B, cfg.Hq, cfg.D, generator=g).to(torch.bfloat16))
        oh.fill_(float("nan"))
        plx.parallax_decode_fwd_host(qh, rh, x["k"], x["v"], None, oh, cfg.scale, ws, 0)
        plx.parallax_decode_fwd_ex(qh.cuda(), rh.cuda(), x["k"], x["v"], None, ref, cfg.scale, ws, 0)
        torch.cuda.synchronize()
        assert torch.equal(oh, ref.cpu()), step


def test_config_c1_tiny(plx, oracle):
    cfg = wl.CONFIGS["C1"]
    x = wl.make_inputs(cfg, "cuda")
    want = oracle_full(oracle, x, cfg.scale)
    got = run_fwd(plx, x, cfg, torch.float32)
    assert_parity(got, want, torch.float32, "C1")


def _sample_rows(cfg, n, seed):
    g = np.random.default_rng(seed)
    rows = {(0, 0), (cfg.B - 1, cfg.Hq - 1)}
    while len(rows) < n:
        rows.add((int(g.integers(cfg.B)), int(g.integers(cfg.Hq))))
    return sorted(rows)


@pytest.mark.parametrize("name,nrows", [("C2", 128), ("C3", 1024), ("C4", 32), ("C5", 2048), ("C6", 1024)])
def test_full_size_configs(plx, oracle, name, nrows):
    """The large configurations at full size, in the launch configuration the bench times
    (planned splits, bf16 output): EVERY row of every configuration against the oracle (which computes a row
    at a time from the slab that row needs)."""
    cfg = wl.CONFIGS[name]
    x = wl.make_inputs(cfg, "cuda", poison_padding=(name == "C5"))
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, 0)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    assert torch.isfinite(out.float()).all()
    rows = [(b, h) for b in range(cfg.B) for h in range(cfg.Hq)] if nrows >= cfg.B * cfg.Hq else _sample_rows(cfg, nrows, 7)
    if name == "C5":  # make sure the shortest and the longest context are among the samples
        sl = x["seqlens_host"]
        rows = sorted(set(rows) | {(int(sl.argmin()), 3), (int(sl.argmax()), 12)})
    want = oracle_rows(oracle, x, cfg.scale, rows, x["seqlens_host"])
    got = np.stack([out[b, h].float().cpu().numpy() for (b, h) in rows])
    e = assert_parity(got, want, torch.bfloat16, name)
    print(name, e)


@pytest.mark.parametrize("page_size,T,ns", [(16, 300, 1), (64, 1000, 0), (64, 1000, 5), (256, 4096, 0), (128, 2500, 7)])
def test_paged_kv_cache(plx, oracle, page_size, T, ns):
    """Paged cache (page pools + block table, random page order, NaN in unused pages and page tails)
    against the oracle on the equivalent contiguous cache; ragged lengths."""
    cfg = wl.DecodeConfig("paged", B=5, Hq=4, Hkv=2, D=128, T_max=T, ragged=(1, T), seed=900 + page_size + ns)
    x = wl.make_inputs(cfg, "cuda")
    kp, vp, table = wl.to_paged(x["k"], x["v"], page_size, seed=3)
    want = oracle_full(oracle, x, cfg.scale, x["seqlens_host"])
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    plx.parallax_decode_fwd_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, ns)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    assert_parity(out.cpu().numpy(), want, torch.float32, f"paged ps={page_size} T={T} ns={ns}")
    # and bit-identical to the contiguous entry point with the same chunking
    ref = torch.empty_like(out)
    T_pad = table.shape[1] * page_size
    kc = torch.zeros(cfg.B, cfg.Hkv, T_pad, cfg.D, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    kc[:, :, :T], vc[:, :, :T] = x["k"], x["v"]
    plx.parallax_decode_fwd_ex(x["q"], x["r"], kc, vc, x["seqlens"], ref, cfg.scale, ws, ns)
    torch.cuda.synchronize()
    assert torch.equal(out, ref)


@pytest.mark.parametrize("ranks", [2, 4])
def test_sequence_sharded_combine_on_one_gpu(plx, oracle, ranks):
    """The sequence-sharded path with the ranks emulated on one GPU: the split kernel runs once per
    key slice (no kernel waits on another), the records are laid out exactly as an all-gather would
    leave them, and parallax_decode_combine_gathered merges them; against the oracle on the whole
    context.  Slices have unequal and, for one sequence, zero lengths."""
    cfg = wl.DecodeConfig("seqpar", B=3, Hq=4, Hkv=2, D=128, T_max=1000, seed=950 + ranks)
    x = wl.make_inputs(cfg, "cuda")
    sl = np.array([1000, 417, 130], dtype=np.int32)
    x["seqlens"] = torch.from_numpy(sl).cuda()
    want = oracle_full(oracle, x, cfg.scale, sl)
    T_shard = -(-cfg.T_max // ranks)
    chunk, ns = 128, -(-T_shard // 128)
    stride = plx.parallax_partial_stride(cfg.D)
    gathered = torch.full((ranks, cfg.B, cfg.Hq, ns, stride), float("nan"), dtype=torch.float32, device="cuda")
    for w in range(ranks):
        lo = w * T_shard
        ks = x["k"][:, :, lo:lo + T_shard].contiguous()
        vs = x["v"][:, :, lo:lo + T_shard].contiguous()
        lens = torch.from_numpy(np.clip(sl - lo, 0, ks.shape[2]).astype(np.int32)).cuda()
        plx.parallax_decode_splitkv_partial(x["q"], x["r"], ks, vs, lens, gathered[w], cfg.scale, chunk, ns)
    out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    plx.parallax_decode_combine_gathered(gathered, out, ranks, ns)
    torch.cuda.synchronize()
    assert_parity(out.cpu().numpy(), want, torch.float32, f"sequence-sharded, {ranks} ranks")


def test_sequence_sharded_single_rank_nccl(plx, oracle):
    """decode_sequence_sharded end to end with a one-rank NCCL group (the only group one GPU allows)."""
    import os
    import torch.distributed as dist
    from paper_2605_29157_b200 import sequence_parallel as sp
    import socket
    with socket.socket() as sk:               # a free port: the machine is shared with other jobs
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        cfg = wl.DecodeConfig("seqpar1", B=2, Hq=4, Hkv=2, D=128, T_max=3000, seed=960)
        x = wl.make_inputs(cfg, "cuda")
        out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
        sp.decode_sequence_sharded(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale)
        torch.cuda.synchronize()
        assert_parity(out.cpu().numpy(), oracle_full(oracle, x, cfg.scale), torch.float32, "one-rank NCCL")
    finally:
        if created:
            dist.destroy_process_group()


def test_call_from_a_fresh_host_thread(plx, oracle):
    """A worker thread that has made no CUDA call of its own (an autograd or serving worker) has no
    current driver context; the library has to bind one before it encodes a tensor map there."""
    import threading
    cfg = wl.DecodeConfig("thread", B=2, Hq=4, Hkv=2, D=128, T_max=333, seed=991)
    x = wl.make_inputs(cfg, "cuda")
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    result = {}

    def work():
        try:
            plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, None, 1,
                                       stream=torch.cuda.default_stream(out.device))
            result["ok"] = True
        except Exception as e:  # noqa: BLE001 - reported below
            result["error"] = e

    t = threading.Thread(target=work)
    t.start()
    t.join()
    torch.cuda.synchronize()
    assert "error" not in result, result.get("error")
    assert_parity(out.cpu().numpy(), oracle_full(oracle, x, cfg.scale), torch.float32, "fresh thread")


def test_capture_into_a_cuda_graph_with_buffers_the_library_has_not_seen(plx, oracle):
    """Every entry point may be captured into a CUDA graph, also when the capture is the library's first
    sight of the K/V buffers (their tensor maps are encoded during the capture, where no call that
    synchronises or frees is allowed); replays reproduce the eager result bit for bit."""
    cfg = wl.DecodeConfig("graph", B=3, Hq=8, Hkv=2, D=128, T_max=2100, ragged=(1, 2100), seed=993)
    x = wl.make_inputs(cfg, "cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    eager = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], eager, cfg.scale, ws, 0)
    torch.cuda.synchronize()
    k2, v2 = x["k"].clone(), x["v"].clone()       # fresh addresses
    out = torch.full_like(eager, float("nan"))
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        plx.parallax_decode_fwd_ex(x["q"], x["r"], k2, v2, x["seqlens"], out, cfg.scale, ws, 0,
                                   stream=torch.cuda.current_stream())
    for _ in range(3):
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager)
    assert plx.parallax_workspace_status(ws) == 0
    assert_parity(out.cpu().numpy(), oracle_full(oracle, x, cfg.scale, x["seqlens_host"]), torch.float32, "graph")


@pytest.mark.parametrize("name", ["C3", "C4", "C5"])
def test_full_size_every_row_by_a_property(plx, name):
    """A property that holds at any size and checks EVERY row of a full-size call: the effective weights
    p_j (1 + tbar - t_j) sum to one (Sec. 4, score-pattern analysis), so when all values of a stream are
    one vector c the output row is c whatever q, the probe and the keys are.  The per-key terms reach
    |1 + tbar - t| ~ 30 and cancel, so the bound is loose in absolute terms but tight for a wrong mask,
    a lost tile or a broken merge (those leave O(1) errors)."""
    cfg = wl.CONFIGS[name]
    x = wl.make_inputs(cfg, "cuda", poison_padding=(name == "C5"))
    g = torch.Generator(device="cuda").manual_seed(5)
    c = torch.randn(cfg.B, cfg.Hkv, 1, cfg.D, device="cuda", generator=g).to(torch.bfloat16)
    v = c.expand(cfg.B, cfg.Hkv, cfg.T_max, cfg.D).contiguous()
    if x["seqlens"] is not None:
        for b in range(cfg.B):
            v[b, :, int(x["seqlens_host"][b]):] = float("nan")
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], v, x["seqlens"], out, cfg.scale, ws, 0)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    want = c[:, :, 0].float().repeat_interleave(cfg.G, dim=1)      # [B, Hq, D]
    err = (out - want).abs().max().item()
    assert err <= 2e-3, err


@pytest.mark.parametrize("D,Hq,Hkv", [(128, 16, 2), (128, 12, 2), (64, 32, 4), (128, 10, 2), (128, 14, 2)])
@pytest.mark.parametrize("ns", [1, 0, 5])
def test_large_gqa_groups(plx, oracle, D, Hq, Hkv, ns):
    """Group sizes above 4 (8, 6, 8, 5, 7 query heads per KV head): one CTA serves all heads of a KV head
    (two quads of heads in the 8 MMA columns, each with its own accumulator set)."""
    cfg = wl.DecodeConfig("gqa", B=2, Hq=Hq, Hkv=Hkv, D=D, T_max=1500, ragged=(200, 1500), seed=970 + Hq)
    x = wl.make_inputs(cfg, "cuda", poison_padding=True)
    want = oracle_full(oracle, x, cfg.scale, x["seqlens_host"])
    got = run_fwd(plx, x, cfg, torch.float32, num_splits=ns)
    assert_parity(got, want, torch.float32, f"G={Hq // Hkv} D={D} ns={ns}")


@pytest.mark.parametrize("D,Hq,Hkv,ns", [(128, 32, 2, 0), (128, 64, 1, 3), (64, 48, 3, 0), (128, 260, 2, 0), (128, 18, 2, 1)])
def test_multi_query_groups_go_to_the_tensor_core_kernel(plx, oracle, D, Hq, Hkv, ns):
    """More than eight query heads per KV head (multi-query models; also more than the decode kernel's 64):
    parallax_decode_fwd_ex hands the step to the tensor-core kernel, contiguous and paged, with and without a
    workspace; the bars are the same."""
    cfg = wl.DecodeConfig("mqa", B=3, Hq=Hq, Hkv=Hkv, D=D, T_max=2100, ragged=(1, 2100), seed=980 + Hq)
    x = wl.make_inputs(cfg, "cuda", poison_padding=True)
    want = oracle_full(oracle, x, cfg.scale, x["seqlens_host"])
    got = run_fwd(plx, x, cfg, torch.float32, num_splits=ns)
    assert_parity(got, want, torch.float32, f"G={Hq // Hkv} D={D} ns={ns}")
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, None, 0)
    torch.cuda.synchronize()
    assert_parity(out.cpu().numpy(), want, torch.float32, "no workspace")
    kp, vp, table = wl.to_paged(x["k"], x["v"], 64, seed=11)
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    out.fill_(float("nan"))
    plx.parallax_decode_fwd_paged(x["q"], x["r"], kp, vp, table, x["seqlens"], out, cfg.scale, ws, ns)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    assert_parity(out.cpu().numpy(), want, torch.float32, "paged")
    # host-buffer entry point
    qh, rh = x["q"].cpu().pin_memory(), x["r"].cpu().pin_memory()
    oh = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32).pin_memory()
    plx.parallax_decode_fwd_host(qh, rh, x["k"], x["v"], x["seqlens"], oh, cfg.scale, ws, ns)
    assert_parity(oh.numpy(), want, torch.float32, "host entry")


def test_one_million_key_context(plx, oracle):
    """One sequence of 2^20 keys (4 GiB of K and V): split planning, chunk arithmetic and the fused merge at a
    context eight times the longest benchmark configuration; sampled rows against the oracle, every row finite."""
    cfg = wl.DecodeConfig("1M", B=1, Hq=16, Hkv=8, D=128, T_max=1 << 20, seed=4321)
    x = wl.make_inputs(cfg, "cuda")
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0)
    torch.cuda.synchronize()
    assert plx.parallax_workspace_status(ws) == 0
    assert torch.isfinite(out).all()
    rows = [(0, 0), (0, 7), (0, 15)]
    want = oracle_rows(oracle, x, cfg.scale, rows)
    got = np.stack([out[b, h].cpu().numpy() for (b, h) in rows])
    assert_parity(got, want, torch.float32, "2^20 keys")
