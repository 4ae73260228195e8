"""The workspace-free entry point, for callers that cannot allocate device memory where they
decode (inside regions where cudaMalloc is illegal, under a host framework's memory pool, in
allocator-averse latency loops).  It keeps its split scratch in a fixed array inside the library.

Collected last on purpose: a run that stops at the first failure has then already run everything
else.  Passes alone in a fresh process as well as after the other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import MAX_ABS_TOL, MEAN_ABS_TOL, assert_parity, oracle_full


def test_explicit_split_count_beyond_the_array_is_rejected():
    """Host-side check, no device needed: 1024 splits of a 64 x 16 x 128 problem need ~1 GiB."""
    from paper_2605_29157_b200 import build, binding
    build.build()
    fake = ctypes.c_void_p(0x1000)
    rc = binding._lib.parallax_decode_fwd_static(fake, fake, fake, fake, None, fake, 64, 16, 8, 128, 1 << 17, 0.1,
                                                 0, 1024, None)
    assert rc == binding.PLX_ERR_STATIC_SCRATCH
    assert "static" in binding.status_string(rc)


@pytest.mark.gpu
def test_static_scratch_entry_matches_workspace_entry(cuda_device, oracle):
    """Two calls in a row on different inputs and split counts, each against the workspace-taking
    entry point on the same inputs and against the fp64 oracle, within the parity tolerances used
    throughout the suite.  The second call reuses the array the first one filled, so stale records
    would show here."""
    from paper_2605_29157_b200 import binding as plx
    cases = [
        (wl.DecodeConfig("na1", B=4, Hq=16, Hkv=8, D=128, T_max=3000, seed=71), 6, torch.float32),
        (wl.DecodeConfig("na2", B=3, Hq=8, Hkv=2, D=64, T_max=1100, ragged=(1, 1100), seed=72), 0, torch.bfloat16),
    ]
    for cfg, ns, dt in cases:
        x = wl.make_inputs(cfg, "cuda", poison_padding=True)
        ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
        ref = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=dt, device="cuda")
        got = torch.full_like(ref, float("nan"))
        plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], ref, cfg.scale, ws, ns)
        plx.parallax_decode_fwd_static(x["q"], x["r"], x["k"], x["v"], x["seqlens"], got, cfg.scale, ns)
        torch.cuda.synchronize()
        a, b = got.float().cpu().numpy(), ref.float().cpu().numpy()
        assert np.isfinite(a).all() and np.isfinite(b).all()
        diff = np.abs(a.astype(np.float64) - b)
        assert diff.max() <= MAX_ABS_TOL and diff.mean() <= MEAN_ABS_TOL, (cfg.name, diff.max(), diff.mean())
        assert_parity(a, oracle_full(oracle, x, cfg.scale, x["seqlens_host"]), dt, f"static entry, {cfg.name}")


@pytest.mark.gpu
def test_planned_splits_are_clamped_to_the_array(cuda_device, oracle):
    """A shape whose planned split records would not fit the 8 MiB array (many short ragged sequences on
    a long padded cache): the entry point plans fewer splits instead of failing, and the result stands."""
    from paper_2605_29157_b200 import binding as plx
    cfg = wl.DecodeConfig("na3", B=96, Hq=16, Hkv=8, D=128, T_max=16384, ragged=(1, 700), seed=73)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    _, planned = plx.parallax_decode_plan(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T_max, sms, True)
    rec_bytes = cfg.B * cfg.Hq * planned * plx.parallax_partial_stride(cfg.D) * 4
    assert rec_bytes > plx.PLX_STATIC_SCRATCH_BYTES, "the case must exceed the array for the clamp to act"
    x = wl.make_inputs(cfg, "cuda", poison_padding=True)
    got = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    plx.parallax_decode_fwd_static(x["q"], x["r"], x["k"], x["v"], x["seqlens"], got, cfg.scale, 0)
    torch.cuda.synchronize()
    assert_parity(got.cpu().numpy(), oracle_full(oracle, x, cfg.scale, x["seqlens_host"]), torch.float32, "clamped plan")


@pytest.mark.gpu
def test_empty_sequence_among_split_ones(cuda_device):
    """seqlens[b] == 0 with several splits: no CTA writes a record for that sequence, so its row of
    zeros has to come from the merge seeing no record at all (exact zeros, not stale scratch)."""
    from paper_2605_29157_b200 import binding as plx
    cfg = wl.DecodeConfig("na4", B=3, Hq=8, Hkv=4, D=128, T_max=2048, seed=74)
    x = wl.make_inputs(cfg, "cuda")
    lens = torch.tensor([2048, 0, 777], dtype=torch.int32, device="cuda")
    for _ in range(2):     # the second call finds the first call's records in the array
        got = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
        plx.parallax_decode_fwd_static(x["q"], x["r"], x["k"], x["v"], lens, got, cfg.scale, 4)
        torch.cuda.synchronize()
        assert torch.equal(got[1], torch.zeros_like(got[1]))
        assert torch.isfinite(got).all()
