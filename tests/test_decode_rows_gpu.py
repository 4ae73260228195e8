"""GPU parity of the keys-on-lanes tensor-core kernel for multi-token decode steps (parallax_decode_fwd_rows:
up to 64 rows per KV head) against the fp64 oracle of the multi-token causal forward."""
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


@pytest.mark.parametrize("G,Lq", [(2, 8), (2, 16), (2, 32), (4, 16), (1, 64), (2, 5), (4, 3), (8, 8), (1, 1), (2, 12), (3, 7)])
@pytest.mark.parametrize("T", [128, 129, 200, 256, 1000])
def test_rows_single_split(plx, oracle, G, Lq, T):
    """One CTA per KV head: full and ragged last tiles, the last Lq - 1 keys straddling a tile boundary."""
    cfg = wl.DecodeConfig("rows", B=2, Hq=2 * G, Hkv=2, D=128, T_max=T, seed=2100 + T + Lq)
    run_rows(plx, oracle, cfg, Lq, ns=1)
