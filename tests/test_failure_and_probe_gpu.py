"""The failure path the kernels have (a bounded device-side wait that gives up) and the read-only
streaming probe, both through the C ABI.

No GPU fault is provoked anywhere here: the wait test polls a barrier on which nothing is in flight
for a bounded number of attempts and returns in the ordinary way.
"""
import numpy as np
import pytest
import torch

from paper_2605_29157_b200 import workloads as wl
from parity_util import assert_parity, oracle_full

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def plx(cuda_device):
    from paper_2605_29157_b200 import binding
    return binding


@pytest.mark.parametrize("attempts", [1, 1024])
def test_bounded_wait_runs_out_and_the_stream_stays_usable(plx, oracle, attempts):
    """A wait that nothing completes ends after its limit, writes PLX_ERR_DEVICE_TIMEOUT to the status
    word and the kernel returns; the next decode call on the same stream is correct and reports no error."""
    stream = torch.cuda.current_stream()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    polls = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    plx.plx_test_bounded_wait(status, attempts, polls, stream)
    cfg = wl.DecodeConfig("after-timeout", B=2, Hq=4, Hkv=2, D=128, T_max=1500, seed=4242)
    x = wl.make_inputs(cfg, "cuda")
    out = torch.full((cfg.B, cfg.Hq, cfg.D), float("nan"), dtype=torch.float32, device="cuda")
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, 8, "cuda")
    plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 3, stream)
    torch.cuda.synchronize()
    assert int(status.item()) == plx.PLX_ERR_DEVICE_TIMEOUT
    assert int(polls.item()) == attempts
    assert "wait" in plx.status_string(int(status.item()))
    assert plx.parallax_workspace_status(ws) == 0          # the decode call's own status word is clean
    assert_parity(out.cpu().numpy(), oracle_full(oracle, x, cfg.scale), torch.float32, "decode after a timed-out wait")


def test_bounded_wait_hook_rejects_long_waits(plx):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(plx.ParallaxError):
        plx.plx_test_bounded_wait(status, 1 << 20)
    with pytest.raises(plx.ParallaxError):
        plx.plx_test_bounded_wait(status, 0)
    torch.cuda.synchronize()
    assert int(status.item()) == 0


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("ctas", [0, 7, 1000])
def test_read_probe_reads_every_byte_once(plx, mode, ctas):
    """The probe is a measurement aid, so what matters is that it reads exactly the bytes it is credited
    with.  Checked through its side channel: the XOR of the 16-byte words it stores per CTA (vector mode)
    equals the XOR of the whole buffer; the bulk mode folds one word per 8 KiB chunk and lane."""
    n = 24 * 8192 + (8192 if ctas == 7 else 0)             # chunks that do not divide evenly among the CTAs
    g = torch.Generator(device="cuda").manual_seed(3)
    buf = torch.randint(-2**31, 2**31 - 1, (n // 4,), dtype=torch.int32, device="cuda", generator=g)
    sink = torch.zeros(plx.PLX_PROBE_SINK_BYTES // 4, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    plx.parallax_read_probe(buf, sink, mode, ctas, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = np.bitwise_xor.reduce(sink.cpu().numpy().view(np.uint32).reshape(-1, 4), axis=0)
    words = buf.cpu().numpy().view(np.uint32)
    if mode == plx.PLX_PROBE_VECTOR_LOADS:
        want = np.bitwise_xor.reduce(words.reshape(-1, 4), axis=0)
        assert (got == want).all()
    else:
        # lane l of the warp that owns a chunk folds word l of that chunk; the warp stores the lane-0 value
        want0 = np.bitwise_xor.reduce(words.reshape(-1, 2048)[:, 0])
        assert got[0] == want0 and (got[1:] == 0).all()


def test_read_probe_argument_checks(plx):
    buf = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    sink = torch.zeros(plx.PLX_PROBE_SINK_BYTES, dtype=torch.uint8, device="cuda")
    with pytest.raises(plx.ParallaxError):
        plx.parallax_read_probe(buf, sink, 0, 0, None, None, nbytes=100)        # not a multiple of 8192
    with pytest.raises(plx.ParallaxError):
        plx.parallax_read_probe(buf, sink, 5)                                    # unknown mode
    with pytest.raises(plx.ParallaxError):
        plx.parallax_read_probe(buf, sink[:100])                                 # sink too small
