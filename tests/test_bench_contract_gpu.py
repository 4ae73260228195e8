"""The one JSON line `bench.py` prints: keys and plausibility, on the small 0.6B-shaped configuration."""
import json
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
pytestmark = pytest.mark.gpu


def _line(*flags):
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), *flags], capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-3000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_decode_line_has_the_contract_keys(cuda_device):
    d = _line("--workload", "C2", "--steps", "5", "--warmup", "3", "--no-other-configs", "--cpu-seconds", "1")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "gpu_launches", "clocks", "cpu_baseline",
                "sustained", "timing"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 5 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["data"] == "synthetic" and d["scaling"] == "weak" and "workload" in d["config"]
    r = d["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic", "traffic_source", "peak_read_probe", "frac_of_read_probe"):
        assert key in r, key
    assert r["bound"] == "hbm" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    # (timing bounds are loose: this test is about the line's shape, and C2 is a 30 us call on a shared box)
    assert 0.2 < r["frac_of_read_probe"] < 1.15                    # a kernel that only reads cannot beat the read probe
    by_bytes = r["read_probe"]["GBps_by_call_bytes"]               # the probe on calls of C2's and C4's size
    assert 3000 < by_bytes[str(128 << 20)] < 1.05 * by_bytes[str(1 << 30)] <= 1.1 * r["peak_read_probe"]
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == 2 * 8 * 16 * 128 * 2 and e["d2h_bytes_per_step"] == 8 * 16 * 128 * 2
    assert 0 < e["value"] <= d["value"] * 1.15                      # end to end is never faster than the device time
    assert d["gpu_launches"] >= d["steps"] and d["clocks"]["samples"] >= 20
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and "single_thread_C2" in c
    # value = algorithmic bytes / time
    kv_bytes = 8 * 8 * 4096 * 128 * 4
    assert abs(d["value"] - kv_bytes / (d["ms_per_step"] * 1e-3) / 1e12) < 0.02 * d["value"]


def test_default_line_has_every_section(cuda_device):
    """The default invocation's shape (short steps, short CPU sample): the other decode configurations, the tensor-core
    workloads, the multi-token steps and the CPU baseline are all there."""
    d = _line("--workload", "C2", "--steps", "5", "--warmup", "3", "--cpu-seconds", "1")
    assert set(d["other_configs"]) == {"C1", "C3", "C4", "C5", "C6"}
    ow = d["other_workloads"]
    assert {"P2", "T1", "C2_new_tokens_2", "C2_new_tokens_4", "C2_new_tokens_8"} <= set(ow)
    assert ow["C2_new_tokens_8"]["kernel"] == "plx_decode_rows_kernel" and ow["C2_new_tokens_2"]["kernel"] == "plx_decode_kernel"
    assert ow["C2_new_tokens_4"]["kernel"] == "plx_decode_rows_kernel"      # eight rows per KV head at D = 128
    assert d["cpu_baseline"]["kind"] == "oracle" and d["sustained"]["value"] > 0


def test_sharded_line_on_one_rank(cuda_device):
    d = _line("--gpus", "1", "--shard-keys", "--workload", "C2", "--steps", "5")
    assert d["scaling"] == "strong" and d["n_gpus"] == 1 and d["e2e"]["value"] > 0
    assert d["config"]["T_shard"] == 4096 and d["gpu_launches"] >= 10
