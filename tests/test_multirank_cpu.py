"""World-size-2 check of the bench's multi-rank path on CPU (gloo): ranks draw different
sequences, the reported time is the slowest rank's, and the value is the whole job's."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np
import torch
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, str(ROOT))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    import bench
    from paper_2605_29157_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.scaled(wl.CONFIGS["C1"], seed=bench.rank_seed(0, rank))
    x = wl.make_inputs(cfg, "cpu")
    digest = float(x["k"].float().abs().sum())
    ms_local = 2.0 + 3.0 * rank                       # rank 1 is the slow one
    ms = bench.max_over_ranks(ms_local, world, "cpu")
    value = bench.whole_job_value(10**9, world, ms)
    dist.barrier()
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([digest, ms, value]))
    dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(world))
    assert r0[0] != r1[0]                             # different sequences per rank
    assert r0[1] == r1[1] == 5.0                      # max over ranks
    assert r0[2] == r1[2] == 2 * 10**9 / 5e-3 / 1e12  # both ranks' bytes over the slowest time


def _seq_worker(rank, world, port, out_dir):
    """Sequence-sharded decode, host side: each rank builds the records of its KV slice (with the
    oracle's per-split state standing in for the split kernel), the product's gather routine
    exchanges them over gloo, and the gathered layout merges to the full-context answer."""
    sys.path.insert(0, str(ROOT))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    from oracle import parallax_oracle as po
    from paper_2605_29157_b200 import sequence_parallel as sp
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = np.random.default_rng(5)                      # same inputs on every rank
    B, Hq, Hkv, D, T, ns = 2, 4, 2, 8, 37, 3
    q, r = g.standard_normal((B, Hq, D)), g.standard_normal((B, Hq, D))
    K, V = g.standard_normal((B, Hkv, T, D)), g.standard_normal((B, Hkv, T, D))
    cuts = [0, 20, 37]                                # rank 0 holds keys 0..19, rank 1 keys 20..36
    lo, hi = cuts[rank], cuts[rank + 1]
    chunk = -(-(hi - lo) // ns)
    stride = 2 * D + 4
    rec = np.zeros((B, Hq, ns, stride), dtype=np.float32)
    for b in range(B):
        for h in range(Hq):
            for s in range(ns):
                k0, k1 = min(lo + s * chunk, hi), min(lo + (s + 1) * chunk, hi)
                m, d1, d2, O1, O2 = po.partial_state(q[b, h], r[b, h], K[b, h // 2], V[b, h // 2], 0.4, k0, k1)
                rec[b, h, s, 0], rec[b, h, s, 1], rec[b, h, s, 2] = m, d1, d2
                rec[b, h, s, 4:4 + D], rec[b, h, s, 4 + D:] = O1, O2
    gathered = sp.gather_partials(torch.from_numpy(rec)).numpy().astype(np.float64)
    assert gathered.shape == (world, B, Hq, ns, stride)
    want, _ = po.decode_f64(q, r, K, V, None, 0.4)
    for b in range(B):
        for h in range(Hq):
            states = [(gathered[w, b, h, s, 0], gathered[w, b, h, s, 1], gathered[w, b, h, s, 2],
                       gathered[w, b, h, s, 4:4 + D], gathered[w, b, h, s, 4 + D:]) for w in range(world) for s in range(ns)]
            np.testing.assert_allclose(po.merge_partials(states), want[b, h], rtol=0, atol=1e-5)
    dist.barrier()
    np.save(os.path.join(out_dir, f"s{rank}.npy"), np.array([1.0]))
    dist.destroy_process_group()


def test_sequence_sharded_gather_two_ranks_gloo(tmp_path):
    world = 2
    mp.spawn(_seq_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"s{r}.npy").exists() for r in range(world))


def _run_bench(*flags):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    return subprocess.run([sys.executable, str(ROOT / "bench.py"), *flags], capture_output=True, text=True, timeout=600,
                          env=env)


def test_bench_launcher_starts_the_ranks_itself():
    """`bench.py --gpus 2` outside torchrun has to start two ranks, bring them through the rendezvous and
    the max-over-ranks reduction, and have rank 0 print ONE line with n_gpus = 2.  Rehearsed on CPU ranks
    (gloo, no kernel, value null): the launcher, the per-rank seeding and the aggregation are the same
    code a GPU run takes."""
    for flags in ((), ("--shard-keys",)):
        res = _run_bench("--gpus", "2", "--steps", "3", "--launcher-selftest", *flags)
        assert res.returncode == 0, res.stderr[-2000:]
        lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
        assert len(lines) == 1, res.stdout
        line = json.loads(lines[0])
        assert line["n_gpus"] == 2 and line["gpu_launches"] == 0 and line["value"] is None
        assert line["distinct_rank_inputs"] is True
        assert line["stand_in_ms_max_over_ranks"] == 2.0          # ranks "took" 1 and 2 ms
        assert line["scaling"] == ("strong" if flags else "weak")
        if flags:
            assert line["gathered_layout_ok"] is True


def test_bench_refuses_to_run_fewer_ranks_than_asked():
    """More ranks than visible GPUs: a non-zero exit and no JSON line, never a silent one-rank run."""
    import torch
    n = torch.cuda.device_count() + 1 if torch.cuda.is_available() else 2
    res = _run_bench("--gpus", str(max(n, 2)), "--steps", "3")
    assert res.returncode != 0
    assert not [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert "refusing" in res.stderr


def test_rank_count_mismatch_under_torchrun_is_an_error():
    env_flags = dict(RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    env = {**os.environ, **env_flags}
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--launcher-selftest"], capture_output=True,
                         text=True, timeout=300, env=env)
    assert res.returncode != 0 and "--gpus 2" in res.stderr
