#!/usr/bin/env python
"""Benchmark of the Parallax decode forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl ours|reference]
                    [--shard-keys]

One step = one full decode call (one fused launch: split kernel whose last CTA per stream merges) over one batch of the
named synthetic workload.  Prints ONE JSON line (rank 0).  The headline value is
achieved KV-read bandwidth (algorithmic K+V bytes / device time, summed over
GPUs); ms_per_step carries the latency (us/call = 1000 * ms_per_step).

Several GPUs: `--gpus N` without a torchrun environment starts N ranks itself (one process per GPU,
NCCL); under torchrun (WORLD_SIZE set) the process is one of the ranks.  Two partitions of the path:
  default       every rank runs the same per-GPU workload on its own seeded sequences (weak scaling:
                sequences are independent, there is no data-path collective);
  --shard-keys  ONE batch whose keys are divided among the ranks (strong scaling): every rank turns
                its slice of each context into partial states, the records are all-gathered, every
                rank merges them.
The time is the slowest rank's; a block of exactly K steps is timed between barriers and repeated
until at least 200 ms of device time have been measured (median block reported, spread beside it).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2605_29157_b200 import workloads as wl  # noqa: E402

METRIC = "parallax_decode_kv_read_bandwidth"
KV_LAYOUT = ["contiguous [B,Hkv,T,D]"]
UNIT = "TB/s"
L2_BYTES = 126 * 1024 * 1024
MIN_TIMED_MS = 200.0     # device time every reported number rests on, whatever --steps is
MAX_BLOCKS = 4000

# DRAM traffic of the dominant kernel per launch (dram__bytes_read.sum + dram__bytes_write.sum of one
# ncu capture).  NOT measured in this run: each entry says which kernel instantiation and which capture
# size it comes from and how it was scaled to a full launch (sequences are independent, so traffic grows
# in proportion to the batch).  An entry goes stale when its kernel changes; the bench line carries the
# provenance string beside the number.
NCU_TRAFFIC = {
    "C2": (134_500_000, "plx_decode_kernel<128,2,3,2,0>, full-size capture (cache sets rotated, so reads miss L2)"),
    "C3": (2_157_500_000, "plx_decode_kernel<128,2,3,2,0>, capture at B=32 scaled x2"),
    "C4": (1_077_300_000, "plx_decode_kernel<128,2,3,2,0>, full-size capture (before the prologue was split around the "
                          "dependency wait; byte counts unaffected)"),
    "C5": (7_661_000_000, "plx_decode_kernel<128,2,3,2,0>, capture at B=16 (887.0 MB for 883.04 MB of K/V) scaled by the key count"),
    "C6": (2 * 541_600_000, "plx_decode_kernel<64,2,2,4,0>, capture at B=32 scaled x2 (before the prologue change)"),
    "P1": (8 * 51_000_000, "plx_prefill_kernel<true,128>, capture at B=1 scaled x8"),
    "T1": (4 * 513_000_000, "plx_bwd_prep/row/col kernels, capture at B=2 scaled x4"),
}
NCU_TRAFFIC_FP8 = {"C3": (2 * 540_800_000, "plx_decode_kernel<128,2,2,4,fp8>, capture at B=32 scaled x2")}


def ncu_traffic(name, fp8=False):
    """(bytes per launch or None, provenance or None) for a workload's dominant kernel."""
    entry = (NCU_TRAFFIC_FP8 if fp8 else NCU_TRAFFIC).get(name)
    return (entry[0], "ncu capture, not measured in this run: " + entry[1]) if entry else (None, None)


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ----------------------------------------------------------------------------------------------
# clocks sampled during the timed regions (read-only NVML queries)
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    """SM clock and clock-event reasons polled every 5 ms through NVML (read-only queries) while `active`
    is set.  `mark()` / `summary(since)` give the statistics of one timed region."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int):
        self.samples, self.bits = [], []
        self.active = threading.Event()
        self.stop = threading.Event()
        self.handle, self.max_mhz = None, None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        while not self.stop.is_set():
            if self.handle is not None and self.active.is_set():
                try:
                    mhz = int(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM))
                    try:
                        bits = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                    except Exception:
                        bits = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                    self.samples.append(mhz)
                    self.bits.append(bits)
                except Exception:
                    pass
            time.sleep(0.005)

    def mark(self) -> int:
        return len(self.samples)

    def summary(self, since: int = 0):
        samples, bits = self.samples[since:], self.bits[since:]
        if not samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        seen = 0
        for x in bits:
            seen |= x
        reasons = [name for bit, name in self.REASONS.items() if seen & bit]
        return {"sm_mhz": float(np.median(samples)), "sm_min_mhz": float(min(samples)), "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(samples)}

    def close(self):
        self.stop.set()
        self.thread.join(timeout=1.0)


# ----------------------------------------------------------------------------------------------
# timed regions
# ----------------------------------------------------------------------------------------------
class BlockTimer:
    """Times blocks of exactly `steps` calls with CUDA events on the launching stream, each block between a
    barrier + device synchronisation on both sides, the slowest rank's time taken per block; blocks are
    repeated until `min_ms` of device time have been measured (the same count on every rank: the
    decision uses the reduced times).  Reports the median block."""

    def __init__(self, stream, sampler, world=1, device="cuda"):
        self.stream, self.sampler, self.world, self.device = stream, sampler, world, device

    def barrier(self):
        if self.world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def block(self, fn, steps, offset=0):
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for i in range(steps):
            fn(offset + i)
        e1.record(self.stream)
        self.barrier()
        return max_over_ranks(e0.elapsed_time(e1), self.world, self.device)

    def sustained(self, fn, steps, load_ms=1200.0, timed_ms=400.0):
        """The same blocks after `load_ms` of uninterrupted running of this very call: an HBM-saturating kernel
        brings a B200 to its 1000 W cap within a few hundred milliseconds and the SM clock then settles near
        1.5-1.7 GHz (`sw_power_cap`), which a single-wave call (one CTA per SM) feels and a multi-wave one barely
        does.  -> dict like run()."""
        total, k = 0.0, 0
        while total < load_ms and k < MAX_BLOCKS:
            total += self.block(fn, steps, offset=k * steps)
            k += 1
        return self.run(fn, steps, min_ms=timed_ms)

    def run(self, fn, steps, min_ms=MIN_TIMED_MS):
        """-> dict: ms_per_step (median block / steps), blocks, ms_total, spread (min, max of the blocks'
        ms per step) and the clock summary of the region."""
        since = self.sampler.mark() if self.sampler else 0
        if self.sampler:
            self.sampler.active.set()
        times, total = [], 0.0
        while (total < min_ms and len(times) < MAX_BLOCKS) or not times:
            t = self.block(fn, steps, offset=len(times) * steps)
            times.append(t)
            total += t
        if self.sampler:
            self.sampler.active.clear()
        per = np.array(times) / steps
        return {"ms_per_step": float(np.median(per)), "blocks": len(times), "ms_total": float(total),
                "ms_per_step_min": float(per.min()), "ms_per_step_max": float(per.max()),
                "clocks": self.sampler.summary(since) if self.sampler else None}


def cool_down(seconds=1.0):
    """Idle pause between two measurements that are each meant as a burst figure: a B200 that has streamed from
    HBM for a few hundred milliseconds sits at its power cap with a lowered SM clock; a second of idling lets it
    leave that state, so that the kernel-only timing and the read-only probe start from the same footing as the
    headline."""
    torch.cuda.synchronize()
    time.sleep(seconds)


def timing_note(t):
    return {"timed_blocks": t["blocks"], "device_ms_timed": round(t["ms_total"], 2),
            "us_per_step_min": round(t["ms_per_step_min"] * 1e3, 2), "us_per_step_max": round(t["ms_per_step_max"] * 1e3, 2)}


def free_port() -> int:
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


# ----------------------------------------------------------------------------------------------
# CPU oracle leg (the only place outside tests/smoke that runs oracle/)
# ----------------------------------------------------------------------------------------------
def oracle_sample_time(cfg, x, seqlens_host, target_seconds=12.0, max_streams=None, wall_seconds=None, start=0):
    """Times the fp64 oracle, as it stands, on whole (b, kv-head) streams of the workload until
    about `target_seconds` of CPU work have been done (and, if given, at most `wall_seconds` of wall
    time including the marshalling of its inputs; at least one stream is always timed).  `start` rotates
    the stream order so that consecutive small samples cover different streams.  Returns (seconds,
    algorithmic KV bytes covered, threads, description)."""
    from oracle import parallax_oracle as po
    po.build()
    G = cfg.G
    streams = [(b, h) for b in range(cfg.B) for h in range(cfg.Hkv)]
    g = np.random.default_rng(0)
    g.shuffle(streams)
    streams = streams[start % len(streams):] + streams[:start % len(streams)]
    wall0 = time.perf_counter()
    if max_streams:
        streams = streams[:max_streams]
    done_bytes, elapsed, n, threads = 0, 0.0, 0, 1
    batch = 1
    i = 0
    # go through the streams (again from the start if the workload is small) until the target has been spent
    while elapsed < target_seconds:
        if wall_seconds is not None and n > 0 and time.perf_counter() - wall0 >= wall_seconds:
            break
        if i >= len(streams):
            i = 0
        group = streams[i:i + batch]
        i += len(group)
        # one oracle call over `len(group)` independent single-stream problems (B = group size)
        Ls = [cfg.T_max if seqlens_host is None else int(seqlens_host[b]) for (b, _) in group]
        Tm = max(max(Ls), 1)
        q = np.stack([wl.bf16_bits(x["q"][b, h * G:(h + 1) * G]) for (b, h) in group])
        r = np.stack([wl.bf16_bits(x["r"][b, h * G:(h + 1) * G]) for (b, h) in group])
        k = np.stack([wl.bf16_bits(x["k"][b, h:h + 1, :Tm]) for (b, h) in group])
        v = np.stack([wl.bf16_bits(x["v"][b, h:h + 1, :Tm]) for (b, h) in group])
        sl = np.array(Ls, dtype=np.int32)
        t0 = time.perf_counter()
        _, threads = po.decode_bf16(q, r, k, v, sl, cfg.scale)
        dt = time.perf_counter() - t0
        elapsed += dt
        n += len(group)
        done_bytes += sum(Ls) * cfg.D * 2 * 2
        if dt < 1.0:
            batch = min(batch * 2, 64)
    desc = (f"{n} (sequence, kv-head) streams of {cfg.name} ({cfg.B * cfg.Hkv} distinct, revisited when the "
            f"workload is shorter than the time budget), {G} query heads each")
    return elapsed, done_bytes, threads, desc


# ----------------------------------------------------------------------------------------------
# multi-rank aggregation (weak scaling: every rank runs its own batch; no data-path collective)
# ----------------------------------------------------------------------------------------------
def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own sequences."""
    return base_seed + 1000 * rank


def max_over_ranks(ms: float, world: int, device="cpu") -> float:
    """Slowest rank's device time (all ranks get the same number back)."""
    if world <= 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(bytes_per_rank: int, world: int, ms_per_step: float) -> float:
    """TB/s over all ranks: every rank moved bytes_per_rank in the slowest rank's time."""
    return bytes_per_rank * world / (ms_per_step * 1e-3) / 1e12


PROBE_CALL_BYTES = (128 << 20, 1 << 30)   # the K/V bytes of one C2 call and of one C4 / C6 call


def read_probe(dev, stream, sampler):
    """Read-only streaming bandwidth of this GPU, measured in this run with the library's own probe kernel:
    2 GiB buffers, two of them read alternately (4 GiB between two reads of a byte vs 0.123 GiB of L2), each
    variant timed for >= 100 ms.  Returns the per-variant GB/s and the best of them: the ceiling of a kernel
    that only reads."""
    from paper_2605_29157_b200 import binding as plx
    nbytes = 2 << 30
    bufs = [torch.empty(nbytes // 4, dtype=torch.int32, device=dev).random_() for _ in range(2)]
    sink = torch.empty(plx.PLX_PROBE_SINK_BYTES, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    timer = BlockTimer(stream, sampler)
    variants = {
        "vector_loads_8_ctas_per_sm": (plx.PLX_PROBE_VECTOR_LOADS, 0),
        "vector_loads_64KiB_per_cta": (plx.PLX_PROBE_VECTOR_LOADS, nbytes // 65536),
        "bulk_copies_2_ctas_per_sm": (plx.PLX_PROBE_BULK_COPIES, 0),
        "bulk_copies_1MiB_per_cta": (plx.PLX_PROBE_BULK_COPIES, nbytes >> 20),
    }
    out = {}
    for name, (mode, ctas) in variants.items():
        def call(i, mode=mode, ctas=ctas):
            plx.parallax_read_probe(bufs[i % 2], sink, mode, ctas, status, stream)
        cool_down(0.5)       # every variant from the same footing (see cool_down)
        for i in range(3):
            call(i)
        t = timer.run(call, 10, min_ms=100.0)
        out[name] = round(nbytes / (t["ms_per_step"] * 1e-3) / 1e9, 1)
    # The same probe on calls of the size of the smaller decode configurations: a launch that reads 128 MiB
    # spends a visible part of its time filling and draining the device, so its ceiling is lower than the
    # 2 GiB figure.  Each call reads the next `size` bytes of the two buffers (4 GiB between two reads of a byte).
    by_bytes = {}
    for size in PROBE_CALL_BYTES:
        per_buf = nbytes // size
        best_small = 0.0
        for mode, ctas in ((plx.PLX_PROBE_VECTOR_LOADS, 0), (plx.PLX_PROBE_VECTOR_LOADS, size // 65536),
                           (plx.PLX_PROBE_BULK_COPIES, 0)):
            def call(i, mode=mode, ctas=ctas):
                j = i % (2 * per_buf)
                src = bufs[j // per_buf][(j % per_buf) * (size // 4):(j % per_buf + 1) * (size // 4)]
                plx.parallax_read_probe(src, sink, mode, ctas, status, stream)
            cool_down(0.3)
            for i in range(3):
                call(i)
            t = timer.run(call, 2 * per_buf, min_ms=60.0)
            best_small = max(best_small, size / (t["ms_per_step"] * 1e-3) / 1e9)
        by_bytes[str(size)] = round(best_small, 1)
    assert int(status.item()) == 0, "read probe: a bounded wait ran out"
    best = max(out, key=out.get)
    return {"GBps": out, "best": best, "peak": out[best], "bytes_per_launch": nbytes,
            "l2_policy": "two 2 GiB buffers read alternately",
            "GBps_by_call_bytes": by_bytes}


def describe(cfg, seqlens_host, nsets, chunk, ns):
    return {
        "workload": f"{cfg.name}: {cfg.note}; B={cfg.B} Hq={cfg.Hq} Hkv={cfg.Hkv} D={cfg.D} context="
                    + (f"{cfg.T_max} uniform" if seqlens_host is None else
                       f"ragged U[{cfg.ragged[0]},{cfg.ragged[1]}] (sum {int(seqlens_host.sum())}) over T_max={cfg.T_max}")
                    + "; q,r,K,V bf16 N(0,1), contiguous [B,Hkv,T,D] cache, bf16 output, scale 1/sqrt(D)",
        "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D, "T_max": cfg.T_max,
        "chunk_len": chunk, "num_splits": ns, "kv_layout": KV_LAYOUT[0],
        "l2_policy": f"{nsets} KV cache set(s) used round-robin, "
                     f"{nsets * cfg.B * cfg.Hkv * cfg.T_max * cfg.D * 4 / 2**30:.3f} GiB touched between two uses "
                     f"of the same set vs 0.123 GiB L2"
                     + ("" if nsets * cfg.B * cfg.Hkv * cfg.T_max * cfg.D * 4 > 2 * L2_BYTES else
                        " (this workload is smaller than L2: launch-bound, not an HBM measurement)"),
        "parallelism": "independent sequences per GPU, no collective",
    }


def run_ours(args, rank, world, local_rank):
    from paper_2605_29157_b200 import binding as plx

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    cfg = wl.CONFIGS[args.workload]
    cfg = wl.scaled(cfg, seed=rank_seed(cfg.seed, rank))
    if args.batch:
        cfg = wl.scaled(cfg, B=args.batch, name=f"{cfg.name}(B={args.batch})", note=cfg.note + ", reduced batch")
    kv_set_bytes = cfg.B * cfg.Hkv * cfg.T_max * cfg.D * 4
    nsets = args.kv_sets or min(16, max(2 if kv_set_bytes < (8 << 30) else 1, -(-(1 << 30) // kv_set_bytes)))
    sets = []
    for i in range(nsets):
        x = wl.make_inputs(wl.scaled(cfg, seed=cfg.seed + 17 * i), dev)
        sets.append(x)
    if args.page_size:
        KV_LAYOUT[0] = f"paged, page_size {args.page_size}, random page order"
        for i, x in enumerate(sets):          # scatter each cache into page pools (random page order)
            x["kp"], x["vp"], x["table"] = wl.to_paged(x["k"], x["v"], args.page_size, seed=i)
            x["k"] = x["v"] = None
    if args.fp8_kv:
        KV_LAYOUT[0] = "contiguous [B,Hkv,T,D] e4m3 (per-tensor scales); bytes counted at 1 byte per element"
        for x in sets:
            x["k8"], x["ks"] = wl.quantize_e4m3(x["k"])
            x["v8"], x["vs"] = wl.quantize_e4m3(x["v"])
            x["k"] = x["v"] = None
    Lq = args.new_tokens
    if Lq > 1:        # several new tokens per sequence and step: q, r [B, Hq, Lq, D] on the decode kernel
        KV_LAYOUT[0] += f"; {Lq} new tokens per sequence and step (parallax_decode_fwd_multi)"
        for i, x in enumerate(sets):
            g = torch.Generator(device=dev).manual_seed(cfg.seed + 1000 + i)
            for n in ("q", "r"):
                x[n] = torch.randn(cfg.B, cfg.Hq, Lq, cfg.D, generator=g, device=dev).to(torch.bfloat16)
    x0 = sets[0]
    seqlens_host = x0["seqlens_host"]
    for x in sets[1:]:                      # one set of lengths for all cache sets
        x["seqlens"], x["seqlens_host"] = x0["seqlens"], seqlens_host
    kv_bytes = cfg.kv_bytes(seqlens_host) // (2 if args.fp8_kv else 1)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    chunk, ns = plx.parallax_decode_plan(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T_max, sms, seqlens_host is not None)
    if args.splits:
        ns = args.splits
        chunk = -(-(-(-cfg.T_max // ns)) // 64) * 64
        ns = -(-cfg.T_max // chunk)
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, plx.PLX_MAX_SPLITS, dev)
    out = torch.empty((cfg.B, cfg.Hq, Lq, cfg.D) if Lq > 1 else (cfg.B, cfg.Hq, cfg.D), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()

    def step(i, st=None):
        x, st = sets[i % nsets], st or stream
        if Lq > 1 and args.fp8_kv:      # several tokens over an e4m3 cache: the options-struct entry (decode kernel)
            plx.parallax_decode_fwd_args(x["q"], x["r"], x["k8"], x["v8"], x["seqlens"], out, cfg.scale, k_scale=x["ks"],
                                         v_scale=x["vs"], workspace=ws, num_splits=args.splits, stream=st)
        elif Lq > 1 and args.page_size:
            plx.parallax_decode_fwd_multi_paged(x["q"], x["r"], x["kp"], x["vp"], x["table"], x["seqlens"], out, cfg.scale,
                                                ws, args.splits, st)
        elif Lq > 1:
            plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, args.splits, st)
        elif args.page_size:
            plx.parallax_decode_fwd_paged(x["q"], x["r"], x["kp"], x["vp"], x["table"], x["seqlens"], out, cfg.scale,
                                          ws, args.splits, st)
        elif args.fp8_kv:
            plx.parallax_decode_fwd_fp8(x["q"], x["r"], x["k8"], x["v8"], x["seqlens"], out, cfg.scale, x["ks"], x["vs"],
                                        ws, args.splits, st)
        else:
            plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, args.splits, st)

    sampler = ClockSampler(local_rank)
    timer = BlockTimer(stream, sampler, world, dev)
    for i in range(args.warmup):
        step(i)
    t_call = timer.run(step, args.steps)
    ms_per_step = t_call["ms_per_step"]
    # one launch per call, except steps the library hands to a tensor-core kernel and splits (kernel + merge)
    route = "decode" if args.fp8_kv else multi_token_route(cfg, Lq, args.page_size)
    launches_per_step = (rows_kernel_launches(cfg, Lq, sms, args.page_size) if route == "rows" else
                         tensor_core_launches(cfg, Lq, sms) if route == "row-major" and not args.page_size else 1)
    value = whole_job_value(kv_bytes, world, ms_per_step)
    assert plx.parallax_workspace_status(ws) == 0, "device-side wait timed out"
    us_graph = graph_replay_us(step, nsets)

    # dominant kernel alone (the split kernel, same chunking; the combine is excluded)
    stride = plx.parallax_partial_stride(cfg.D)
    partials = torch.empty(cfg.B * cfg.Hq * ns * stride, dtype=torch.float32, device=dev)

    def main_only(i):
        x = sets[i % nsets]
        if args.page_size or args.fp8_kv or Lq > 1:
            step(i)      # paged / fp8 cache / several tokens: the fused call is the one kernel
        elif ns == 1:
            plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, 1, stream)
        else:
            plx.parallax_decode_splitkv_partial(x["q"], x["r"], x["k"], x["v"], x["seqlens"], partials, cfg.scale,
                                                chunk, ns, None, stream)
    cool_down()
    for i in range(max(3, args.warmup)):
        main_only(i)
    t_kernel = timer.run(main_only, args.steps)
    ms_kernel = t_kernel["ms_per_step"]
    peak, peak_src = measured_peaks()
    achieved = kv_bytes / (ms_kernel * 1e-3) / 1e9
    traffic, traffic_src = ((None, None) if (args.page_size or Lq > 1 or args.batch or args.splits) else
                            ncu_traffic(cfg.name, args.fp8_kv))
    roofline = {"bound": "hbm", "kernel": {"decode": "plx_decode_kernel", "rows": "plx_decode_rows_kernel",
                                           "row-major": "plx_prefill_kernel"}[route],
                "achieved": round(achieved, 1), "peak": peak,
                "peak_source": f"{peak_src} copy bandwidth (read + write)", "unit": "GB/s", "frac": round(achieved / peak, 4),
                "frac_of_8TBps_nominal": round(achieved / 8000.0, 4),
                "us_per_launch": round(ms_kernel * 1e3, 2),
                "algorithmic_bytes_per_launch": kv_bytes,
                "traffic": traffic, "traffic_source": traffic_src, **timing_note(t_kernel)}
    if rank == 0 and not args.no_read_probe:
        cool_down()
        probe = read_probe(dev, stream, sampler)
        roofline["peak_read_probe"] = probe["peak"]
        roofline["frac_of_read_probe"] = round(achieved / probe["peak"], 4)
        roofline["read_probe"] = probe

    # end to end through the host-buffer entry point: q, r from pinned host memory, out to host
    qh = [x["q"].cpu().pin_memory() for x in sets]
    rh = [x["r"].cpu().pin_memory() for x in sets]
    oh = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()

    def e2e_step(i):
        x = sets[i % nsets]
        if args.page_size or args.fp8_kv or Lq > 1:     # no host-buffer entry point for these: stage by hand
            x["q"].copy_(qh[i % nsets], non_blocking=True)
            x["r"].copy_(rh[i % nsets], non_blocking=True)
            step(i)
            oh.copy_(out, non_blocking=True)
            stream.synchronize()
            return
        plx.parallax_decode_fwd_host(qh[i % nsets], rh[i % nsets], x["k"], x["v"], x["seqlens"], oh, cfg.scale, ws,
                                     args.splits, stream)
    e2e_steps = max(10, args.steps // 4)
    for i in range(3):
        e2e_step(i)
    t_e2e = timer.run(e2e_step, e2e_steps)
    ms_e2e = t_e2e["ms_per_step"]
    n_qr = cfg.B * cfg.Hq * Lq * cfg.D * 2
    e2e = {"value": round(whole_job_value(kv_bytes, world, ms_e2e), 4), "unit": UNIT,
           "us_per_call": round(ms_e2e * 1e3, 2), "h2d_bytes_per_step": 2 * n_qr, "d2h_bytes_per_step": n_qr,
           "note": ("q and r copied from pinned host memory and the output copied back every step (copy commands "
                    "around the device call: this variant has no host-buffer entry point); "
                    if (args.page_size or args.fp8_kv or Lq > 1) else
                    "q and r read from pinned host memory and the output written to pinned host memory every step "
                    "(both by the attention kernel itself, over the host link: one launch, no copy command); ") +
                   "the KV cache is device-resident state of a decode step", **timing_note(t_e2e)}
    clocks = t_call["clocks"]
    # last, so that it heats nothing that is measured as a burst
    t_sus = timer.sustained(step, args.steps) if not args.no_sustained else None

    result = {
        "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 6), "us_per_call": round(ms_per_step * 1e3, 2),
        "us_per_call_graph_replay": round(us_graph, 2),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp16 products on an e4m3 cache" if args.fp8_kv else "bf16",
        "data": "synthetic", "config": describe(cfg, seqlens_host, nsets, chunk, ns),
        "roofline": roofline, "e2e": e2e, "gpu_launches": launches_per_step * args.steps * t_call["blocks"],
        "clocks": clocks, "timing": {"protocol": f"blocks of exactly {args.steps} steps between barriers, repeated until "
                                                 f">= {MIN_TIMED_MS:.0f} ms of device time; median block reported",
                                     **timing_note(t_call)},
    }
    if t_sus is not None:
        result["sustained"] = {"us_per_call": round(t_sus["ms_per_step"] * 1e3, 2),
                               "value": round(whole_job_value(kv_bytes, world, t_sus["ms_per_step"]), 4), "unit": UNIT,
                               "protocol": "the same call timed for 400 ms after 1.2 s of uninterrupted running of it "
                                           "(the board at its power cap; the headline above is the first 200 ms)",
                               "clocks": t_sus["clocks"], **timing_note(t_sus)}
    if args.fp8_kv:   # the e4m3 variant plans its own splits inside the library
        result["config"]["chunk_len"] = result["config"]["num_splits"] = "planned inside the library for the e4m3 variant"
    if Lq > 1:
        result["config"]["new_tokens_per_step"] = Lq
        result["config"]["chunk_len"] = result["config"]["num_splits"] = "planned inside the library for Hq * new tokens rows"
        result["tokens_per_s"] = round(world * cfg.B * Lq / (ms_per_step * 1e-3), 1)
    if rank == 0 and world == 1 and args.all_configs and not args.fp8_kv and Lq == 1:
        del sets
        torch.cuda.empty_cache()
        read_peak = roofline.get("peak_read_probe")
        by_bytes = roofline.get("read_probe", {}).get("GBps_by_call_bytes")
        result["other_configs"] = {n: quick_config(n, sampler, read_peak, by_bytes) for n in sorted(wl.CONFIGS) if n != args.workload}
        result["other_workloads"] = {n: quick_tensor_workload(n, local_rank) for n in ("P2", "T1")}
        for new_tokens in (2, 4, 8):   # multi-token decode steps on the headline shape: 4, 8 and 16 rows per KV head
            result["other_workloads"][f"{args.workload}_new_tokens_{new_tokens}"] = quick_multi_token(args.workload, new_tokens,
                                                                                                   sampler, read_peak)
            torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.fp8_kv and Lq == 1:
        secs, nbytes, threads, desc = oracle_sample_time(cfg, x0, seqlens_host, args.cpu_seconds)
        result["cpu_baseline"] = {"value": round(nbytes / secs / 1e12, 8), "unit": UNIT, "cores": threads,
                                  "kind": "oracle", "sample": desc, "seconds": round(secs, 2),
                                  "single_thread_C2": single_thread_oracle_c2()}
    sampler.close()
    return result


def multi_token_route(cfg, Lq, page_size=0):
    """The kernel the library runs for a multi-token step of this shape (asked of the library itself, only to name
    the kernel and count launches): "decode", "rows" (keys-on-lanes tensor-core kernel) or "row-major"."""
    from paper_2605_29157_b200 import binding as plx
    kernel, _ = plx.parallax_decode_multi_plan(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lq, cfg.T_max, page_size)
    return {plx.PLX_MULTI_KERNEL_DECODE: "decode", plx.PLX_MULTI_KERNEL_ROWS: "rows",
            plx.PLX_MULTI_KERNEL_ROW_MAJOR: "row-major"}[kernel]


def routed_to_tensor_core(cfg, Lq):
    return multi_token_route(cfg, Lq) != "decode"


def rows_kernel_launches(cfg, Lq, sms, page_size=0):
    """Launches per call of the keys-on-lanes kernel: 2 when the library splits the keys (kernel + merge), else 1."""
    from paper_2605_29157_b200 import binding as plx
    _, ns = plx.parallax_decode_multi_plan(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, Lq, cfg.T_max, page_size)
    return 2 if ns > 1 else 1


def tensor_core_launches(cfg, Lq, sms):
    """Launches per call of the multi-token tensor-core kernel: 2 when the library splits the keys (kernel +
    merge), else 1.  Mirrors the library's rule only to count launches."""
    pack = cfg.G if (cfg.G > 1 and cfg.G * Lq <= 128) else 1
    base_ctas = (1 if pack > 1 else -(-Lq // 128)) * cfg.B * (cfg.Hkv if pack > 1 else cfg.Hq)
    planned = min(sms // base_ctas, max(1, -(-cfg.T_max // 64) // 8), 64) if base_ctas < sms else 1
    return 2 if planned > 1 else 1


def graph_replay_us(step, nsets, reps=5):
    """Device time per call when 2 * nsets calls are replayed from one CUDA graph (the second of the paper's
    two timers: no per-call launch cost on the host)."""
    per_graph = 2 * nsets
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(per_graph):
                step(i, side)
        graph.replay()
        side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        for _ in range(reps):
            graph.replay()
        e1.record(side)
        side.synchronize()
    return e0.elapsed_time(e1) / (reps * per_graph) * 1e3


def quick_config(name, sampler, read_peak=None, read_by_bytes=None, steps=20, warmup=5):
    """Device-timed run of one decode configuration (library plan, L2-cold by rotating cache sets, blocks of
    `steps` calls repeated until >= 200 ms of device time): us per call, KV-read TB/s, its fractions of the
    measured copy bandwidth, of this run's read-only probe and of 8 TB/s, and the clocks of its own region."""
    from paper_2605_29157_b200 import binding as plx
    cfg = wl.CONFIGS[name]
    kv_set_bytes = cfg.B * cfg.Hkv * cfg.T_max * cfg.D * 4
    nsets = min(16, max(2 if kv_set_bytes < (8 << 30) else 1, -(-(1 << 30) // kv_set_bytes)))
    sets = [wl.make_inputs(wl.scaled(cfg, seed=cfg.seed + 17 * i), "cuda") for i in range(nsets)]
    for x in sets[1:]:
        x["seqlens"], x["seqlens_host"] = sets[0]["seqlens"], sets[0]["seqlens_host"]
    kv_bytes = cfg.kv_bytes(sets[0]["seqlens_host"])
    ws = plx.alloc_workspace(cfg.B, cfg.Hq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.float32 if cfg.out_dtype == "f32" else torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i, st=None):
        x = sets[i % nsets]
        plx.parallax_decode_fwd_ex(x["q"], x["r"], x["k"], x["v"], x["seqlens"], out, cfg.scale, ws, 0, st or stream)
    for i in range(warmup):
        step(i)
    t = BlockTimer(stream, sampler).run(step, steps)
    us = t["ms_per_step"] * 1e3
    peak, _ = measured_peaks()
    traffic, traffic_src = ncu_traffic(name)
    res = {"us_per_call": round(us, 2), "us_per_call_graph_replay": round(graph_replay_us(step, nsets), 2),
           "kv_read_TBps": round(kv_bytes / us / 1e6, 4),
           "frac_of_measured_copy_bw": round(kv_bytes / us / 1e3 / peak, 4),
           "frac_of_8TBps_nominal": round(kv_bytes / us / 1e3 / 8000.0, 4), "kv_bytes": kv_bytes,
           "traffic": traffic, "traffic_source": traffic_src, "clocks": t["clocks"], **timing_note(t)}
    if read_peak:
        res["frac_of_read_probe"] = round(kv_bytes / us / 1e3 / read_peak, 4)
    if read_by_bytes and str(kv_bytes) in read_by_bytes:   # the probe reading exactly this call's bytes per launch
        res["read_probe_same_bytes_GBps"] = read_by_bytes[str(kv_bytes)]
        res["frac_of_read_probe_same_bytes"] = round(kv_bytes / us / 1e3 / read_by_bytes[str(kv_bytes)], 4)
    return res


def quick_tensor_workload(name, local_rank=0):
    """Short run of a tensor-core workload (multi-token forward or backward) for the default line: value,
    roofline fraction against the sustained bf16 peak, clocks."""
    def one(mode):
        ns = argparse.Namespace(workload=name, steps=5, warmup=3, batch=0, kv_sets=0, plain_bf16_p=False, p_precision=mode,
                                no_cpu_baseline=True, cpu_seconds=0.0)
        runner = run_prefill if name in wl.PREFILL_CONFIGS else run_backward
        r = runner(ns, 0, 1, local_rank)
        torch.cuda.empty_cache()
        return {"metric": r["metric"], "value": r["value"], "unit": r["unit"], "ms_per_step": r["ms_per_step"],
                "roofline_frac_of_sustained_bf16": r["roofline"]["frac"], "roofline_kernel": r["roofline"]["kernel"],
                "workload": r["config"]["workload"], "clocks": r["clocks"], **r["timing"]}
    res = one("residual")
    if name in wl.PREFILL_CONFIGS:   # the same workload with residual products only where rows see few keys
        res["p_precision"] = "bf16+residual"
        res["adaptive_p_precision"] = one("adaptive")
    return res


def quick_multi_token(name, Lq, sampler, read_peak=None, steps=20, warmup=5):
    """Device-timed multi-token decode step (Lq new tokens per sequence through parallax_decode_fwd_multi, which
    picks the kernel) on a decode configuration, for the default line: us per step, KV-read TB/s, tokens/s, kernel."""
    from paper_2605_29157_b200 import binding as plx
    cfg = wl.CONFIGS[name]
    sets = [wl.make_prefill_inputs(wl.scaled(cfg, seed=cfg.seed + 17 * i), Lq, "cuda") for i in range(2)]
    kv_bytes = cfg.kv_bytes(None)
    ws = plx.alloc_workspace(cfg.B, cfg.Hq * Lq, cfg.D, plx.PLX_MAX_SPLITS, "cuda")
    out = torch.empty(cfg.B, cfg.Hq, Lq, cfg.D, dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        x = sets[i % 2]
        plx.parallax_decode_fwd_multi(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0, stream)
    for i in range(warmup):
        step(i)
    t = BlockTimer(stream, sampler).run(step, steps)
    assert plx.parallax_workspace_status(ws) == 0, "device-side wait timed out"
    us = t["ms_per_step"] * 1e3
    route = multi_token_route(cfg, Lq)
    res = {"new_tokens_per_step": Lq, "rows_per_kv_head": cfg.G * Lq, "us_per_step": round(us, 2),
           "kv_read_TBps": round(kv_bytes / us / 1e6, 4), "tokens_per_s": round(cfg.B * Lq / (us * 1e-6), 1),
           "kernel": {"decode": "plx_decode_kernel", "rows": "plx_decode_rows_kernel", "row-major": "plx_prefill_kernel"}[route],
           "clocks": t["clocks"], **timing_note(t)}
    if read_peak:
        res["frac_of_read_probe"] = round(kv_bytes / us / 1e3 / read_peak, 4)
    return res


def single_thread_oracle_c2():
    """The fp64 oracle on the whole C2 call with ONE thread (seconds per call)."""
    from oracle import parallax_oracle as po
    po.build()
    cfg = wl.CONFIGS["C2"]
    x = wl.make_inputs(cfg, "cuda" if torch.cuda.is_available() else "cpu")
    bits = {n: wl.bf16_bits(x[n]) for n in ("q", "r", "k", "v")}
    t0 = time.perf_counter()
    _, threads = po.decode_bf16(bits["q"], bits["r"], bits["k"], bits["v"], None, cfg.scale, threads=1)
    secs = time.perf_counter() - t0
    return {"seconds_per_call": round(secs, 4), "value": round(cfg.kv_bytes() / secs / 1e12, 8), "unit": UNIT,
            "cores": threads, "sample": "the whole C2 call (64 (sequence, kv-head) streams of 4096 keys), one thread"}


def run_prefill(args, rank, world, local_rank):
    """Multi-token causal forward (tcgen05 kernel): value = algorithmic TFLOP/s."""
    from paper_2605_29157_b200 import binding as plx

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    cfg, Lq = wl.PREFILL_CONFIGS[args.workload]
    cfg = wl.scaled(cfg, seed=rank_seed(cfg.seed, rank))
    if args.batch:
        cfg = wl.scaled(cfg, B=args.batch, name=f"{cfg.name}(B={args.batch})", note=cfg.note + ", reduced batch")
    nsets = args.kv_sets or 2
    sets = [wl.make_prefill_inputs(wl.scaled(cfg, seed=cfg.seed + 17 * i), Lq, dev) for i in range(nsets)]
    flops = wl.prefill_flops(cfg, Lq)
    mode = "plain" if args.plain_bf16_p else getattr(args, "p_precision", "residual")
    prec = {"plain": plx.PLX_P_BF16, "residual": plx.PLX_P_BF16_RESIDUAL, "adaptive": plx.PLX_P_BF16_ADAPTIVE}[mode]
    # executed / algorithmic tensor work: the residual products add half; in the adaptive mode only in the row
    # tiles in which some row sees fewer than PLX_P_ADAPTIVE_MIN_KEYS keys
    if mode == "adaptive":
        i = np.arange(Lq, dtype=np.int64)
        vis = np.maximum(cfg.T_max - Lq + i + 1, 0)
        first = np.maximum(cfg.T_max - Lq + 128 * (i // 128) + 1, 0)
        mma_factor = 1.0 + 0.5 * float(vis[first < plx.PLX_P_ADAPTIVE_MIN_KEYS].sum()) / float(vis.sum())
    else:
        mma_factor = 1.0 if mode == "plain" else 1.5
    out = torch.empty(cfg.B, cfg.Hq, Lq, cfg.D, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    # room for the split-KV records: the library splits the keys only when the row tiles alone leave SMs idle
    ws = torch.empty(min(plx.parallax_prefill_workspace_bytes(cfg.B, cfg.Hq, cfg.D, Lq, 64), 1 << 30), dtype=torch.uint8,
                     device=dev)

    launches_per_step = tensor_core_launches(cfg, Lq, torch.cuda.get_device_properties(dev).multi_processor_count)

    def step(i):
        x = sets[i % nsets]
        plx.parallax_prefill_fwd_ex(x["q"], x["r"], x["k"], x["v"], None, out, cfg.scale, ws, 0, status, stream, prec)

    sampler = ClockSampler(local_rank)
    timer = BlockTimer(stream, sampler, world, dev)
    for i in range(args.warmup):
        step(i)
    t_call = timer.run(step, args.steps)
    ms = t_call["ms_per_step"]
    assert int(status.item()) == 0, "device-side wait timed out"
    value = flops * world / (ms * 1e-3) / 1e12

    # end to end: q, r from pinned host memory, output back to host, every step (the caches are resident)
    qh = [x["q"].cpu().pin_memory() for x in sets]
    rh = [x["r"].cpu().pin_memory() for x in sets]
    oh = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
    qd, rd = torch.empty_like(sets[0]["q"]), torch.empty_like(sets[0]["r"])

    def e2e_step(i):
        x = sets[i % nsets]
        qd.copy_(qh[i % nsets], non_blocking=True)
        rd.copy_(rh[i % nsets], non_blocking=True)
        plx.parallax_prefill_fwd_ex(qd, rd, x["k"], x["v"], None, out, cfg.scale, ws, 0, status, stream, prec)
        oh.copy_(out, non_blocking=True)
        stream.synchronize()
    e2e_steps = max(5, args.steps // 10)
    for i in range(2):
        e2e_step(i)
    ms_e2e = timer.run(e2e_step, e2e_steps)["ms_per_step"]
    clocks = t_call["clocks"]
    sampler.close()

    peaks = json.loads((ROOT / "MEASURED_PEAKS.json").read_text()) if (ROOT / "MEASURED_PEAKS.json").exists() else None
    peak = float(peaks["bf16_tflops_sustained"]) if peaks else 1400.0
    burst = float(peaks["bf16_tflops"]) if peaks else 1590.0
    achieved = flops / (ms * 1e-3) / 1e12
    n_q = cfg.B * cfg.Hq * Lq * cfg.D * 2
    kv_b = cfg.B * cfg.Hkv * cfg.T_max * cfg.D * 4
    result = {
        "metric": "parallax_prefill_throughput", "value": round(value, 2), "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.note}; B={cfg.B} Hq={cfg.Hq} Hkv={cfg.Hkv} D={cfg.D} Lq={Lq} "
                               f"context={cfg.T_max}, causal; q,r,K,V bf16 N(0,1), bf16 output, scale 1/sqrt(D)",
                   "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D, "Lq": Lq, "T_max": cfg.T_max,
                   "l2_policy": f"{nsets} input sets used round-robin; {(3 * n_q + kv_b) * nsets / 2**20:.0f} MiB touched "
                                f"between two uses of a set vs 126 MiB L2",
                   "parallelism": "independent sequences per GPU, no collective"},
        "roofline": {"bound": "tensor", "kernel": "plx_prefill_kernel", "achieved": round(achieved, 1), "peak": peak,
                     "peak_source": ("measured" if peaks else "fallback") + " cuBLAS bf16, sustained (kernel timed back to back for the whole step)",
                     "unit": "TFLOP/s", "frac": round(achieved / peak, 4), "frac_of_burst_peak": round(achieved / burst, 4),
                     "executed_tflops_incl_residual_mmas": round(achieved * mma_factor, 1),
                     "p_precision": {"plain": "bf16", "residual": "bf16+residual",
                                     "adaptive": f"bf16+residual in row tiles with a row of fewer than {plx.PLX_P_ADAPTIVE_MIN_KEYS} "
                                                 "keys, plain bf16 elsewhere"}[mode],
                     "algorithmic_flops_per_launch": flops,
                     "traffic": None if args.batch else ncu_traffic(cfg.name)[0],
                     "traffic_source": None if args.batch else ncu_traffic(cfg.name)[1]},
        "e2e": {"value": round(flops * world / (ms_e2e * 1e-3) / 1e12, 2), "unit": "TFLOP/s",
                "ms_per_step": round(ms_e2e, 4), "h2d_bytes_per_step": 2 * n_q, "d2h_bytes_per_step": n_q,
                "note": "q and r copied from pinned host memory and the output copied back every step"},
        "gpu_launches": launches_per_step * args.steps * t_call["blocks"], "clocks": clocks, "timing": timing_note(t_call),
    }
    if launches_per_step > 1:
        result["config"]["split_kv"] = ("the row tiles alone leave SMs idle: the library divides each tile's keys among "
                                        "CTAs and finishes the rows with its merge kernel (second launch)")
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import parallax_oracle as po
        po.build()
        x = sets[0]
        G, tail = cfg.G, min(Lq, 128)
        done, secs, n, threads = 0, 0.0, 0, 1
        g = np.random.default_rng(0)
        while secs < args.cpu_seconds and n < cfg.B * cfg.Hkv:
            b, h = int(g.integers(cfg.B)), int(g.integers(cfg.Hkv))
            qb = wl.bf16_bits(x["q"][b:b + 1, h * G:(h + 1) * G, Lq - tail:])
            rb = wl.bf16_bits(x["r"][b:b + 1, h * G:(h + 1) * G, Lq - tail:])
            kb, vb = wl.bf16_bits(x["k"][b:b + 1, h:h + 1]), wl.bf16_bits(x["v"][b:b + 1, h:h + 1])
            t0 = time.perf_counter()
            _, threads = po.prefill_bf16(qb, rb, kb, vb, None, cfg.scale)
            secs += time.perf_counter() - t0
            i = np.arange(tail, dtype=np.int64)
            done += int((cfg.T_max - tail + i + 1).sum()) * G * cfg.D * 8
            n += 1
        result["cpu_baseline"] = {"value": round(done / secs / 1e12, 6), "unit": "TFLOP/s", "cores": threads,
                                  "kind": "oracle", "seconds": round(secs, 2),
                                  "sample": f"last {tail} query tokens of {n} (sequence, kv-head) groups of {cfg.name}"}
    return result


def run_backward(args, rank, world, local_rank):
    """Backward of the multi-token causal forward (projection kernel + tcgen05 row and column passes):
    value = algorithmic TFLOP/s of the backward call (16*D flop per visible (query, key) pair)."""
    from paper_2605_29157_b200 import binding as plx

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    cfg, Lq = wl.BACKWARD_CONFIGS[args.workload]
    cfg = wl.scaled(cfg, seed=rank_seed(cfg.seed, rank))
    if args.batch:
        cfg = wl.scaled(cfg, B=args.batch, name=f"{cfg.name}(B={args.batch})", note=cfg.note + ", reduced batch")
    B, Hq, Hkv, D, T = cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T_max
    nsets = args.kv_sets or 2
    stream = torch.cuda.current_stream()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    sets = []
    for i in range(nsets):
        x = wl.make_prefill_inputs(wl.scaled(cfg, seed=cfg.seed + 17 * i), Lq, dev)
        g = torch.Generator(device=dev).manual_seed(cfg.seed + 1000 + i)
        x["dout"] = torch.randn(B, Hq, Lq, D, device=dev, generator=g).to(torch.bfloat16)
        x["out"] = torch.empty(B, Hq, Lq, D, dtype=torch.bfloat16, device=dev)
        x["vbar"] = torch.empty_like(x["out"])
        x["lse"] = torch.empty(B, Hq, Lq, dtype=torch.float32, device=dev)
        x["tbar"] = torch.empty_like(x["lse"])
        plx.parallax_prefill_fwd_save(x["q"], x["r"], x["k"], x["v"], None, x["out"], x["lse"], x["tbar"], x["vbar"],
                                      cfg.scale, status, stream)
        sets.append(x)
    dq = torch.empty(B, Hq, Lq, D, dtype=torch.bfloat16, device=dev)
    dr = torch.empty_like(dq)
    dk = torch.empty(B, Hkv, T, D, dtype=torch.bfloat16, device=dev)
    dv = torch.empty_like(dk)
    ws = torch.empty(plx.parallax_prefill_bwd_workspace_bytes(B, Hq, Lq), dtype=torch.uint8, device=dev)
    flops = wl.backward_flops(cfg, Lq)

    def step(i, dout=None):
        x = sets[i % nsets]
        plx.parallax_prefill_bwd(x["q"], x["r"], x["k"], x["v"], x["dout"] if dout is None else dout, x["out"], x["lse"],
                                 x["tbar"], x["vbar"], None, dq, dr, dk, dv, cfg.scale, ws, status, stream)

    sampler = ClockSampler(local_rank)
    timer = BlockTimer(stream, sampler, world, dev)
    for i in range(args.warmup):
        step(i)
    t_call = timer.run(step, args.steps)
    ms = t_call["ms_per_step"]
    assert int(status.item()) == 0, "device-side wait timed out"
    value = flops * world / (ms * 1e-3) / 1e12

    # end to end: the upstream gradient comes from pinned host memory, the four gradients go back, every step
    gh = [x["dout"].cpu().pin_memory() for x in sets]
    gd = torch.empty_like(sets[0]["dout"])
    back = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (dq, dr, dk, dv)]

    def e2e_step(i):
        gd.copy_(gh[i % nsets], non_blocking=True)
        step(i, gd)
        for h, t in zip(back, (dq, dr, dk, dv)):
            h.copy_(t, non_blocking=True)
        stream.synchronize()
    e2e_steps = max(3, args.steps // 10)
    for i in range(2):
        e2e_step(i)
    ms_e2e = timer.run(e2e_step, e2e_steps)["ms_per_step"]
    clocks = t_call["clocks"]
    sampler.close()

    peaks = json.loads((ROOT / "MEASURED_PEAKS.json").read_text()) if (ROOT / "MEASURED_PEAKS.json").exists() else None
    peak = float(peaks["bf16_tflops_sustained"]) if peaks else 1400.0
    burst = float(peaks["bf16_tflops"]) if peaks else 1590.0
    achieved = flops / (ms * 1e-3) / 1e12
    n_q = B * Hq * Lq * D * 2
    n_kv = B * Hkv * T * D * 2
    result = {
        "metric": "parallax_backward_throughput", "value": round(value, 2), "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.note}; B={B} Hq={Hq} Hkv={Hkv} D={D} Lq=context={T}, causal; "
                               f"q,r,K,V,dO bf16 N(0,1), bf16 gradients, scale 1/sqrt(D); forward state saved beforehand",
                   "B": B, "Hq": Hq, "Hkv": Hkv, "D": D, "Lq": Lq, "T_max": T,
                   "l2_policy": f"{nsets} input sets used round-robin; {(6 * n_q + 4 * n_kv) * nsets / 2**20:.0f} MiB touched "
                                f"between two uses of a set vs 126 MiB L2",
                   "parallelism": "independent sequences per GPU, no collective"},
        "roofline": {"bound": "tensor", "kernel": "plx_bwd_row_kernel + plx_bwd_col_kernel", "achieved": round(achieved, 1),
                     "peak": peak,
                     "peak_source": ("measured" if peaks else "fallback") + " cuBLAS bf16, sustained (kernels timed back to back for the whole step)",
                     "unit": "TFLOP/s", "frac": round(achieved / peak, 4), "frac_of_burst_peak": round(achieved / burst, 4),
                     "executed_tflops_incl_recomputed_scores": round(achieved * 22.0 / 16.0, 1),
                     "algorithmic_flops_per_launch": flops,
                     "traffic": None if args.batch else ncu_traffic(cfg.name)[0],
                     "traffic_source": None if args.batch else ncu_traffic(cfg.name)[1]},
        "e2e": {"value": round(flops * world / (ms_e2e * 1e-3) / 1e12, 2), "unit": "TFLOP/s",
                "ms_per_step": round(ms_e2e, 4), "h2d_bytes_per_step": n_q, "d2h_bytes_per_step": 2 * n_q + 2 * n_kv,
                "note": "dO copied from pinned host memory and dq, dr, dk, dv copied back every step"},
        "gpu_launches": 3 * args.steps * t_call["blocks"], "clocks": clocks, "timing": timing_note(t_call),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import parallax_oracle as po
        po.build()
        x = sets[0]
        n_rows = min(Lq, 2048)
        secs, done, n = 0.0, 0, 0
        threads = min(po.max_threads(), Hkv)  # the oracle runs one thread per (sequence, kv-head) group
        while secs < args.cpu_seconds and n < B:
            sl = slice(0, n_rows)  # the first n_rows tokens of a sequence form a complete causal problem
            qb, rb, gb = (wl.bf16_bits(x[name][n:n + 1, :, sl]) for name in ("q", "r", "dout"))
            kb, vb = wl.bf16_bits(x["k"][n:n + 1, :, sl]), wl.bf16_bits(x["v"][n:n + 1, :, sl])
            t0 = time.perf_counter()
            po.backward_bf16(qb, rb, kb, vb, gb, None, cfg.scale)
            secs += time.perf_counter() - t0
            done += (n_rows * (n_rows + 1) // 2) * Hq * D * 16
            n += 1
        result["cpu_baseline"] = {"value": round(done / secs / 1e12, 6), "unit": "TFLOP/s", "cores": threads,
                                  "kind": "oracle", "seconds": round(secs, 2),
                                  "sample": f"first {n_rows} tokens, all heads, of {n} sequences of {cfg.name}"}
    return result


def run_grid(args):
    """The paper's decode profiling grid (Sec. 3.3 "Profiling Result": batch 1..2048 x context 128..32768,
    head dimension 128 and 64) for this library.  One JSON line per cell: device time per call for
    back-to-back stream launches and under CUDA-graph replay (the paper's two timers), KV-read TB/s."""
    from paper_2605_29157_b200 import binding as plx
    torch.cuda.set_device(0)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    Hq, Hkv = 16, 8

    def device_time(fn, n, warm=3):
        for i in range(warm):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n * 1e3

    for D in (128, 64):
        for B in (1, 4, 16, 64, 256, 1024, 2048):
            for T in (128, 512, 2048, 8192, 32768):
                kvb = B * Hkv * T * D * 4
                if kvb > 24 * 2 ** 30:
                    continue
                nsets = max(int(min(8, max(1, (1 << 30) // kvb))), 2 if kvb < (4 << 30) else 1)
                g = torch.Generator(device="cuda").manual_seed(B * 131 + T + D)
                q = torch.randn(B, Hq, D, generator=g, device="cuda").to(torch.bfloat16)
                r = torch.randn(B, Hq, D, generator=g, device="cuda").to(torch.bfloat16)
                ks = [torch.empty(B, Hkv, T, D, dtype=torch.bfloat16, device="cuda").uniform_(-1.7, 1.7, generator=g)
                      for _ in range(nsets)]
                vs = [torch.empty(B, Hkv, T, D, dtype=torch.bfloat16, device="cuda").uniform_(-1.7, 1.7, generator=g)
                      for _ in range(nsets)]
                out = torch.empty(B, Hq, D, dtype=torch.bfloat16, device="cuda")
                ws = plx.alloc_workspace(B, Hq, D, plx.PLX_MAX_SPLITS, "cuda")
                _, ns = plx.parallax_decode_plan(B, Hq, Hkv, D, T, sms, False)
                scale = 1.0 / float(np.sqrt(D))

                def call(i):
                    plx.parallax_decode_fwd_ex(q, r, ks[i % nsets], vs[i % nsets], None, out, scale, ws, 0)
                n = 200 if kvb < (1 << 28) else (50 if kvb < (1 << 31) else 10)
                us_stream = device_time(call, n)
                graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
                with torch.cuda.stream(side):
                    call(0)
                    torch.cuda.synchronize()
                    with torch.cuda.graph(graph, stream=side):
                        for i in range(nsets * 2):
                            call(i)
                torch.cuda.synchronize()
                us_graph = device_time(lambda i: graph.replay(), max(2, n // (nsets * 2)), warm=1) / (nsets * 2)
                us = min(us_stream, us_graph)
                print(json.dumps({"D": D, "B": B, "context": T, "num_splits": ns, "us_stream_launch": round(us_stream, 2),
                                  "us_graph_replay": round(us_graph, 2), "kv_read_TBps": round(kvb / us / 1e6, 3)}), flush=True)
                del ks, vs


def run_sharded(args, rank, world, local_rank):
    """--shard-keys: ONE batch whose keys are divided among the ranks (strong scaling).  Every rank holds
    T/world keys of every sequence and, per step: split kernel on its slice -> all-gather of the ~1 KB
    records (NCCL; skipped on one rank) -> combine kernel over all ranks' records.  value = the whole
    context's K/V bytes / the slowest rank's time."""
    from paper_2605_29157_b200 import binding as plx
    from paper_2605_29157_b200 import sequence_parallel as sp

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    cfg = wl.CONFIGS[args.workload]
    if cfg.ragged is not None:
        raise SystemExit("--shard-keys needs a uniform-context workload (C4 is the one it is meant for)")
    if cfg.T_max % (world * 64):
        raise SystemExit(f"--shard-keys: context {cfg.T_max} is not a multiple of 64 * {world} ranks")
    T_shard = cfg.T_max // world
    shard_cfg = wl.scaled(cfg, T_max=T_shard)
    set_bytes = cfg.B * cfg.Hkv * T_shard * cfg.D * 4
    nsets = args.kv_sets or min(16, max(2, -(-(1 << 30) // set_bytes)))
    # q, r are replicated (same seed on every rank); each rank draws its own slice of the caches
    qr = wl.make_inputs(wl.scaled(shard_cfg, T_max=64), dev)
    sets = [wl.make_inputs(wl.scaled(shard_cfg, seed=rank_seed(cfg.seed, rank) + 17 * i), dev, kv_only=True)
            for i in range(nsets)]
    chunk, ns = sp.plan_shard(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, T_shard, dev)
    stride = plx.parallax_partial_stride(cfg.D)
    partials = torch.empty(cfg.B, cfg.Hq, ns, stride, dtype=torch.float32, device=dev)
    out = torch.empty(cfg.B, cfg.Hq, cfg.D, dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()
    kv_bytes = cfg.kv_bytes()

    def step(i):
        x = sets[i % nsets]
        sp.decode_sequence_sharded(qr["q"], qr["r"], x["k"], x["v"], None, out, cfg.scale, chunk, None, partials)

    def local_only(i):
        x = sets[i % nsets]
        plx.parallax_decode_splitkv_partial(qr["q"], qr["r"], x["k"], x["v"], None, partials, cfg.scale, chunk, ns,
                                            None, stream)
    sampler = ClockSampler(local_rank)
    timer = BlockTimer(stream, sampler, world, dev)
    for i in range(args.warmup):
        step(i)
    t_call = timer.run(step, args.steps)
    for i in range(3):
        local_only(i)
    t_kernel = timer.run(local_only, args.steps)
    # end to end: q, r from pinned host memory, the result back to pinned host memory, every step
    qh, rh = qr["q"].cpu().pin_memory(), qr["r"].cpu().pin_memory()
    oh = torch.empty(out.shape, dtype=out.dtype).pin_memory()

    def e2e_step(i):
        qr["q"].copy_(qh, non_blocking=True)
        qr["r"].copy_(rh, non_blocking=True)
        step(i)
        oh.copy_(out, non_blocking=True)
        stream.synchronize()
    for i in range(3):
        e2e_step(i)
    t_e2e = timer.run(e2e_step, max(10, args.steps // 4))
    n_qr = cfg.B * cfg.Hq * cfg.D * 2
    peak, peak_src = measured_peaks()
    achieved = kv_bytes / world / (t_kernel["ms_per_step"] * 1e-3) / 1e9
    ms = t_call["ms_per_step"]
    result = {
        "metric": METRIC, "value": round(kv_bytes / (ms * 1e-3) / 1e12, 4), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 6), "us_per_call": round(ms * 1e3, 2),
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.note}; B={cfg.B} Hq={cfg.Hq} Hkv={cfg.Hkv} D={cfg.D} context={cfg.T_max} "
                               f"uniform, keys sharded over {world} rank(s) ({T_shard} keys per sequence and rank)",
                   "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D, "T_max": cfg.T_max, "T_shard": T_shard,
                   "chunk_len": chunk, "num_splits_per_rank": ns,
                   "l2_policy": f"{nsets} cache slices per rank used round-robin ({nsets * set_bytes / 2**30:.3f} GiB vs 0.123 GiB L2)",
                   "parallelism": f"keys of every sequence sharded over {world} rank(s); per step: split kernel -> "
                                  "all-gather of the partial records -> combine kernel on every rank",
                   "collective_bytes_per_rank": cfg.B * cfg.Hq * ns * stride * 4},
        "roofline": {"bound": "hbm", "kernel": "plx_decode_kernel (one rank's slice)", "achieved": round(achieved, 1),
                     "peak": peak, "peak_source": f"{peak_src} copy bandwidth (read + write)", "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "us_per_launch": round(t_kernel["ms_per_step"] * 1e3, 2),
                     "algorithmic_bytes_per_launch": kv_bytes // world, "traffic": None},
        "e2e": {"value": round(kv_bytes / (t_e2e["ms_per_step"] * 1e-3) / 1e12, 4), "unit": UNIT,
                "us_per_call": round(t_e2e["ms_per_step"] * 1e3, 2), "h2d_bytes_per_step": 2 * n_qr, "d2h_bytes_per_step": n_qr,
                "note": "every rank copies q and r from pinned host memory and its copy of the result back, every step; "
                        "the KV slices are device-resident state", **timing_note(t_e2e)},
        "gpu_launches": 2 * args.steps * t_call["blocks"], "clocks": t_call["clocks"],
        "timing": timing_note(t_call),
    }
    sampler.close()
    return result


def run_launcher_selftest(args, rank, world):
    """Rehearsal of the multi-rank plumbing on CPU ranks (gloo): the same launcher, rendezvous, per-rank
    seeding, max-over-ranks reduction, record gather and one-line report as a GPU run, with NO kernel and
    therefore no measurement (value is null).  Exists so that the launcher can be tested without GPUs."""
    from paper_2605_29157_b200 import sequence_parallel as sp
    cfg = wl.scaled(wl.CONFIGS["C1"], seed=rank_seed(0, rank))
    x = wl.make_inputs(cfg, "cpu")
    digest = float(x["k"].float().abs().sum())
    digests = [None] * world
    torch.distributed.all_gather_object(digests, digest)
    ms = max_over_ranks(1.0 + rank, world, "cpu")            # stand-in times: rank r "took" 1 + r ms
    gathered_ok = None
    if args.shard_keys:                                        # the exchange step on CPU tensors
        rec = torch.full((2, 4, 3, 20), float(rank))
        g = sp.gather_partials(rec)
        gathered_ok = bool(tuple(g.shape) == (world, 2, 4, 3, 20) and all(float(g[w].mean()) == w for w in range(world)))
    return {"metric": METRIC, "value": None, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong" if args.shard_keys else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "gpu_launches": 0,
            "selftest": "launcher rehearsal on CPU ranks (gloo): no kernel ran, nothing here is a measurement",
            "distinct_rank_inputs": len(set(digests)) == world, "stand_in_ms_max_over_ranks": ms,
            "gathered_layout_ok": gathered_ok, "config": {"workload": "none (launcher rehearsal)"}}


def launch_ranks(args, argv):
    """`--gpus N` outside a torchrun environment: start N ranks of this script (one process per GPU) under
    torch.distributed.run and pass their exit code on.  Never runs fewer ranks than asked for."""
    n = args.gpus
    if not args.launcher_selftest:
        have = torch.cuda.device_count()
        if have < n:
            print(f"bench.py: --gpus {n} asked for, {have} CUDA device(s) visible; refusing to run fewer ranks", file=sys.stderr)
            return 2
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), str(Path(__file__).resolve())] + argv
    return subprocess.call(cmd)


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    if args.workload in wl.PREFILL_CONFIGS or args.workload in wl.BACKWARD_CONFIGS:
        raise SystemExit("--impl reference covers the decode workloads C1..C5 (the metric the baseline names)")
    cfg = wl.CONFIGS[args.workload]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    small = cfg
    if dev == "cpu" and cfg.B * cfg.Hkv * cfg.T_max * cfg.D * 4 > (2 << 30):
        small = wl.scaled(cfg, B=max(1, cfg.B // 16))   # host-only box: draw a slice of the batch
    x = wl.make_inputs(small, dev)
    for name in ("q", "r", "k", "v"):   # the oracle reads host memory: stage the tensors there once
        x[name] = x[name].cpu()
    seqlens_host = x["seqlens_host"]
    # the whole run (all warm-up and timed steps, input marshalling included) is held to about 2.5 minutes
    per_step = min(20.0, 150.0 / max(1, args.steps + args.warmup))
    times, nbytes_all, threads, desc, n_seen = [], [], 1, "", 0
    for i in range(args.warmup + args.steps):
        secs, nbytes, threads, desc = oracle_sample_time(small, x, seqlens_host, per_step, max_streams=None,
                                                         wall_seconds=per_step, start=n_seen)
        n_seen += int(desc.split()[0])
        if i >= args.warmup:
            times.append(secs)
            nbytes_all.append(nbytes)
    value = sum(nbytes_all) / sum(times) / 1e12
    ms = 1e3 * sum(times) / len(times)
    return {
        "impl": "reference", "metric": METRIC, "value": round(value, 8), "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.note} (bounded sample per step: {desc})"},
        "cpu_baseline": {"value": round(value, 8), "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": round(value, 8), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default=None, choices=sorted(wl.CONFIGS) + sorted(wl.PREFILL_CONFIGS) + sorted(wl.BACKWARD_CONFIGS),
                    help="default C3 (C4 with --shard-keys)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--shard-keys", action="store_true",
                    help="strong scaling: the keys of every sequence are divided among the ranks (split kernel, "
                         "all-gather of the partial records, combine)")
    ap.add_argument("--fp8-kv", action="store_true", help="decode workloads over an e4m3 KV cache")
    ap.add_argument("--splits", type=int, default=0, help="force the split count (0 = library plan)")
    ap.add_argument("--kv-sets", type=int, default=0, help="number of KV cache sets rotated between steps")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (profiling captures on a smaller case)")
    ap.add_argument("--plain-bf16-p", action="store_true", help="prefill workloads: PLX_P_BF16 (no residual tiles)")
    ap.add_argument("--p-precision", default="residual", choices=["residual", "adaptive", "plain"],
                    help="prefill workloads: precision of the softmax weights on their way into the value product")
    ap.add_argument("--new-tokens", type=int, default=1,
                    help="decode workloads: this many new tokens per sequence and step (parallax_decode_fwd_multi)")
    ap.add_argument("--page-size", type=int, default=0, help="decode workloads: run over a paged KV cache with this page size")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--grid", action="store_true", help="decode sweep over the paper's batch x context grid (one JSON line per cell)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-read-probe", action="store_true", help="skip the read-only streaming probe (profiling captures)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the sustained (power-capped) timing of the headline call")
    ap.add_argument("--no-other-configs", dest="all_configs", action="store_false",
                    help="skip the short runs of the other decode configurations that ride along in the default line")
    ap.add_argument("--launcher-selftest", action="store_true",
                    help="rehearse the multi-rank plumbing on CPU ranks (gloo): no kernel, no measurement")
    args = ap.parse_args(argv)
    if args.warmup < 3:
        args.warmup = 3
    if args.workload is None:
        args.workload = "C4" if args.shard_keys else "C3"
    if args.gpus < 1:
        ap.error("--gpus must be >= 1")

    in_torchrun = "WORLD_SIZE" in os.environ
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return 0
    if args.grid:
        if rank == 0:
            run_grid(args)
        return 0
    if not in_torchrun and args.gpus > 1:
        return launch_ranks(args, argv)
    if in_torchrun and world != args.gpus:
        print(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)", file=sys.stderr)
        return 2

    if args.launcher_selftest:
        if world > 1:
            torch.distributed.init_process_group("gloo")
        result = run_launcher_selftest(args, rank, world) if world > 1 else {"selftest": "one rank: nothing to rehearse", "n_gpus": 1}
    else:
        if not torch.cuda.is_available() or torch.cuda.device_count() <= local_rank:
            print("bench.py: no CUDA device for this rank (the CUDA library is the only implementation)", file=sys.stderr)
            return 2
        if world > 1:
            torch.cuda.set_device(local_rank)
            torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        if args.shard_keys:
            if args.workload not in wl.CONFIGS:
                ap.error("--shard-keys applies to the decode workloads")
            runner = run_sharded
        else:
            runner = (run_prefill if args.workload in wl.PREFILL_CONFIGS else
                      run_backward if args.workload in wl.BACKWARD_CONFIGS else run_ours)
        result = runner(args, rank, world, local_rank)
    if rank == 0:
        print(json.dumps(result), flush=True)
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
