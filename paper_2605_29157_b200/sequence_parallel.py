"""Decode over a context whose KEYS are sharded across GPUs (one process per GPU).

The path has exactly one exchange step: every rank turns its slice of each sequence into partial
states with the split kernel, the ~1 KB records are all-gathered over NCCL (NVLink / NVSwitch), and
every rank merges all records locally with the combine kernel.  The gathered records land in local
HBM before any kernel touches them; no kernel ever reads a peer's memory.

Softmax weights are permutation invariant, so a rank needs no knowledge of where its slice sits in
the sequence: only the number of valid keys it holds (`shard_lens`).
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def gather_partials(partials: torch.Tensor, group: Optional[dist.ProcessGroup] = None) -> torch.Tensor:
    """All-gather of per-rank partial records [B, Hq, num_splits, stride] into
    [world, B, Hq, num_splits, stride] (rank-major), the layout parallax_decode_combine_gathered reads.
    Works on any backend (NCCL on GPUs, gloo on CPU tensors)."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    partials = partials.contiguous()
    if world == 1:
        return partials.unsqueeze(0)
    gathered = torch.empty((world,) + tuple(partials.shape), dtype=partials.dtype, device=partials.device)
    dist.all_gather_into_tensor(gathered.view(-1), partials.view(-1), group=group)
    return gathered


def plan_shard(B, Hq, Hkv, D, T_shard, device, has_lens=False):
    """(chunk_len, num_splits) the library plans for one rank's slice."""
    from . import binding as plx
    sms = torch.cuda.get_device_properties(device).multi_processor_count
    chunk_len, _ = plx.parallax_decode_plan(B, Hq, Hkv, D, T_shard, sms, has_lens)
    return chunk_len, -(-T_shard // chunk_len)


def decode_sequence_sharded(q, r, k_shard, v_shard, shard_lens, out, scale, chunk_len: int = 0,
                            group: Optional[dist.ProcessGroup] = None, partials: Optional[torch.Tensor] = None):
    """q, r [B,Hq,D] (replicated), k_shard, v_shard [B,Hkv,T_shard,D] (this rank's slice of every
    sequence), shard_lens int32 [B] valid keys in the slice (None = T_shard).  Every rank ends with the
    full result in `out`.

    All three steps (split kernel, all-gather, combine kernel) are enqueued on torch's CURRENT stream:
    the collective is ordered against that stream only, so a caller that wants another stream wraps the
    call in `with torch.cuda.stream(s):`.  `partials` may pass a reusable [B,Hq,num_splits,stride] fp32
    buffer (steady-state loops allocate nothing then, apart from the gather's output)."""
    from . import binding as plx
    B, Hq, D = q.shape
    T_shard = k_shard.shape[2]
    if chunk_len <= 0:
        chunk_len, _ = plan_shard(B, Hq, k_shard.shape[1], D, T_shard, q.device, shard_lens is not None)
    num_splits = -(-T_shard // chunk_len)
    stride = plx.parallax_partial_stride(D)
    if partials is None:
        partials = torch.empty(B, Hq, num_splits, stride, dtype=torch.float32, device=q.device)
    stream = torch.cuda.current_stream(q.device)
    plx.parallax_decode_splitkv_partial(q, r, k_shard, v_shard, shard_lens, partials, scale, chunk_len, num_splits,
                                        None, stream)
    gathered = gather_partials(partials, group)
    plx.parallax_decode_combine_gathered(gathered, out, gathered.shape[0], num_splits, stream)
    return out
