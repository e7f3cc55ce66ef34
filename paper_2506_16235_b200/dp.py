"""Data-parallel plumbing around the single-GPU path (torch.distributed only).

The hot path shards by bucket and by worker with no data-path collective: every
rank compresses its own buckets.  What ranks must share is small host state:
the ratio the controller picked (all ranks have to compress at the same ratio,
so that payloads have one size and can be all-gathered), and timings.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def _device_for(group=None):
    return torch.device("cuda", torch.cuda.current_device()) if dist.get_backend(group) == "nccl" else torch.device("cpu")


def agree_ratio(ratio: float, group=None, src: int = 0) -> float:
    """Rank `src`'s controller decides; every rank returns that ratio (exact double)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(ratio)
    t = torch.tensor([float(ratio)], dtype=torch.float64, device=_device_for(group))
    dist.broadcast(t, src=src, group=group)
    return float(t.item())


def max_over_ranks(value: float, group=None) -> float:
    """Slowest rank's value (used for step times: a step ends when the last rank ends)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device_for(group))
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def whole_job_gbps(world: int, steps: int, bytes_per_rank_step: float, slowest_ms: float) -> float:
    """Aggregate throughput of `world` ranks doing the same work per step (weak scaling)."""
    return world * steps * bytes_per_rank_step / (slowest_ms * 1e-3) / 1e9


def payload_slots(world: int, payload_bytes: int):
    """Byte ranges of the W equal-size payloads inside an all-gather buffer (16-byte aligned slots)."""
    slot = (payload_bytes + 15) // 16 * 16
    return [(r * slot, r * slot + payload_bytes) for r in range(world)], slot * world
