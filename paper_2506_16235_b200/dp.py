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


def exchange_payloads(payload: torch.Tensor, group=None):
    """The exchange step of the sparse path (Section 5.3: top-k payloads travel by AllGather):
    every rank contributes its payload (uint8 tensor; all ranks' payloads have the same size because
    they compressed equally long buckets at the agreed ratio) and receives all of them.
    Returns (buffer, [one view per rank]); view r is rank r's payload, 16-byte aligned, ready for
    nsml_decompress_accumulate.  One fixed-size all-gather, NCCL on CUDA tensors, gloo on CPU ones."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    nbytes = payload.numel()
    slots, total = payload_slots(world, nbytes)
    slot = total // world
    buf = torch.empty(total, dtype=torch.uint8, device=payload.device)
    if world == 1:
        buf[:nbytes].copy_(payload)
    else:
        rank = dist.get_rank(group)
        mine = buf[rank * slot:(rank + 1) * slot]
        mine[:nbytes].copy_(payload)
        if slot > nbytes:
            mine[nbytes:].zero_()
        dist.all_gather_into_tensor(buf, mine.clone(), group=group)
    return buf, [buf[a:b] for a, b in slots]


class _HostClock:
    def __init__(self):
        import time

        self._now, self._marks = time.perf_counter, []

    def mark(self):
        self._marks.append(self._now())

    def phases_ms(self):
        return [1e3 * (b - a) for a, b in zip(self._marks, self._marks[1:])]


class _CudaClock:
    def __init__(self):
        self._marks = []

    def mark(self):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        self._marks.append(ev)

    def phases_ms(self):
        self._marks[-1].synchronize()
        return [a.elapsed_time(b) for a, b in zip(self._marks, self._marks[1:])]


def exchange_round(ctrl, last, dense_bytes_all_ranks: float, compress, accumulate, on_cuda: bool, group=None):
    """One step of the data-parallel exchange (Fig. 1, Alg. 1 Step 2 and Section 5.3 put together).

    ctrl      this rank's controller (only rank 0's decision is used: ranks must compress at one ratio so that
              the payloads have one size)
    last      (bytes, seconds) of the previous step's transfer as this function returned it; (0, 0) at first
    compress(ratio) -> this rank's payload (uint8 tensor); accumulate(views) sums the gathered payloads
    Returns (agreed ratio, [compress, all-gather, sum] times in ms each MAX-reduced over the ranks, new `last`):
    the transfer the controller sees next is all ranks' payload bytes and the slowest rank's all-gather time."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    ratio = agree_ratio(ctrl.select_ratio(last[0], last[1], dense_bytes_all_ranks), group)
    clock = _CudaClock() if on_cuda else _HostClock()
    clock.mark()
    payload = compress(ratio)
    clock.mark()
    _, views = exchange_payloads(payload, group)
    clock.mark()
    accumulate(views)
    clock.mark()
    phases = [max_over_ranks(ms, group) for ms in clock.phases_ms()]
    return ratio, phases, (float(world * payload.numel()), max(phases[1] * 1e-3, 1e-9))


class GradientExchange:
    """One bucket's data-parallel gradient exchange, every step (Fig. 1 and Alg. 1-2 of the paper put
    together): rank 0's controller picks the ratio from the last measured transfer, every rank compresses
    its bucket at that ratio, the payloads are all-gathered, every rank sums them into its dense
    gradient, and the measured transfer (bytes of all payloads, slowest rank's device time of the
    all-gather) is what the controller sees next step.  CUDA only: the compression and the sum run in
    libnsml."""

    def __init__(self, n: int, bits: int = 8, group=None, device=None, **ctrl_overrides):
        import paper_2506_16235_b200 as nsml

        self.nsml, self.n, self.bits, self.group = nsml, int(n), int(bits), group
        self.device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.ctrl = nsml.Controller(**ctrl_overrides)
        self.ws = nsml.alloc_bytes(nsml.nsml_workspace_bytes(self.n), self.device)
        self.aws = nsml.alloc_bytes(nsml.nsml_accumulate_workspace_bytes(self.n, self.world), self.device)
        self.last = (0.0, 0.0)
        self.ratio = None

    def step(self, grad: torch.Tensor, dense: torch.Tensor) -> float:
        """dense <- sum over ranks of their compressed `grad`; returns the ratio used."""
        nsml = self.nsml
        self.ratio, self.phases_ms, self.last = exchange_round(
            self.ctrl, self.last, 4.0 * self.n * self.world,
            lambda ratio: nsml.nsml_compress(grad, ratio, self.bits, workspace=self.ws),
            lambda views: nsml.nsml_decompress_accumulate(views, dense, zero_first=True, workspace=self.aws, sized=True),
            on_cuda=True, group=self.group)
        return self.ratio
