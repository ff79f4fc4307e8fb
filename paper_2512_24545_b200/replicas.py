"""Host-side plumbing for running the forward on several GPUs.

One MDBF layer lives on one GPU and its forward has no exchange step, so the
path does not shard: N GPUs run N independent replicas (independent layers or
requests), one process per GPU.  The only cross-rank traffic is bookkeeping:
which replica takes which work items, and the max-over-ranks of the device
times.  Nothing here touches the data path; it works with any
torch.distributed backend (nccl on GPUs, gloo on CPU).
"""
from __future__ import annotations

from typing import List, Sequence

import torch


def shard_units(n_units: int, rank: int, world: int) -> List[int]:
    """Indices of the independent work items (layers, requests) replica `rank` of
    `world` takes: a contiguous, balanced split; the first n_units % world ranks
    get one more item."""
    if world < 1 or not 0 <= rank < world or n_units < 0:
        raise ValueError(f"bad split: n_units={n_units} rank={rank} world={world}")
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def max_over_ranks(values: Sequence[float], dist=None, device: str = "cpu") -> List[float]:
    """Element-wise maximum of per-rank timings (a job is as slow as its slowest
    replica).  `dist` is torch.distributed (initialised) or None for one process."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_throughput(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job throughput of `world` replicas that each processed
    `units_per_rank` units while the slowest one took `seconds_max`."""
    if seconds_max <= 0:
        raise ValueError("non-positive time")
    return world * units_per_rank / seconds_max
