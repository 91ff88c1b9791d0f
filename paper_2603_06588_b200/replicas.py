"""Multi-GPU plumbing of the benchmark: the hooked attention path has no exchange step (sequences
and KV heads are independent), so N GPUs run N independent replicas.  The only communication is
the bookkeeping of the measurement: a barrier around the timed region and the maximum of the
per-rank durations.  Works on any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def max_over_ranks(values: Sequence[float], device: torch.device) -> list:
    """Element-wise maximum of a few per-rank scalars (durations) over all ranks."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def replica_throughput(units_per_rank: float, seconds: float, world_size: int) -> float:
    """Whole-job throughput of `world_size` replicas that each process `units_per_rank` units in
    `seconds` (the slowest rank's time)."""
    return world_size * units_per_rank / seconds
