"""Multi-GPU runs are independent replicas: (sequence, head) pairs never exchange data, so ranks only
agree on a common time.  These helpers hold that host logic (used by bench.py; tested on CPU with gloo)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world_size() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's value: a job of replicas is as slow as its slowest replica."""
    if world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds_local: float, device="cpu") -> float:
    """Whole-job throughput of identical replicas: all ranks' units over the slowest rank's time."""
    return world_size() * float(units_per_rank) / max_over_ranks(seconds_local, device)
