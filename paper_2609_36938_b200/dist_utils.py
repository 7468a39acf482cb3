"""Multi-process plumbing for the benchmark: sessions are independent problems, so ranks share no data path.

Each rank runs its own sessions; the only exchange is the timing reduction (maximum elapsed time over ranks, sum of
the units processed).  Works with any torch.distributed backend (nccl on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_units(n_units: int, rank: int, world: int) -> List[int]:
    """Unit ids (sessions) owned by `rank`: round-robin, every unit owned exactly once."""
    return list(range(rank, n_units, world))


def aggregate_throughput(units_local: float, elapsed_ms_local: float, device: str = "cpu") -> Tuple[float, float, float]:
    """Whole-job throughput from per-rank measurements: (units/s, max elapsed ms, total units).
    The job is as slow as its slowest rank, so the time is the maximum over ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return units_local / (elapsed_ms_local * 1e-3), elapsed_ms_local, units_local
    t = torch.tensor([elapsed_ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()) / (float(t.item()) * 1e-3), float(t.item()), float(u.item())
