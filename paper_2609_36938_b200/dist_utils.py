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


def or_reduce_bitmap(bitmap: torch.Tensor, union_into=None) -> torch.Tensor:
    """Union of the ranks' page bitmaps (Sec. 4.2, Eq. 3: each rank predicts on its own disjoint history shard and keeps its
    own page set; the union is only needed when the exact pass asks which pages nobody predicted).

    The one exchange of the key-sharded partition: an all-gather of the bitmaps (a few KB to a few tens of KB each; works
    with nccl and gloo alike, where a bitwise-OR all-reduce is a gloo-only operation) followed by a local OR.
    ``union_into(dst, src)`` does the local OR in place (on a GPU: the library's janus_page_union); without it the OR is a
    torch op (CPU tests).  Returns a new tensor; every rank gets the same union."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return bitmap.clone()
    world = dist.get_world_size()
    flat = torch.empty((world * bitmap.numel(),), dtype=bitmap.dtype, device=bitmap.device)
    dist.all_gather_into_tensor(flat, bitmap.contiguous().view(-1))
    gathered = flat.view(world, bitmap.numel())
    union = gathered[0].clone()
    for r in range(1, world):
        if union_into is not None:
            union_into(union, gathered[r])
        else:
            union |= gathered[r]
    return union
