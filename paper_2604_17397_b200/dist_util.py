"""Rank plumbing for multi-GPU runs.  The path has no exchange step: ranks are independent
replicas (one video each), so the only collectives are the barrier and the max over ranks
that bracket a timed region."""
from __future__ import annotations

import torch
import torch.distributed as dist


def barrier(world: int) -> None:
    if world > 1 and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest rank)."""
    if world <= 1 or not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_heads(heads: int, world: int, rank: int) -> range:
    """Heads owned by `rank` if one problem were sharded by head (heads are independent in
    rope, attention and commit; no collective is needed inside the path)."""
    if heads % world:
        raise ValueError("heads must divide evenly over ranks")
    per = heads // world
    return range(rank * per, (rank + 1) * per)


def aggregate_throughput(per_rank_units: float, ms_max: float, world: int) -> float:
    """Whole-job units per second: every rank processed per_rank_units in at most ms_max."""
    return world * per_rank_units / (ms_max * 1e-3)
