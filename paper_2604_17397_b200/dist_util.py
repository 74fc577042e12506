"""Rank plumbing for multi-GPU runs.

The path has no exchange step: heads are independent in rope, attention and commit, and videos are
independent of each other.  Ranks are therefore either replicas (one video each) or own a slice of
the heads of one problem, and the only collectives are the barrier and the max over ranks that
bracket a timed region.  This module launches the ranks (one process per GPU), reads a rank's
place from the environment the launcher set, and does those two collectives.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import Optional, Sequence

import torch
import torch.distributed as dist


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def launched_by_rank_launcher() -> bool:
    """True inside a process that torch.distributed.run (or an equivalent launcher) started."""
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def rank_env() -> tuple:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def spawn_ranks(n: int, script_argv: Sequence[str], port: Optional[int] = None, extra_env: Optional[dict] = None,
                timeout: Optional[float] = None) -> subprocess.CompletedProcess:
    """Run ``python script_argv...`` as ``n`` ranks on this node, one process per GPU (LOCAL_RANK = GPU index),
    rendezvous on 127.0.0.1.  stdout/stderr of the ranks pass through to the caller's."""
    if n < 1:
        raise ValueError("need at least one rank")
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")          # the communicator's own log states how many ranks joined
    if extra_env:
        env.update(extra_env)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), *script_argv]
    return subprocess.run(cmd, env=env, timeout=timeout)


def init_ranks(backend: str, device=None) -> tuple:
    """Join the process group the launcher prepared (no-op for a single process); returns rank_env()."""
    rank, local, world = rank_env()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)
    return rank, local, world


def shutdown_ranks() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()


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


def gather_objects(obj, world: int) -> list:
    """`obj` of every rank, in rank order, on every rank."""
    if world <= 1 or not dist.is_initialized():
        return [obj]
    out = [None] * world
    dist.all_gather_object(out, obj)
    return out


def shard_heads(heads: int, world: int, rank: int) -> range:
    """Heads owned by `rank` when one problem is sharded by head (heads are independent in
    rope, attention and commit; no collective is needed inside the path)."""
    if heads % world:
        raise ValueError("heads must divide evenly over ranks")
    per = heads // world
    return range(rank * per, (rank + 1) * per)


def aggregate_throughput(per_rank_units: float, ms_max: float, world: int) -> float:
    """Whole-job units per second: every rank processed per_rank_units in at most ms_max."""
    return world * per_rank_units / (ms_max * 1e-3)
