"""Rank plumbing for running independent replicas of the path on several GPUs.

The path does not shard: each rank processes its own batch against its own copy of
the weights and there is no data-path collective.  The only communication is the
barrier around the timed region and the reduction of the timing itself.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init_from_env(backend: str | None = None):
    """(rank, world, local_rank); initialises the process group when WORLD_SIZE > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"),
                                rank=rank, world_size=world)
    return rank, world, local


def barrier():
    if dist.is_initialized():
        dist.barrier()


def aggregate(units: float, elapsed_ms: float, device="cpu"):
    """Whole-job totals: sum of the units every rank processed and the slowest rank's time."""
    if not dist.is_initialized():
        return float(units), float(elapsed_ms)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(u.item()), float(t.item())
