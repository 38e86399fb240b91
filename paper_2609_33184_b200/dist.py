"""Multi-GPU plumbing: the path shards by request, so there is no data-path collective.

Every rank runs the same per-GPU workload on its own requests; the only communication is
the barrier around the timed region and the max-over-ranks reduction of its duration.
"""
from __future__ import annotations

import dataclasses
import os

import torch


def env_rank():
    """(rank, local_rank, world_size) from the torchrun environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def rank_config(cfg, rank: int):
    """The workload of one rank: same shapes, its own requests (rank-specific seed)."""
    return cfg if rank == 0 else dataclasses.replace(cfg, seed=cfg.seed + 0x100 * rank)


def shard_requests(n_requests: int, rank: int, world: int):
    """Contiguous block of request indices owned by `rank` when a fixed batch is split
    (strong scaling); sizes differ by at most one."""
    base, rem = divmod(n_requests, world)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a per-rank scalar (a duration) over all ranks; identity without a process group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    """Sum of a per-rank scalar (bytes processed) over all ranks; identity without a process group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier(cuda: bool = False):
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()
