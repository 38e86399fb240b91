"""Multi-GPU plumbing.

The path shards by request (the cohort axis), so the benchmark has no data-path collective:
every rank runs the same per-GPU workload on its own requests and the only communication is
the barrier around the timed region and the max-over-ranks reduction of its duration.

One optional exchange is provided for a history that is sharded by CHUNKS over the ranks
(context-parallel style): each rank reduces its own chunks of every request to a merged state
(ss_verify_export_state), `allgather_states` exchanges the states with one all-gather, and the
peers' states are added to the open round with ss_verify_import_state before finalize.  The
merge is order-free (Eq. 17), so every rank ends with the full result.  The all-gather writes
into this rank's own memory; the kernels never read a peer's memory.
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


def chunk_shard(n_chunks: int, rank: int, world: int):
    """Chunk indices of a request's history owned by `rank` (round-robin: every rank gets
    early and late chunks, so ragged lengths stay balanced)."""
    return range(rank, n_chunks, world)


def allgather_states(ml: torch.Tensor, a: torch.Tensor, group=None):
    """Exchange exported round states between the ranks of `group` with one all-gather each
    for ml [rows, 2] and a [rows, d] (fp32; device tensors over NCCL, CPU tensors over gloo).

    Returns the list [(ml_r, a_r) for every OTHER rank r], in rank order: the states to hand
    to ss_verify_import_state.  Without a process group the list is empty.
    """
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return []
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    ml_all = [torch.empty_like(ml) for _ in range(world)]
    a_all = [torch.empty_like(a) for _ in range(world)]
    dist.all_gather(ml_all, ml.contiguous(), group=group)
    dist.all_gather(a_all, a.contiguous(), group=group)
    return [(ml_all[r], a_all[r]) for r in range(world) if r != rank]


def import_peer_states(ctx, ml: torch.Tensor, a: torch.Tensor, group=None, stream=None) -> int:
    """Export this rank's state of the open round is given as (ml, a); gather the peers'
    states and add them to the round.  Returns the number of states imported."""
    peers = allgather_states(ml, a, group)
    for ml_r, a_r in peers:
        ctx.ss_verify_import_state(ml_r, a_r, stream)
    return len(peers)


@dataclasses.dataclass
class ChunkShardPlan:
    """What one rank does in a round whose history is sharded by chunks."""
    chunks: list            # chunk indices this rank reduces
    owns_local: bool        # the local candidate segment is attended to once, by rank 0
    rows: int               # query rows of the round: B * H_q * T_q
    d: int
    state_bytes: int        # bytes of one exported state (ml [rows, 2] + a [rows, d], fp32)


def chunk_shard_plan(cfg, n_chunks: int, rank: int, world: int) -> ChunkShardPlan:
    rows = cfg.B * cfg.H_q * cfg.T_q
    return ChunkShardPlan(list(chunk_shard(n_chunks, rank, world)), rank == 0, rows, cfg.d,
                          rows * (cfg.d + 2) * 4)


def state_buffers(plan: ChunkShardPlan, device):
    """Export buffers of a round state in the library's format."""
    return (torch.empty(plan.rows, 2, dtype=torch.float32, device=device),
            torch.empty(plan.rows, plan.d, dtype=torch.float32, device=device))


def chunk_sharded_round(ctx, ssb, cfg, Q, my_chunks, K_loc, V_loc, bits, O, LSE, plan, ml, a, group=None):
    """One round with the history sharded by chunks over the ranks (the merge of Eq. 14 is
    order-free, Eq. 17): this rank's chunks (and, on rank 0, the local segment) -> exported
    state -> one all-gather of the states (they land in this rank's own memory) -> the peers'
    states imported as further partials -> finalize.  Every rank ends with the full result.
    my_chunks: [(K, V, valid_len), ...] for plan.chunks, in that order."""
    kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
    ctx.ss_verify_begin(Q, cfg.scale)
    for K, V, vl in my_chunks:
        ctx.ss_verify_chunk(K, V, vl)
    if plan.owns_local:
        ctx.ss_verify_local(K_loc, V_loc, kind, bits if cfg.mask == "tree" else None)
    ctx.ss_verify_export_state(ml, a)
    import_peer_states(ctx, ml, a, group)
    ctx.ss_verify_finalize(O, LSE)
