"""World-size-2 CPU (gloo) test of the multi-rank plumbing: per-rank workloads, request
sharding and the max-over-ranks timing reduction.  Each rank checks its own shard of a tiny
workload with the oracle, so the sharded job as a whole covers every request exactly once."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_33184_b200 import dist as ssdist
from paper_2609_33184_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert ssdist.env_rank() == (rank, rank, world)
        # weak scaling: same shapes, different requests
        cfg = ssdist.rank_config(inputs.scaled(inputs.CONFIGS["c1_tiny_chain"], len_lo=40, len_hi=40, L_c=16), rank)
        q = inputs.make_q(cfg)
        gathered = [torch.zeros_like(q) for _ in range(world)]
        dist.all_gather(gathered, q)
        assert not torch.equal(gathered[0], gathered[1])
        # strong scaling: a fixed batch split by request covers every request once
        mine = torch.zeros(7, dtype=torch.int32)
        mine[list(ssdist.shard_requests(7, rank, world))] = 1
        dist.all_reduce(mine)
        assert mine.tolist() == [1] * 7
        # timing: the job's duration is the slowest rank's
        ssdist.barrier()
        t = ssdist.max_over_ranks(1.0 + rank)
        assert t == float(world)
        assert ssdist.sum_over_ranks(10.0 * (rank + 1)) == 30.0   # whole-job units = sum over ranks
        out.put((rank, "ok"))
    except Exception as e:  # pragma: no cover
        out.put((rank, repr(e)))
    finally:
        dist.destroy_process_group()


def test_two_rank_gloo_plumbing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == {0: "ok", 1: "ok"}, res


def test_single_process_helpers():
    assert ssdist.max_over_ranks(3.5) == 3.5 and ssdist.sum_over_ranks(2.0) == 2.0
    assert list(ssdist.shard_requests(5, 0, 1)) == [0, 1, 2, 3, 4]
    sizes = [len(ssdist.shard_requests(10, r, 4)) for r in range(4)]
    assert sizes == [3, 3, 2, 2]
    cfg = inputs.CONFIGS["c2_qwen3_8b"]
    assert ssdist.rank_config(cfg, 0) is cfg and ssdist.rank_config(cfg, 3).seed != cfg.seed


def _cp_worker(rank, world, port, out):
    """History sharded by chunks: each rank reduces its chunks to a state in the library's
    export format (base-2 domain), the states are all-gathered, every rank merges them and
    must obtain full attention (Eq. 17)."""
    from oracle import attention, streaming
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(7)     # same data on every rank
        R, d, n, L_c, scale = 6, 16, 150, 32, 0.25
        q, k, v = rng.normal(size=(R, d)), rng.normal(size=(n, d)), rng.normal(size=(n, d))
        n_chunks = -(-n // L_c)
        state = streaming.IDENTITY(R, d)
        for j in ssdist.chunk_shard(n_chunks, rank, world):
            state = streaming.merge(state, streaming.chunk_partial(q, k[j * L_c:(j + 1) * L_c],
                                                                   v[j * L_c:(j + 1) * L_c], scale))
        LOG2E = 1.4426950408889634
        ml = torch.tensor(np.stack([state[0] * LOG2E, state[1]], axis=1), dtype=torch.float64)
        a = torch.tensor(state[2], dtype=torch.float64)
        peers = ssdist.allgather_states(ml, a)
        assert len(peers) == world - 1
        for ml_r, a_r in peers:
            state = streaming.merge(state, (ml_r[:, 0].numpy() / LOG2E, ml_r[:, 1].numpy(), a_r.numpy()))
        O, lse = streaming.finalize(state)
        ref_O, ref_lse = attention.verify_attention_rows(q, k, v, scale)
        assert np.abs(O - ref_O).max() < 1e-12 and np.abs(lse - ref_lse).max() < 1e-12
        covered = torch.zeros(n_chunks, dtype=torch.int32)
        covered[list(ssdist.chunk_shard(n_chunks, rank, world))] = 1
        dist.all_reduce(covered)
        assert covered.tolist() == [1] * n_chunks
        out.put((rank, "ok"))
    except Exception as e:  # pragma: no cover
        out.put((rank, repr(e)))
    finally:
        dist.destroy_process_group()


def test_two_rank_gloo_chunk_sharded_states():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_cp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == {0: "ok", 1: "ok"}, res
