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


def _plan_worker(rank, world, port, out):
    """bench.py --shard chunks as far as a CPU goes: argument plumbing, the per-rank plan, shard
    coverage, the shapes of the exchanged states, and the round's sequence of calls (recorded by a
    stand-in context) with the all-gather running over gloo."""
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        args = bench.arg_parser().parse_args(["--gpus", str(world), "--shard", "chunks", "--workload", "c4_tree"])
        assert args.shard == "chunks" and bench.arg_parser().parse_args([]).shard == "requests"
        cfg = inputs.scaled(inputs.CONFIGS[args.workload], len_lo=5 * 4096, len_hi=5 * 4096)
        lens = inputs.history_lengths(cfg)
        n_chunks = inputs.num_chunks(cfg, lens)
        plan = ssdist.chunk_shard_plan(cfg, n_chunks, rank, world)
        assert plan.chunks == list(range(rank, n_chunks, world)) and plan.owns_local == (rank == 0)
        assert plan.rows == cfg.B * cfg.H_q * cfg.T_q and plan.state_bytes == plan.rows * (cfg.d + 2) * 4
        covered = torch.zeros(n_chunks, dtype=torch.int32)
        covered[plan.chunks] = 1
        dist.all_reduce(covered)
        assert covered.tolist() == [1] * n_chunks
        ml, a = ssdist.state_buffers(plan, "cpu")
        assert ml.shape == (plan.rows, 2) and a.shape == (plan.rows, cfg.d)

        class Recorder:   # stands in for the library's context: records the calls of a round
            def __init__(self):
                self.calls = []

            def __getattr__(self, name):
                def call(*args, **kw):
                    self.calls.append(name)
                    if name == "ss_verify_export_state":
                        args[0].fill_(float(rank + 1))
                        args[1].fill_(float(10 * (rank + 1)))
                    if name == "ss_verify_import_state":   # a peer's state arrived intact
                        peer = 1 - rank
                        assert bool((args[0] == float(peer + 1)).all()) and bool((args[1] == float(10 * (peer + 1))).all())
                return call

        class Consts:
            SS_MASK_TREE_BITS, SS_MASK_CHAIN = 1, 0

        rec = Recorder()
        mine = [(None, None, None)] * len(plan.chunks)
        ssdist.chunk_sharded_round(rec, Consts, cfg, None, mine, None, None, None, None, None, plan, ml, a)
        want = (["ss_verify_begin"] + ["ss_verify_chunk"] * len(plan.chunks) +
                (["ss_verify_local"] if rank == 0 else []) + ["ss_verify_export_state"] +
                ["ss_verify_import_state"] * (world - 1) + ["ss_verify_finalize"])
        assert rec.calls == want, rec.calls
        out.put((rank, "ok"))
    except Exception as e:  # pragma: no cover
        out.put((rank, repr(e)))
    finally:
        dist.destroy_process_group()


def test_two_rank_gloo_chunk_sharded_bench_path():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_plan_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == {0: "ok", 1: "ok"}, res
