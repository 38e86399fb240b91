"""The five workloads at their full sizes, in the launch configuration bench.py times
(overlapped chunk kernels), checked on sampled query rows the oracle computes one by one."""
import random

import pytest
import torch

import bench
from paper_2609_33184_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _samples(cfg, lens, n, seed):
    rng = random.Random(seed)
    out = []
    bs = sorted(range(cfg.B), key=lambda b: lens[b])
    pick_b = [bs[0], bs[-1]] + [rng.randrange(cfg.B) for _ in range(n)]
    for k in range(n):
        out.append((pick_b[k % len(pick_b)], rng.randrange(cfg.H_q), rng.randrange(cfg.T_q)))
    # always include a first and a last candidate row (mask extremes)
    out.append((pick_b[0], 0, 0))
    out.append((pick_b[1], cfg.H_q - 1, cfg.T_q - 1))
    return out


def _resident(name, n_samples):
    from paper_2609_33184_b200 import binding as ssb
    cfg = inputs.CONFIGS[name]
    lens = inputs.history_lengths(cfg)
    Q, chunks, K_loc, V_loc, bits = bench.build_resident(cfg, lens, DEV)
    ctx = ssb.Context(cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, cfg.T_q, cfg.L_c, max_chunks=len(chunks),
                      flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    hints = bench.host_valid(cfg, lens, len(chunks)) if len(set(lens)) > 1 else None   # as bench.py does
    for _ in range(2):
        bench.run_round(ctx, ssb, cfg, Q, chunks, K_loc, V_loc, bits, O, LSE, hints=hints)
    torch.cuda.synchronize()
    st, dev_bits = ctx.ss_poll_status()
    assert st == 0, dev_bits
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    samples = _samples(cfg, lens, n_samples, cfg.seed)
    ref = util.oracle_samples(cfg, lens, Q, chunks, K_loc, V_loc, bits, samples)
    worst = util.compare_samples(O, LSE, ref)
    print(name, ctx.last_chunk_kernel(), worst)
    ctx.close()


def test_c2_qwen3_8b_full():
    _resident("c2_qwen3_8b", 16)


def test_c3_internlm25_7b_ragged_full():
    _resident("c3_internlm25_7b_ragged", 10)


def test_c4_tree_full():
    _resident("c4_tree", 16)


def test_c5_streamed_full():
    import numpy as np
    import oracle
    from paper_2609_33184_b200 import binding as ssb
    from tests.test_gpu_commit_stream import _stream_case, _u16
    cfg = inputs.CONFIGS["c5_streamed"]
    lens = sorted(inputs.history_lengths(cfg), reverse=True)   # active requests stay a prefix
    ctx, case, O, LSE, bufs, acc, stats, _ = _stream_case(cfg, lens)
    assert stats.h2d_bytes == sum(lens) * cfg.H_kv * cfg.d * 4
    samples = _samples(cfg, lens, 10, cfg.seed)
    ref = util.oracle_samples(cfg, lens, *case, samples)
    worst = util.compare_samples(O, LSE, ref)
    zero = np.zeros((cfg.B, cfg.H_kv, cfg.T_q, cfg.d), np.uint16)
    ko, vo = oracle.commit_gather(_u16(case[2]), _u16(case[3]), acc["idx_host"].numpy(), acc["cnt_host"].numpy(),
                                  zero, zero, np.zeros(cfg.B, np.int32))
    assert np.array_equal(_u16(acc["hk"]), ko) and np.array_equal(_u16(acc["hv"]), vo)
    print("c5", worst, "GB/s", stats.h2d_bytes / stats.ms_device / 1e6)
    ctx.close()


def test_sweep_tool_runs_a_small_shape():
    # the sizing aid goes through the same C ABI; keep it working
    from paper_2609_33184_b200 import sweep
    for d, page in ((128, 0), (64, 0), (128, 16)):
        gbps, ms, kernel = sweep.measure(rows=8, d=d, page_size=page, B=2, H_kv=2, L_c=512, tokens=2048,
                                         flags=0, rounds=2, dev="cuda:0")
        assert gbps > 0 and ms > 0 and kernel.startswith("tcgen05")
