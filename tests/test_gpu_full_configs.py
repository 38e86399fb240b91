"""The five workloads at their full sizes, in the launch configurations bench.py times
(overlapped chunk kernels, host length hints, a round's chunks with one call or one by one), checked on whole (request, kv-head) groups: every
query row of the group, all head dims and the LSE, against the oracle.  A whole group covers
every row tile, replica and token split the full-size launch uses for that kv-head."""
import random

import numpy as np
import pytest
import torch

from paper_2609_33184_b200 import harness, inputs
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _groups(cfg, lens, n_random, seed):
    """(request, kv-head) groups to compare: the shortest and the longest request, a request
    whose last chunk is partial (if any), and n_random others; kv-heads vary, first and last
    included."""
    rng = random.Random(seed)
    order = sorted(range(cfg.B), key=lambda b: lens[b])
    reqs = [order[0], order[-1]]
    partial = [b for b in range(cfg.B) if lens[b] % cfg.L_c]
    if partial:
        reqs.append(partial[rng.randrange(len(partial))])
    reqs += [rng.randrange(cfg.B) for _ in range(n_random)]
    heads = [0, cfg.H_kv - 1] + [rng.randrange(cfg.H_kv) for _ in range(len(reqs))]
    out = []
    for k, b in enumerate(reqs):
        g = (b, heads[k])
        if g not in out:
            out.append(g)
    return out


def _assert_contract(cfg, O, LSE, ref):
    """The unscaled contract bounds, stated explicitly: max |dO| <= 1e-2, mean |dO| <= 1e-3 per
    group, |dLSE| <= 1e-3 (the workloads' outputs are far below 1 in magnitude)."""
    G = cfg.G
    Og, Lg = util.f64(O), util.f64(LSE)
    for (b, kvh), (Or, Lr) in ref.items():
        err = np.abs(Og[b, kvh * G:(kvh + 1) * G] - Or)
        assert err.max() <= 1e-2 and err.mean() <= 1e-3, (b, kvh, err.max(), err.mean())
        assert np.abs(Lg[b, kvh * G:(kvh + 1) * G] - Lr).max() <= 1e-3, (b, kvh)


def _resident(name, n_random, one_call=True, kernel=None):
    """one_call: the round's chunks go in with one ss_verify_chunks call and the host's copy of the
    lengths, as bench.py does by default (one launch for the whole list where the library takes
    it); False: one call per chunk (bench.py --chunk-calls separate)."""
    from paper_2609_33184_b200 import binding as ssb
    cfg = inputs.CONFIGS[name]
    lens = inputs.history_lengths(cfg)
    Q, chunks, K_loc, V_loc, bits = harness.build_resident(cfg, lens, DEV)
    ctx = ssb.Context(cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, cfg.T_q, cfg.L_c, max_chunks=len(chunks),
                      flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    hints = harness.host_valid(cfg, lens, len(chunks))   # as bench.py does
    descs = ctx.chunk_descs([chunks], hints) if one_call else None
    for _ in range(2):
        harness.run_round(ctx, ssb, cfg, Q, chunks, K_loc, V_loc, bits, O, LSE, hints=hints, descs=descs)
    torch.cuda.synchronize()
    if kernel:
        assert ctx.last_chunk_kernel() == kernel, ctx.last_chunk_kernel()
    st, dev_bits = ctx.ss_poll_status()
    assert st == 0, dev_bits
    assert torch.isfinite(O.float()).all() and torch.isfinite(LSE).all()
    groups = _groups(cfg, lens, n_random, cfg.seed)
    ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits, groups=groups)
    _assert_contract(cfg, O, LSE, ref)
    worst = util.compare(cfg, O, LSE, ref)   # the tighter elementwise gate and the cosine check
    print(name, ctx.last_chunk_kernel(), len(groups), "groups", worst)
    ctx.close()


def test_c2_qwen3_8b_full():
    _resident("c2_qwen3_8b", 2, kernel="tcgen05-keys-round")


def test_c2_qwen3_8b_full_one_call_per_chunk():
    _resident("c2_qwen3_8b", 2, one_call=False, kernel="tcgen05-keys")


def test_c3_internlm25_7b_ragged_full():
    # ragged, lengths known to the host: one launch whose CTAs share all requests' tiles
    _resident("c3_internlm25_7b_ragged", 1, kernel="tcgen05-keys-round")


def test_c3_internlm25_7b_ragged_full_one_call_per_chunk():
    _resident("c3_internlm25_7b_ragged", 1, one_call=False, kernel="tcgen05-keys")


def test_c5_resident_full():
    # the streamed workload's batch (32 requests, 8,192 to 65,536 tokens) with its history in HBM
    _resident("c5_streamed", 1, kernel="tcgen05-keys-round")


def test_c4_tree_full():
    # 320 rows per group: all three row tiles of a kv-head, the 64-row remainder tile included;
    # the whole list of chunks in one launch (three token splits per row tile)
    _resident("c4_tree", 0, kernel="tcgen05-round")


def test_c4_tree_full_one_call_per_chunk():
    _resident("c4_tree", 0, one_call=False, kernel="tcgen05")


def test_c5_streamed_full():
    import oracle
    from tests.test_gpu_commit_stream import _stream_case, _u16
    cfg = inputs.CONFIGS["c5_streamed"]
    lens = sorted(inputs.history_lengths(cfg), reverse=True)   # active requests stay a prefix
    ctx, case, O, LSE, bufs, acc, stats, _ = _stream_case(cfg, lens)
    assert stats.h2d_bytes == sum(lens) * cfg.H_kv * cfg.d * 4
    groups = _groups(cfg, lens, 1, cfg.seed)
    ref = util.oracle_case(cfg, lens, *case, groups=groups)
    _assert_contract(cfg, O, LSE, ref)
    worst = util.compare(cfg, O, LSE, ref)
    zero = np.zeros((cfg.B, cfg.H_kv, cfg.T_q, cfg.d), np.uint16)
    ko, vo = oracle.commit_gather(_u16(case[2]), _u16(case[3]), acc["idx_host"].numpy(), acc["cnt_host"].numpy(),
                                  zero, zero, np.zeros(cfg.B, np.int32))
    assert np.array_equal(_u16(acc["hk"]), ko) and np.array_equal(_u16(acc["hv"]), vo)
    print("c5", len(groups), "groups", worst, "GB/s", stats.h2d_bytes / stats.ms_device / 1e6)
    ctx.close()
