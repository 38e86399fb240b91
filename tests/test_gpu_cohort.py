"""Cohort batching on the GPU: requests of a scheduled batch are grouped by ss_cohort_build,
each cohort runs as ONE batched verification round (per-request history lengths and query
counts of the cohort), and every request's result equals the result of running it alone:
requests in a cohort keep independent KV extents and softmax states."""
import ctypes as C
import dataclasses

import pytest
import torch

from paper_2609_33184_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
H_Q, H_KV, D, L_C = 8, 2, 128, 256


def _request(r, width, hist_len):
    """One request: its own seed, T_q = width + 1 candidate queries, its own history."""
    cfg = inputs.VerifyConfig(f"req{r}", 0x900 + r, 1, H_Q, H_KV, D, L_C, width + 1, hist_len, hist_len, k_mult=2.0)
    return cfg, util.gen_case(cfg, [hist_len], DEV, fill=0.0)


def test_cohorts_run_batched_and_match_single_request_rounds():
    from paper_2609_33184_b200 import binding as ssb
    lib = ssb.load()
    spec = [(4, 700), (8, 300), (4, 1500), (4, 0), (8, 1100), (4, 257), (8, 64)]   # (width, history tokens)
    reqs = [_request(r, w, n) for r, (w, n) in enumerate(spec)]
    tasks = (ssb.ss_task * len(spec))(*[ssb.ss_task(0, w, 0, H_KV, D, L_C, r, n) for r, (w, n) in enumerate(spec)])
    order = (C.c_int32 * len(spec))()
    start = (C.c_int32 * (len(spec) + 1))()
    n_cohorts = lib.ss_cohort_build(tasks, len(spec), 16, order, start)
    cohorts = [list(order[start[c]:start[c + 1]]) for c in range(n_cohorts)]
    assert cohorts == [[2, 0, 5, 3], [4, 1, 6]]          # by width, longest history first

    # every request alone (B = 1)
    alone = {}
    for r, (cfg, case) in enumerate(reqs):
        ctx = util.make_ctx(cfg)
        alone[r] = util.gpu_case(ctx, cfg, *case)
        ctx.close()

    for members in cohorts:
        cfg0 = reqs[members[0]][0]
        lens = [spec[r][1] for r in members]
        cfg = dataclasses.replace(cfg0, B=len(members))
        n_chunks = inputs.num_chunks(cfg, lens)
        cat = lambda ts: torch.cat(ts, dim=0).contiguous()
        Q = cat([reqs[r][1][0] for r in members])
        K_loc = cat([reqs[r][1][2] for r in members])
        V_loc = cat([reqs[r][1][3] for r in members])
        bits = cat([reqs[r][1][4] for r in members])
        chunks = []
        for j in range(n_chunks):
            ks, vs, vl = [], [], []
            for r in members:
                ch = reqs[r][1][1]
                if j < len(ch):
                    ks.append(ch[j][0]); vs.append(ch[j][1]); vl.append(int(ch[j][2][0]))
                else:   # this request has ended: its slot of the batch holds nothing valid
                    ks.append(torch.full((1, H_KV, L_C, D), float("nan"), dtype=torch.bfloat16, device=DEV))
                    vs.append(ks[-1]); vl.append(0)
            chunks.append((cat(ks), cat(vs), torch.tensor(vl, dtype=torch.int32, device=DEV)))
        ctx = util.make_ctx(cfg)
        O, LSE = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
        assert ctx.ss_poll_status() == (0, 0)
        ctx.close()
        for b, r in enumerate(members):
            Oa, La = alone[r]
            d = (O[b].float() - Oa[0].float()).abs().max().item()
            assert d <= 2.0 ** -7 * max(1.0, Oa.float().abs().max().item()), (r, d)
            assert (LSE[b] - La[0]).abs().max().item() <= 1e-4, r
        # and against the oracle, for the longest and the shortest member
        ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits, groups=[(0, 0), (len(members) - 1, 1)])
        util.compare(cfg, O, LSE, ref)
