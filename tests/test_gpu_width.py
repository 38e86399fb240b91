"""The verification-width controller driven by round times measured on this library's
streamed path (history in pinned host memory) and a synthetic acceptance model: no Draft or
Target model is involved, so this is a simulation of the controller's loop, not of a system."""
import dataclasses
import statistics

import pytest
import torch

from paper_2609_33184_b200 import harness
from paper_2609_33184_b200 import inputs
from tests import util
from tests.test_width_controller import LibController

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
WIDTHS = [2, 4, 6, 8]


def _measured_round_ms():
    """Per width q (T_q = q + 1): median transfer and compute time (ms) of a streamed
    verification round, from the library's own phase counters (ss_get_stats)."""
    from paper_2609_33184_b200 import binding as ssb
    base = inputs.VerifyConfig("v", 0x77, 4, 8, 2, 128, 512, 9, 4096, 4096)
    lens = [4096] * base.B
    ctx = ssb.Context(base.B, base.H_q, base.H_kv, base.d, 9, 9, base.L_c, flags=ssb.SS_FLAG_STREAM_TIMING)
    out = {}
    # the first configuration of a process is measured twice and its first pass dropped: its
    # pinned buffers and the link take a few dozen rounds to reach their steady rate
    for n_pass, q in enumerate([WIDTHS[0]] + WIDTHS):
        cfg = dataclasses.replace(base, T_q=q + 1)
        Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV, fill=0.0)
        host = harness.pinned_history(cfg, lens, chunks)
        bufs = harness.stream_buffers(cfg, DEV, len(chunks))
        O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
        LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
        desc = harness.make_stream_desc(ssb, cfg, lens, host, DEV, Q, K_loc, V_loc, bits, O, LSE, bufs)
        tr, co = [], []
        for _ in range(7):
            stats = ctx.ss_stream_round(desc)
            st = ctx.ss_get_stats()
            # the phases lie inside the round and account for it: transfers run beside the
            # chunk kernels, the tail comes after both
            assert 0 < st.last_transfer_ns <= st.last_round_ns
            assert 0 < st.last_chunk_ns and 0 < st.last_tail_ns
            assert st.last_chunk_ns + st.last_tail_ns + st.last_wait_ns == st.last_round_ns
            assert abs(st.last_round_ns * 1e-6 - stats.ms_device) < 1e-3
            tr.append(st.last_transfer_ns * 1e-6)
            co.append((st.last_chunk_ns + st.last_tail_ns) * 1e-6)
        assert ctx.ss_poll_status() == (0, 0)
        st = ctx.ss_get_stats()
        assert st.rounds >= 7 and st.chunk_calls >= 7 * len(chunks) and st.kv_bytes > 0
        if n_pass > 0:
            out[q] = (statistics.median(tr[2:]), statistics.median(co[2:]))
    ctx.close()
    return out


@pytest.mark.parametrize("alpha,draft_ms_per_token", [(0.9, 0.02), (0.2, 0.2)])
def test_controller_converges_to_the_argmin_of_measured_cost(alpha, draft_ms_per_token):
    phases = _measured_round_ms()
    # overlapped time is counted once (the controller's T_V = max(t_transfer, t_compute))
    t_round = {q: max(phases[q]) for q in WIDTHS}
    # the history transfer does not depend on q, so the measured round is nearly flat in q
    assert max(t_round.values()) < 1.5 * min(t_round.values())
    committed = {q: sum(alpha ** i for i in range(q + 1)) for q in WIDTHS}      # expected tokens per round
    cost = {q: (q * draft_ms_per_token + t_round[q]) / committed[q] for q in WIDTHS}
    best = min(WIDTHS, key=lambda q: (cost[q], q))
    ctl = LibController(WIDTHS, 2, 0.0, 0.5)
    q = None
    for _ in range(40):
        q = ctl.next()
        # committed tokens as the nearest integer count; the expectation is fed through repeats
        ctl.observe(q, q * draft_ms_per_token, phases[q][0], phases[q][1], 0.0, max(1, round(committed[q] * 100)))
    ctl.close()
    # the integer scaling by 100 keeps the ratios, so the minimiser is unchanged
    assert q == best
    if alpha >= 0.9:
        assert best == 8          # good drafts, transfer-dominated rounds: verify wide (Section 4.2)
    if alpha <= 0.2 and draft_ms_per_token >= 0.2:
        assert best == 2          # poor drafts: the extra candidates only cost drafting time
