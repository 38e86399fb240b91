"""Verification-width controller: the library's host logic against the plain-Python oracle,
a hand-worked example and a noiseless simulation whose optimum is known in closed form."""
import ctypes as C
import os
import random

import pytest

import oracle
from paper_2609_33184_b200 import binding as ssb
from paper_2609_33184_b200 import build as ssbuild

GOLD = os.path.join(os.path.dirname(__file__), "golden", "width_hand_example.txt")


class LibController:
    def __init__(self, widths, sample_rounds, thr, ema):
        ssbuild.build()
        self.lib = ssb.load()
        cfg = ssb.ss_width_config(len(widths), (C.c_int32 * 8)(*widths), sample_rounds, thr, ema)
        self.h = C.c_void_p()
        assert self.lib.ss_width_create(C.byref(self.h), C.byref(cfg)) == 0

    def observe(self, q, td, tt, tc, to, u):
        obs = ssb.ss_width_obs(td, tt, tc, to, u)
        assert self.lib.ss_width_observe(self.h, q, C.byref(obs)) == 0

    def next(self):
        return self.lib.ss_width_next(self.h)

    def estimate(self, q):
        t, u, c, n = C.c_double(), C.c_double(), C.c_double(), C.c_int32()
        assert self.lib.ss_width_estimate(self.h, q, C.byref(t), C.byref(u), C.byref(c), C.byref(n)) == 0
        return t.value, u.value, c.value, n.value

    def close(self):
        self.lib.ss_width_destroy(self.h)


def _steps():
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        yield f[0], [float(x) for x in f[1:]]


@pytest.mark.parametrize("impl", ["oracle", "library"])
def test_hand_example(impl):
    ctl = (oracle.WidthController([2, 4, 6, 8], 1, 0.05, 0.5) if impl == "oracle"
           else LibController([2, 4, 6, 8], 1, 0.05, 0.5))
    assert ctl.next() == 2
    for kind, v in _steps():
        if kind == "obs":
            # committed is fractional in the example: the oracle takes it as is, the library's
            # observation is an integer count, so the library is fed tenths (same ratios)
            if impl == "oracle":
                ctl.observe(int(v[0]), v[1], v[2], v[3], v[4], v[5])
            else:
                ctl.observe(int(v[0]), v[1], v[2], v[3], v[4], int(round(v[5] * 10)))
        else:
            assert ctl.next() == int(v[0]), (impl, kind, v)


def test_overlapped_time_is_counted_once():
    ctl = LibController([4], 1, 0.0, 1.0)
    ctl.observe(4, 1.0, 10.0, 9.0, 0.5, 3)
    t, u, c, n = ctl.estimate(4)
    assert abs(t - 11.5) < 1e-6 and u == 3 and abs(c - 11.5 / 3) < 1e-6 and n == 1
    ctl.observe(4, 1.0, 2.0, 9.0, 0.5, 3)       # compute-bound round: max picks the compute time
    assert abs(ctl.estimate(4)[0] - 10.5) < 1e-6
    ctl.close()


def test_library_matches_oracle_on_random_rounds():
    rng = random.Random(3)
    for trial in range(20):
        widths = rng.choice([[2, 4, 6, 8], [1, 3], [8, 4, 2], [5]])
        sr, thr, ema = rng.randint(1, 3), rng.choice([0.0, 0.05, 0.2]), rng.choice([1.0, 0.5, 0.1])
        a, b = oracle.WidthController(widths, sr, thr, ema), LibController(widths, sr, thr, ema)
        for _ in range(60):
            qa, qb = a.next(), b.next()
            assert qa == qb
            # values exactly representable in float32 keep both sides on identical arithmetic
            td, tt, tc, to = (rng.randint(0, 64) / 8.0 for _ in range(4))
            u = rng.randint(1, qa + 1)
            a.observe(qa, td, tt, tc, to, u)
            b.observe(qb, td, tt, tc, to, u)
        b.close()


def test_invalid_arguments():
    ssbuild.build()
    lib = ssb.load()
    h = C.c_void_p()
    bad = ssb.ss_width_config(2, (C.c_int32 * 8)(4, 4), 1, 0.05, 0.5)        # duplicate width
    assert lib.ss_width_create(C.byref(h), C.byref(bad)) == ssb.SS_ERR_ARG
    bad = ssb.ss_width_config(2, (C.c_int32 * 8)(2, 4), 0, 0.05, 0.5)        # no sampling rounds
    assert lib.ss_width_create(C.byref(h), C.byref(bad)) == ssb.SS_ERR_ARG
    ctl = LibController([2, 4], 1, 0.05, 0.5)
    obs = ssb.ss_width_obs(1, 1, 1, 1, 1)
    assert lib.ss_width_observe(ctl.h, 3, C.byref(obs)) == ssb.SS_ERR_ARG     # not a candidate
    ctl.close()


@pytest.mark.parametrize("alpha,transfer", [(0.3, 40.0), (0.8, 40.0), (0.8, 0.5), (0.95, 40.0)])
def test_noiseless_simulation_finds_the_closed_form_optimum(alpha, transfer):
    # acceptance probability alpha per draft token: committed(q) = 1 + alpha + ... + alpha^q;
    # draft time 1 per token, compute 0.2 (q + 1), history transfer independent of q
    widths = [2, 4, 6, 8]
    committed = {q: sum(alpha ** i for i in range(q + 1)) for q in widths}
    t_round = {q: q * 1.0 + max(transfer, 0.2 * (q + 1)) + 0.3 for q in widths}
    best = min(widths, key=lambda q: (t_round[q] / committed[q], q))
    ctl = oracle.WidthController(widths, 2, 0.0, 0.5)
    q = None
    for _ in range(40):
        q = ctl.next()
        ctl.observe(q, q * 1.0, transfer, 0.2 * (q + 1), 0.3, committed[q])
    assert q == best
    # long transfers and good drafts favour wide verification, short transfers or poor drafts narrow
    if transfer > 10 and alpha >= 0.8:
        assert best >= 6
    if alpha <= 0.3 and transfer < 1:
        assert best == 2


def test_cohort_builder_against_oracle_and_a_hand_case():
    ssbuild.build()
    lib = ssb.load()

    def run(tasks, max_batch):
        arr = (ssb.ss_task * len(tasks))(*[ssb.ss_task(t["layer"], t["width"], t["dtype"], t["n_kv"], t["d_h"],
                                                      t["chunk_size"], i, t["hist_len"]) for i, t in enumerate(tasks)])
        order = (C.c_int32 * max(1, len(tasks)))()
        start = (C.c_int32 * (len(tasks) + 1))()
        n = lib.ss_cohort_build(arr, len(tasks), max_batch, order, start)
        return [list(order[start[c]:start[c + 1]]) for c in range(n)]

    base = dict(layer=3, width=4, dtype=0, n_kv=8, d_h=128, chunk_size=2048)
    # hand case: tasks 0,2,3 are compatible (sorted by length: 2,0,3), task 1 differs in width
    tasks = [dict(base, hist_len=500), dict(base, width=8, hist_len=900), dict(base, hist_len=700),
             dict(base, hist_len=100)]
    assert run(tasks, 16) == [[2, 0, 3], [1]] == oracle.cohort_build(tasks, 16)
    assert run(tasks, 2) == [[2, 0], [3], [1]] == oracle.cohort_build(tasks, 2)
    assert run([], 4) == []
    rng = random.Random(9)
    for _ in range(30):
        tasks = [dict(layer=rng.randint(0, 2), width=rng.choice([2, 4]), dtype=0, n_kv=rng.choice([4, 8]),
                      d_h=128, chunk_size=rng.choice([1024, 2048]), hist_len=rng.randint(0, 50))
                 for _ in range(rng.randint(1, 40))]
        mb = rng.randint(1, 8)
        got = run(tasks, mb)
        assert got == oracle.cohort_build(tasks, mb)
        assert sorted(i for c in got for i in c) == list(range(len(tasks)))     # every task exactly once
    assert lib.ss_cohort_build(None, 1, 1, None, None) == -1
    # the binding's wrappers marshal the same calls
    assert ssb.cohort_build(tasks, mb) == got
    wc = ssb.WidthController([2, 4], sample_rounds=1, switch_threshold=0.0, ema=1.0)
    for q, t in ((2, 1.0), (4, 1.2)):
        assert wc.next() == q
        wc.observe(q, 0.0, t, 0.0, 0.0, q)
    assert wc.next() == 4 and wc.estimate(4)[2] == pytest.approx(0.3)
    wc.close()
