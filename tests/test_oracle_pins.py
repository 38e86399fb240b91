"""Pins for the CPU oracle: it is checked against things other than itself.

 * a pure-Python brute force (full score matrix, explicit loops, math.exp)
 * closed forms (equal keys, single key), invariants (shift, causality, GQA
   replication, one-hot values), the tree/chain path equivalence
 * scipy's logsumexp/softmax on unmasked cases
 * a hand-derived example of Eq. 13-14 and hand cases of Eq. 9 (tests/golden)
 * the chunked routine (Eq. 13-14) against the direct definition (Eq. 17)
"""
import math
import os
import random

import numpy as np
import pytest

import oracle
from oracle import streaming

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand_case(rng, B, H_q, H_kv, T_q, d, lens, tree=False, kscale=1.0):
    Q = rng.standard_normal((B, H_q, T_q, d))
    Kh = [kscale * rng.standard_normal((H_kv, n, d)) for n in lens]
    Vh = [rng.standard_normal((H_kv, n, d)) for n in lens]
    Kl = kscale * rng.standard_normal((B, H_kv, T_q, d))
    Vl = rng.standard_normal((B, H_kv, T_q, d))
    mask = np.zeros((B, T_q, T_q), dtype=bool)
    for b in range(B):
        if tree:
            par = [-1] + [int(rng.integers(0, i)) for i in range(1, T_q)]
            for i in range(T_q):
                j = i
                while j >= 0:
                    mask[b, i, j] = True
                    j = par[j]
        else:
            mask[b] = np.tril(np.ones((T_q, T_q), dtype=bool))
    return Q, Kh, Vh, Kl, Vl, mask


def _brute(Q, Kh, Vh, Kl, Vl, mask, scale):
    """Independent pure-Python implementation: explicit loops and math.exp only."""
    B, H_q, T_q, d = Q.shape
    H_kv = Kl.shape[1]
    G = H_q // H_kv
    O = [[[[0.0] * d for _ in range(T_q)] for _ in range(H_q)] for _ in range(B)]
    L = [[[-math.inf] * T_q for _ in range(H_q)] for _ in range(B)]
    for b in range(B):
        n = Kh[b].shape[1]
        for h in range(H_q):
            g = h // G
            for i in range(T_q):
                keys = [Kh[b][g, t] for t in range(n)] + [Kl[b, g, j] for j in range(T_q) if mask[b, i, j]]
                vals = [Vh[b][g, t] for t in range(n)] + [Vl[b, g, j] for j in range(T_q) if mask[b, i, j]]
                if not keys:
                    continue
                s = [scale * sum(float(Q[b, h, i, c]) * float(k[c]) for c in range(d)) for k in keys]
                mx = max(s)
                w = [math.exp(x - mx) for x in s]
                tot = sum(w)
                for c in range(d):
                    O[b][h][i][c] = sum(w[t] * float(vals[t][c]) for t in range(len(w))) / tot
                L[b][h][i] = mx + math.log(tot)
    return np.array(O), np.array(L)


@pytest.mark.parametrize("tree", [False, True])
@pytest.mark.parametrize("lens", [[0, 1], [17, 5], [3, 0]])
def test_brute_force_tiny(tree, lens):
    rng = np.random.default_rng(11 + sum(lens) + tree)
    case = _rand_case(rng, 2, 4, 2, 5, 8, lens, tree=tree, kscale=2.0)
    O, L = oracle.verify_attention(*case, scale=0.37)
    Ob, Lb = _brute(*case, scale=0.37)
    assert np.abs(O - Ob).max() < 1e-12
    assert np.abs(L - Lb).max() < 1e-12


def test_uniform_keys_closed_form():
    # all visible keys equal -> O = mean of visible V, LSE = scale*q.k + ln(n_vis);
    # with the chain mask n_vis(i) = len_b + i + 1 (pins the inclusive diagonal and ragged len)
    rng = np.random.default_rng(3)
    B, H_q, H_kv, T_q, d = 2, 4, 2, 5, 8
    lens = [7, 0]
    Q, Kh, Vh, Kl, Vl, mask = _rand_case(rng, B, H_q, H_kv, T_q, d, lens)
    kvec = rng.standard_normal((B, H_kv, d))
    Kh = [np.broadcast_to(kvec[b][:, None, :], (H_kv, lens[b], d)).copy() for b in range(B)]
    Kl = np.broadcast_to(kvec[:, :, None, :], (B, H_kv, T_q, d)).copy()
    scale = 0.5
    O, L = oracle.verify_attention(Q, Kh, Vh, Kl, Vl, mask, scale)
    for b in range(B):
        for h in range(H_q):
            g = h // (H_q // H_kv)
            for i in range(T_q):
                vis_v = np.concatenate([Vh[b][g], Vl[b, g, :i + 1]], axis=0)
                assert np.abs(O[b, h, i] - vis_v.mean(axis=0)).max() < 1e-12
                want = scale * Q[b, h, i] @ kvec[b, g] + math.log(lens[b] + i + 1)
                assert abs(L[b, h, i] - want) < 1e-12


def test_single_visible_key():
    rng = np.random.default_rng(4)
    Q, Kh, Vh, Kl, Vl, mask = _rand_case(rng, 1, 2, 1, 3, 4, [0])
    O, L = oracle.verify_attention(Q, Kh, Vh, Kl, Vl, mask, 0.7)
    for h in range(2):
        assert np.array_equal(O[0, h, 0], Vl[0, 0, 0])
        assert abs(L[0, h, 0] - 0.7 * Q[0, h, 0] @ Kl[0, 0, 0]) < 1e-14


def test_empty_row_is_zero():
    rng = np.random.default_rng(5)
    Q, Kh, Vh, Kl, Vl, mask = _rand_case(rng, 1, 2, 1, 3, 4, [0])
    mask[:] = False
    O, L = oracle.verify_attention(Q, Kh, Vh, Kl, Vl, mask, 1.0)
    assert np.all(O == 0) and np.all(L == -np.inf)


def test_shift_invariance_pins_lse():
    rng = np.random.default_rng(6)
    case = list(_rand_case(rng, 1, 4, 2, 4, 8, [9]))
    scale = 0.3
    O, L = oracle.verify_attention(*case, scale=scale)
    delta = rng.standard_normal(8)
    case2 = list(case)
    case2[1] = [k + delta for k in case[1]]
    case2[3] = case[3] + delta
    O2, L2 = oracle.verify_attention(*case2, scale=scale)
    assert np.abs(O - O2).max() < 1e-12
    assert np.abs((L2 - L) - scale * (case[0] @ delta)).max() < 1e-12


def test_causality_and_last_row_unmasked():
    rng = np.random.default_rng(7)
    Q, Kh, Vh, Kl, Vl, mask = _rand_case(rng, 1, 2, 1, 5, 8, [6])
    O, L = oracle.verify_attention(Q, Kh, Vh, Kl, Vl, mask, 0.4)
    Kl2, Vl2 = Kl.copy(), Vl.copy()
    Kl2[:, :, 3:] += 5.0
    Vl2[:, :, 3:] -= 2.0
    O2, L2 = oracle.verify_attention(Q, Kh, Vh, Kl2, Vl2, mask, 0.4)
    assert np.array_equal(O[:, :, :3], O2[:, :, :3]) and np.array_equal(L[:, :, :3], L2[:, :, :3])
    assert not np.array_equal(O[:, :, 3:], O2[:, :, 3:])
    # last chain row == unmasked attention over everything (scipy as the textbook routine)
    from scipy.special import logsumexp, softmax
    for h in range(2):
        k = np.concatenate([Kh[0][0], Kl[0, 0]], axis=0)
        v = np.concatenate([Vh[0][0], Vl[0, 0]], axis=0)
        s = 0.4 * (k @ Q[0, h, 4])
        assert abs(L[0, h, 4] - logsumexp(s)) < 1e-12
        assert np.abs(O[0, h, 4] - softmax(s) @ v).max() < 1e-12


def test_gqa_equals_mha_with_replicated_kv():
    rng = np.random.default_rng(8)
    B, H_q, H_kv, T_q, d = 1, 6, 2, 3, 4
    Q, Kh, Vh, Kl, Vl, mask = _rand_case(rng, B, H_q, H_kv, T_q, d, [5])
    O, L = oracle.verify_attention(Q, Kh, Vh, Kl, Vl, mask, 0.6)
    G = H_q // H_kv
    rep = lambda x, ax: np.repeat(x, G, axis=ax)  # consecutive q-heads share a kv-head
    O2, L2 = oracle.verify_attention(Q, [rep(k, 0) for k in Kh], [rep(v, 0) for v in Vh],
                                     rep(Kl, 1), rep(Vl, 1), mask, 0.6)
    assert np.array_equal(O, O2) and np.array_equal(L, L2)
    # and head h really uses kv-head h // G: perturbing kv-head 1 leaves heads 0..G-1 alone
    Kh2 = [k.copy() for k in Kh]
    Kh2[0][1] += 1.0
    O3, _ = oracle.verify_attention(Q, Kh2, Vh, Kl, Vl, mask, 0.6)
    assert np.array_equal(O3[:, :G], O[:, :G]) and not np.array_equal(O3[:, G:], O[:, G:])


def test_one_hot_values_give_probabilities():
    rng = np.random.default_rng(9)
    n, T_q = 6, 3
    d = n + T_q
    Q, Kh, Vh, Kl, Vl, mask = _rand_case(rng, 1, 1, 1, T_q, d, [n])
    eye = np.eye(d)
    Vh = [eye[None, :n]]
    Vl = eye[None, None, n:]
    O, L = oracle.verify_attention(Q, Kh, Vh, Kl, Vl, mask, 0.5)
    assert np.abs(O.sum(-1) - 1).max() < 1e-13
    assert np.all(O >= 0)
    for i in range(T_q):
        assert np.all(O[0, 0, i, n + i + 1:] == 0)      # invisible local keys get no mass
        s = 0.5 * np.concatenate([Kh[0][0], Kl[0, 0, :i + 1]]) @ Q[0, 0, i]
        assert np.abs(np.log(O[0, 0, i, :n + i + 1]) - (s - L[0, 0, i])).max() < 1e-12


def test_tree_row_equals_chain_on_root_path():
    rng = np.random.default_rng(10)
    B, H_q, H_kv, T_q, d = 1, 2, 1, 9, 4
    Q, Kh, Vh, Kl, Vl, mask = _rand_case(rng, B, H_q, H_kv, T_q, d, [5], tree=True)
    O, L = oracle.verify_attention(Q, Kh, Vh, Kl, Vl, mask, 0.5)
    for i in range(T_q):
        path = np.nonzero(mask[0, i])[0]          # ancestors in increasing index = root..i
        n = len(path)
        Qc = Q[:, :, path]
        cm = np.tril(np.ones((n, n), dtype=bool))[None]
        Oc, Lc = oracle.verify_attention(Qc, Kh, Vh, Kl[:, :, path], Vl[:, :, path], cm, 0.5)
        assert np.abs(Oc[0, :, -1] - O[0, :, i]).max() < 1e-12
        assert np.abs(Lc[0, :, -1] - L[0, :, i]).max() < 1e-12
    # perturbing a node outside row i's path does not change row i
    i = T_q - 1
    out = [j for j in range(T_q) if not mask[0, i, j]]
    if out:
        Kl2 = Kl.copy()
        Kl2[0, 0, out] += 3.0
        O2, _ = oracle.verify_attention(Q, Kh, Vh, Kl2, Vl, mask, 0.5)
        assert np.array_equal(O2[0, :, i], O[0, :, i])


# ---- Eq. 13 / Eq. 14 routine ------------------------------------------------

def _read_kv(path):
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split()
        out[k] = float(v)
    return out


def test_hand_example_eq13_eq14():
    g = _read_kv(os.path.join(GOLD, "merge_hand_example.txt"))
    q = np.array([[1.0]])
    k = np.array([[0.0], [math.log(2)], [math.log(3)]])
    v = np.array([[6.0], [12.0], [18.0]])
    A = streaming.chunk_partial(q, k[:2], v[:2], 1.0)
    Bp = streaming.chunk_partial(q, k[2:], v[2:], 1.0)
    for name, st in (("A", A), ("B", Bp), ("M", streaming.merge(A, Bp))):
        assert abs(st[0][0] - g[name + "_m"]) < 1e-15
        assert abs(st[1][0] - g[name + "_l"]) < 1e-15
        assert abs(st[2][0, 0] - g[name + "_a"]) < 1e-14
    o, lse = streaming.finalize(streaming.merge(A, Bp))
    assert abs(o[0, 0] - g["O"]) < 1e-14 and abs(lse[0] - g["LSE"]) < 1e-15
    # the direct definition gives the same numbers
    O, L = oracle.verify_attention(q[None, None], [k[None]], [v[None]], np.zeros((1, 1, 0, 1)),
                                   np.zeros((1, 1, 0, 1)), np.zeros((1, 1, 0), dtype=bool), 1.0)
    assert abs(O[0, 0, 0, 0] - g["O"]) < 1e-14 and abs(L[0, 0, 0] - g["LSE"]) < 1e-15


def test_merge_algebra():
    rng = np.random.default_rng(12)
    R, dv = 5, 3

    def rnd():
        return (rng.standard_normal(R) * 3, rng.random(R) + 0.1, rng.standard_normal((R, dv)))

    def close(x, y):
        return all(np.allclose(a, b, rtol=1e-13, atol=1e-13) for a, b in zip(x, y))

    x, y, z = rnd(), rnd(), rnd()
    e = streaming.IDENTITY(R, dv)
    assert close(streaming.merge(x, e), x) and close(streaming.merge(e, x), x)
    me = streaming.merge(e, e)
    assert np.all(me[0] == -np.inf) and np.all(me[1] == 0) and np.all(me[2] == 0)
    # states are equivalent when they describe the same (lse, a/l): compare finalised values
    f = streaming.finalize
    assert close(f(streaming.merge(x, y)), f(streaming.merge(y, x)))
    assert close(f(streaming.merge(streaming.merge(x, y), z)), f(streaming.merge(x, streaming.merge(y, z))))


@pytest.mark.parametrize("L_c", [1, 3, 13, 18])
def test_chunked_equals_direct(L_c):
    rng = np.random.default_rng(13)
    R, d, n, T = 6, 8, 13, 4
    q = rng.standard_normal((R, d))
    kh, vh = 2 * rng.standard_normal((n, d)), rng.standard_normal((n, d))
    kl, vl = 2 * rng.standard_normal((T, d)), rng.standard_normal((T, d))
    vis = rng.random((R, T)) < 0.6
    vis[:, 0] = True
    J = (n + L_c - 1) // L_c
    want_o = np.zeros((R, d))
    want_l = np.zeros(R)
    for r in range(R):
        k = np.concatenate([kh, kl[vis[r]]])
        v = np.concatenate([vh, vl[vis[r]]])
        o, l = oracle.verify_attention_rows(q[r:r + 1], k, v, 0.35)
        want_o[r], want_l[r] = o[0], l[0]
    pyr = random.Random(L_c)
    for trial in range(4):
        order = list(range(J))
        if trial:
            pyr.shuffle(order)
        local_at = [None, 0, J // 2, J][trial]
        o, l = oracle.streamed_verify_attention(q, kh, vh, kl, vl, vis, 0.35, L_c, order, local_at)
        assert np.abs(o - want_o).max() < 1e-12 and np.abs(l - want_l).max() < 1e-12


def test_chunk_with_no_visible_key_is_identity():
    rng = np.random.default_rng(14)
    q = rng.standard_normal((3, 4))
    k, v = rng.standard_normal((5, 4)), rng.standard_normal((5, 4))
    vis = np.ones((3, 5), dtype=bool)
    vis[1] = False
    m, l, a = streaming.chunk_partial(q, k, v, 1.0, vis)
    assert m[1] == -np.inf and l[1] == 0 and np.all(a[1] == 0)
    m0, l0, a0 = streaming.chunk_partial(q, k[:0], v[:0], 1.0)
    assert np.all(m0 == -np.inf) and np.all(l0 == 0)


# ---- commit gather / Eq. 9 ---------------------------------------------------

def test_commit_gather_against_python_loops():
    rng = np.random.default_rng(15)
    B, H, T, d, cap = 3, 2, 5, 4, 9
    kl = rng.integers(0, 65536, (B, H, T, d), dtype=np.uint16)
    vl = rng.integers(0, 65536, (B, H, T, d), dtype=np.uint16)
    kd = rng.integers(0, 65536, (B, H, cap, d), dtype=np.uint16)
    vd = rng.integers(0, 65536, (B, H, cap, d), dtype=np.uint16)
    idx = np.array([[0, 2, 4, 1, 3], [4, 3, 2, 1, 0], [1, 1, 1, 1, 1]], dtype=np.int32)
    cnt = np.array([3, 0, 5], dtype=np.int32)
    off = np.array([2, 7, 4], dtype=np.int32)
    ko, vo = oracle.commit_gather(kl, vl, idx, cnt, kd, vd, off)
    want_k, want_v = kd.copy(), vd.copy()
    want_k[0, :, 2], want_k[0, :, 3], want_k[0, :, 4] = kl[0, :, 0], kl[0, :, 2], kl[0, :, 4]
    want_v[0, :, 2], want_v[0, :, 3], want_v[0, :, 4] = vl[0, :, 0], vl[0, :, 2], vl[0, :, 4]
    for k in range(5):
        want_k[2, :, 4 + k] = kl[2, :, 1]
        want_v[2, :, 4 + k] = vl[2, :, 1]
    assert np.array_equal(ko, want_k) and np.array_equal(vo, want_v)
    # identity permutation is a plain copy; inputs are not modified
    ko2, _ = oracle.commit_gather(kl, vl, np.tile(np.arange(T, dtype=np.int32), (B, 1)),
                                  np.full(B, T, np.int32), kd, vd, np.zeros(B, np.int32))
    assert np.array_equal(ko2[:, :, :T], kl) and np.array_equal(ko2[:, :, T:], kd[:, :, T:])
    # out-of-range rows are skipped
    bad = idx.copy()
    bad[0, 1] = 9
    ko3, _ = oracle.commit_gather(kl, vl, bad, cnt, kd, vd, off)
    assert np.array_equal(ko3[0, :, 3], kd[0, :, 3]) and np.array_equal(ko3[0, :, 4], kl[0, :, 4])


def test_migration_endpoint_hand_cases():
    for line in open(os.path.join(GOLD, "migration_endpoint.txt")):
        if line.startswith("#") or not line.strip():
            continue
        H, C, T, g, E = map(int, line.split())
        assert oracle.migration_endpoint(H, C, T, g) == E
    rng = random.Random(1)
    for _ in range(500):
        g = rng.choice([1, 16, 128])
        H = g * rng.randrange(0, 20)
        C = H + rng.randrange(0, 3000)
        T = rng.randrange(0, 1024)
        E = oracle.migration_endpoint(H, C, T, g)
        assert E % g == 0 and H <= E <= max(H, C - T) and (E == H or C - T - E < g)
