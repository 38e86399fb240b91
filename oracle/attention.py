"""Direct definition of the verification-attention result (Eq. 12, Section 4.2).

TEST INFRASTRUCTURE ONLY (see the package docstring).

For request b, query head h (kv-head h // G, consecutive query heads share a
kv-head) and candidate query i, the visible set is every committed history
token of the request plus the local candidate KV j allowed by the mask row
(chain: j <= i; tree: j is i or an ancestor of i).  The result is the plain
softmax-weighted mean of the visible values with scores scale * <q, k>, and
LSE = log(sum(exp(scores))) (natural log).  Everything is fp64; bf16 inputs are
widened exactly by the caller.  Two passes (max, then sums); no chunking and
no online rescaling - the streamed method reaches the same value up to
rounding order (Eq. 17), so the oracle is the definition itself.

A row with an empty visible set returns O = 0 and LSE = -inf.

Every part of this file is pinned by tests/test_oracle_pins.py (pure-Python
brute force, closed forms, invariants, a hand-derived example).
"""
import numpy as np


def verify_attention_rows(q, k_vis, v_vis, scale):
    """One (request, kv-head) group with a common visible set.

    q [R, d], k_vis [n, d], v_vis [n, d] (fp64).  Returns O [R, d], LSE [R].
    """
    R = q.shape[0]
    n = k_vis.shape[0]
    if n == 0:
        return np.zeros((R, v_vis.shape[1])), np.full(R, -np.inf)
    s = scale * (q @ k_vis.T)                    # [R, n]
    m = s.max(axis=1, keepdims=True)
    p = np.exp(s - m)
    l = p.sum(axis=1, keepdims=True)
    o = (p @ v_vis) / l
    return o, (m + np.log(l))[:, 0]


def verify_attention(Q, K_hist, V_hist, K_loc, V_loc, mask, scale):
    """Eq. 12 for a ragged batch.

    Q      [B, H_q, T_q, d]            fp64
    K_hist list of B arrays [H_kv, len_b, d] (len_b may be 0), same for V_hist
    K_loc  [B, H_kv, T_loc, d], V_loc likewise (T_loc may be 0)
    mask   [B, T_q, T_loc] bool - local visibility
    Returns O [B, H_q, T_q, d] fp64, LSE [B, H_q, T_q] fp64.
    """
    Q = np.asarray(Q, dtype=np.float64)
    B, H_q, T_q, _ = Q.shape
    H_kv = K_loc.shape[1]
    G = H_q // H_kv
    assert G * H_kv == H_q
    dv = V_loc.shape[-1]
    O = np.zeros((B, H_q, T_q, dv))
    LSE = np.full((B, H_q, T_q), -np.inf)
    for b in range(B):
        for h in range(H_q):
            kvh = h // G
            kh = np.asarray(K_hist[b][kvh], dtype=np.float64)
            vh = np.asarray(V_hist[b][kvh], dtype=np.float64)
            for i in range(T_q):
                vis = np.nonzero(mask[b, i])[0]
                k = np.concatenate([kh, np.asarray(K_loc[b, kvh][vis], dtype=np.float64)], axis=0)
                v = np.concatenate([vh, np.asarray(V_loc[b, kvh][vis], dtype=np.float64)], axis=0)
                o, lse = verify_attention_rows(Q[b, h, i:i + 1], k, v, scale)
                O[b, h, i] = o[0]
                LSE[b, h, i] = lse[0]
    return O, LSE
