"""Chunk-local states and their merge, written out literally (Eq. 13 and Eq. 14).

TEST INFRASTRUCTURE ONLY (see the package docstring).

This second routine exists only to test the invariances the paper claims for
the chunked reduction (Eq. 17): independence of chunk size, chunk order and of
where the local segment is merged.  It follows the paper's steps and notation:
accumulators (m, l, a) per query row start at (-inf, 0, 0); each chunk yields
(m_j, l_j, a_j); merging rescales both sides to the common maximum.

Reading of the paper for -inf arithmetic (Eq. 14 gives exp(-inf - -inf) when
both sides are empty): merging with an empty state is the identity, i.e. when
the common maximum is -inf both factors are taken as 0.
"""
import numpy as np


def IDENTITY(R, dv):
    return (np.full(R, -np.inf), np.zeros(R), np.zeros((R, dv)))


def chunk_partial(q, k, v, scale, visible=None):
    """Eq. 13 for one chunk.  q [R, d], k/v [n, d]; visible [R, n] bool or None (all).

    Returns (m_j [R], l_j [R], a_j [R, dv]).  Rows with no visible key give the
    identity (-inf, 0, 0).
    """
    R = q.shape[0]
    n = k.shape[0]
    dv = v.shape[1]
    m = np.full(R, -np.inf)
    l = np.zeros(R)
    a = np.zeros((R, dv))
    if n == 0:
        return m, l, a
    s = scale * (q @ k.T)
    if visible is not None:
        s = np.where(visible, s, -np.inf)
    for r in range(R):
        mr = s[r].max()
        if mr == -np.inf:
            continue
        p = np.exp(s[r] - mr)
        m[r] = mr
        l[r] = p.sum()
        a[r] = p @ v
    return m, l, a


def merge(x, y):
    """Eq. 14: (m, l, a) <- merge of two partial states."""
    m1, l1, a1 = x
    m2, l2, a2 = y
    mn = np.maximum(m1, m2)
    with np.errstate(invalid="ignore"):
        alpha = np.where(mn == -np.inf, 0.0, np.exp(m1 - mn))
        beta = np.where(mn == -np.inf, 0.0, np.exp(m2 - mn))
    return mn, alpha * l1 + beta * l2, alpha[:, None] * a1 + beta[:, None] * a2


def finalize(state):
    """O = a / l and LSE = m + ln l; empty rows give O = 0, LSE = -inf."""
    m, l, a = state
    with np.errstate(invalid="ignore", divide="ignore"):
        o = np.where(l[:, None] > 0, a / l[:, None], 0.0)
        lse = np.where(l > 0, m + np.log(l), -np.inf)
    return o, lse


def streamed_verify_attention(q, k_hist, v_hist, k_loc, v_loc, vis_loc, scale, L_c,
                              order=None, local_at=None):
    """One (request, kv-head) group processed the streamed way.

    q [R, d]; k_hist/v_hist [len, d]; k_loc/v_loc [T_loc, d]; vis_loc [R, T_loc] bool.
    The history is cut into chunks of L_c tokens (last one partial), taken in
    ``order`` (default arrival order); the local segment is merged after
    ``local_at`` history chunks (default: last, as in the paper).
    """
    n = k_hist.shape[0]
    J = (n + L_c - 1) // L_c
    order = list(range(J)) if order is None else list(order)
    local_at = J if local_at is None else local_at
    state = IDENTITY(q.shape[0], v_loc.shape[1])
    for pos in range(J + 1):
        if pos == local_at:
            state = merge(state, chunk_partial(q, k_loc, v_loc, scale, vis_loc))
        if pos < J:
            j = order[pos]
            sl = slice(j * L_c, min(n, (j + 1) * L_c))
            state = merge(state, chunk_partial(q, k_hist[sl], v_hist[sl], scale))
    return finalize(state)
