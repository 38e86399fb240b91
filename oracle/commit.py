"""Commit-side data movement, as plain loops.

TEST INFRASTRUCTURE ONLY (see the package docstring).

commit_gather: at the end of a round the accepted candidates' KV joins the
committed prefix (Section 4.1: accepted candidates move into the Active Tail
and the rest of the speculative frontier is released).  The paper describes
this as a boundary move in a paged pool; here it is an explicit ordered copy
of cnt_b local rows to the committed buffer at offset dst_off_b, as raw 16-bit
words, every other word untouched.

migration_endpoint: Eq. 9, E = max(H, g * floor(max(0, C_r - T) / g)).
"""
import numpy as np


def commit_gather(k_loc, v_loc, accept_idx, accept_cnt, k_dst, v_dst, dst_off):
    """k_loc/v_loc [B, H_kv, T_loc, d] uint16; k_dst/v_dst [B, H_kv, cap, d] uint16 (copied).

    Rows whose index is outside [0, T_loc) or whose destination is outside
    [0, cap) are skipped.  Returns new (k_dst, v_dst).
    """
    k_out = np.array(k_dst, copy=True)
    v_out = np.array(v_dst, copy=True)
    B, H_kv, T_loc, _ = k_loc.shape
    cap = k_out.shape[2]
    for b in range(B):
        cnt = min(max(int(accept_cnt[b]), 0), accept_idx.shape[1])
        for k in range(cnt):
            src = int(accept_idx[b, k])
            dst = int(dst_off[b]) + k
            if not (0 <= src < T_loc) or not (0 <= dst < cap):
                continue
            for h in range(H_kv):
                k_out[b, h, dst, :] = k_loc[b, h, src, :]
                v_out[b, h, dst, :] = v_loc[b, h, src, :]
    return k_out, v_out


def migration_endpoint(H, C_r, T, g):
    """Eq. 9: end of the next batched offload interval [H, E)."""
    return max(H, g * (max(0, C_r - T) // g))


def cohort_build(tasks, max_batch):
    """Cohort batching (Section 4.2): group tasks with equal (layer, width, dtype, n_kv, d_h,
    chunk_size); inside a group order by decreasing history length (stable); groups keep the
    order of their first task; groups larger than max_batch are cut into consecutive pieces.
    tasks: list of dicts.  Returns a list of cohorts, each a list of task indices."""
    key = lambda t: (t["layer"], t["width"], t["dtype"], t["n_kv"], t["d_h"], t["chunk_size"])
    groups = {}
    for i, t in enumerate(tasks):
        groups.setdefault(key(t), []).append(i)
    out = []
    for idx in groups.values():                       # dicts keep insertion order
        idx = sorted(idx, key=lambda i: -tasks[i]["hist_len"])   # sorted() is stable
        out += [idx[k:k + max_batch] for k in range(0, len(idx), max_batch)]
    return out
