"""Test helpers: run a workload through the CUDA library and through the CPU oracle.

The two sides share only the input tensors produced by the seeded generators.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_33184_b200 import inputs

# contract tolerances (bf16 outputs against the fp64 oracle)
TOL_MAX_O, TOL_MEAN_O, TOL_LSE = 1e-2, 1e-3, 1e-3


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().double().numpy()


def gen_case(cfg: inputs.VerifyConfig, lens, device, fill=None):
    """All tensors of one round on ``device``: Q, list of chunks, local KV, mask bits."""
    Q = inputs.make_q(cfg, device)
    K_loc, V_loc = inputs.make_local(cfg, device)
    bits = inputs.make_mask_bits(cfg, device)
    chunks = [inputs.make_history_chunk(cfg, j, lens, device, fill)
              for j in range(inputs.num_chunks(cfg, lens))]
    return Q, chunks, K_loc, V_loc, bits


def oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits, groups=None):
    """fp64 oracle on the same tensors.  ``groups`` = list of (b, kvh) to evaluate (default all);
    returns dict {(b, kvh): (O [G,T_q,d], LSE [G,T_q])}."""
    import oracle
    G = cfg.G
    mask = inputs.mask_bits_to_bool(bits, cfg.T_q).numpy()
    out = {}
    if groups is None:
        groups = [(b, h) for b in range(cfg.B) for h in range(cfg.H_kv)]
    for b, kvh in groups:
        ks, vs = [], []
        for K, V, vl in chunks:
            n = int(vl[b])
            if n:
                ks.append(f64(K[b, kvh, :n]))
                vs.append(f64(V[b, kvh, :n]))
        d = cfg.d
        kh = np.concatenate(ks) if ks else np.zeros((0, d))
        vh = np.concatenate(vs) if vs else np.zeros((0, d))
        assert kh.shape[0] == lens[b]
        q = f64(Q[b:b + 1, kvh * G:(kvh + 1) * G])
        O, L = oracle.verify_attention(q, [kh[None]], [vh[None]], f64(K_loc[b:b + 1, kvh:kvh + 1]),
                                       f64(V_loc[b:b + 1, kvh:kvh + 1]), mask[b:b + 1], cfg.scale)
        out[(b, kvh)] = (O[0], L[0])
    return out


def gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits, order=None, local_at=None):
    from paper_2609_33184_b200 import binding as ssb
    kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=Q.device)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=Q.device)
    order = list(range(len(chunks))) if order is None else order
    local_at = len(order) if local_at is None else local_at
    ctx.ss_verify_begin(Q, cfg.scale)
    for pos in range(len(order) + 1):
        if pos == local_at:
            ctx.ss_verify_local(K_loc, V_loc, kind, bits if cfg.mask == "tree" else None)
        if pos < len(order):
            K, V, vl = chunks[order[pos]]
            ctx.ss_verify_chunk(K, V, vl)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    return O, LSE


def make_ctx(cfg, flags=0, max_chunks=0, max_B=None, max_Lc=None):
    from paper_2609_33184_b200 import binding as ssb
    return ssb.Context(max_B or cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, max(cfg.T_q, 1),
                       max_Lc or cfg.L_c, max_chunks=max_chunks, flags=flags)


def compare(cfg, O, LSE, ref, strict=True):
    """Element-by-element comparison of the GPU result with the oracle groups in ``ref``."""
    G = cfg.G
    Og, Lg = f64(O), f64(LSE)
    worst = dict(max_o=0.0, mean_o=0.0, lse=0.0)
    for (b, kvh), (Or, Lr) in ref.items():
        og = Og[b, kvh * G:(kvh + 1) * G]
        lg = Lg[b, kvh * G:(kvh + 1) * G]
        assert np.isfinite(og).all(), f"non-finite O in group {(b, kvh)}"
        err = np.abs(og - Or)
        worst["max_o"] = max(worst["max_o"], err.max())
        worst["mean_o"] = max(worst["mean_o"], err.mean())
        fin = np.isfinite(Lr)
        assert np.array_equal(np.isfinite(lg), fin), f"LSE finiteness differs in {(b, kvh)}"
        if fin.any():
            worst["lse"] = max(worst["lse"], np.abs(lg[fin] - Lr[fin]).max())
        # contract tolerances hold for |O| <= 1 (the workloads); a bf16 output in [2^k, 2^(k+1)) has a
        # half-ulp of 2^(k-8), so for larger magnitudes the bound scales with max|O_ref|
        mag = max(1.0, float(np.abs(Or).max()))
        assert err.max() <= TOL_MAX_O * mag and err.mean() <= TOL_MEAN_O * mag, (b, kvh, err.max(), err.mean())
        if strict:
            # tighter than the contract: bf16 rounding of O (2^-9 relative) and of P leave a 4x margin
            rms = float(np.sqrt((Or ** 2).mean()))
            bound = 2.0 ** -7 * (np.abs(Or) + rms) + 1e-5
            assert (err <= bound).all(), (b, kvh, err.max(), rms, float((err / bound).max()))
            for g in range(G):
                a, r = og[g].ravel(), Or[g].ravel()
                if np.linalg.norm(r) > 0:
                    cos = a @ r / (np.linalg.norm(a) * np.linalg.norm(r) + 1e-300)
                    assert cos >= 0.9999, (b, kvh, g, cos)
    assert worst["lse"] <= TOL_LSE, worst
    return worst


def oracle_samples(cfg, lens, Q, chunks, K_loc, V_loc, bits, samples):
    """fp64 oracle for individual query rows.  samples = [(b, h_q, i), ...];
    returns {(b, h_q, i): (O [d], LSE)} - used at full workload sizes."""
    import oracle
    mask = inputs.mask_bits_to_bool(bits, cfg.T_q).numpy()
    cache = {}
    out = {}
    for b, h, i in samples:
        kvh = h // cfg.G
        if (b, kvh) not in cache:
            ks = [f64(K[b, kvh, :int(vl[b])]) for K, V, vl in chunks if int(vl[b])]
            vs = [f64(V[b, kvh, :int(vl[b])]) for K, V, vl in chunks if int(vl[b])]
            cache = {(b, kvh): (np.concatenate(ks) if ks else np.zeros((0, cfg.d)),
                                np.concatenate(vs) if vs else np.zeros((0, cfg.d)))}
        kh, vh = cache[(b, kvh)]
        O, L = oracle.verify_attention(f64(Q[b:b + 1, h:h + 1, i:i + 1]), [kh[None]], [vh[None]],
                                       f64(K_loc[b:b + 1, kvh:kvh + 1]), f64(V_loc[b:b + 1, kvh:kvh + 1]),
                                       mask[b:b + 1, i:i + 1], cfg.scale)
        out[(b, h, i)] = (O[0, 0, 0], L[0, 0, 0])
    return out


def compare_samples(O, LSE, ref):
    Og, Lg = O.detach().cpu().double().numpy(), LSE.detach().cpu().double().numpy()
    worst = dict(max_o=0.0, mean_o=0.0, lse=0.0)
    for (b, h, i), (Or, Lr) in ref.items():
        err = np.abs(Og[b, h, i] - Or)
        mag = max(1.0, float(np.abs(Or).max()))
        assert err.max() <= TOL_MAX_O * mag and err.mean() <= TOL_MEAN_O * mag, (b, h, i, err.max())
        rms = float(np.sqrt((Or ** 2).mean()))
        bound = 2.0 ** -7 * (np.abs(Or) + rms) + 1e-5
        assert (err <= bound).all(), (b, h, i, err.max(), rms)
        assert abs(Lg[b, h, i] - Lr) <= TOL_LSE, (b, h, i, Lg[b, h, i], Lr)
        worst["max_o"] = max(worst["max_o"], err.max())
        worst["mean_o"] = max(worst["mean_o"], err.mean())
        worst["lse"] = max(worst["lse"], abs(Lg[b, h, i] - Lr))
    return worst
