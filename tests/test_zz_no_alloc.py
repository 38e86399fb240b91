"""ss_verify_round_static: a whole round for callers that cannot allocate device memory.

Plug-ins that do not own the process's memory pool, code in regions that must not synchronise
the device and start-up paths that run before an allocator exists cannot give the library a
workspace.  This entry point keeps its partial-state scratch inside the library's device
image.  The test calls it through the C ABI twice in a row (the second call finds the first
call's contents in the shared scratch) and checks each result against the regular
begin/chunk/local/finalize entry points.  This file is collected last on purpose.
"""
import ctypes as C

import pytest
import torch

from paper_2609_33184_b200 import inputs
from tests import util

DEV = "cuda:0"


def _static_round(ssb, cfg, Q, K, V, vl, K_loc, V_loc, bits, O, LSE, status=None):
    r = ssb.ss_static_round()
    r.B, r.H_q, r.H_kv, r.d, r.T_q = cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q
    r.T_loc = K_loc.shape[2] if K_loc is not None else 0
    r.L_c = K.shape[2] if K is not None else 0
    r.scale = cfg.scale
    r.Q = ssb.as_ss_tensor(Q)
    if K is not None:
        r.K, r.V = ssb.as_ss_tensor(K), ssb.as_ss_tensor(V)
        r.valid_len = vl.data_ptr() if vl is not None else None
    if K_loc is not None:
        r.K_loc, r.V_loc = ssb.as_ss_tensor(K_loc), ssb.as_ss_tensor(V_loc)
    r.mask_kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
    r.mask_bits = bits.data_ptr() if cfg.mask == "tree" else None
    r.O, r.LSE = O.data_ptr(), LSE.data_ptr() if LSE is not None else None
    r.status = status.data_ptr() if status is not None else None
    return ssb.load().ss_verify_round_static(C.byref(r), torch.cuda.current_stream().cuda_stream)


@pytest.mark.gpu
def test_static_round_matches_regular_entry_points_twice_in_a_row():
    from paper_2609_33184_b200 import binding as ssb
    cases = [inputs.VerifyConfig("n1", 0x71, 2, 8, 2, 128, 192, 6, 60, 192, mask="chain", k_mult=2.0),
             inputs.VerifyConfig("n2", 0x72, 1, 4, 1, 64, 320, 9, 320, 320, mask="tree")]
    for cfg in cases:            # two calls in a row on the shared scratch
        lens = inputs.history_lengths(cfg)
        Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
        K, V, vl = chunks[0]
        assert len(chunks) == 1
        O = torch.full((cfg.B, cfg.H_q, cfg.T_q, cfg.d), float("nan"), dtype=torch.bfloat16, device=DEV)
        LSE = torch.full((cfg.B, cfg.H_q, cfg.T_q), float("nan"), dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        st = _static_round(ssb, cfg, Q, K, V, vl, K_loc, V_loc, bits, O, LSE, status)
        assert st == ssb.SS_OK, st
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # the regular entry points on the same inputs
        ctx = util.make_ctx(cfg)
        O_ref, LSE_ref = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
        ctx.close()
        mag = max(1.0, float(O_ref.float().abs().max()))
        err = (O.float() - O_ref.float()).abs()
        assert float(err.max()) <= util.TOL_MAX_O * mag and float(err.mean()) <= util.TOL_MEAN_O * mag
        assert float((LSE - LSE_ref).abs().max()) <= util.TOL_LSE
        # and the oracle, so that both paths being wrong together cannot pass
        util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))


@pytest.mark.gpu
def test_static_round_optional_parts_after_a_larger_call():
    """The branches a plain round does not take - no history chunk, no local segment, no valid
    lengths, no status word - each right after a larger call, so that the partial states the
    larger call left in the shared scratch are there to be (wrongly) picked up."""
    import oracle
    from paper_2609_33184_b200 import binding as ssb
    big = inputs.VerifyConfig("big", 0x73, 2, 8, 2, 128, 256, 8, 256, 256)
    lens_big = inputs.history_lengths(big)
    Qb, chunks_b, Klb, Vlb, bits_b = util.gen_case(big, lens_big, DEV)
    Ob = torch.empty(big.B, big.H_q, big.T_q, big.d, dtype=torch.bfloat16, device=DEV)
    Lb = torch.empty(big.B, big.H_q, big.T_q, dtype=torch.float32, device=DEV)

    def dirty():   # a larger call that fills the scratch
        assert _static_round(ssb, big, Qb, *chunks_b[0], Klb, Vlb, bits_b, Ob, Lb) == ssb.SS_OK

    cfg = inputs.VerifyConfig("small", 0x74, 1, 4, 2, 128, 128, 4, 100, 100)
    lens = inputs.history_lengths(cfg)
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV, fill=0.0)   # finite padding: one case reads it
    K, V, vl = chunks[0]
    mask = inputs.mask_bits_to_bool(bits, cfg.T_q).numpy()
    f64 = util.f64
    G = cfg.G

    def check(O, LSE, k_hist, v_hist, kl, vl_, msk):
        Or, Lr = oracle.verify_attention(f64(Q), k_hist, v_hist, kl, vl_, msk, cfg.scale)
        ref = {(b, h): (Or[b, h * G:(h + 1) * G], Lr[b, h * G:(h + 1) * G]) for b in range(cfg.B)
               for h in range(cfg.H_kv)}
        util.compare(cfg, O, LSE, ref)

    hist = ([f64(K[b, :, :lens[b]]) for b in range(cfg.B)], [f64(V[b, :, :lens[b]]) for b in range(cfg.B)])
    none = ([f64(K[b, :, :0]) for b in range(cfg.B)], [f64(V[b, :, :0]) for b in range(cfg.B)])
    new = lambda: (torch.full((cfg.B, cfg.H_q, cfg.T_q, cfg.d), float("nan"), dtype=torch.bfloat16, device=DEV),
                   torch.full((cfg.B, cfg.H_q, cfg.T_q), float("nan"), dtype=torch.float32, device=DEV))
    # no history chunk (L_c = 0): local segment only, no status word
    dirty()
    O, LSE = new()
    assert _static_round(ssb, cfg, Q, None, None, None, K_loc, V_loc, bits, O, LSE) == ssb.SS_OK
    torch.cuda.synchronize()
    check(O, LSE, *none, f64(K_loc), f64(V_loc), mask)
    # no local segment (T_loc = 0): history only, ragged valid lengths, status word
    dirty()
    O, LSE = new()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert _static_round(ssb, cfg, Q, K, V, vl, None, None, bits, O, LSE, status) == ssb.SS_OK
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check(O, LSE, *hist, f64(K_loc[:, :, :0]), f64(V_loc[:, :, :0]), mask[:, :, :0])
    # no valid lengths (NULL: every token of the chunk counts) and no LSE
    dirty()
    O, _ = new()
    full = ([f64(K[b]) for b in range(cfg.B)], [f64(V[b]) for b in range(cfg.B)])
    assert _static_round(ssb, cfg, Q, K, V, None, K_loc, V_loc, bits, O, None) == ssb.SS_OK
    torch.cuda.synchronize()
    Or, _ = oracle.verify_attention(f64(Q), *full, f64(K_loc), f64(V_loc), mask, cfg.scale)
    assert float((O.double().cpu() - torch.from_numpy(Or)).abs().max()) <= util.TOL_MAX_O
    # an out-of-range valid length with no status word: clamped, the call still completes
    bad = torch.tensor([10 ** 6] * cfg.B, dtype=torch.int32, device=DEV)
    O, LSE = new()
    assert _static_round(ssb, cfg, Q, K, V, bad, K_loc, V_loc, bits, O, LSE) == ssb.SS_OK
    torch.cuda.synchronize()
    check(O, LSE, *full, f64(K_loc), f64(V_loc), mask)


def test_static_round_rejects_bad_shapes_on_the_host():
    # all decided before any device work, so this runs without a GPU too
    from paper_2609_33184_b200 import binding as ssb
    from paper_2609_33184_b200 import build as ssbuild
    ssbuild.build()
    call = ssb.load().ss_verify_round_static
    fake = ssb.ss_tensor(4096, 1 << 20, 1 << 16, 128)

    def make(**kw):
        r = ssb.ss_static_round()
        r.B, r.H_q, r.H_kv, r.d, r.T_q, r.T_loc, r.L_c, r.scale = 1, 8, 2, 128, 4, 4, 128, 1.0
        r.Q = r.K = r.V = r.K_loc = r.V_loc = fake
        r.O = 4096
        for k, v in kw.items():
            setattr(r, k, v)
        return r

    assert call(C.byref(make(mask_kind=7)), None) == ssb.SS_ERR_ARG             # unknown mask kind
    assert call(C.byref(make(T_loc=3)), None) == ssb.SS_ERR_ARG                 # chain with T_loc < T_q
    assert call(C.byref(make(mask_kind=ssb.SS_MASK_TREE_BITS)), None) == ssb.SS_ERR_ARG   # tree without bits
    assert call(C.byref(make(T_q=2048, T_loc=2048)), None) == ssb.SS_ERR_SHAPE  # T_q * G > 4096
    assert call(C.byref(make(B=1 << 30, H_q=1 << 10, H_kv=1 << 10)), None) == ssb.SS_ERR_SHAPE   # rows >= 2^31
    # products that overflow 32 bits must end in a clean rejection, not a wrapped split count
    assert call(C.byref(make(B=1 << 20, H_q=1 << 9, H_kv=1 << 9, T_q=2, T_loc=2)), None) == ssb.SS_ERR_CAPACITY
    assert call(C.byref(make(H_q=9)), None) == ssb.SS_ERR_SHAPE                 # H_q % H_kv
    assert call(C.byref(make(scale=0.0)), None) == ssb.SS_ERR_ARG


def test_static_round_rejects_rounds_beyond_its_scratch():
    # decided on the host before any device work, so this runs without a GPU too
    from paper_2609_33184_b200 import binding as ssb
    from paper_2609_33184_b200 import build as ssbuild
    ssbuild.build()
    r = ssb.ss_static_round()
    r.B, r.H_q, r.H_kv, r.d, r.T_q, r.T_loc, r.L_c, r.scale = 64, 32, 8, 128, 8, 8, 2048, 1.0
    fake = ssb.ss_tensor(4096, 1 << 20, 1 << 16, 128)
    r.Q = r.K = r.V = r.K_loc = r.V_loc = fake
    r.O = 4096
    assert ssb.load().ss_verify_round_static(C.byref(r), None) == ssb.SS_ERR_CAPACITY
    assert ssb.load().ss_verify_round_static(None, None) == ssb.SS_ERR_ARG
