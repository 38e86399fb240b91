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
    r.B, r.H_q, r.H_kv, r.d, r.T_q, r.T_loc = cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, cfg.T_q
    r.L_c = K.shape[2] if K is not None else 0
    r.scale = cfg.scale
    r.Q = ssb.as_ss_tensor(Q)
    if K is not None:
        r.K, r.V = ssb.as_ss_tensor(K), ssb.as_ss_tensor(V)
        r.valid_len = vl.data_ptr() if vl is not None else None
    r.K_loc, r.V_loc = ssb.as_ss_tensor(K_loc), ssb.as_ss_tensor(V_loc)
    r.mask_kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
    r.mask_bits = bits.data_ptr() if cfg.mask == "tree" else None
    r.O, r.LSE = O.data_ptr(), LSE.data_ptr()
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
