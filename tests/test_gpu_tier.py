"""Commit-aware KV tiering on the GPU: many verification rounds with acceptance, commit-gather
into the on-GPU Active Tail, batched offload of [H, E) by Eq. 9 and streamed attention over
host history + tail + candidates, checked every round against the oracle (attention over the
true committed sequence, Eq. 9 boundaries, bit-exact placement of every committed token)."""

import numpy as np
import pytest
import torch

from paper_2609_33184_b200 import harness
import oracle
from paper_2609_33184_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_tiering_rounds_match_oracle_and_eq9():
    from paper_2609_33184_b200 import binding as ssb
    B, H_q, H_kv, d, T_q, L_c = 3, 8, 2, 128, 8, 32
    T, g, cap = 32, 16, 64
    max_tokens = 256
    cfg = inputs.VerifyConfig("tier", 0x7E, B, H_q, H_kv, d, L_c, T_q, 0, 0)
    host = [torch.full((max_tokens // L_c, 2, H_kv, L_c, d), float("nan"), dtype=torch.bfloat16).pin_memory()
            for _ in range(B)]
    tier = ssb.Tier(B, H_kv, d, L_c, T, g, cap, host, DEV)
    tier.reset([0] * B, [0] * B)
    ctx = ssb.Context(B, H_q, H_kv, d, T_q, T_q, max(L_c, cap))
    bufs = harness.stream_buffers(cfg, DEV, max_tokens // L_c)
    O = torch.empty(B, H_q, T_q, d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(B, H_q, T_q, dtype=torch.float32, device=DEV)
    bits = inputs.make_mask_bits(cfg, DEV)
    seq_k = [torch.zeros(H_kv, 0, d, dtype=torch.bfloat16) for _ in range(B)]   # the true committed KV
    seq_v = [torch.zeros(H_kv, 0, d, dtype=torch.bfloat16) for _ in range(B)]
    rng = np.random.default_rng(5)
    H_sim, C_sim = [0] * B, [0] * B
    saw_pending = False
    for rnd in range(36):
        Q = inputs.normal_bf16(100 + rnd, inputs.TID_Q, (B, H_q, T_q, d), device=DEV)
        K_loc = inputs.normal_bf16(100 + rnd, inputs.TID_KLOC, (B, H_kv, T_q, d), device=DEV)
        V_loc = inputs.normal_bf16(100 + rnd, inputs.TID_VLOC, (B, H_kv, T_q, d), device=DEV)
        cnt = [int(rng.integers(1, T_q + 1)) if b != 1 or rnd % 3 else 0 for b in range(B)]
        idx = torch.arange(T_q, dtype=torch.int32).repeat(B, 1).to(DEV)
        cnt_dev = torch.tensor(cnt, dtype=torch.int32, device=DEV)
        Hs, Cs, _, _ = tier.get()
        tk, tv, tK, tV = tier.tail()
        desc = harness.make_stream_desc(ssb, cfg, Hs, host, DEV, Q, K_loc, V_loc,
                                      bits, O, LSE, bufs)
        desc.tail_K, desc.tail_V, desc.tail_Lc, desc.tail_len = tK, tV, cap, tier.len_dev.data_ptr()
        desc.accept_idx, desc.accept_cnt = idx.data_ptr(), cnt_dev.data_ptr()
        desc.zero_off = tier.len_dev.data_ptr()          # append at the tail's current length
        desc.commit_k, desc.commit_v, desc.commit_cap = tk.data_ptr(), tv.data_ptr(), cap
        ctx.ss_stream_round(desc)
        st, dev_bits = ctx.ss_poll_status()
        assert st == 0, dev_bits
        # attention over the true committed sequence + candidates
        mask = inputs.mask_bits_to_bool(bits, T_q).numpy()
        Oo, Lo = oracle.verify_attention(util.f64(Q), [util.f64(k) for k in seq_k], [util.f64(v) for v in seq_v],
                                         util.f64(K_loc), util.f64(V_loc), mask, cfg.scale)
        err = np.abs(util.f64(O) - Oo)
        assert err.max() <= util.TOL_MAX_O * max(1.0, np.abs(Oo).max()) and err.mean() <= util.TOL_MEAN_O
        assert np.abs(util.f64(LSE) - Lo).max() <= util.TOL_LSE
        # commit: the accepted rows were appended to the tail by the round's commit-gather
        for b in range(B):
            seq_k[b] = torch.cat([seq_k[b], K_loc[b, :, :cnt[b]].cpu()], dim=1)
            seq_v[b] = torch.cat([seq_v[b], V_loc[b, :, :cnt[b]].cpu()], dim=1)
            C_sim[b] += cnt[b]
        tier.commit(cnt)
        moved = tier.migrate()
        Hn, Cn, En, _ = tier.get()
        assert Hn == H_sim and Cn == C_sim            # H does not move before the copy is confirmed
        E_sim = [oracle.migration_endpoint(H_sim[b], C_sim[b], T, g) for b in range(B)]
        assert En == E_sim and moved == sum(e > h for e, h in zip(E_sim, H_sim))
        saw_pending |= moved > 0
        tier.poll(wait=True)
        torch.cuda.synchronize()
        H_sim = E_sim
        Hn, Cn, En, cur = tier.get()
        assert Hn == H_sim and Cn == C_sim and En == H_sim
        tk, tv, _, _ = tier.tail()
        assert tier.len_dev.tolist() == [c - h for c, h in zip(C_sim, H_sim)]
        for b in range(B):
            assert H_sim[b] % g == 0 and 0 <= C_sim[b] - H_sim[b] <= cap
            assert C_sim[b] - H_sim[b] < T + g or C_sim[b] <= T
            # every committed token sits where the boundaries say, bit for bit
            hk = host[b][:, 0].permute(1, 0, 2, 3).reshape(H_kv, -1, d)[:, :H_sim[b]]
            hv = host[b][:, 1].permute(1, 0, 2, 3).reshape(H_kv, -1, d)[:, :H_sim[b]]
            n_tail = C_sim[b] - H_sim[b]
            full_k = torch.cat([hk, tk[b, :, :n_tail].cpu()], dim=1)
            full_v = torch.cat([hv, tv[b, :, :n_tail].cpu()], dim=1)
            assert torch.equal(full_k.view(torch.int16), seq_k[b].view(torch.int16))
            assert torch.equal(full_v.view(torch.int16), seq_v[b].view(torch.int16))
    assert saw_pending and max(H_sim) >= 4 * g
    assert tier.d2h_bytes() == sum(H_sim) * H_kv * d * 2 * 2
    tier.close()
    ctx.close()
