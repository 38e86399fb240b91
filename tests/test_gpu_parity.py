"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle,
element by element on the same seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2609_33184_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _ssb():
    from paper_2609_33184_b200 import binding
    return binding


def _run(cfg, lens=None, flags=0, fill=None, order=None, local_at=None, strict=True, kernel=None,
         max_chunks=0):
    lens = inputs.history_lengths(cfg) if lens is None else lens
    case = util.gen_case(cfg, lens, DEV, fill)
    ctx = util.make_ctx(cfg, flags=flags, max_chunks=max_chunks)
    O, LSE = util.gpu_case(ctx, cfg, *case, order=order, local_at=local_at)
    st, bits = ctx.ss_poll_status()
    assert st == 0 and bits == 0, (st, bits)
    if kernel and case[1]:
        assert ctx.last_chunk_kernel().startswith(kernel)
    ref = util.oracle_case(cfg, lens, *case)
    worst = util.compare(cfg, O, LSE, ref, strict=strict)
    ctx.close()
    return O, LSE, worst


@pytest.mark.parametrize("flags,kernel", [(0, "simt"), (8, "tcgen05-keys")])
def test_c1_tiny_chain_exact_config(flags, kernel):
    cfg = inputs.CONFIGS["c1_tiny_chain"]
    _run(cfg, flags=flags, kernel=kernel)


def _small(name, **kw):
    return inputs.scaled(inputs.CONFIGS[name], **kw)


def test_c2_shape_scaled_tensor_core_path():
    cfg = _small("c2_qwen3_8b", B=2, H_q=8, H_kv=2, L_c=256, len_lo=1000, len_hi=1000)
    _run(cfg, kernel="tcgen05")


def test_c3_shape_scaled_ragged_nan_padding():
    cfg = _small("c3_internlm25_7b_ragged", B=3, H_q=8, H_kv=2, L_c=256, len_lo=65, len_hi=700)
    _run(cfg, kernel="tcgen05")  # padding past valid_len is NaN by default


@pytest.mark.parametrize("flags", [0, 8])
def test_c4_shape_scaled_tree(flags):
    cfg = _small("c4_tree", B=2, H_q=10, H_kv=2, L_c=256, len_lo=600, len_hi=600)
    _run(cfg, flags=flags, kernel="tcgen05-keys" if flags else "tcgen05")


@pytest.mark.parametrize("flags", [0, 1, 4])   # keys-on-M, CUDA cores, rows-on-M
@pytest.mark.parametrize("n", [0, 1, 15, 16, 17, 63, 64, 65, 127, 129, 255, 256, 257])
def test_short_histories(flags, n):
    # short histories give the masks and the local segment real weight
    cfg = _small("c2_qwen3_8b", B=2, H_q=8, H_kv=2, L_c=128, len_lo=n, len_hi=n, k_mult=1.0)
    _run(cfg, flags=flags)


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("G", [1, 4, 5, 8])
@pytest.mark.parametrize("mask", ["chain", "tree"])
def test_group_sizes_and_head_dims(d, G, mask):
    cfg = inputs.VerifyConfig("v", 0x77 + G + d, 2, 2 * G, 2, d, 96, 7, 40, 300, mask=mask, k_mult=2.0)
    _run(cfg)
    if d == 128:
        _run(cfg, flags=8)   # keys-on-M kernel for every row count


@pytest.mark.parametrize("flags", [0, 8])
@pytest.mark.parametrize("T_q", [1, 2, 3, 5, 9, 16, 25, 33])
def test_query_counts_odd_rows(T_q, flags):
    # R = 4 T_q rows per kv-head: 4 .. 132 (one and two row groups, 4 / 8 / 16 softmax warps)
    cfg = inputs.VerifyConfig("v", 0x99 + T_q, 2, 8, 2, 128, 128, T_q, 100, 400, k_mult=2.0)
    _run(cfg, flags=flags, kernel="tcgen05-keys" if flags else "tcgen05")


@pytest.mark.parametrize("k_mult", [4.0, 8.0])
@pytest.mark.parametrize("flags", [0, 1, 4])
def test_peaked_softmax(k_mult, flags):
    cfg = inputs.VerifyConfig("v", 0x1234, 2, 8, 2, 128, 192, 8, 50, 700, k_mult=k_mult)
    _run(cfg, flags=flags)


@pytest.mark.parametrize("flags", [0, 1, 4, 8])
@pytest.mark.parametrize("T_q", [8, 20])
def test_one_hot_softmax_large_scores(flags, T_q):
    # K x 32: scaled scores of several hundred, the softmax is one-hot up to ties and the
    # reference maximum jumps by far more than the lazy-rescale thresholds on most tiles
    cfg = inputs.VerifyConfig("v", 0x2222 + T_q, 2, 8, 2, 128, 192, T_q, 300, 1000, k_mult=32.0)
    _run(cfg, flags=flags)


@pytest.mark.parametrize("flags", [0, 1, 4])
def test_equal_keys_closed_form_without_the_oracle(flags):
    # every history key and every local key of a kv-head equals one vector k: the softmax is
    # uniform over the visible keys, so O_i = mean of the visible V rows and
    # LSE_i = scale * q_i . k + ln(n_vis(i)) with n_vis(i) = len_b + i + 1 (inclusive chain mask)
    cfg = inputs.VerifyConfig("v", 0x3131, 3, 8, 2, 128, 192, 6, 0, 700)
    lens = [0, 385, 700]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV, fill=0.0)
    kvec = K_loc[:, :, :1, :].clone()                       # [B, H_kv, 1, d]
    K_loc.copy_(kvec.expand_as(K_loc))
    for K, V, vl in chunks:
        K.copy_(kvec.expand_as(K))
    ctx = util.make_ctx(cfg, flags=flags)
    O, LSE = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    ctx.close()
    G = cfg.G
    for b in range(cfg.B):
        for h in range(cfg.H_q):
            kvh = h // G
            vh = np.concatenate([util.f64(V[b, kvh, :int(vl[b])]) for K, V, vl in chunks] + [np.zeros((0, cfg.d))])
            assert vh.shape[0] == lens[b]
            for i in range(cfg.T_q):
                vis = np.concatenate([vh, util.f64(V_loc[b, kvh, :i + 1])])
                want_o = vis.mean(axis=0)
                want_lse = cfg.scale * float(util.f64(Q[b, h, i]) @ util.f64(kvec[b, kvh, 0])) + np.log(len(vis))
                got = util.f64(O[b, h, i])
                assert np.abs(got - want_o).max() <= 2.0 ** -7 * (np.abs(want_o).max() + 1e-3), (b, h, i)
                assert abs(float(LSE[b, h, i]) - want_lse) <= 1e-3, (b, h, i)


@pytest.mark.parametrize("flags", [0, 1])
def test_single_visible_key_returns_its_value_bit_exact(flags):
    # no history, chain mask: row 0 sees local key 0 only, so O = V_0 exactly (the weight is
    # exp2(0) = 1, the row sum 1) and LSE = scale * q . k_0
    cfg = inputs.VerifyConfig("v", 0x3232, 2, 8, 2, 128, 64, 5, 0, 0)
    lens = [0, 0]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=flags)
    O, LSE = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    ctx.close()
    for h in range(cfg.H_q):
        kvh = h // cfg.G
        assert torch.equal(O[:, h, 0].view(torch.int16), V_loc[:, kvh, 0].view(torch.int16))
        want = cfg.scale * (util.f64(Q[:, h, 0]) * util.f64(K_loc[:, kvh, 0])).sum(axis=1)
        assert np.abs(util.f64(LSE[:, h, 0]) - want).max() <= 1e-4


@pytest.mark.parametrize("flags", [0, 4])
def test_later_candidates_do_not_change_earlier_rows(flags):
    # causality of the chain mask: rewriting local K/V at positions j > i leaves row i
    # bit-identical (the kernels are deterministic)
    cfg = inputs.VerifyConfig("v", 0x3333, 2, 8, 2, 128, 128, 8, 200, 500)
    lens = inputs.history_lengths(cfg)
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=flags)
    O1, L1 = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    O1, L1 = O1.clone(), L1.clone()
    i = 3
    K2, V2 = K_loc.clone(), V_loc.clone()
    K2[:, :, i + 1:] = -K2[:, :, i + 1:] * 3
    V2[:, :, i + 1:] = V2[:, :, i + 1:] + 5
    O2, L2 = util.gpu_case(ctx, cfg, Q, chunks, K2, V2, bits)
    ctx.close()
    assert torch.equal(O1[:, :, :i + 1].view(torch.int16), O2[:, :, :i + 1].view(torch.int16))
    assert torch.equal(L1[:, :, :i + 1], L2[:, :, :i + 1])
    assert not torch.equal(O1[:, :, i + 1:], O2[:, :, i + 1:])


def test_tree_row_equals_chain_over_its_root_path():
    # a tree node sees the history and its ancestors-or-self: row i of a tree round equals the
    # LAST row of a chain round whose candidates are the path root -> i (other subtrees are
    # invisible to it)
    import dataclasses
    cfg = inputs.VerifyConfig("v", 0x3434, 1, 8, 2, 128, 128, 24, 300, 300, mask="tree", k_mult=2.0)
    lens = [300]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg)
    O_t, L_t = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    ctx.close()
    vis = inputs.mask_bits_to_bool(bits, cfg.T_q)[0]          # [T_q, T_loc]
    for i in (0, 7, 23):
        path = [j for j in range(cfg.T_q) if bool(vis[i, j])]
        assert path[-1] == i and path[0] == 0
        ccfg = dataclasses.replace(cfg, T_q=len(path), mask="chain")
        idx = torch.tensor(path, device=DEV)
        Qc = Q[:, :, idx].contiguous()
        Kc, Vc = K_loc[:, :, idx].contiguous(), V_loc[:, :, idx].contiguous()
        cctx = util.make_ctx(ccfg)
        O_c, L_c = util.gpu_case(cctx, ccfg, Qc, chunks, Kc, Vc, inputs.make_mask_bits(ccfg, DEV))
        cctx.close()
        d = (O_t[:, :, i].float() - O_c[:, :, -1].float()).abs().max().item()
        assert d <= 2.0 ** -7 * max(1.0, O_t[:, :, i].float().abs().max().item()), (i, d)
        assert (L_t[:, :, i] - L_c[:, :, -1]).abs().max().item() <= 1e-4, i


def test_gqa_equals_mha_with_replicated_kv_heads():
    # consecutive query heads share a kv-head: replicating every kv-head G times and running
    # with H_kv = H_q gives the same result
    import dataclasses
    cfg = inputs.VerifyConfig("v", 0x3535, 2, 8, 2, 128, 128, 6, 200, 450, k_mult=2.0)
    lens = inputs.history_lengths(cfg)
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg)
    O_g, L_g = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    ctx.close()
    G = cfg.G
    rep = lambda t: t.repeat_interleave(G, dim=1).contiguous()
    mcfg = dataclasses.replace(cfg, H_kv=cfg.H_q)
    mchunks = [(rep(K), rep(V), vl) for K, V, vl in chunks]
    mctx = util.make_ctx(mcfg)
    O_m, L_m = util.gpu_case(mctx, mcfg, Q, mchunks, rep(K_loc), rep(V_loc), bits)
    mctx.close()
    assert (O_g.float() - O_m.float()).abs().max().item() <= 2.0 ** -7 * max(1.0, O_g.float().abs().max().item())
    assert (L_g - L_m).abs().max().item() <= 1e-4


def test_needle_keys_and_rescale_path():
    # one key per request with a score ~ +20 above the rest, placed late in the history, so the
    # running maximum jumps by more than the rescale threshold after many tiles
    cfg = inputs.VerifyConfig("v", 0x4321, 2, 8, 2, 128, 256, 8, 900, 900)
    lens = [900, 900]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    for b, (j, t) in enumerate([(3, 100), (2, 255)]):
        K = chunks[j][0]
        for h in range(cfg.H_kv):
            q = Q[b, h * cfg.G].float().mean(0)
            K[b, h, t] = (q / q.norm() * 30.0).to(torch.bfloat16)
    # and one needle in the local segment
    K_loc[0, 0, 2] = (Q[0, 0, 5].float() / Q[0, 0, 5].float().norm() * 25.0).to(torch.bfloat16)
    for flags in (0, 1, 4):
        ctx = util.make_ctx(cfg, flags=flags)
        O, LSE = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
        ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits)
        util.compare(cfg, O, LSE, ref)
        ctx.close()


def test_empty_chunks_reverse_order_local_first():
    cfg = inputs.VerifyConfig("v", 0x55, 3, 8, 2, 128, 128, 6, 0, 600)
    lens = [600, 0, 130]
    n = inputs.num_chunks(cfg, lens)
    O1, L1, _ = _run(cfg, lens=lens)
    O2, L2, _ = _run(cfg, lens=lens, order=list(range(n))[::-1], local_at=0)
    assert (O1.float() - O2.float()).abs().max() < 2e-2
    assert (L1 - L2).abs().max() < 1e-4


def test_more_chunk_calls_than_partial_sets_folds():
    cfg = inputs.VerifyConfig("v", 0x56, 2, 8, 2, 128, 64, 5, 500, 700)
    _run(cfg, max_chunks=3)


@pytest.mark.parametrize("flags", [0, 1, 4])
def test_deterministic_bitwise(flags):
    cfg = inputs.VerifyConfig("v", 0x57, 2, 8, 2, 128, 256, 8, 300, 900)
    lens = inputs.history_lengths(cfg)
    case = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=flags)
    O1, L1 = util.gpu_case(ctx, cfg, *case)
    O1, L1 = O1.clone(), L1.clone()
    O2, L2 = util.gpu_case(ctx, cfg, *case)
    assert torch.equal(O1.view(torch.int16), O2.view(torch.int16)) and torch.equal(L1, L2)
    ctx.close()


@pytest.mark.parametrize("flags,T_q,B,H_q,k_mult", [
    (0, 8, 16, 32, 2.0), (0, 24, 16, 32, 2.0), (0, 40, 16, 32, 2.0), (8, 24, 16, 32, 2.0),
    (0, 64, 4, 40, 1.0)])  # the last: 320 rows per kv-head (row tiles of 128 + 128 + 64), the tree workload's score spread
def test_many_rounds_stay_bitwise_identical_and_never_stall(flags, T_q, B, H_q, k_mult):
    # Hand-off races between the TMA, MMA and softmax roles show up as a rare wrong tile or as
    # a bounded wait that runs out (status word), typically once in 10^5 CTAs and only when the
    # SMs are full (two CTAs per SM, overlapping launches): repeat rounds of a launch shape
    # that fills the GPU and compare every round with the first, bit for bit.
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x5A + T_q, B, H_q, 8, 128, 1024, T_q, 3000, 4096, k_mult=k_mult)
    lens = inputs.history_lengths(cfg)
    case = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=flags | ssb.SS_FLAG_OVERLAP_CHUNKS)
    O1, L1 = util.gpu_case(ctx, cfg, *case)   # the first launches of this context
    O1, L1 = O1.clone(), L1.clone()
    for i in range(400):
        O2, L2 = util.gpu_case(ctx, cfg, *case)
        if i % 50 == 49:
            assert ctx.ss_poll_status() == (0, 0)
            assert torch.equal(O1.view(torch.int16), O2.view(torch.int16)) and torch.equal(L1, L2)
    ref = util.oracle_case(cfg, lens, *case, groups=[(0, 0), (B - 1, 7)])
    util.compare(cfg, O1, L1, ref)
    ctx.close()


def test_simt_and_tensor_core_kernels_agree():
    cfg = inputs.VerifyConfig("v", 0x58, 2, 16, 4, 128, 320, 8, 100, 1200, k_mult=2.0)
    lens = inputs.history_lengths(cfg)
    case = util.gen_case(cfg, lens, DEV)
    outs = []
    for flags, name in ((0, "tcgen05-keys"), (1, "simt"), (4, "tcgen05")):
        ctx = util.make_ctx(cfg, flags=flags)
        O, L = util.gpu_case(ctx, cfg, *case)
        assert ctx.last_chunk_kernel() == name
        outs.append((O.float(), L))
        ctx.close()
    for k in (1, 2):
        assert (outs[0][0] - outs[k][0]).abs().max() < 2e-2
        assert (outs[0][1] - outs[k][1]).abs().max() < 1e-4


def test_overlap_flag_same_result():
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x59, 4, 16, 4, 128, 512, 8, 1500, 2500)
    lens = inputs.history_lengths(cfg)
    case = util.gen_case(cfg, lens, DEV)
    torch.cuda.synchronize()
    res = []
    for flags in (0, ssb.SS_FLAG_OVERLAP_CHUNKS):
        ctx = util.make_ctx(cfg, flags=flags)
        for _ in range(3):
            O, L = util.gpu_case(ctx, cfg, *case)
        res.append((O.clone(), L.clone()))
        st, bits = ctx.ss_poll_status()
        assert st == 0
        ctx.close()
    assert torch.equal(res[0][0].view(torch.int16), res[1][0].view(torch.int16))
    assert torch.equal(res[0][1], res[1][1])
    ref = util.oracle_case(cfg, lens, *case, groups=[(0, 0), (3, 3)])
    util.compare(cfg, res[1][0], res[1][1], ref)


def test_strided_inputs():
    # K/V chunks that are views into a larger buffer (token stride > d, head stride padded)
    cfg = inputs.VerifyConfig("v", 0x5A, 2, 8, 2, 128, 128, 4, 128, 128)
    lens = [128, 128]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    K, V, vl = chunks[0]
    big_k = torch.full((2, 2, 160, 256), float("nan"), dtype=torch.bfloat16, device=DEV)
    big_v = torch.full_like(big_k, float("nan"))
    big_k[:, :, 16:144, 128:] = K
    big_v[:, :, 16:144, :128] = V
    Kv, Vv = big_k[:, :, 16:144, 128:], big_v[:, :, 16:144, :128]
    for flags in (0, 1, 4):
        ctx = util.make_ctx(cfg, flags=flags)
        O, L = util.gpu_case(ctx, cfg, Q, [(Kv, Vv, vl)], K_loc, V_loc, bits)
        ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits)
        util.compare(cfg, O, L, ref)
        ctx.close()


@pytest.mark.parametrize("d", [64, 128])
def test_token_major_layouts(d):
    # K/V (and Q, local KV) stored token-major, [B, tokens, heads, d], passed as permuted views:
    # the head stride is then smaller than the token stride
    cfg = inputs.VerifyConfig("v", 0x5B + d, 2, 8, 2, d, 256, 12, 300, 700, k_mult=2.0)
    lens = [700, 300]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)

    def token_major(t):     # same values, [B, T, H, d] memory, [B, H, T, d] view
        return t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)

    chunks_tm = [(token_major(K), token_major(V), vl) for K, V, vl in chunks]
    assert chunks_tm[0][0].stride(1) < chunks_tm[0][0].stride(2)
    ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits)
    for flags in (0, 1, 4, 8):
        ctx = util.make_ctx(cfg, flags=flags)
        O, L = util.gpu_case(ctx, cfg, token_major(Q), chunks_tm, token_major(K_loc), token_major(V_loc), bits)
        assert ctx.ss_poll_status() == (0, 0)
        util.compare(cfg, O, L, ref)
        ctx.close()


def test_bad_valid_len_sets_status_and_is_clamped():
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x5B, 2, 8, 2, 128, 128, 4, 128, 128)
    lens = [128, 128]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    K, V, vl = chunks[0]
    bad = torch.tensor([500, -3], dtype=torch.int32, device=DEV)
    ctx = util.make_ctx(cfg)
    util.gpu_case(ctx, cfg, Q, [(K, V, bad)], K_loc, V_loc, bits)
    st, b = ctx.ss_poll_status()
    assert st == ssb.SS_ERR_DEVICE_FLAG and b & ssb.SS_DEV_BAD_VALID_LEN
    st, b = ctx.ss_poll_status()
    assert st == 0 and b == 0  # cleared
    ctx.close()


def test_hinted_chunk_calls_match_unhinted():
    # host copies of valid_len only change the split sizes, never the result's correctness
    cfg = inputs.VerifyConfig("v", 0x5C, 6, 8, 2, 128, 512, 8, 10, 1500)
    lens = [1500, 10, 700, 513, 0, 1024]
    case = util.gen_case(cfg, lens, DEV)
    Q, chunks, K_loc, V_loc, bits = case
    ref = util.oracle_case(cfg, lens, *case)
    from paper_2609_33184_b200 import harness
    hints = harness.host_valid(cfg, lens, len(chunks))
    ssb = _ssb()
    ctx = util.make_ctx(cfg)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    harness.run_round(ctx, ssb, cfg, Q, chunks, K_loc, V_loc, bits, O, LSE, hints=hints)
    torch.cuda.synchronize()
    st, dev_bits = ctx.ss_poll_status()
    assert st == 0, dev_bits
    util.compare(cfg, O, LSE, ref)
    ctx.close()


@pytest.mark.parametrize("flags", [0, 1, 4])
@pytest.mark.parametrize("max_chunks", [0, 2])
def test_hinted_calls_skip_requests_without_tokens(flags, max_chunks):
    # With a host copy of the lengths, requests that have no tokens in a chunk get no thread
    # blocks in that call and the merge skips that call's partial set for them - also after the
    # sets were folded (max_chunks = 2 forces folds), with a NaN-poisoned workspace (a skipped
    # slot holds whatever an earlier round left there), with a chunk nobody has tokens in, and
    # through an exported state.
    from paper_2609_33184_b200 import harness
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x5E, 6, 8, 2, 128, 256, 12, 0, 1300, k_mult=2.0)
    lens = [900, 0, 300, 1300, 0, 257]
    case = util.gen_case(cfg, lens, DEV, fill=float("nan"))
    Q, chunks, K_loc, V_loc, bits = case
    ref = util.oracle_case(cfg, lens, *case)
    hints = harness.host_valid(cfg, lens, len(chunks))
    empty = (torch.zeros_like(chunks[0][0]), torch.zeros_like(chunks[0][1]), torch.zeros_like(chunks[0][2]))
    ctx = util.make_ctx(cfg, flags=flags, max_chunks=max_chunks)
    ctx.workspace[4096:].view(torch.float32)[:] = float("nan")   # past the status word and trace region
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ml = torch.empty(cfg.B * cfg.H_q * cfg.T_q, 2, dtype=torch.float32, device=DEV)
    a = torch.empty(cfg.B * cfg.H_q * cfg.T_q, cfg.d, dtype=torch.float32, device=DEV)
    for use_export in (False, True):
        ctx.ss_verify_begin(Q, cfg.scale)
        for j, (K, V, vl) in enumerate(chunks):
            ctx.ss_verify_chunk_hinted(K, V, vl, hints[j])
            if j == 1:
                ctx.ss_verify_chunk_hinted(*empty, [0] * cfg.B)       # nobody has tokens here
        if use_export:                                                  # state out, round dropped, state back in
            ctx.ss_verify_export_state(ml, a)
            ctx.ss_verify_abort()
            ctx.ss_verify_begin(Q, cfg.scale)
            ctx.ss_verify_import_state(ml, a)
        ctx.ss_verify_local(K_loc, V_loc)
        ctx.ss_verify_finalize(O, LSE)
        torch.cuda.synchronize()
        assert ctx.ss_poll_status() == (0, 0)
        util.compare(cfg, O, LSE, ref)
    ctx.close()


def test_hinted_calls_with_a_batch_of_more_than_64_requests():
    # request lists and the merge's "absent" bits cover batches of up to 256 requests
    from paper_2609_33184_b200 import harness
    ssb = _ssb()
    B = 130
    cfg = inputs.VerifyConfig("v", 0x5F, B, 4, 2, 128, 128, 4, 0, 400, k_mult=2.0)
    lens = [(37 * b) % 401 if b % 3 else 0 for b in range(B)]
    lens[129] = 400
    case = util.gen_case(cfg, lens, DEV, fill=float("nan"))
    Q, chunks, K_loc, V_loc, bits = case
    hints = harness.host_valid(cfg, lens, len(chunks))
    ctx = util.make_ctx(cfg)
    ctx.workspace[8192:].view(torch.float32)[:] = float("nan")
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    harness.run_round(ctx, ssb, cfg, Q, chunks, K_loc, V_loc, bits, O, LSE, hints=hints)
    torch.cuda.synchronize()
    assert ctx.ss_poll_status() == (0, 0)
    groups = [(0, 0), (1, 1), (64, 0), (65, 1), (127, 0), (128, 1), (129, 0), (129, 1)]
    util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, *case, groups=groups))
    assert torch.isfinite(O.float()).all()
    ctx.close()


@pytest.mark.parametrize("seed", range(24))
def test_random_ragged_shapes(seed):
    # seeded sweep over batch, GQA group, candidate count, head dim, chunk size, ragged lengths,
    # mask kind and kernel choice; short and peaked cases give the masks real weight
    import random
    rng = random.Random(1000 + seed)
    d = rng.choice([64, 128, 128])
    H_kv = rng.choice([1, 2, 3])
    G = rng.choice([1, 2, 4, 5, 8])
    T_q = rng.randint(1, 12)
    B = rng.randint(1, 4)
    L_c = rng.choice([64, 96, 128, 200, 256, 448])
    hi = rng.choice([0, 40, 300, 900])
    mask = rng.choice(["chain", "tree"])
    cfg = inputs.VerifyConfig("rnd", 0xA000 + seed, B, H_kv * G, H_kv, d, L_c, T_q, 0, hi, mask=mask,
                              k_mult=rng.choice([1.0, 2.0, 6.0]))
    lens = [rng.randint(0, hi) for _ in range(B)]
    flags = rng.choice([0, 0, 1, 4, 8]) | rng.choice([0, 2])
    n = inputs.num_chunks(cfg, lens)
    order = list(range(n))
    rng.shuffle(order)
    _run(cfg, lens=lens, flags=flags, order=order, local_at=rng.randint(0, n), max_chunks=rng.choice([0, 2]))


@pytest.mark.parametrize("page_size,flags", [(128, 0), (128, 4), (64, 0), (64, 8), (64, 4), (32, 0), (32, 4), (16, 0),
                                             (16, 4), (16, 8), (8, 0), (8, 4), (4, 0), (128, 1), (16, 1), (256, 0), (256, 4)])
def test_paged_chunks_match_contiguous_and_oracle(page_size, flags):
    # the chunk's tokens live in shuffled pages of a pool; same result as the gathered chunk
    ssb = _ssb()
    cfg = inputs.VerifyConfig("pg", 0x5D + page_size, 3, 8, 2, 128, 512, 6, 40, 1500, k_mult=2.0)
    lens = [1500, 40, 1024]
    case = util.gen_case(cfg, lens, DEV, fill=float("nan"))
    Q, chunks, K_loc, V_loc, bits = case
    ref = util.oracle_case(cfg, lens, *case)
    ppr = cfg.L_c // page_size
    g = torch.Generator().manual_seed(page_size)
    ctx = util.make_ctx(cfg, flags=flags)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    for K, V, vl in chunks:
        n_pages = cfg.B * ppr + 3                      # a few unused pages
        perm = torch.randperm(n_pages, generator=g)[:cfg.B * ppr].to(torch.int32)
        table = perm.view(cfg.B, ppr).contiguous()
        K_pool = torch.full((n_pages, cfg.H_kv, page_size, cfg.d), float("nan"), dtype=torch.bfloat16, device=DEV)
        V_pool = torch.full_like(K_pool, float("nan"))
        Kp = K.view(cfg.B, cfg.H_kv, ppr, page_size, cfg.d).permute(0, 2, 1, 3, 4).reshape(-1, cfg.H_kv, page_size, cfg.d)
        Vp = V.view(cfg.B, cfg.H_kv, ppr, page_size, cfg.d).permute(0, 2, 1, 3, 4).reshape(-1, cfg.H_kv, page_size, cfg.d)
        K_pool[table.view(-1).long()] = Kp
        V_pool[table.view(-1).long()] = Vp
        ctx.ss_verify_chunk_paged(K_pool, V_pool, table.to(DEV), vl, vl.tolist())
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    st, dev_bits = ctx.ss_poll_status()
    assert st == 0, dev_bits
    # pages of 8 tokens and more are gathered into the tensor-core kernels' tiles
    expect = "simt" if (flags & 1 or page_size < 8) else ("tcgen05" if flags & 4 else "tcgen05-keys")
    assert ctx.last_chunk_kernel() == expect, (ctx.last_chunk_kernel(), expect)
    util.compare(cfg, O, LSE, ref)
    ctx.close()


def test_paged_chunk_bad_page_id_is_flagged():
    ssb = _ssb()
    cfg = inputs.VerifyConfig("pg", 0x5E, 2, 8, 2, 128, 256, 4, 256, 256)
    lens = [256, 256]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    K, V, vl = chunks[0]
    table = torch.tensor([[0, 7], [1, -2]], dtype=torch.int32, device=DEV)      # pool has 2 pages
    K_pool = K.view(2, 2, 2, 128, 128)[:, :, 0].contiguous()
    V_pool = V.view(2, 2, 2, 128, 128)[:, :, 0].contiguous()
    for flags in (0, 1):
        ctx = util.make_ctx(cfg, flags=flags)
        O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
        ctx.ss_verify_begin(Q, cfg.scale)
        ctx.ss_verify_chunk_paged(K_pool, V_pool, table, None)
        ctx.ss_verify_finalize(O, None)
        st, dev_bits = ctx.ss_poll_status()
        assert st == ssb.SS_ERR_DEVICE_FLAG and dev_bits & ssb.SS_DEV_BAD_PAGE
        assert torch.isfinite(O.float()).all()
        ctx.close()


@pytest.mark.parametrize("flags", [0, 4, 1])
def test_small_pages_bad_ids_and_unused_table_entries(flags):
    # pages of 16 tokens: a bad id among the pages that hold valid tokens is flagged and reads as
    # zeros; entries past the valid length hold garbage ids and must never be looked up
    ssb = _ssb()
    cfg = inputs.VerifyConfig("pg", 0x60, 2, 8, 2, 128, 256, 4, 100, 100)
    lens = [100, 37]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    K, V, vl = chunks[0]
    ps, ppr = 16, 16
    Kp = K.view(2, 2, ppr, ps, 128).permute(0, 2, 1, 3, 4).reshape(-1, 2, ps, 128).contiguous()
    Vp = V.view(2, 2, ppr, ps, 128).permute(0, 2, 1, 3, 4).reshape(-1, 2, ps, 128).contiguous()
    table = torch.arange(2 * ppr, dtype=torch.int32).view(2, ppr).clone()
    table[0, 7:] = 1 << 30          # request 0 has 100 tokens = 7 pages (6 full + 4 tokens): rest unused
    table[1, 3:] = -5               # request 1 has 37 tokens = 3 pages
    table = table.to(DEV)
    ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits)
    ctx = util.make_ctx(cfg, flags=flags)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunk_paged(Kp, Vp, table, vl, vl.tolist())
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_finalize(O, LSE)
    assert ctx.ss_poll_status() == (0, 0)
    util.compare(cfg, O, LSE, ref)
    # now break a page that is in use
    table[0, 2] = 2 * ppr + 9
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunk_paged(Kp, Vp, table, vl, vl.tolist())
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_finalize(O, LSE)
    st, dev_bits = ctx.ss_poll_status()
    assert st == ssb.SS_ERR_DEVICE_FLAG and dev_bits & ssb.SS_DEV_BAD_PAGE
    assert torch.isfinite(O.float()).all()
    ctx.close()


@pytest.mark.parametrize("flags", [0, 4, 1])
def test_paged_pool_stored_token_major(flags):
    # the pool as paged KV caches commonly store it, [n_pages, page_size, H_kv, d], passed as a
    # permuted view [n_pages, H_kv, page_size, d]
    cfg = inputs.VerifyConfig("pg", 0x61, 3, 8, 2, 128, 256, 6, 30, 700, k_mult=2.0)
    lens = [700, 30, 512]
    case = util.gen_case(cfg, lens, DEV, fill=float("nan"))
    Q, chunks, K_loc, V_loc, bits = case
    ref = util.oracle_case(cfg, lens, *case)
    ps, ppr = 16, cfg.L_c // 16
    g = torch.Generator().manual_seed(5)
    ctx = util.make_ctx(cfg, flags=flags)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    for K, V, vl in chunks:
        n_pages = cfg.B * ppr + 2
        table = torch.randperm(n_pages, generator=g)[:cfg.B * ppr].to(torch.int32).view(cfg.B, ppr).contiguous()
        pools = []
        for X in (K, V):
            pool = torch.full((n_pages, ps, cfg.H_kv, cfg.d), float("nan"), dtype=torch.bfloat16, device=DEV)
            pool[table.view(-1).long()] = X.view(cfg.B, cfg.H_kv, ppr, ps, cfg.d).permute(0, 2, 3, 1, 4).reshape(-1, ps, cfg.H_kv, cfg.d)
            pools.append(pool.permute(0, 2, 1, 3))
        ctx.ss_verify_chunk_paged(pools[0], pools[1], table.to(DEV), vl, vl.tolist())
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_finalize(O, LSE)
    assert ctx.ss_poll_status() == (0, 0)
    util.compare(cfg, O, LSE, ref)
    ctx.close()


def test_round_can_be_captured_in_a_cuda_graph():
    # the calls only enqueue on the stream: a captured round replays bit-identically
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x5F, 2, 8, 2, 128, 256, 8, 300, 700)
    lens = inputs.history_lengths(cfg)
    case = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    O_ref, L_ref = util.gpu_case(ctx, cfg, *case)
    O_ref, L_ref = O_ref.clone(), L_ref.clone()
    Q, chunks, K_loc, V_loc, bits = case
    O = torch.zeros_like(O_ref)
    LSE = torch.zeros_like(L_ref)

    def one_round():
        ctx.ss_verify_begin(Q, cfg.scale)
        for K, V, vl in chunks:
            ctx.ss_verify_chunk(K, V, vl)
        ctx.ss_verify_local(K_loc, V_loc)
        ctx.ss_verify_finalize(O, LSE)

    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        one_round()
    for _ in range(3):
        O.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(O.view(torch.int16), O_ref.view(torch.int16)) and torch.equal(LSE, L_ref)
    ctx.close()


@pytest.mark.parametrize("lens", [[5000, 4900, 5000], [5000, 700, 2300]])
def test_chunk_list_round_can_be_captured_in_a_cuda_graph(lens):
    """A round whose list of chunks is one launch (equally long histories: equal splits per
    request; a ragged batch: shares across requests) replays from a CUDA graph bit-identically,
    also after the inputs were refreshed in place."""
    import ctypes as C
    ssb = _ssb()
    cfg = inputs.VerifyConfig("gl", 0x61, len(lens), 8, 2, 128, 1024, 8, 0, max(lens))
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    hints = [(C.c_int32 * cfg.B)(*vl.tolist()) for (_, _, vl) in chunks]
    descs = ctx.chunk_descs([chunks], hints)
    O, LSE = (torch.zeros(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV),
              torch.zeros(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV))

    def one_round():
        ctx.ss_verify_round(Q, cfg.scale, chunks, K_loc, V_loc, ssb.SS_MASK_CHAIN, None, O, LSE, descs=descs)

    one_round()   # (the list of tensor maps is sent on first use: outside the capture)
    torch.cuda.synchronize()
    assert ctx.last_chunk_kernel() == "tcgen05-keys-round"
    O_ref, L_ref = O.clone(), LSE.clone()
    util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        one_round()
    for _ in range(3):
        O.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(O.view(torch.int16), O_ref.view(torch.int16)) and torch.equal(LSE, L_ref)
    # new queries in place: the replay equals a fresh call
    Q.copy_(inputs.normal_bf16(cfg.seed + 1, inputs.TID_Q, tuple(Q.shape), device=DEV))
    g.replay()
    torch.cuda.synchronize()
    O_g, L_g = O.clone(), LSE.clone()
    one_round()
    torch.cuda.synchronize()
    assert torch.equal(O.view(torch.int16), O_g.view(torch.int16)) and torch.equal(LSE, L_g)
    O_ref, L_ref = O.clone(), LSE.clone()
    # The launch reads its chunks' tensor maps from a list in the workspace, of which there are four:
    # a list a capture used stays, however many other lists the context sees afterwards
    O2, L2 = torch.empty_like(O), torch.empty_like(LSE)
    keep = []   # (alive, so that no later buffer takes an address a list already holds)
    for k in range(6):
        other = [(K.clone(), V.clone(), vl) for (K, V, vl) in chunks]
        keep.append(other)
        ctx.ss_verify_round(Q, cfg.scale, other, K_loc, V_loc, ssb.SS_MASK_CHAIN, None, O2, L2, hints=hints)
        torch.cuda.synchronize()
        assert ctx.last_chunk_kernel() == "tcgen05-keys-round"
        assert torch.equal(O2.view(torch.int16), O_ref.view(torch.int16))
    O.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(O.view(torch.int16), O_ref.view(torch.int16)) and torch.equal(LSE, L_ref)
    # a list first seen inside a capture is not sent from there: the chunks go out one by one
    fresh = [(K.clone(), V.clone(), vl) for (K, V, vl) in chunks]
    fresh_descs = ctx.chunk_descs([fresh], hints)
    g2 = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g2):
        ctx.ss_verify_round(Q, cfg.scale, fresh, K_loc, V_loc, ssb.SS_MASK_CHAIN, None, O2, L2, descs=fresh_descs)
    assert ctx.last_chunk_kernel() == "tcgen05-keys"
    g2.replay()
    torch.cuda.synchronize()
    util.compare(cfg, O2, L2, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))
    ctx.close()


def test_two_contexts_on_two_streams_do_not_interfere():
    # Two contexts (own workspaces) whose rounds interleave call by call on two streams give,
    # bit for bit, what each gives alone: no state is shared between contexts.
    ssb = _ssb()
    cfgs = [inputs.VerifyConfig("v", 0x71, 4, 16, 4, 128, 512, 8, 900, 2000),
            inputs.VerifyConfig("v", 0x72, 3, 8, 2, 128, 256, 24, 500, 1500, mask="tree")]
    cases, alone, ctxs = [], [], []
    for cfg in cfgs:
        lens = inputs.history_lengths(cfg)
        case = util.gen_case(cfg, lens, DEV)
        ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
        O, L = util.gpu_case(ctx, cfg, *case)
        cases.append(case)
        alone.append((O.clone(), L.clone()))
        ctxs.append(ctx)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [(torch.zeros_like(o), torch.zeros_like(l)) for o, l in alone]
    for rep in range(20):
        for i in (0, 1):
            ctxs[i].ss_verify_begin(cases[i][0], cfgs[i].scale, streams[i])
        n = max(len(c[1]) for c in cases)
        for j in range(n):
            for i in (0, 1):
                if j < len(cases[i][1]):
                    K, V, vl = cases[i][1][j]
                    ctxs[i].ss_verify_chunk(K, V, vl, streams[i])
        for i in (0, 1):
            Q, chunks, K_loc, V_loc, bits = cases[i]
            tree = cfgs[i].mask == "tree"
            ctxs[i].ss_verify_local(K_loc, V_loc, ssb.SS_MASK_TREE_BITS if tree else ssb.SS_MASK_CHAIN,
                                    bits if tree else None, streams[i])
            ctxs[i].ss_verify_finalize(outs[i][0], outs[i][1], streams[i])
    torch.cuda.synchronize()
    for i in (0, 1):
        assert ctxs[i].ss_poll_status() == (0, 0)
        assert torch.equal(outs[i][0].view(torch.int16), alone[i][0].view(torch.int16))
        assert torch.equal(outs[i][1], alone[i][1])
        ctxs[i].close()


@pytest.mark.parametrize("flags", [0, 4])
def test_rounds_narrower_than_the_context_limit(flags):
    # A context sized for max_Tq candidates runs rounds with fewer: the partial-state rows of a
    # slot then have room past the round's last row (the rows-on-M kernel's write-out may put
    # padding there), and a later, wider round must not see anything of it.
    ssb = _ssb()
    wide = inputs.VerifyConfig("v", 0x81, 2, 16, 4, 128, 512, 40, 700, 1500, k_mult=2.0)
    ctx = ssb.Context(wide.B, wide.H_q, wide.H_kv, wide.d, wide.T_q, wide.T_q, wide.L_c, flags=flags)
    for T_q in (40, 20, 9, 33, 40):
        cfg = inputs.VerifyConfig("v", 0x81 + T_q, 2, 16, 4, 128, 512, T_q, 700, 1500, k_mult=2.0)
        lens = inputs.history_lengths(cfg)
        case = util.gen_case(cfg, lens, DEV)
        O, LSE = util.gpu_case(ctx, cfg, *case)
        assert ctx.ss_poll_status() == (0, 0)
        ref = util.oracle_case(cfg, lens, *case, groups=[(0, 0), (1, 3)])
        util.compare(cfg, O, LSE, ref)
    ctx.close()


@pytest.mark.parametrize("T_q,G,n", [(2, 4, 300), (5, 4, 129), (8, 4, 1000), (9, 4, 127), (7, 8, 640), (33, 2, 500),
                                      (17, 8, 257), (40, 4, 384), (3, 1, 1), (6, 4, 0)])
@pytest.mark.parametrize("flags", [0, 8])
def test_head_dim_64_runs_on_the_tensor_cores(T_q, G, n, flags):
    # head dim 64: one 64-column box per tile in both tensor-core kernels (the keys-on-M kernel's
    # output MMA pads M with rows that are never read), every row-group width, ragged tails,
    # several chunks; flags = 8 takes the keys-on-M kernel for every row count
    cfg = inputs.VerifyConfig("v", 0x90 + T_q + G + n, 3, 2 * G, 2, 64, 256, T_q, n, n, k_mult=2.0,
                              mask="tree" if T_q % 2 else "chain")
    lens = [n, max(0, n - 77), n // 2]
    want = "tcgen05-keys" if (flags or T_q * G <= 16) else "tcgen05"
    O, LSE, _ = _run(cfg, lens=lens, flags=flags, fill=float("nan"), kernel=want)
    # and the CUDA-core kernel agrees
    case = util.gen_case(cfg, lens, DEV, float("nan"))
    ctx = util.make_ctx(cfg, flags=1)
    O2, L2 = util.gpu_case(ctx, cfg, *case)
    ctx.close()
    assert (O.float() - O2.float()).abs().max() < 2e-2
    fin = torch.isfinite(L2)
    assert torch.equal(torch.isfinite(LSE), fin) and (LSE[fin] - L2[fin]).abs().max() < 1e-4


@pytest.mark.parametrize("page_size", [8, 16, 64, 128])
def test_head_dim_64_paged(page_size):
    ssb = _ssb()
    cfg = inputs.VerifyConfig("pg", 0xA0 + page_size, 3, 8, 2, 64, 512, 6, 40, 1500, k_mult=2.0)
    lens = [1500, 40, 1024]
    case = util.gen_case(cfg, lens, DEV, fill=float("nan"))
    Q, chunks, K_loc, V_loc, bits = case
    ref = util.oracle_case(cfg, lens, *case)
    ppr = cfg.L_c // page_size
    g = torch.Generator().manual_seed(page_size)
    ctx = util.make_ctx(cfg)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    for K, V, vl in chunks:
        n_pages = cfg.B * ppr + 3
        table = torch.randperm(n_pages, generator=g)[:cfg.B * ppr].to(torch.int32).view(cfg.B, ppr).contiguous()
        K_pool = torch.full((n_pages, cfg.H_kv, page_size, cfg.d), float("nan"), dtype=torch.bfloat16, device=DEV)
        V_pool = torch.full_like(K_pool, float("nan"))
        K_pool[table.view(-1).long()] = K.view(cfg.B, cfg.H_kv, ppr, page_size, cfg.d).permute(0, 2, 1, 3, 4).reshape(-1, cfg.H_kv, page_size, cfg.d)
        V_pool[table.view(-1).long()] = V.view(cfg.B, cfg.H_kv, ppr, page_size, cfg.d).permute(0, 2, 1, 3, 4).reshape(-1, cfg.H_kv, page_size, cfg.d)
        ctx.ss_verify_chunk_paged(K_pool, V_pool, table.to(DEV), vl, vl.tolist())
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    assert ctx.ss_poll_status() == (0, 0)
    assert ctx.last_chunk_kernel() == "tcgen05"      # 24 rows per kv-head: rows on M at head dim 64
    util.compare(cfg, O, LSE, ref)
    ctx.close()


def test_graph_round_helper_replays_with_refreshed_inputs():
    # the binding's GraphRound: capture once, refresh the inputs in place, replay
    ssb = _ssb()
    cfg = inputs.CONFIGS["c1_tiny_chain"]
    lens = inputs.history_lengths(cfg)
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    g = ssb.GraphRound(ctx, Q, chunks, K_loc, V_loc, cfg.scale)
    O, LSE = g.replay()
    torch.cuda.synchronize()
    util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))
    # new contents in the same buffers
    cfg2 = inputs.VerifyConfig(cfg.name, cfg.seed + 1, cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.L_c, cfg.T_q,
                               cfg.len_lo, cfg.len_hi)
    Q2, chunks2, K_loc2, V_loc2, bits2 = util.gen_case(cfg2, lens, DEV)
    Q.copy_(Q2); K_loc.copy_(K_loc2); V_loc.copy_(V_loc2)
    for (K, V, vl), (K2, V2, vl2) in zip(chunks, chunks2):
        K.copy_(K2); V.copy_(V2); vl.copy_(vl2)
    O, LSE = g.replay()
    torch.cuda.synchronize()
    assert ctx.ss_poll_status() == (0, 0)
    util.compare(cfg2, O, LSE, util.oracle_case(cfg2, lens, Q2, chunks2, K_loc2, V_loc2, bits2))
    ctx.close()


@pytest.mark.parametrize("T_q,T_loc,G", [(4, 9, 4), (8, 40, 2), (1, 17, 8)])
def test_chain_with_more_local_tokens_than_queries(T_q, T_loc, G):
    """The GPU-resident pass over Active Tail + Speculative Frontier (Section 4.2): T_loc - T_q
    leading local tokens every query sees, then the causal part.  The chain rule is computed in
    the kernel; the oracle gets the explicit boolean mask j <= i + (T_loc - T_q)."""
    import oracle
    from paper_2609_33184_b200 import binding as ssb
    cfg = inputs.VerifyConfig("tail", 0x90 + T_q, 2, 2 * G, 2, 128, 128, T_q, 0, 200, k_mult=2.0)
    lens = [200, 37]
    Q, chunks, _, _, _ = util.gen_case(cfg, lens, DEV)
    shape = (cfg.B, cfg.H_kv, T_loc, cfg.d)
    K_loc = inputs.normal_bf16(cfg.seed, inputs.TID_KLOC, shape, mult=2.0, device=DEV)
    V_loc = inputs.normal_bf16(cfg.seed, inputs.TID_VLOC, shape, device=DEV)
    ctx = ssb.Context(cfg.B, cfg.H_q, cfg.H_kv, cfg.d, T_q, T_loc, cfg.L_c)
    O = torch.empty(cfg.B, cfg.H_q, T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    for K, V, vl in chunks:
        ctx.ss_verify_chunk(K, V, vl)
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    i, j = np.arange(T_q)[:, None], np.arange(T_loc)[None, :]
    mask = np.broadcast_to(j <= i + (T_loc - T_q), (cfg.B, T_q, T_loc))
    f64 = util.f64
    kh = [np.concatenate([f64(K[b, :, :int(vl[b])]) for K, V, vl in chunks], axis=1) for b in range(cfg.B)]
    vh = [np.concatenate([f64(V[b, :, :int(vl[b])]) for K, V, vl in chunks], axis=1) for b in range(cfg.B)]
    Or, Lr = oracle.verify_attention(f64(Q), kh, vh, f64(K_loc), f64(V_loc), mask, cfg.scale)
    ref = {(b, h): (Or[b, h * G:(h + 1) * G], Lr[b, h * G:(h + 1) * G]) for b in range(cfg.B)
           for h in range(cfg.H_kv)}
    util.compare(cfg, O, LSE, ref)
    # fewer local tokens than queries under the chain rule is rejected, not silently run
    ctx.ss_verify_begin(Q, cfg.scale)
    if T_q > 1:
        with pytest.raises(ssb.SpecStreamError):
            ctx.ss_verify_local(K_loc[:, :, :T_q - 1], V_loc[:, :, :T_q - 1])
    ctx.ss_verify_abort()
    ctx.close()


@pytest.mark.parametrize("name,cfg,lens", [
    ("tiny chain", inputs.CONFIGS["c1_tiny_chain"], None),
    ("ragged, G=4, d=128", inputs.VerifyConfig("r1", 0xa1, 3, 8, 2, 128, 256, 7, 0, 700, k_mult=2.0), [700, 0, 257]),
    ("tree, one row tile of 8", inputs.VerifyConfig("r2", 0xa2, 2, 2, 2, 64, 128, 8, 0, 300, mask="tree"), [300, 64]),
    ("tree, G=5", inputs.VerifyConfig("r3", 0xa3, 2, 10, 2, 128, 192, 12, 0, 500, mask="tree"), [1, 500]),
    ("plain decode", inputs.VerifyConfig("r4", 0xa4, 4, 16, 2, 64, 512, 1, 0, 1500), [1500, 511, 512, 513]),
])
@pytest.mark.parametrize("merge", ["cluster", "ticket"])
def test_whole_round_in_one_call_small(name, cfg, lens, merge, monkeypatch):
    """ss_verify_round on rounds small enough for its single-launch kernel: equal to the oracle
    and (within rounding) to the separate calls.  The token splits of a (request, kv-head, row
    tile) merge inside a thread-block cluster through distributed shared memory, or (clusters
    turned off) through scratch memory and a ticket counter; both give the same bits."""
    from paper_2609_33184_b200 import binding as ssb
    lens = lens or inputs.history_lengths(cfg)
    if merge == "ticket":
        monkeypatch.setenv("SS_ROUND_CLUSTER", "never")   # (read when the context is created)
    else:
        monkeypatch.delenv("SS_ROUND_CLUSTER", raising=False)
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg)
    kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
    O = torch.full((cfg.B, cfg.H_q, cfg.T_q, cfg.d), float("nan"), dtype=torch.bfloat16, device=DEV)
    LSE = torch.full((cfg.B, cfg.H_q, cfg.T_q), float("nan"), dtype=torch.float32, device=DEV)
    ctx.ss_verify_round(Q, cfg.scale, chunks, K_loc, V_loc, kind, bits if cfg.mask == "tree" else None, O, LSE)
    torch.cuda.synchronize()
    assert ctx.last_chunk_kernel() == "simt-round"
    assert ctx.ss_poll_status() == (0, 0)
    ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits)
    util.compare(cfg, O, LSE, ref)
    if merge == "cluster":   # the other merge path sums the same states in the same order
        monkeypatch.setenv("SS_ROUND_CLUSTER", "never")
        ctx_t = util.make_ctx(cfg)
        Ot, Lt = torch.empty_like(O), torch.empty_like(LSE)
        for _ in range(3):
            ctx_t.ss_verify_round(Q, cfg.scale, chunks, K_loc, V_loc, kind, bits if cfg.mask == "tree" else None, Ot, Lt)
            ctx.ss_verify_round(Q, cfg.scale, chunks, K_loc, V_loc, kind, bits if cfg.mask == "tree" else None, O, LSE)
        torch.cuda.synchronize()
        assert torch.equal(O.view(torch.int16), Ot.view(torch.int16)) and torch.equal(LSE.view(torch.int32), Lt.view(torch.int32))
        ctx_t.close()
    O2, L2 = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    mag = max(1.0, float(O2.float().abs().max()))
    assert float((O.float() - O2.float()).abs().max()) <= util.TOL_MAX_O * mag
    assert float((LSE - L2).abs().max()) <= util.TOL_LSE
    # no local segment, no LSE, chunks in reverse order: still Eq. 12 over the history alone
    O3 = torch.empty_like(O)
    ctx.ss_verify_round(Q, cfg.scale, chunks[::-1], None, None, kind, None, O3, None)
    torch.cuda.synchronize()
    ctx.ss_verify_begin(Q, cfg.scale)
    for K, V, vl in chunks:
        ctx.ss_verify_chunk(K, V, vl)
    O4, L4 = torch.empty_like(O), torch.empty_like(LSE)
    ctx.ss_verify_finalize(O4, L4)
    torch.cuda.synchronize()
    assert float((O3.float() - O4.float()).abs().max()) <= util.TOL_MAX_O * max(1.0, float(O4.float().abs().max()))
    ctx.close()


def test_whole_round_in_one_call_large_and_errors():
    """A round too large for the single launch goes through the separate kernels (bit-identical
    to calling them one by one); errors leave the context idle."""
    from paper_2609_33184_b200 import binding as ssb
    cfg = inputs.VerifyConfig("big", 0xa5, 2, 8, 2, 128, 1024, 8, 0, 5000)
    lens = [5000, 1025]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    O, LSE = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    O2, L2 = torch.empty_like(O), torch.empty_like(LSE)
    ctx.ss_verify_round(Q, cfg.scale, chunks, K_loc, V_loc, ssb.SS_MASK_CHAIN, None, O2, L2)
    torch.cuda.synchronize()
    assert ctx.last_chunk_kernel().startswith("tcgen05")
    assert torch.equal(O, O2) and torch.equal(LSE, L2)
    util.compare(cfg, O2, L2, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))
    # a failing call (chunk longer than the context allows) leaves no round open
    big = torch.zeros(2, 2, 2048, 128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(ssb.SpecStreamError):
        ctx.ss_verify_round(Q, cfg.scale, chunks + [(big, big, None)], K_loc, V_loc, ssb.SS_MASK_CHAIN, None, O2, L2)
    ctx.ss_verify_begin(Q, cfg.scale)          # idle again: a new round can start
    with pytest.raises(ssb.SpecStreamError):   # and ss_verify_round refuses to run over it
        ctx.ss_verify_round(Q, cfg.scale, chunks, K_loc, V_loc, ssb.SS_MASK_CHAIN, None, O2, L2)
    ctx.ss_verify_abort()
    ctx.close()


@pytest.mark.parametrize("d,T_q,H_q,H_kv", [(128, 40, 8, 2), (128, 24, 16, 2), (64, 40, 8, 2), (128, 64, 10, 2),
                                             (128, 8, 8, 2), (128, 3, 4, 4), (64, 4, 8, 2)])
def test_chunk_list_in_one_launch(d, T_q, H_q, H_kv, monkeypatch):
    """ss_verify_chunks where the whole list of chunks goes out as one launch whose CTAs walk tiles
    across chunk boundaries: more than 128 rows per kv-head (rows-on-M kernel) and up to 32 rows
    (keys-on-M kernel).  Checked against the oracle with the list in history order and reversed
    (the ragged chunk and the empty ones then come first and a partly filled chunk sits in the
    middle of a CTA's walk), against the separate calls, and for bit-identical repeats."""
    from paper_2609_33184_b200 import binding as ssb
    keys = T_q * (H_q // H_kv) <= (32 if d == 128 else 16)
    one, each = ("tcgen05-keys-round", "tcgen05-keys") if keys else ("tcgen05-round", "tcgen05")
    monkeypatch.setenv("SS_HISTORY_LAUNCH", "always")   # (the routing has a test of its own; these lengths are ragged)
    cfg = inputs.VerifyConfig("hist", 0xb7 + d + T_q, 4, H_q, H_kv, d, 512, T_q, 0, 3000)
    lens = [3000, 1, 1537, 0]     # ragged, a single token, one token past a chunk boundary, nothing
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    assert len(chunks) == 6
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    O5, L5 = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    assert ctx.last_chunk_kernel() == each
    ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits)
    util.compare(cfg, O5, L5, ref)
    outs = []
    import ctypes as C
    for order, with_host_lengths in ((list(range(6)), False), (list(range(5, -1, -1)), True), ([2, 5, 0, 3, 1, 4], True)):
        lst = [chunks[j] for j in order]
        # with the host's copy of the lengths a ragged batch is cut into pieces of about equal length
        # (a request-dependent number of them); without, every request into equally many pieces
        hints = [(C.c_int32 * cfg.B)(*vl.tolist()) for (_, _, vl) in lst] if with_host_lengths else None
        descs = ctx.chunk_descs([lst], hints)
        O, LSE = torch.empty_like(O5), torch.empty_like(L5)
        for rep in range(3):
            ctx.ss_verify_begin(Q, cfg.scale)
            ctx.ss_verify_chunks(descs, len(lst))
            ctx.ss_verify_local(K_loc, V_loc, ssb.SS_MASK_CHAIN, None)
            ctx.ss_verify_finalize(O, LSE)
            torch.cuda.synchronize()
            assert ctx.last_chunk_kernel() == one
            assert ctx.ss_poll_status() == (0, 0)
            if rep == 0:
                O0, L0 = O.clone(), LSE.clone()
            else:
                assert torch.equal(O0.view(torch.int16), O.view(torch.int16)) and torch.equal(L0, LSE)
        util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, lst, K_loc, V_loc, bits))
        outs.append(O0)
    # the same through ss_verify_round
    O, LSE = torch.empty_like(O5), torch.empty_like(L5)
    ctx.ss_verify_round(Q, cfg.scale, chunks, K_loc, V_loc, ssb.SS_MASK_CHAIN, None, O, LSE)
    torch.cuda.synchronize()
    assert ctx.last_chunk_kernel() == one
    assert torch.equal(O.view(torch.int16), outs[0].view(torch.int16))
    # a bad valid length is flagged and clamped; a chunk beyond the context's size is refused and
    # leaves the round open
    bad = [(K, V, vl.clone()) for (K, V, vl) in chunks]
    bad[1][2][0] = 9999
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunks(ctx.chunk_descs([bad]), 6)
    ctx.ss_verify_local(K_loc, V_loc, ssb.SS_MASK_CHAIN, None)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    st, bits_ = ctx.ss_poll_status()
    assert bits_ & ssb.SS_DEV_BAD_VALID_LEN
    big = torch.zeros(4, H_kv, 1024, d, dtype=torch.bfloat16, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    with pytest.raises(ssb.SpecStreamError):
        ctx.ss_verify_chunks(ctx.chunk_descs([chunks[:2] + [(big, big, None)]]), 3)
    ctx.ss_verify_abort()
    ctx.close()


@pytest.mark.parametrize("d,T_q,H_q,H_kv,lens", [
    (128, 8, 8, 2, [6000, 300, 3100, 1500, 5000]),      # 32 rows; five requests over 15 CTAs per kv-head
    (128, 3, 4, 4, [129, 6000, 128, 127, 1, 4000]),     # requests of a tile or two between long ones
    (64, 4, 8, 2, [2000, 2100, 5900, 2200, 6000]),
    (128, 5, 12, 4, [6000, 5000]),                      # 15 rows; fewer requests than CTAs
])
def test_chunk_list_ragged_batch_shares_across_requests(d, T_q, H_q, H_kv, lens, monkeypatch):
    """A batch the host knows to be ragged, up to 32 rows per kv-head: one launch whose CTAs take
    equal shares of all requests' tiles laid end to end, so a CTA may end one request and begin the
    next and a request has as many partial states as CTAs touched it.  Against the oracle and the
    separate calls, with the chunk list in two orders, with host lengths that are out of date (the
    shares are then scaled to the lengths on the device), and for bit-identical repeats."""
    import ctypes as C
    from paper_2609_33184_b200 import binding as ssb
    monkeypatch.setenv("SS_HISTORY_LAUNCH", "always")   # (a history of a few dozen tiles: not routed by itself)
    cfg = inputs.VerifyConfig("walk", 0xe9 + d + T_q, len(lens), H_q, H_kv, d, 512, T_q, 0, max(lens))
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    keys = T_q * (H_q // H_kv) <= (32 if d == 128 else 16)
    one, each = ("tcgen05-keys-round", "tcgen05-keys") if keys else ("tcgen05-round", "tcgen05")
    O5, L5 = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    assert ctx.last_chunk_kernel() == each
    ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits)
    util.compare(cfg, O5, L5, ref)
    n = len(chunks)
    stale = [max(1, (l * 3) // 5 if i % 2 else min(max(lens), l + 700)) for i, l in enumerate(lens)]
    for order, host_lens in ((list(range(n)), lens), (list(range(n - 1, -1, -1)), lens), (list(range(n)), stale)):
        lst = [chunks[j] for j in order]
        hints = []
        for j in order:   # the host's idea of chunk j's valid lengths
            hints.append((C.c_int32 * cfg.B)(*[max(0, min(cfg.L_c, hl - j * cfg.L_c)) for hl in host_lens]))
        descs = ctx.chunk_descs([lst], hints)
        O, LSE = torch.empty_like(O5), torch.empty_like(L5)
        for rep in range(3):
            ctx.ss_verify_begin(Q, cfg.scale)
            ctx.ss_verify_chunks(descs, n)
            ctx.ss_verify_local(K_loc, V_loc, ssb.SS_MASK_CHAIN, None)
            ctx.ss_verify_finalize(O, LSE)
            torch.cuda.synchronize()
            assert ctx.last_chunk_kernel() == one
            assert ctx.ss_poll_status() == (0, 0)
            if rep == 0:
                O0, L0 = O.clone(), LSE.clone()
            else:
                assert torch.equal(O0.view(torch.int16), O.view(torch.int16)) and torch.equal(L0, LSE)
        util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, lst, K_loc, V_loc, bits))
        assert float((O.float() - O5.float()).abs().max()) <= 2.0 ** -7 * max(1.0, float(O5.float().abs().max()))
        assert float((LSE - L5).abs().max()) <= 1e-4
    # a bad valid length on the device is flagged and clamped
    bad = [(K, V, vl.clone()) for (K, V, vl) in chunks]
    bad[1][2][0] = 9999
    hints = [(C.c_int32 * cfg.B)(*vl.tolist()) for (_, _, vl) in chunks]
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunks(ctx.chunk_descs([bad], hints), n)
    ctx.ss_verify_local(K_loc, V_loc, ssb.SS_MASK_CHAIN, None)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    assert ctx.last_chunk_kernel() == one
    assert ctx.ss_poll_status()[1] & ssb.SS_DEV_BAD_VALID_LEN
    ctx.close()


@pytest.mark.parametrize("B,seed", [(3, 1), (7, 2), (16, 3), (32, 4), (32, 5)])
def test_chunk_list_ragged_batch_random_lengths(B, seed):
    """Shares across requests on random batches with 8 kv-heads (37 CTAs per kv-head, or one per
    eight tiles): lengths from one token to the full history, so requests of a tile or two sit
    between long ones and a request is cut into one to a dozen pieces.  Every request against
    the separate calls, a sample of (request, kv-head) groups against the oracle."""
    import ctypes as C
    from paper_2609_33184_b200 import binding as ssb
    rng = np.random.default_rng(1000 + seed)
    hi = 9000
    lens = [int(x) for x in rng.integers(1, hi + 1, size=B)]
    lens[int(rng.integers(0, B))] = hi                     # one request has the full history
    if B > 3:
        lens[int(rng.integers(0, B))] = int(rng.integers(1, 129))   # and one a single tile
    cfg = inputs.VerifyConfig("walkr", 0xf300 + seed, B, 8, 8, 128, 1024, 4, 0, hi)
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    n = len(chunks)
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    O5, L5 = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    hints = [(C.c_int32 * B)(*vl.tolist()) for (_, _, vl) in chunks]
    O, LSE = torch.empty_like(O5), torch.empty_like(L5)
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunks(ctx.chunk_descs([chunks], hints), n)
    ctx.ss_verify_local(K_loc, V_loc, ssb.SS_MASK_CHAIN, None)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    assert ctx.last_chunk_kernel() == "tcgen05-keys-round"
    assert ctx.ss_poll_status() == (0, 0)
    # the two paths sum the same weights in another order: far inside the oracle tolerances
    assert float((O.float() - O5.float()).abs().max()) <= 2.0 ** -7 * max(1.0, float(O5.float().abs().max()))
    assert float((LSE - L5).abs().max()) <= 1e-4
    groups = [(int(rng.integers(0, B)), int(rng.integers(0, 8))) for _ in range(4)]
    groups += [(int(np.argmax(lens)), 0), (int(np.argmin(lens)), 7)]
    util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits, groups=groups))
    ctx.close()


@pytest.mark.parametrize("T_q,H_q", [(8, 8), (40, 8)])
def test_chunk_list_of_32_chunks(T_q, H_q, monkeypatch):
    """The longest list a launch takes (32 chunks: every entry of the kernels' chunk tables in
    use), keys-on-M and rows-on-M kernel, the last chunks ragged and one request's empty."""
    import ctypes as C
    from paper_2609_33184_b200 import binding as ssb
    monkeypatch.setenv("SS_HISTORY_LAUNCH", "always")
    cfg = inputs.VerifyConfig("l32", 0x7a + T_q, 2, H_q, 2, 128, 128, T_q, 0, 4096)
    lens = [4096, 3900]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    assert len(chunks) == 32
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
    hints = [(C.c_int32 * cfg.B)(*vl.tolist()) for (_, _, vl) in chunks]
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunks(ctx.chunk_descs([chunks], hints), 32)
    ctx.ss_verify_local(K_loc, V_loc, ssb.SS_MASK_CHAIN, None)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    assert ctx.last_chunk_kernel() == ("tcgen05-keys-round" if T_q == 8 else "tcgen05-round")
    assert ctx.ss_poll_status() == (0, 0)
    util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))
    ctx.close()


def test_chunk_list_after_separate_chunks_with_one_partial_set(monkeypatch):
    """A context with a single partial set: a chunk call, then a list of chunks in one launch (the
    set in use is folded first), then another chunk call; against the oracle."""
    from paper_2609_33184_b200 import binding as ssb
    monkeypatch.setenv("SS_HISTORY_LAUNCH", "always")   # (a short list: not routed by itself)
    cfg = inputs.VerifyConfig("hist1", 0xc3, 2, 8, 2, 128, 512, 40, 0, 2500)
    lens = [2500, 900]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    assert len(chunks) == 5
    ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS, max_chunks=1)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunk(*chunks[0])
    ctx.ss_verify_chunks(ctx.chunk_descs([chunks[1:4]]), 3)
    assert ctx.last_chunk_kernel() == "tcgen05-round"
    ctx.ss_verify_chunk(*chunks[4])
    ctx.ss_verify_local(K_loc, V_loc, ssb.SS_MASK_CHAIN, None)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    assert ctx.ss_poll_status() == (0, 0)
    util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))
    ctx.close()


def test_two_chunk_calls_with_max_chunks_one():
    """max_chunks = 1 still leaves room to fold: a second chunk call must not land on the local
    segment's partial set."""
    cfg = inputs.VerifyConfig("v", 0x59, 2, 8, 2, 128, 256, 8, 600, 700)
    _run(cfg, max_chunks=1)


def test_chunk_list_routing():
    """Which lists go out as one launch: histories the host knows to be equally long at any row
    count; up to 32 rows per kv-head also a batch it knows to be ragged (no request empty); more than
    128 rows per kv-head at head dim 128 also when it knows nothing, but not a batch it knows to be
    ragged; never a history of a few tiles."""
    import ctypes as C
    from paper_2609_33184_b200 import binding as ssb

    def kernel_for(d, T_q, H_q, H_kv, lens, host_lengths, L_c=512):
        cfg = inputs.VerifyConfig("route", 0xd1 + T_q, len(lens), H_q, H_kv, d, L_c, T_q, 0, max(lens))
        Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV, fill=0.0)
        ctx = util.make_ctx(cfg, flags=ssb.SS_FLAG_OVERLAP_CHUNKS)
        hints = [(C.c_int32 * cfg.B)(*vl.tolist()) for (_, _, vl) in chunks] if host_lengths else None
        ctx.ss_verify_begin(Q, cfg.scale)
        ctx.ss_verify_chunks(ctx.chunk_descs([chunks], hints), len(chunks))
        ctx.ss_verify_abort()
        torch.cuda.synchronize()
        k = ctx.last_chunk_kernel()
        ctx.close()
        return k

    even, ragged = [4096, 4096, 4000], [4096, 1000, 2500]
    assert kernel_for(128, 8, 8, 2, even, True) == "tcgen05-keys-round"      # 32 rows, known equal
    assert kernel_for(128, 8, 8, 2, even, False) == "tcgen05-keys"           # lengths only on the device
    assert kernel_for(128, 8, 8, 2, ragged, True) == "tcgen05-keys-round"    # known ragged: shares across requests
    assert kernel_for(128, 8, 8, 2, [4096, 0, 2500], True) == "tcgen05-keys"  # ... not with an empty request
    assert kernel_for(128, 8, 16, 2, even, True) == "tcgen05-round"          # 64 rows, known equal
    assert kernel_for(128, 8, 16, 2, even, False) == "tcgen05"
    assert kernel_for(64, 8, 16, 2, even, True) == "tcgen05-round"           # head dim 64, 64 rows
    assert kernel_for(128, 40, 8, 2, even, False) == "tcgen05-round"         # 160 rows: whatever the host knows
    assert kernel_for(128, 40, 8, 2, ragged, True) == "tcgen05"              # ... unless it knows the batch is ragged
    assert kernel_for(64, 40, 8, 2, even, True) == "tcgen05"                 # head dim 64, 160 rows: not taken
    assert kernel_for(128, 8, 8, 2, [300, 300], True, L_c=256) == "tcgen05-keys"   # a few tiles in all
