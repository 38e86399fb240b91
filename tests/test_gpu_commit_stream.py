"""GPU tests of commit-gather (bit exact), the streamed round, the call-order state machine
and the trace facility, all through the C ABI."""
import ctypes as C
import time

import numpy as np
import pytest
import torch

from paper_2609_33184_b200 import harness
from paper_2609_33184_b200 import inputs
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _ssb():
    from paper_2609_33184_b200 import binding
    return binding


def _u16(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("d", [64, 128])
def test_commit_gather_bit_exact(d):
    import oracle
    ssb = _ssb()
    B, H_kv, T, cap = 5, 3, 9, 20
    ctx = ssb.Context(B, 2 * H_kv, H_kv, d, T, T, 64)
    g = torch.Generator().manual_seed(d)
    rnd = lambda *s: torch.randint(-32768, 32767, s, generator=g, dtype=torch.int16)
    K_loc, V_loc = rnd(B, H_kv, T, d).to(DEV).view(torch.bfloat16), rnd(B, H_kv, T, d).to(DEV).view(torch.bfloat16)
    # destination: a strided view into a larger canary-filled buffer
    Kbig, Vbig = rnd(B, H_kv, cap + 4, d + 8).to(DEV), rnd(B, H_kv, cap + 4, d + 8).to(DEV)
    K0, V0 = Kbig.clone(), Vbig.clone()
    K_dst = Kbig.view(torch.bfloat16)[:, :, 2:2 + cap, 8:]
    V_dst = Vbig.view(torch.bfloat16)[:, :, 2:2 + cap, :d]
    idx = torch.tensor([[0, 1, 2, 3, 4, 5, 6, 7, 8], [8, 6, 4, 2, 0, 1, 3, 5, 7], [3, 3, 3, 3, 3, 3, 3, 3, 3],
                        [0, 4, 8, 0, 0, 0, 0, 0, 0], [1, 2, 0, 0, 0, 0, 0, 0, 0]], dtype=torch.int32)
    cnt = torch.tensor([9, 5, 9, 3, 0], dtype=torch.int32)
    off = torch.tensor([0, 15, 11, 7, 19], dtype=torch.int32)
    ctx.ss_commit_gather(K_loc, V_loc, idx.to(DEV), cnt.to(DEV), K_dst, V_dst, off.to(DEV))
    st, bits = ctx.ss_poll_status()
    assert st == 0, bits
    ko, vo = oracle.commit_gather(_u16(K_loc), _u16(V_loc), idx.numpy(), cnt.numpy(),
                                  _u16(K0.view(torch.bfloat16)[:, :, 2:2 + cap, 8:]),
                                  _u16(V0.view(torch.bfloat16)[:, :, 2:2 + cap, :d]), off.numpy())
    assert np.array_equal(_u16(K_dst), ko) and np.array_equal(_u16(V_dst), vo)
    # nothing outside the destination view changed
    Kchk, Vchk = Kbig.clone(), Vbig.clone()
    Kchk.view(torch.bfloat16)[:, :, 2:2 + cap, 8:] = K0.view(torch.bfloat16)[:, :, 2:2 + cap, 8:]
    Vchk.view(torch.bfloat16)[:, :, 2:2 + cap, :d] = V0.view(torch.bfloat16)[:, :, 2:2 + cap, :d]
    assert torch.equal(Kchk, K0) and torch.equal(Vchk, V0)
    ctx.close()


def test_commit_gather_device_detected_errors():
    import oracle
    ssb = _ssb()
    B, H_kv, T, d, cap = 3, 2, 4, 128, 6
    ctx = ssb.Context(B, 2 * H_kv, H_kv, d, T, T, 64)
    K_loc = inputs.normal_bf16(1, 1, (B, H_kv, T, d), device=DEV)
    V_loc = inputs.normal_bf16(1, 2, (B, H_kv, T, d), device=DEV)
    K_dst = torch.zeros(B, H_kv, cap, d, dtype=torch.bfloat16, device=DEV)
    V_dst = torch.zeros_like(K_dst)
    idx = torch.tensor([[0, 7, 2, 3], [0, 1, 2, 3], [0, -1, 2, 3]], dtype=torch.int32)
    cnt = torch.tensor([3, 4, 9], dtype=torch.int32)     # request 2: count out of range
    off = torch.tensor([0, 4, 0], dtype=torch.int32)     # request 1: rows 2,3 overflow cap
    ctx.ss_commit_gather(K_loc, V_loc, idx.to(DEV), cnt.to(DEV), K_dst, V_dst, off.to(DEV))
    st, bits = ctx.ss_poll_status()
    assert st == ssb.SS_ERR_DEVICE_FLAG
    assert bits & ssb.SS_DEV_BAD_ACCEPT and bits & ssb.SS_DEV_DST_OVERFLOW
    ko, vo = oracle.commit_gather(_u16(K_loc), _u16(V_loc), idx.numpy(), cnt.numpy(),
                                  np.zeros((B, H_kv, cap, d), np.uint16), np.zeros((B, H_kv, cap, d), np.uint16),
                                  off.numpy())
    assert np.array_equal(_u16(K_dst), ko) and np.array_equal(_u16(V_dst), vo)   # offending rows skipped
    ctx.close()


def test_call_order_and_argument_errors():
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x61, 2, 8, 2, 128, 128, 4, 128, 128)
    lens = [128, 128]
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    K, V, vl = chunks[0]
    O = torch.empty(2, 8, 4, 128, dtype=torch.bfloat16, device=DEV)
    ctx = util.make_ctx(cfg)

    def status(fn, *a):
        with pytest.raises(ssb.SpecStreamError) as e:
            fn(*a)
        return e.value.status

    assert status(ctx.ss_verify_chunk, K, V, vl) == ssb.SS_ERR_STATE          # before begin
    assert status(ctx.ss_verify_finalize, O, None) == ssb.SS_ERR_STATE
    ctx.ss_verify_begin(Q, cfg.scale)
    assert status(ctx.ss_verify_begin, Q, cfg.scale) == ssb.SS_ERR_STATE       # begin twice
    ctx.ss_verify_local(K_loc, V_loc)
    assert status(ctx.ss_verify_local, K_loc, V_loc) == ssb.SS_ERR_STATE       # local twice
    other = torch.cuda.Stream()
    assert status(ctx.ss_verify_chunk, K, V, vl, other) == ssb.SS_ERR_STATE    # another stream
    big = torch.zeros(2, 2, 256, 128, dtype=torch.bfloat16, device=DEV)
    assert status(ctx.ss_verify_chunk, big, big, None) == ssb.SS_ERR_SHAPE     # L_c > max_Lc
    mis = torch.zeros(2 * 2 * 128 * 128 + 8, dtype=torch.bfloat16, device=DEV)[4:-4].view(2, 2, 128, 128)
    assert status(ctx.ss_verify_chunk, mis, V, vl) == ssb.SS_ERR_ALIGN         # base not 16-byte aligned
    assert status(ctx.ss_verify_local, K_loc, V_loc, ssb.SS_MASK_TREE_BITS, None) in (ssb.SS_ERR_ARG, ssb.SS_ERR_STATE)
    ctx.ss_verify_finalize(O, None)                                            # LSE may be NULL
    torch.cuda.synchronize()
    # no chunk at all and no local: every row is empty -> O = 0
    ctx.ss_verify_begin(Q, cfg.scale)
    L = torch.empty(2, 8, 4, dtype=torch.float32, device=DEV)
    ctx.ss_verify_finalize(O, L)
    torch.cuda.synchronize()
    assert (O == 0).all() and torch.isinf(L).all() and (L < 0).all()
    too_many = torch.zeros(3, 8, 4, 128, dtype=torch.bfloat16, device=DEV)
    assert status(ctx.ss_verify_begin, too_many, cfg.scale) == ssb.SS_ERR_SHAPE
    # an aborted round leaves nothing behind: the next round sees only its own calls
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_chunk(K, V, vl)
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_abort()
    assert status(ctx.ss_verify_finalize, O, None) == ssb.SS_ERR_STATE
    ctx.ss_verify_abort()                                                      # no round open: no-op
    ctx.ss_verify_begin(Q, cfg.scale)
    ctx.ss_verify_finalize(O, L)
    torch.cuda.synchronize()
    assert (O == 0).all() and torch.isinf(L).all()
    O2, L2 = util.gpu_case(ctx, cfg, Q, chunks, K_loc, V_loc, bits)
    ref = util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits, groups=[(1, 1)])
    util.compare(cfg, O2, L2, ref)
    ctx.close()
    with pytest.raises(ssb.SpecStreamError):
        ssb.Context(2, 9, 2, 128, 4, 4, 128)       # H_q % H_kv != 0


def _stream_case(cfg, lens, batch_chunks=1, copy_only=0, accept=True, fused=True):
    ssb = _ssb()
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV, fill=0.0)
    host = harness.pinned_history(cfg, lens, chunks)
    # poison the padding of partial host blocks: those tokens must never be read into results
    for b in range(cfg.B):
        j, r = divmod(lens[b], cfg.L_c)
        if r and j < host.shape[1]:
            host[b, j, :, :, r:] = float("nan")
    bufs = harness.stream_buffers(cfg, DEV, len(chunks), batch_chunks, fused=fused)
    for s in range(2):
        bufs["stage_k"][s].fill_(float("nan"))
        bufs["stage_v"][s].fill_(float("nan"))
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    acc = None
    if accept:
        idx, cnt = inputs.make_accept(cfg)
        shape = (cfg.B, cfg.H_kv, cfg.T_q, cfg.d)
        acc = {"idx": idx.to(DEV), "cnt": cnt.to(DEV), "zero": torch.zeros(cfg.B, dtype=torch.int32, device=DEV),
               "ck": torch.zeros(shape, dtype=torch.bfloat16, device=DEV),
               "cv": torch.zeros(shape, dtype=torch.bfloat16, device=DEV),
               "hk": torch.zeros(shape, dtype=torch.bfloat16).pin_memory(),
               "hv": torch.zeros(shape, dtype=torch.bfloat16).pin_memory(), "cnt_host": cnt, "idx_host": idx}
    ctx = ssb.Context(cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, cfg.T_q,
                      cfg.L_c * (1 if fused == "blocks" else batch_chunks))
    desc = harness.make_stream_desc(ssb, cfg, lens, host, DEV, Q, K_loc, V_loc, bits, O, LSE, bufs,
                                  batch_chunks=batch_chunks, accept=acc, copy_only=copy_only)
    stats = ctx.ss_stream_round(desc)
    st, dev_bits = ctx.ss_poll_status()
    assert st == 0, dev_bits
    return ctx, (Q, chunks, K_loc, V_loc, bits), O, LSE, bufs, acc, stats, desc


@pytest.mark.parametrize("fused", [True, False, "blocks"])   # K|V fused / separate / block-major fills
@pytest.mark.parametrize("batch_chunks", [1, 2, 3])
def test_stream_round_matches_oracle_ragged(batch_chunks, fused):
    import oracle
    cfg = inputs.VerifyConfig("v", 0x62, 5, 8, 2, 128, 128, 8, 0, 900, accept=True)
    lens = [900, 0, 128, 257, 513]
    ctx, case, O, LSE, bufs, acc, stats, _ = _stream_case(cfg, lens, batch_chunks, fused=fused)
    n_blocks = sum(-(-l // cfg.L_c) for l in lens)
    n_fills = (max(lens) + cfg.L_c * batch_chunks - 1) // (cfg.L_c * batch_chunks)
    if fused == "blocks":   # per request and fill: one copy for the full blocks, one for a partial block
        want = 0
        for l in lens:
            for f in range(n_fills):
                rem = l - f * batch_chunks * cfg.L_c
                if rem > 0:
                    nfull = min(batch_chunks, rem // cfg.L_c)
                    want += (1 if nfull else 0) + (1 if nfull < batch_chunks and rem - nfull * cfg.L_c > 0 else 0)
        assert stats.copies == want
    else:
        assert stats.copies == (n_blocks if fused else 2 * n_blocks)
    ref = util.oracle_case(cfg, lens, *case)
    util.compare(cfg, O, LSE, ref)
    assert torch.equal(bufs["O_host"], O.cpu()) and torch.equal(bufs["LSE_host"], LSE.cpu())
    assert stats.h2d_bytes == sum(lens) * cfg.H_kv * cfg.d * 4
    assert stats.chunk_calls == (-(-max(lens) // cfg.L_c) if fused == "blocks" else n_fills)
    # committed rows arrived on the host, bit exact
    zero = np.zeros((cfg.B, cfg.H_kv, cfg.T_q, cfg.d), np.uint16)
    ko, vo = oracle.commit_gather(_u16(case[2]), _u16(case[3]), acc["idx_host"].numpy(), acc["cnt_host"].numpy(),
                                  zero, zero, np.zeros(cfg.B, np.int32))
    assert np.array_equal(_u16(acc["hk"]), ko) and np.array_equal(_u16(acc["hv"]), vo)
    ctx.close()


def test_stream_round_head_dim_64():
    # the streamed round with 64-wide heads (host block layout, staging strides and kernels follow d)
    cfg = inputs.VerifyConfig("v", 0x63, 4, 8, 2, 64, 256, 8, 0, 1500, accept=True)
    lens = [1500, 0, 256, 700]
    ctx, case, O, LSE, bufs, acc, stats, _ = _stream_case(cfg, lens, 2, fused="blocks")
    ref = util.oracle_case(cfg, lens, *case)
    util.compare(cfg, O, LSE, ref)
    assert ctx.last_chunk_kernel().startswith("tcgen05")
    assert stats.h2d_bytes == sum(lens) * cfg.H_kv * cfg.d * 4
    ctx.close()


def test_stream_round_copy_only_and_reuse():
    cfg = inputs.VerifyConfig("v", 0x63, 3, 8, 2, 128, 256, 6, 300, 1500)
    lens = inputs.history_lengths(cfg)
    ctx, case, O, LSE, bufs, acc, stats, desc = _stream_case(cfg, lens, accept=False)
    O1 = O.clone()
    desc.copy_only = 1
    s2 = ctx.ss_stream_round(desc)
    assert s2.chunk_calls == 0 and s2.h2d_bytes == stats.h2d_bytes and s2.copies == stats.copies
    desc.copy_only = 0
    ctx.ss_stream_round(desc)        # the context is reusable and deterministic
    assert torch.equal(O.view(torch.int16), O1.view(torch.int16))
    ctx.close()


def test_trace_records_tile_loop():
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x64, 1, 4, 1, 128, 8192, 8, 8192, 8192)
    lens = [8192]
    case = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg)
    ctx.ss_trace_enable(True)
    util.gpu_case(ctx, cfg, *case)
    tr = ctx.ss_trace_read()
    ctx.ss_trace_enable(False)
    for role in (1, 2):      # MMA issuer and softmax lane 0 stamp event 0 at the top of every tile
        tops = [t[0] for t in tr[role] if t[0]]
        assert len(tops) >= 2 and all(b > a for a, b in zip(tops, tops[1:]))
    ctx.close()


def test_export_import_state_shards_the_history_by_chunks():
    """Two contexts each reduce half of the history chunks (what two GPUs would do), export
    their merged states, a third imports both, adds the local segment and finalizes: the result
    equals full attention (Eq. 17: the merge is order-free)."""
    from oracle import streaming
    cfg = inputs.VerifyConfig("v", 0x65, 2, 8, 2, 128, 256, 6, 700, 1500, k_mult=2.0)
    lens = inputs.history_lengths(cfg)
    Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg, lens, DEV)
    rows = cfg.B * cfg.H_q * cfg.T_q
    from paper_2609_33184_b200 import dist as ssdist
    states = []
    shards = [[chunks[j] for j in ssdist.chunk_shard(len(chunks), r, 2)] for r in range(2)]
    assert shards[0] == chunks[0::2] and shards[1] == chunks[1::2]
    for part in shards:
        ctx = util.make_ctx(cfg)
        ml = torch.empty(rows, 2, dtype=torch.float32, device=DEV)
        a = torch.empty(rows, cfg.d, dtype=torch.float32, device=DEV)
        ctx.ss_verify_begin(Q, cfg.scale)
        for K, V, vl in part:
            ctx.ss_verify_chunk(K, V, vl)
        ctx.ss_verify_export_state(ml, a)
        assert ssdist.import_peer_states(ctx, ml, a) == 0   # no process group: no peers
        O_part = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
        ctx.ss_verify_finalize(O_part, None)      # the round stays usable after an export
        torch.cuda.synchronize()
        states.append((ml, a))
        ctx.close()
    # an exported state is (m, l, a) of Eq. 13/14 up to the common reference: check a/l and
    # m + log2 l of one shard against the literal chunk-state routine of the oracle
    ml0, a0 = states[0]
    b, h, i = 1, 5, 3
    row = (b * cfg.H_q + h) * cfg.T_q + i
    kvh = h // cfg.G
    st = streaming.IDENTITY(1, cfg.d)
    for K, V, vl in chunks[0::2]:
        n = int(vl[b])
        st = streaming.merge(st, streaming.chunk_partial(util.f64(Q[b, h, i:i + 1]), util.f64(K[b, kvh, :n]),
                                                         util.f64(V[b, kvh, :n]), cfg.scale))
    o_ref, lse_ref = streaming.finalize(st)
    m, l = ml0[row].tolist()
    assert abs((m + np.log2(l)) * np.log(2.0) - lse_ref[0]) < 1e-3
    assert np.abs(a0[row].cpu().double().numpy() / l - o_ref[0]).max() < 2e-2 * max(1.0, np.abs(o_ref).max())
    # combine the shards
    ctx = util.make_ctx(cfg)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
    ctx.ss_verify_begin(Q, cfg.scale)
    for ml, a in states:
        ctx.ss_verify_import_state(ml, a)
    ctx.ss_verify_local(K_loc, V_loc)
    ctx.ss_verify_finalize(O, LSE)
    torch.cuda.synchronize()
    util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits))
    ctx.close()


def _layer_descs(ssb, cfg, lens, n_layers, bufs, batch_chunks=1):
    """One stream descriptor per layer: own history / Q / local KV / outputs, shared staging."""
    import dataclasses
    layers = []
    for l in range(n_layers):
        cfg_l = dataclasses.replace(cfg, seed=cfg.seed + 17 * l)
        Q, chunks, K_loc, V_loc, bits = util.gen_case(cfg_l, lens, DEV, fill=0.0)
        host = harness.pinned_history(cfg_l, lens, chunks)
        O = torch.zeros(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=DEV)
        LSE = torch.zeros(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=DEV)
        lb = dict(bufs)
        lb["O_host"] = torch.zeros(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16).pin_memory()
        lb["LSE_host"] = torch.zeros(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32).pin_memory()
        desc = harness.make_stream_desc(ssb, cfg_l, lens, host, DEV, Q, K_loc, V_loc, bits, O, LSE, lb,
                                      batch_chunks=batch_chunks)
        layers.append(dict(cfg=cfg_l, case=(Q, chunks, K_loc, V_loc, bits), host=host, O=O, LSE=LSE, desc=desc,
                           bufs=lb))
    return layers


@pytest.mark.parametrize("fused_restore,fills", [(False, 1), (True, 1), (True, 3)])
def test_stream_layers_modes_match_oracle_and_each_other(fused_restore, fills):
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x66, 3, 8, 2, 128, 256, 8, 200, 1300)
    lens = [1300, 200, 777]
    n_chunks = inputs.num_chunks(cfg, lens)
    if fills > 1:   # block-major fills of `fills` chunks, one copy per request and fill
        bufs = harness.stream_buffers(cfg, DEV, n_chunks, fills, fused="blocks")
    else:
        bufs = harness.stream_buffers(cfg, DEV, n_chunks)
    layers = _layer_descs(ssb, cfg, lens, 3, bufs, batch_chunks=fills)
    ctx = ssb.Context(cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, cfg.T_q, cfg.L_c)
    if fused_restore:   # K and V of a request next to each other in one buffer
        rk = torch.full((cfg.B, 2, cfg.H_kv, n_chunks * cfg.L_c, cfg.d), float("nan"), dtype=torch.bfloat16,
                        device=DEV)
        rv = None
    else:
        rk = torch.full((cfg.B, cfg.H_kv, n_chunks * cfg.L_c, cfg.d), float("nan"), dtype=torch.bfloat16, device=DEV)
        rv = torch.full_like(rk, float("nan"))
    outs = {}
    for mode in (ssb.SS_LAYERS_PREFETCH, ssb.SS_LAYERS_STREAM, ssb.SS_LAYERS_RESTORE):
        for L in layers:
            L["O"].zero_()
            L["LSE"].zero_()
        restore = (rk, rv) if mode == ssb.SS_LAYERS_RESTORE else (None, None)
        stats = ctx.ss_stream_layers([L["desc"] for L in layers], mode, *restore)
        st, dev_bits = ctx.ss_poll_status()
        assert st == 0, dev_bits
        assert stats.h2d_bytes == 3 * sum(lens) * cfg.H_kv * cfg.d * 4
        assert stats.chunk_calls == 3 * n_chunks
        outs[mode] = [(L["O"].clone(), L["LSE"].clone()) for L in layers]
        for L in layers:
            assert torch.equal(L["bufs"]["O_host"], L["O"].cpu())
    for L, (O, LSE) in zip(layers, outs[ssb.SS_LAYERS_PREFETCH]):
        util.compare(L["cfg"], O, LSE, util.oracle_case(L["cfg"], lens, *L["case"]))
    for mode in (ssb.SS_LAYERS_STREAM, ssb.SS_LAYERS_RESTORE):
        for (O0, L0), (O1, L1) in zip(outs[ssb.SS_LAYERS_PREFETCH], outs[mode]):
            assert torch.equal(O0.view(torch.int16), O1.view(torch.int16)) and torch.equal(L0, L1)
    ctx.close()


def test_probe_read_folds_every_word_once():
    # the read-bandwidth probe must touch every 16-byte vector of every segment exactly once:
    # its sink is the XOR of all 32-bit words
    import numpy as np
    ssb = _ssb()
    g = torch.Generator(device="cpu").manual_seed(5)
    sizes = [16, 4096 + 16, (1 << 20) + 48, 3 * (1 << 17)]   # bytes: below, across and past a 128 KiB slab
    segs = [torch.randint(-2**31, 2**31 - 1, (n // 4,), dtype=torch.int32, generator=g) for n in sizes]
    want = 0
    for t in segs:
        want ^= int(np.bitwise_xor.reduce(t.numpy().view(np.uint32)))
    dev_segs = [t.to(DEV) for t in segs]
    sink = torch.zeros(1, dtype=torch.int64, device=DEV)
    ssb.ss_probe_read(dev_segs, sink)
    torch.cuda.synchronize()
    assert int(sink.item()) == want
    with pytest.raises(ssb.SpecStreamError):
        ssb.ss_probe_read([dev_segs[1][1:]], sink)   # 4-byte offset: not 16-byte aligned


def test_a_wait_that_nothing_satisfies_gives_up_and_the_context_stays_usable():
    # the chunk kernels bound every wait and report SS_DEV_WAIT_EXPIRED instead of hanging; the
    # self-test kernel makes that routine run out on a barrier nobody completes (50 ms limit)
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x70, 2, 8, 2, 128, 128, 4, 100, 300)
    lens = inputs.history_lengths(cfg)
    case = util.gen_case(cfg, lens, DEV)
    ctx = util.make_ctx(cfg)
    O1, L1 = util.gpu_case(ctx, cfg, *case)
    O1 = O1.clone()
    gave_up = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0 = time.time()
    ctx.ss_selftest_wait_expiry(50, gave_up)
    st, bits = ctx.ss_poll_status(timeout_ms=5000)
    assert time.time() - t0 < 3.0
    assert st == ssb.SS_ERR_DEVICE_FLAG and bits & 8          # SS_DEV_WAIT_EXPIRED
    assert int(gave_up.item()) == 64                          # every waiting thread returned
    assert ctx.ss_poll_status() == (0, 0)                     # reading cleared the word
    O2, _ = util.gpu_case(ctx, cfg, *case)                    # and the context still works
    assert torch.equal(O1.view(torch.int16), O2.view(torch.int16))
    ctx.close()


def test_stream_round_leaves_an_open_round_alone():
    """The streamed entry points refuse to run while the caller has a round open, and the open
    round survives the refusal."""
    ssb = _ssb()
    cfg = inputs.VerifyConfig("v", 0x6a, 2, 8, 2, 128, 128, 4, 0, 300)
    lens = [300, 129]
    ctx, case, O, LSE, bufs, acc, stats, desc = _stream_case(cfg, lens)
    Q, chunks, K_loc, V_loc, bits = case
    O_stream, L_stream = O.clone(), LSE.clone()
    ctx.ss_verify_begin(Q, cfg.scale)
    K, V, vl = chunks[0]
    ctx.ss_verify_chunk(K, V, vl)
    st = ssb.ss_stream_stats()
    assert ctx.lib.ss_stream_round(ctx.handle, C.byref(desc), C.byref(st)) == ssb.SS_ERR_STATE
    arr = (ssb.ss_stream_desc * 1)(desc)
    ld = ssb.ss_layers_desc(1, arr, ssb.SS_LAYERS_STREAM, None, None, 0)
    assert ctx.lib.ss_stream_layers(ctx.handle, C.byref(ld), C.byref(st)) == ssb.SS_ERR_STATE
    # the caller's round is still open and complete-able
    for K, V, vl in chunks[1:]:
        ctx.ss_verify_chunk(K, V, vl)
    ctx.ss_verify_local(K_loc, V_loc)
    O2, L2 = torch.empty_like(O), torch.empty_like(LSE)
    ctx.ss_verify_finalize(O2, L2)
    torch.cuda.synchronize()
    util.compare(cfg, O2, L2, util.oracle_case(cfg, lens, *case))
    assert float((O2.float() - O_stream.float()).abs().max()) <= util.TOL_MAX_O
    ctx.close()
