"""Round drivers shared by bench.py and the GPU tests: the tensors of a workload resident in
HBM, one verification round through the C ABI, and the buffers / descriptor of the streamed
round.  Argument marshalling only: every step of the path runs in the library's kernels."""
from __future__ import annotations

import ctypes as C

import torch

from . import inputs


def kv_bytes(cfg, lens):
    return sum(lens) * cfg.H_kv * cfg.d * 2 * 2


def build_resident(cfg, lens, dev):
    """History as distinct per-chunk device buffers + the round's other tensors."""
    Q = inputs.make_q(cfg, dev)
    K_loc, V_loc = inputs.make_local(cfg, dev)
    bits = inputs.make_mask_bits(cfg, dev)
    chunks = [inputs.make_history_chunk(cfg, j, lens, dev, fill=0.0)
              for j in range(inputs.num_chunks(cfg, lens))]
    return Q, chunks, K_loc, V_loc, bits


def host_valid(cfg, lens, n_chunks):
    """Host copies of every chunk call's valid lengths (scheduling hint), as ctypes arrays."""
    return [(C.c_int32 * cfg.B)(*[max(0, min(cfg.L_c, l - j * cfg.L_c)) for l in lens])
            for j in range(n_chunks)]


def paged_views(cfg, chunks, page_size, dev):
    """Every chunk's own memory re-read as a pool of pages [n_pages, H_kv, page_size, d] with a
    shuffled page table (for throughput runs of the paged chunk call: the tokens a request sees
    are a permutation of the batch's, so the outputs are not those of the contiguous chunks)."""
    assert cfg.L_c % page_size == 0
    ppr = cfg.L_c // page_size
    g = torch.Generator().manual_seed(page_size)
    n_pages = cfg.B * ppr
    out = []
    for K, V, vl in chunks:
        table = torch.randperm(n_pages, generator=g).to(torch.int32).view(cfg.B, ppr).contiguous().to(dev)
        shape = (n_pages, cfg.H_kv, page_size, cfg.d)
        out.append((K.reshape(-1).view(shape), V.reshape(-1).view(shape), table))
    return out


def run_round(ctx, ssb, cfg, Q, chunks, K_loc, V_loc, bits, O, LSE, ev_pair=None, hints=None, paged=None,
              descs=None):
    """One round through the separate calls.  descs (a Context.chunk_descs array for `chunks`):
    the chunks go in with one ss_verify_chunks call instead of one call each."""
    kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
    ctx.ss_verify_begin(Q, cfg.scale)
    if ev_pair:
        ev_pair[0].record()
    if descs is not None and paged is None:
        ctx.ss_verify_chunks(descs, len(chunks))
    for j, (K, V, vl) in enumerate(chunks if (descs is None or paged is not None) else ()):
        if paged is not None:
            Kp, Vp, table = paged[j]
            ctx.ss_verify_chunk_paged(Kp, Vp, table, vl, hints[j] if hints is not None else None)
        elif hints is not None:
            ctx.ss_verify_chunk_hinted(K, V, vl, hints[j])
        else:
            ctx.ss_verify_chunk(K, V, vl)
    if ev_pair:
        ev_pair[1].record()
    ctx.ss_verify_local(K_loc, V_loc, kind, bits if cfg.mask == "tree" else None)
    ctx.ss_verify_finalize(O, LSE)


def pinned_history(cfg, lens, chunks):
    """Host layout of ss_stream_round: per request, per chunk, [2][H_kv][L_c][d] bf16, pinned."""
    J = len(chunks)
    host = torch.empty(cfg.B, J, 2, cfg.H_kv, cfg.L_c, cfg.d, dtype=torch.bfloat16).pin_memory()
    for j, (K, V, _) in enumerate(chunks):
        host[:, j, 0].copy_(K)
        host[:, j, 1].copy_(V)
    torch.cuda.synchronize()
    return host


def make_stream_desc(ssb, cfg, lens, host, dev, Q, K_loc, V_loc, bits, O, LSE, bufs, batch_chunks=1,
                     accept=None, copy_only=0):
    d = ssb.ss_stream_desc()
    d.B, d.T_q, d.L_c, d.scale = cfg.B, cfg.T_q, cfg.L_c, cfg.scale
    ptrs = (C.c_void_p * cfg.B)(*[host[b].data_ptr() for b in range(cfg.B)])
    hl = (C.c_int32 * cfg.B)(*lens)
    d.hist = C.cast(ptrs, C.POINTER(C.c_void_p))
    d.hist_len = C.cast(hl, C.POINTER(C.c_int32))
    d.batch_chunks = batch_chunks
    for s in range(2):
        d.stage_k[s] = bufs["stage_k"][s].data_ptr()
        d.stage_v[s] = bufs["stage_v"][s].data_ptr()
    d.stage_fused = 2 if bufs.get("fused") == "blocks" else (1 if bufs.get("fused") else 0)
    d.scratch_fills = bufs["fills"]
    d.valid_len_host = bufs["vl_host"].data_ptr()
    d.valid_len_dev = bufs["vl_dev"].data_ptr()
    d.Q, d.K_loc, d.V_loc = ssb.as_ss_tensor(Q), ssb.as_ss_tensor(K_loc), ssb.as_ss_tensor(V_loc)
    d.mask_kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
    d.mask_bits = bits.data_ptr() if cfg.mask == "tree" else None
    d.O, d.LSE = O.data_ptr(), LSE.data_ptr()
    if accept is not None:
        d.accept_idx, d.accept_cnt = accept["idx"].data_ptr(), accept["cnt"].data_ptr()
        d.zero_off = accept["zero"].data_ptr()
        d.commit_k, d.commit_v = accept["ck"].data_ptr(), accept["cv"].data_ptr()
        d.host_commit_k, d.host_commit_v = accept["hk"].data_ptr(), accept["hv"].data_ptr()
    d.O_host, d.LSE_host = bufs["O_host"].data_ptr(), bufs["LSE_host"].data_ptr()
    d.copy_only = copy_only
    d._keep = (ptrs, hl)  # keep the ctypes arrays alive
    return d


def stream_buffers(cfg, dev, n_chunks, batch_chunks=1, fused=True):
    """Device staging + scratch of ss_stream_round.  fused: one buffer [B][2 (K,V)][H_kv][Ls][d]
    per slot (each (request, chunk) block is then one copy); fused = "blocks": one buffer
    [B][batch_chunks][2][H_kv][L_c][d] per slot (the adjacent blocks of a request in one copy);
    else separate K and V buffers."""
    Ls = cfg.L_c * batch_chunks
    fills = (n_chunks + batch_chunks - 1) // batch_chunks + 1
    if fused == "blocks":
        fills = fills * batch_chunks   # one valid-length row per chunk call
        kv = [torch.zeros(cfg.B, batch_chunks, 2, cfg.H_kv, cfg.L_c, cfg.d, dtype=torch.bfloat16, device=dev)
              for _ in range(2)]
        stage_k, stage_v = kv, kv
    elif fused:
        kv = [torch.zeros(cfg.B, 2, cfg.H_kv, Ls, cfg.d, dtype=torch.bfloat16, device=dev) for _ in range(2)]
        stage_k, stage_v = [t[:, 0] for t in kv], [t[:, 1] for t in kv]   # views of the fused buffers
    else:
        stage_k = [torch.zeros(cfg.B, cfg.H_kv, Ls, cfg.d, dtype=torch.bfloat16, device=dev) for _ in range(2)]
        stage_v = [torch.zeros(cfg.B, cfg.H_kv, Ls, cfg.d, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    return {
        "stage_k": stage_k, "stage_v": stage_v, "fused": fused,
        "fills": fills,
        "vl_host": torch.zeros(fills * cfg.B, dtype=torch.int32).pin_memory(),
        "vl_dev": torch.zeros(fills * cfg.B, dtype=torch.int32, device=dev),
        "O_host": torch.zeros(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16).pin_memory(),
        "LSE_host": torch.zeros(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32).pin_memory(),
    }
