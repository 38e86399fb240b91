"""Throughput of one verification round for shapes outside the benchmark's five workloads.

    python -m paper_2609_33184_b200.sweep --rows 8 32 64 128 --head-dim 128 --page-size 0 16

For every combination it builds seeded synthetic inputs (B requests, H_kv kv-heads, equal
history lengths, T_q = 8 candidates, H_q chosen so that T_q * H_q / H_kv gives the row count),
runs rounds through the C ABI with the history resident in HBM and prints the KV GB/s of a
round (history bytes / device time, CUDA events, after warm-up) and which chunk kernel ran.
`--page-size P` (P > 0) passes every chunk as shuffled pages of a pool through
ss_verify_chunk_paged.  The inputs of a round exceed L2 (>= 256 MiB of history).

This is a sizing aid: it measures, it checks nothing (parity lives in tests/).
"""
from __future__ import annotations

import argparse

import torch

from . import binding as ssb
from . import build as ssbuild
from . import inputs


def _paged(cfg, chunks, page_size, dev):
    """Every chunk as (pool views, shuffled page table): the chunk's own memory cut into pages."""
    out = []
    ppr = cfg.L_c // page_size
    g = torch.Generator().manual_seed(page_size)
    n_pages = cfg.B * ppr
    for K, V, vl in chunks:
        table = torch.randperm(n_pages, generator=g).to(torch.int32).view(cfg.B, ppr).contiguous().to(dev)
        shape = (n_pages, cfg.H_kv, page_size, cfg.d)
        out.append((K.reshape(-1).view(shape), V.reshape(-1).view(shape), table, vl, vl.tolist()))
    return out


def measure(rows: int, d: int, page_size: int, B: int, H_kv: int, L_c: int, tokens: int, flags: int,
            rounds: int, dev: str):
    T_q = 8 if rows % 8 == 0 else 1
    G = rows // T_q
    cfg = inputs.VerifyConfig("sweep", 7, B, G * H_kv, H_kv, d, L_c, T_q, tokens, tokens)
    lens = inputs.history_lengths(cfg)
    Q = inputs.make_q(cfg, dev)
    K_loc, V_loc = inputs.make_local(cfg, dev)
    chunks = [inputs.make_history_chunk(cfg, j, lens, dev, fill=0.0) for j in range(inputs.num_chunks(cfg, lens))]
    paged = _paged(cfg, chunks, page_size, dev) if page_size else None
    O = torch.empty(B, cfg.H_q, T_q, d, dtype=torch.bfloat16, device=dev)
    LSE = torch.empty(B, cfg.H_q, T_q, dtype=torch.float32, device=dev)
    ctx = ssb.Context(B, cfg.H_q, H_kv, d, T_q, T_q, L_c, max_chunks=len(chunks),
                      flags=ssb.SS_FLAG_OVERLAP_CHUNKS | flags)

    def one_round():
        ctx.ss_verify_begin(Q, cfg.scale)
        if paged:
            for Kp, Vp, table, vl, vl_host in paged:
                ctx.ss_verify_chunk_paged(Kp, Vp, table, vl, vl_host)
        else:
            for K, V, vl in chunks:
                ctx.ss_verify_chunk(K, V, vl)
        ctx.ss_verify_local(K_loc, V_loc)
        ctx.ss_verify_finalize(O, LSE)

    for _ in range(5):
        one_round()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(rounds):
        one_round()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / rounds
    st, bits = ctx.ss_poll_status()
    kernel = ctx.last_chunk_kernel()
    ctx.close()
    if st != 0:
        raise SystemExit(f"device status word set: {bits}")
    kv_bytes = sum(lens) * H_kv * d * 2 * 2
    return kv_bytes / (ms * 1e-3) / 1e9, ms, kernel


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--rows", type=int, nargs="+", default=[8, 32, 64, 128],
                    help="query rows per kv-head (T_q * H_q / H_kv)")
    ap.add_argument("--head-dim", type=int, nargs="+", default=[128], choices=[64, 128])
    ap.add_argument("--page-size", type=int, nargs="+", default=[0], help="0 = contiguous chunks")
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--chunk-tokens", type=int, default=2048)
    ap.add_argument("--history-tokens", type=int, default=16384)
    ap.add_argument("--flags", type=int, default=0, help="extra SS_FLAG_* bits (1 = CUDA cores, 4 = rows on M, 8 = keys on M)")
    ap.add_argument("--rounds", type=int, default=50)
    ap.add_argument("--device", default="cuda:0")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: there is no CPU path")
    ssbuild.build()
    print(f"B={args.batch} H_kv={args.kv_heads} L_c={args.chunk_tokens} history={args.history_tokens} tokens/request")
    for d in args.head_dim:
        for rows in args.rows:
            for ps in args.page_size:
                if ps and args.chunk_tokens % ps:
                    continue
                gbps, ms, kernel = measure(rows, d, ps, args.batch, args.kv_heads, args.chunk_tokens,
                                           args.history_tokens, args.flags, args.rounds, args.device)
                page = f"pages of {ps}" if ps else "contiguous"
                print(f"d={d:3d} rows={rows:4d} {page:13s} {kernel:13s} {gbps:8.0f} GB/s  {ms:.3f} ms/round")


if __name__ == "__main__":
    main()
