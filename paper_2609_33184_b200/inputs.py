"""Seeded synthetic inputs for streamed-KV verification attention.

This module is the only code shared by the CPU oracle's tests and the CUDA
path's tests/benchmarks.  It holds no attention arithmetic: it only produces
tensors (bf16 Q/K/V, ragged lengths, candidate masks, accept indices) from a
counter-based random generator, so both sides see identical bits.

Generator.  Element ``e`` (flat index in the tensor's canonical layout) of
tensor ``tid`` under ``seed`` is

    bf16_rne(mult * normal(seed, tid, e))

where ``normal`` is Box-Muller over two 24-bit uniforms taken from a 64-bit
mix (splitmix64 finaliser) of ``(seed, tid, e)``.  Being index addressed, any
chunking or host layout of the same logical tensor holds the same bits.  All
integer steps are exact in int64 (wrapping), so CPU and GPU agree on the
uniforms; the float32 log/cos of Box-Muller may differ by an ulp between
devices, which is why a test always widens the *same* tensor for the oracle
instead of regenerating it elsewhere.

The workloads mirror one verification round of one layer (Section 4.2 of the
paper): ``T_q`` candidate queries per request (pending committed token plus
drafts) attend to the committed history (contiguous chunks of ``L_c`` tokens)
and to the ``T_loc = T_q`` on-GPU candidate KV under a chain (causal) or tree
(ancestor) mask.  Shapes follow Qwen3- and InternLM2.5-class GQA layers;
values are Gaussians, not real activations.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import torch

# tensor ids (streams of the counter-based generator)
TID_Q, TID_K, TID_V, TID_KLOC, TID_VLOC, TID_LEN, TID_TREE, TID_ACC = range(1, 9)

_M64 = (1 << 64) - 1


def _to_i64(x: int) -> int:
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = _to_i64(0x9E3779B97F4A7C15)
_MIX1 = _to_i64(0xBF58476D1CE4E5B9)
_MIX2 = _to_i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = x ^ _lsr(x, 30)
    x = x * _MIX1
    x = x ^ _lsr(x, 27)
    x = x * _MIX2
    x = x ^ _lsr(x, 31)
    return x


def _key(seed: int, tid: int) -> int:
    """Scalar stream key, computed in Python ints with the same mixer."""
    x = (seed * 0x9E3779B97F4A7C15 + tid * 0xD1B54A32D192ED03 + 0x632BE59BD9B4E019) & _M64
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & _M64
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & _M64
    x ^= x >> 31
    return _to_i64(x)


def u64_stream(seed: int, tid: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """``count`` raw 64-bit words (as int64) of stream (seed, tid) from index ``start``."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix64((idx + 1) * _GOLD + _key(seed, tid))


def normal_stream(seed: int, tid: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """float32 standard normals for flat indices [start, start+count)."""
    w = u64_stream(seed, tid, start, count, device)
    u1 = (_lsr(w, 40).to(torch.float32) + 1.0) * (1.0 / 16777216.0)       # (0, 1]
    u2 = ((_lsr(w, 16) & 0xFFFFFF).to(torch.float32)) * (1.0 / 16777216.0)  # [0, 1)
    r = torch.sqrt(-2.0 * torch.log(u1))
    return r * torch.cos(6.283185307179586 * u2)


def normal_bf16(seed: int, tid: int, shape, mult: float = 1.0, device="cpu",
                start: int = 0, block: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of ``shape`` whose flat element e is bf16(mult*normal(seed,tid,start+e))."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for lo in range(0, n, block):
        c = min(block, n - lo)
        x = normal_stream(seed, tid, start + lo, c, device)
        if mult != 1.0:
            x = x * mult
        out[lo:lo + c] = x.to(torch.bfloat16)
    return out.view(*shape)


def randint_list(seed: int, tid: int, count: int, lo: int, hi: int, start: int = 0) -> List[int]:
    """``count`` integers uniform in [lo, hi] (inclusive), as Python ints."""
    w = u64_stream(seed, tid, start, count, "cpu")
    span = hi - lo + 1
    return [lo + int((int(v) & _M64) % span) for v in w.tolist()]


# --------------------------------------------------------------------------
# candidate masks
# --------------------------------------------------------------------------

def chain_mask_bits(T_q: int, T_loc: Optional[int] = None) -> List[List[int]]:
    """Chain (causal) visibility: query i sees local j <= i.  One word list per row."""
    T_loc = T_q if T_loc is None else T_loc
    words = (T_loc + 63) // 64
    rows = []
    for i in range(T_q):
        bits = (1 << (min(i, T_loc - 1) + 1)) - 1
        rows.append([(bits >> (64 * w)) & _M64 for w in range(words)])
    return rows


def random_tree(seed: int, sub: int, n_nodes: int = 64, max_depth: int = 6,
                max_children: int = 4) -> List[int]:
    """Parent array of a seeded candidate tree in BFS order (parent < child).

    Node 0 is the root (the pending committed token) at depth 0.  Nodes are
    popped FIFO; a node at depth < max_depth receives U{1..max_children}
    children until ``n_nodes`` exist.  If the frontier empties first the draw
    is repeated with the next sub-seed.
    """
    attempt = 0
    while True:
        draws = randint_list(seed, TID_TREE, 4 * n_nodes, 1, max_children,
                             start=(sub * 1024 + attempt) * 4 * n_nodes)
        parent = [-1]
        depth = [0]
        head = 0
        k = 0
        while head < len(parent) and len(parent) < n_nodes:
            p = head
            head += 1
            if depth[p] >= max_depth:
                continue
            c = min(draws[k], n_nodes - len(parent))
            k += 1
            for _ in range(c):
                parent.append(p)
                depth.append(depth[p] + 1)
        if len(parent) == n_nodes:
            return parent
        attempt += 1


def tree_mask_bits(parent: List[int]) -> List[List[int]]:
    """Ancestor-or-self bit rows: row i has bit j set iff j is i or an ancestor of i."""
    n = len(parent)
    words = (n + 63) // 64
    acc = [0] * n
    for i in range(n):
        acc[i] = (acc[parent[i]] if parent[i] >= 0 else 0) | (1 << i)
    return [[(acc[i] >> (64 * w)) & _M64 for w in range(words)] for i in range(n)]


def mask_bits_tensor(rows_per_request: List[List[List[int]]], device="cpu") -> torch.Tensor:
    """[B, T_q, words] int64 tensor holding the uint64 bit patterns."""
    t = torch.tensor([[[_to_i64(w) for w in row] for row in rows] for rows in rows_per_request],
                     dtype=torch.int64)
    return t.to(device)


def mask_bits_to_bool(bits: torch.Tensor, T_loc: int) -> torch.Tensor:
    """[B, T_q, words] int64 -> [B, T_q, T_loc] bool."""
    b = bits.cpu()
    j = torch.arange(T_loc)
    w = b[:, :, (j // 64)]
    return ((w >> (j % 64)) & 1).bool()


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------

@dataclasses.dataclass
class VerifyConfig:
    name: str
    seed: int
    B: int
    H_q: int
    H_kv: int
    d: int
    L_c: int
    T_q: int
    len_lo: int
    len_hi: int                 # history lengths uniform in [len_lo, len_hi]
    mask: str = "chain"         # "chain" | "tree"
    k_mult: float = 1.0
    accept: bool = False        # draw accept lengths (streamed workload)

    @property
    def G(self) -> int:
        return self.H_q // self.H_kv

    @property
    def scale(self) -> float:
        return 1.0 / float(self.d) ** 0.5


def _seed(c: int) -> int:
    return 0x5EC57000 + c


CONFIGS = {
    # tiny chain verify: 4 chunks of 256, 4 drafts + 1 pending token
    "c1_tiny_chain": VerifyConfig("c1_tiny_chain", _seed(1), 1, 4, 1, 64, 256, 5, 1024, 1024),
    # Qwen3-8B-shaped layer, K scaled by 0.5
    "c2_qwen3_8b": VerifyConfig("c2_qwen3_8b", _seed(2), 16, 32, 8, 128, 2048, 8, 32768, 32768,
                                k_mult=0.5),
    # InternLM2.5-7B-shaped layer, ragged histories, last chunk partial
    "c3_internlm25_7b_ragged": VerifyConfig("c3_internlm25_7b_ragged", _seed(3), 8, 32, 8, 128,
                                            4096, 6, 65536, 131072),
    # 64-node candidate tree
    "c4_tree": VerifyConfig("c4_tree", _seed(4), 4, 40, 8, 128, 4096, 64, 65536, 65536,
                            mask="tree"),
    # streamed end-to-end layer: histories in pinned host memory
    "c5_streamed": VerifyConfig("c5_streamed", _seed(5), 32, 32, 8, 128, 2048, 8, 8192, 65536,
                                accept=True),
}


def history_lengths(cfg: VerifyConfig) -> List[int]:
    if cfg.len_lo == cfg.len_hi:
        return [cfg.len_lo] * cfg.B
    return randint_list(cfg.seed, TID_LEN, cfg.B, cfg.len_lo, cfg.len_hi)


def make_q(cfg: VerifyConfig, device="cpu") -> torch.Tensor:
    return normal_bf16(cfg.seed, TID_Q, (cfg.B, cfg.H_q, cfg.T_q, cfg.d), device=device)


def make_local(cfg: VerifyConfig, device="cpu"):
    shape = (cfg.B, cfg.H_kv, cfg.T_q, cfg.d)
    k = normal_bf16(cfg.seed, TID_KLOC, shape, mult=cfg.k_mult, device=device)
    v = normal_bf16(cfg.seed, TID_VLOC, shape, device=device)
    return k, v


def _req_base(cfg: VerifyConfig, b: int) -> int:
    # element offset of request b's history in the K (or V) stream; requests are
    # spaced by the maximum length so a request's bits do not depend on the others.
    return b * cfg.H_kv * cfg.len_hi * cfg.d


def make_history_block(cfg: VerifyConfig, tid: int, b: int, h: int, t0: int, n: int,
                       device="cpu") -> torch.Tensor:
    """[n, d] bf16: tokens [t0, t0+n) of kv-head h of request b (canonical layout
    history[b][H_kv][len_hi][d])."""
    mult = cfg.k_mult if tid == TID_K else 1.0
    start = _req_base(cfg, b) + (h * cfg.len_hi + t0) * cfg.d
    return normal_bf16(cfg.seed, tid, (n, cfg.d), mult=mult, device=device, start=start)


def make_history_chunk(cfg: VerifyConfig, j: int, lens: List[int], device="cpu",
                       fill: Optional[float] = None):
    """Chunk j for the whole batch: K, V [B, H_kv, L_c, d] bf16 and valid_len [B] int32.

    Tokens past a request's valid length hold ``fill`` (NaN by default on purpose:
    they are invisible and their memory may contain anything).
    """
    fill = float("nan") if fill is None else fill
    K = torch.full((cfg.B, cfg.H_kv, cfg.L_c, cfg.d), fill, dtype=torch.bfloat16, device=device)
    V = torch.full_like(K, fill)
    valid = []
    for b in range(cfg.B):
        n = max(0, min(cfg.L_c, lens[b] - j * cfg.L_c))
        valid.append(n)
        if n == 0:
            continue
        for h in range(cfg.H_kv):
            K[b, h, :n] = make_history_block(cfg, TID_K, b, h, j * cfg.L_c, n, device)
            V[b, h, :n] = make_history_block(cfg, TID_V, b, h, j * cfg.L_c, n, device)
    return K, V, torch.tensor(valid, dtype=torch.int32, device=device)


def num_chunks(cfg: VerifyConfig, lens: List[int]) -> int:
    return max((l + cfg.L_c - 1) // cfg.L_c for l in lens) if lens else 0


def make_mask_bits(cfg: VerifyConfig, device="cpu") -> torch.Tensor:
    if cfg.mask == "chain":
        rows = [chain_mask_bits(cfg.T_q) for _ in range(cfg.B)]
    else:
        rows = [tree_mask_bits(random_tree(cfg.seed, b, cfg.T_q)) for b in range(cfg.B)]
    return mask_bits_tensor(rows, device)


def make_accept(cfg: VerifyConfig):
    """Accepted local rows: a_b ~ U{0..T_q-1} drafts accepted; committed rows are local
    0..a_b (the pending token's KV is always committed), so cnt_b = a_b + 1."""
    a = randint_list(cfg.seed, TID_ACC, cfg.B, 0, cfg.T_q - 1)
    idx = torch.arange(cfg.T_q, dtype=torch.int32).repeat(cfg.B, 1)
    cnt = torch.tensor([x + 1 for x in a], dtype=torch.int32)
    return idx, cnt


def scaled(cfg: VerifyConfig, **kw) -> VerifyConfig:
    """A copy of ``cfg`` with fields replaced (smaller histories for oracle-sized tests)."""
    return dataclasses.replace(cfg, **kw)
