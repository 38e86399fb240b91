"""Benchmark of the streamed-KV verification-attention hot path on B200.

A step is one verification round of one layer over one batch: begin -> one chunk call per
history chunk -> local candidate segment -> finalize.  The headline `value` is verify-attention
KV GB/s (committed-history K/V bytes read per round / round time) with the history resident in
HBM; `e2e` is the same metric through ss_stream_round with the history in pinned HOST memory
(host->device copies and the device->host read of the result inside the timed region).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2_qwen3_8b] [--impl reference]

The headline keys (`value`, `roofline`, `e2e`, `cpu_baseline`, ...) belong to --workload and honour
--steps / --warmup.  On one GPU the line also carries `workloads` (the other four workloads,
each with its resident figures, roofline object and clock sample; the streamed workload also
with its own ss_stream_round figures: ragged requests, accept lengths, commit-gather and the
copies back to the host) and `sustained` (the headline round repeated for more than a second
after a warm-up of half a second, clocks sampled inside).

Prints ONE JSON line on stdout.  With --gpus N > 1 (under torchrun) every rank runs the same
per-GPU workload on its own requests (the path shards by request, no data-path collective).
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2609_33184_b200 import dist as ssdist  # noqa: E402
from paper_2609_33184_b200 import inputs  # noqa: E402
from paper_2609_33184_b200.harness import (build_resident, host_valid, kv_bytes, make_stream_desc,  # noqa: E402
                                            paged_views, pinned_history, run_round, stream_buffers)

METRIC = "verify_attention_kv_GBps"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0
E2E_FILL_CHUNKS = 4   # adjacent history chunks per staging-buffer fill of the streamed leg
L2_BYTES = 126 << 20


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            v = json.load(f).get("hbm_gbs")
        if v:
            return float(v), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def tensor_peak():
    """Dense bf16 TFLOP/s, the sustained figure (the chunk kernel is timed inside a long step)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            v = json.load(f).get("bf16_tflops_sustained")
        if v:
            return float(v), "measured (sustained)"
    return FALLBACK_BF16_TFLOPS, "fallback (sustained)"


def ncu_traffic(workload: str, kernel: str, alg_bytes: float = 0.0):
    """DRAM bytes (read + write) per chunk-kernel launch from the tracked table of ncu captures
    (profiles/ncu_traffic.json: one entry per workload with the kernel it was captured on).
    Returns (bytes or None, note): None with the reason when there is no capture for the
    workload or the kernel routed now is not the captured one."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    try:
        with open(path) as f:
            table = json.load(f)
    except Exception:
        return None, "no traffic table"
    e = table.get(workload)
    if not e:
        return None, "no ncu capture of this workload"
    if isinstance(e, list):   # captures of several kernels: the one this run routed, if any
        e = next((x for x in e if x.get("kernel") == kernel), e[0])
    if e.get("kernel") != kernel:
        return None, f"captured on kernel {e.get('kernel')!r}, this run routed {kernel!r}"
    if "ratio_to_algorithmic" in e:
        return float(e["ratio_to_algorithmic"]) * alg_bytes, e.get("note", "")
    return float(e["dram_bytes_per_launch"]), e.get("note", "")


class ClockSampler:
    """nvidia-smi clocks / throttle reasons while the GPU is under load."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0: float, t1: float):
        sm, mx, reasons = [], [], set()
        for t, line in self.samples:
            if not (t0 <= t <= t1):
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def pcie_link(index: int):
    """Current PCIe generation and width of the GPU (nvidia-smi), for the host-link figures."""
    try:
        out = subprocess.run(["nvidia-smi", f"--id={index}",
                              "--query-gpu=pcie.link.gen.current,pcie.link.width.current,pcie.link.gen.max",
                              "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=20).stdout
        g, w, gm = [x.strip() for x in out.strip().splitlines()[0].split(",")]
        return {"gen_current": g, "width_current": w, "gen_max": gm}
    except Exception:
        return None


def cores_used():
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(cfg, lens, Q, chunks, K_loc, V_loc, bits, budget_s=15.0, max_groups=64):
    """The oracle, as it stands, timed on this machine's host cores on a bounded sample of the
    same workload: whole (request, kv-head) groups until about `budget_s` seconds are spent."""
    from tests import util
    cores = cores_used()
    groups = [(b, h) for b in range(cfg.B) for h in range(cfg.H_kv)]
    done, t0, nbytes = 0, time.perf_counter(), 0
    for g in groups[:max_groups]:
        util.oracle_case(cfg, lens, Q, chunks, K_loc, V_loc, bits, groups=[g])
        done += 1
        nbytes += lens[g[0]] * cfg.d * 2 * 2
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{done} of {len(groups)} (request, kv-head) groups of {cfg.name}, all "
                      f"{cfg.G * cfg.T_q} query rows each, {dt:.1f} s",
            "rounds_per_s": nbytes / dt / kv_bytes(cfg, lens)}


def run_reference(args, cfg, rank):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    if rank != 0:
        return
    lens = inputs.history_lengths(cfg)
    # a sample of 2 (request, kv-head) groups per step keeps the whole run within minutes
    small = inputs.scaled(cfg, B=1, H_kv=2, H_q=2 * cfg.G)
    lens1 = lens[:1]
    Q, chunks, K_loc, V_loc, bits = build_resident(small, lens1, "cpu")
    from tests import util
    times = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        util.oracle_case(small, lens1, Q, chunks, K_loc, V_loc, bits)
        if i >= args.warmup:
            times.append(time.perf_counter() - t0)
    dt = sum(times) / len(times)
    val = kv_bytes(small, lens1) / dt / 1e9
    cores = cores_used()
    sample = f"per step: 2 (request, kv-head) groups of {cfg.name} ({lens1[0]} tokens, {cfg.G * cfg.T_q} rows each)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


class Workload:
    """One workload resident on the device: tensors, context, outputs, and the round driver."""

    def __init__(self, ssb, cfg, dev, local_rank, flags, page_size=0, chunk_calls="one"):
        self.ssb, self.cfg, self.dev = ssb, cfg, dev
        self.page_size = page_size
        self.chunk_calls = chunk_calls
        self.lens = inputs.history_lengths(cfg)
        self.Q, self.chunks, self.K_loc, self.V_loc, self.bits = build_resident(cfg, self.lens, dev)
        self.ctx = ssb.Context(cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, cfg.T_q, cfg.L_c,
                               max_chunks=len(self.chunks) or 1, device=local_rank, flags=flags)
        self.O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=dev)
        self.LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=dev)
        self.nbytes = kv_bytes(cfg, self.lens)
        # the host's copy of the valid lengths goes with every chunk (scheduling hint)
        self.hints = host_valid(cfg, self.lens, len(self.chunks)) if self.chunks else None
        # A workload whose history fits in L2 (the tiny chain: 256 KiB) is timed over rotating
        # copies of its history buffers, more than two L2 capacities in total, so that every round
        # reads HBM; the large workloads stream more than L2 per round by themselves.
        self.n_sets = 1
        if 0 < self.nbytes < 2 * L2_BYTES:
            self.n_sets = min(4096, -(-2 * L2_BYTES // self.nbytes))
        self.chunk_sets = [self.chunks] + [[(K.clone(), V.clone(), vl) for (K, V, vl) in self.chunks]
                                           for _ in range(self.n_sets - 1)]
        # --page-size: the same buffers read through shuffled page tables (ss_verify_chunk_paged)
        self.paged_sets = [paged_views(cfg, cs, page_size, dev) for cs in self.chunk_sets] if page_size else None
        # a round's chunks go in with ONE ss_verify_chunks call (--chunk-calls separate: one call each)
        self.descs = ([self.ctx.chunk_descs([cs], self.hints) for cs in self.chunk_sets]
                      if chunk_calls == "one" and not page_size and self.chunks else None)

    def round(self, i=0, ev_pair=None):
        run_round(self.ctx, self.ssb, self.cfg, self.Q, self.chunk_sets[i % self.n_sets], self.K_loc,
                  self.V_loc, self.bits, self.O, self.LSE, ev_pair=ev_pair, hints=self.hints,
                  paged=self.paged_sets[i % self.n_sets] if self.paged_sets else None,
                  descs=self.descs[i % self.n_sets] if self.descs else None)

    def single_call(self, n_rounds):
        """The same round through ss_verify_round (one host call per round), and both ways from
        a C caller (ss_time_rounds: no binding overhead).  Microseconds per round, device time
        of n_rounds rounds enqueued back to back over the rotating history buffers."""
        ssb, cfg = self.ssb, self.cfg
        kind = ssb.SS_MASK_TREE_BITS if cfg.mask == "tree" else ssb.SS_MASK_CHAIN
        bits = self.bits if cfg.mask == "tree" else None
        per_set = [self.ctx.chunk_descs([cs], self.hints) for cs in self.chunk_sets]
        all_sets = self.ctx.chunk_descs(self.chunk_sets, self.hints)
        n = len(self.chunks)

        def one(i):
            self.ctx.ss_verify_round(self.Q, cfg.scale, self.chunk_sets[i % self.n_sets], self.K_loc, self.V_loc,
                                     kind, bits, self.O, self.LSE, descs=per_set[i % self.n_sets])
        for i in range(10):
            one(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n_rounds):
            one(i)
        e1.record()
        torch.cuda.synchronize()
        out = {"python_us_per_round": e0.elapsed_time(e1) / n_rounds * 1e3, "kernel": self.ctx.last_chunk_kernel(),
               "rounds": n_rounds}
        for key, single in (("c_caller_us_per_round", 1), ("c_caller_separate_calls_us_per_round", 0)):
            args = (self.Q, cfg.scale, all_sets, n, self.n_sets, self.K_loc, self.V_loc, kind, bits, self.O, self.LSE)
            self.ctx.ss_time_rounds(*args, min(n_rounds, 50), single)
            out[key] = self.ctx.ss_time_rounds(*args, n_rounds, single) / n_rounds * 1e3
        out["kv_GBps"] = self.nbytes / (out["c_caller_us_per_round"] * 1e-6) / 1e9
        return out

    def l2_note(self):
        if self.n_sets == 1:
            return ("inputs larger than L2 (each round streams all history chunks, "
                    f"{self.nbytes / 2**20:.0f} MiB, through distinct buffers)")
        return (f"history of {self.nbytes / 2**10:.0f} KiB per round: rounds rotate through {self.n_sets} "
                f"copies of the history buffers ({self.n_sets * self.nbytes / 2**20:.0f} MiB, twice L2)")

    def config(self, overlap):
        cfg = self.cfg
        return {"workload": cfg.name, "B": cfg.B, "H_q": cfg.H_q, "H_kv": cfg.H_kv, "d": cfg.d,
                "T_q": cfg.T_q, "L_c": cfg.L_c,
                "history_tokens": self.lens if len(set(self.lens)) > 1 else self.lens[0],
                "chunks_per_round": len(self.chunks),
                "chunk_calls": ("one ss_verify_chunks call per round" if self.descs else "one call per chunk"),
                "mask": cfg.mask,
                "kv_bytes_per_round": self.nbytes, "l2": self.l2_note(),
                "overlap_chunks": overlap, "host_length_hints": self.hints is not None,
                "page_size": self.page_size or None}

    def close(self):
        self.ctx.close()


def timed_rounds(w, steps, warmup, dev, barrier):
    """`warmup` untimed rounds, then exactly `steps` rounds between two events on the launching
    stream, a barrier + synchronize on both sides; max over ranks.  Returns (ms per step,
    launches inside the timed region, wall-clock window)."""
    for i in range(warmup):
        w.round(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = w.ctx.launch_count()
    t0 = time.time()
    e0.record()
    for i in range(steps):
        w.round(i)
    e1.record()
    barrier()
    t1 = time.time()
    launches = w.ctx.launch_count() - launches0
    ms = ssdist.max_over_ranks(e0.elapsed_time(e1), dev)
    st, dev_bits = w.ctx.ss_poll_status()
    if st != 0:
        raise SystemExit(f"device status word set: {dev_bits}")
    return ms / steps, launches, (t0, t1)


def clocks_for(sampler, w, window):
    """Clock sample of a timed window; a window too short for 3 samples is followed by about a
    second of identical untimed rounds that are sampled instead."""
    clocks = sampler.summary(*window)
    clocks["sampled"] = "timed region"
    if clocks["samples"] < 3:
        t0 = time.time()
        while time.time() - t0 < 1.2:
            for _ in range(20):
                w.round()
            torch.cuda.synchronize()
        clocks = sampler.summary(t0, time.time())
        clocks["sampled"] = "identical rounds run right after the timed region (it was too short)"
    return clocks


def chunk_roofline(w, n_rounds):
    """The dominant kernel: chunk attention.  Average launch duration from events around the
    chunk launches of `n_rounds` rounds (gaps between the launches included), against the
    measured HBM copy bandwidth, or - when a launch's useful flops take longer at the sustained
    bf16 peak than its bytes at the HBM peak (many query rows per kv-head: the tree workload) -
    against the tensor peak."""
    cfg = w.cfg
    n_calls = len(w.chunks)
    if not n_calls:
        return None
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range(n_rounds)]
    for i, p in enumerate(pairs):
        w.round(i, ev_pair=p)
    torch.cuda.synchronize()
    kernel = w.ctx.last_chunk_kernel()
    if kernel in ("tcgen05-round", "tcgen05-keys-round"):   # the whole list of chunks went out as one launch
        n_calls = 1
    chunk_ms = statistics.mean(a.elapsed_time(b) for a, b in pairs) / n_calls
    peak, peak_kind = peaks()
    alg_bytes = w.nbytes / n_calls
    achieved = alg_bytes / (chunk_ms * 1e-3) / 1e9
    traffic, traffic_note = ncu_traffic(cfg.name, kernel, alg_bytes)
    roofline = {"bound": "hbm", "kernel": f"chunk attention ({kernel})",
                "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "traffic_note": traffic_note,
                "algorithmic_bytes_per_launch": alg_bytes, "us_per_launch": chunk_ms * 1e3,
                "launches_timed": n_rounds * n_calls}
    alg_flops = 4.0 * cfg.d * cfg.G * cfg.T_q * (alg_bytes / (cfg.d * 2 * 2))
    tpeak, tpeak_kind = tensor_peak()
    if alg_flops / (tpeak * 1e12) > alg_bytes / (peak * 1e9):
        tf = alg_flops / (chunk_ms * 1e-3) / 1e12
        roofline.update({"bound": "tensor", "achieved": tf, "peak": tpeak, "peak_kind": tpeak_kind,
                         "unit": "TFLOP/s", "frac": tf / tpeak, "algorithmic_flops_per_launch": alg_flops,
                         "kv_GBps": achieved})
    return roofline


def round_distribution(w, n):
    rp = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for i, (a, b_) in enumerate(rp):
        a.record()
        w.round(i)
        b_.record()
    torch.cuda.synchronize()
    r_ms = sorted(a.elapsed_time(b_) for a, b_ in rp)
    med, best = r_ms[len(r_ms) // 2], r_ms[0]
    return {"rounds": n, "median_ms": med, "best_ms": best,
            "median_kv_GBps": w.nbytes / (med * 1e-3) / 1e9 if w.nbytes else None,
            "best_kv_GBps": w.nbytes / (best * 1e-3) / 1e9 if w.nbytes else None}


def read_probe(w):
    """Practical read ceiling: a plain streaming read of the same history buffers, same job,
    same clock state (best of 5 timings of 4 sweeps)."""
    ssb = w.ssb
    sink = torch.zeros(1, dtype=torch.int64, device=w.dev)
    bufs_p = [t for (K, V, _) in w.chunks for t in (K, V)]
    p_bytes = sum(t.numel() * t.element_size() for t in bufs_p)
    if p_bytes <= 2 * L2_BYTES:   # inputs must be larger than L2, else it is not an HBM figure
        return None
    best_p, sweeps = 0.0, 4   # a single 2 GiB sweep is 0.3 ms and still shows its ramp-up
    for _ in range(5):
        pa, pb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pa.record()
        for _s in range(sweeps):
            for k in range(0, len(bufs_p), 64):
                ssb.ss_probe_read(bufs_p[k:k + 64], sink)
        pb.record()
        torch.cuda.synchronize()
        best_p = max(best_p, sweeps * p_bytes / (pa.elapsed_time(pb) * 1e-3) / 1e9)
    return {"GBps": best_p, "bytes": p_bytes,
            "note": "ss_probe_read over the same history buffers (allocated bytes, padding included), "
                    "4 sweeps per timing, best of 5"}


def graph_replay(w, n_rep):
    """The same round replayed from a CUDA graph (launch-bound workloads gain; the calls only
    enqueue on the stream, so a captured round can be replayed without the host API)."""
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            w.round()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            w.round()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(n_rep):
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        g_ms = g0.elapsed_time(g1) / n_rep
        return {"ms_per_round": g_ms, "rounds_per_s": 1e3 / g_ms, "kv_GBps": w.nbytes / (g_ms * 1e-3) / 1e9}
    except Exception as e:  # reported, never fatal for the headline number
        return {"error": str(e)[:200]}


_link_peak = {}


def link_probe(dev):
    """Host-link ceiling of this machine: best single pinned->device copy of 512 MiB, same job."""
    if dev in _link_peak:
        return _link_peak[dev]
    probe_h = torch.zeros(512 << 20, dtype=torch.uint8).pin_memory()
    probe_d = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    best = 0.0
    for i in range(12):  # two warm-up copies, then best of 10
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        probe_d.copy_(probe_h, non_blocking=True)
        b_.record()
        torch.cuda.synchronize()
        if i >= 2:
            best = max(best, (512 << 20) / (a.elapsed_time(b_) * 1e-3) / 1e9)
    _link_peak[dev] = best
    return best


def streamed_leg(w, n_rounds, barrier, local_rank, job_bytes, layers=0, rank=0):
    """End to end through ss_stream_round: the history in pinned HOST memory, two staging
    buffers, the host->device copies of the history, Q and the local KV and the device->host
    copies of O / LSE (and, for a workload with accept lengths, commit-gather and the copy of
    the committed rows back to the host) inside the timed region."""
    ssb, cfg, dev = w.ssb, w.cfg, w.dev
    n_calls = len(w.chunks)
    host = pinned_history(cfg, w.lens, w.chunks)
    # fills of E2E_FILL_CHUNKS adjacent chunks in the host's own block order: one copy per
    # request and fill (32 MiB at c2) instead of one per block
    bufs = stream_buffers(cfg, dev, n_calls, E2E_FILL_CHUNKS, fused="blocks")
    Qh, Klh, Vlh = w.Q.cpu().pin_memory(), w.K_loc.cpu().pin_memory(), w.V_loc.cpu().pin_memory()
    Qd, Kld, Vld = torch.empty_like(w.Q), torch.empty_like(w.K_loc), torch.empty_like(w.V_loc)
    acc = None
    if cfg.accept:
        idx, cnt = inputs.make_accept(cfg)
        shape = (cfg.B, cfg.H_kv, cfg.T_q, cfg.d)
        acc = {"idx": idx.to(dev), "cnt": cnt.to(dev), "zero": torch.zeros(cfg.B, dtype=torch.int32, device=dev),
               "ck": torch.zeros(shape, dtype=torch.bfloat16, device=dev),
               "cv": torch.zeros(shape, dtype=torch.bfloat16, device=dev),
               "hk": torch.zeros(shape, dtype=torch.bfloat16).pin_memory(),
               "hv": torch.zeros(shape, dtype=torch.bfloat16).pin_memory()}
    desc = make_stream_desc(ssb, cfg, w.lens, host, dev, Qd, Kld, Vld, w.bits, w.O, w.LSE, bufs,
                            batch_chunks=E2E_FILL_CHUNKS, accept=acc)
    times, stats = [], None
    for i in range(2 + n_rounds):
        barrier()
        t0 = time.perf_counter()
        Qd.copy_(Qh, non_blocking=True)
        Kld.copy_(Klh, non_blocking=True)
        Vld.copy_(Vlh, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        stats = w.ctx.ss_stream_round(desc)  # returns after the D2H of O and LSE (and committed rows)
        dt = time.perf_counter() - t0
        if i >= 2:
            times.append(dt)
    dt = ssdist.max_over_ranks(statistics.mean(times), dev)
    small_in = (Qh.numel() + Klh.numel() + Vlh.numel()) * 2
    best = link_probe(dev)
    # control: the same copy schedule with the attention calls removed
    desc.copy_only = 1
    co = [w.ctx.ss_stream_round(desc).ms_device for _ in range(3)]
    desc.copy_only = 0
    full = [w.ctx.ss_stream_round(desc).ms_device for _ in range(3)]
    h2d_gbps = stats.h2d_bytes / (min(full) * 1e-3) / 1e9
    e2e = {"value": job_bytes / dt / 1e9, "unit": UNIT,
           "h2d_bytes_per_step": int(stats.h2d_bytes + small_in),
           "d2h_bytes_per_step": int(stats.d2h_bytes), "ms_per_step": dt * 1e3,
           "api": f"ss_stream_round (pinned host history, 2 staging buffers, fills of {E2E_FILL_CHUNKS} chunks"
                  + (", commit-gather of the accepted rows + their copy to the host)" if acc else ")"),
           "pipeline_device_ms": min(full), "copy_only_device_ms": min(co),
           "exposed_attention_ms": min(full) - min(co),
           "h2d_GBps": h2d_gbps, "link_peak_GBps": best, "pct_of_link": 100.0 * h2d_gbps / best,
           "copies_per_round": int(stats.copies), "pcie": pcie_link(local_rank)}
    if layers > 1 and rank == 0:
        # N layers sharing this layer's host history (same lengths); one descriptor each
        descs = [make_stream_desc(ssb, cfg, w.lens, host, dev, Qd, Kld, Vld, w.bits, w.O, w.LSE, bufs,
                                  batch_chunks=E2E_FILL_CHUNKS)
                 for _ in range(layers)]
        # restore buffer in the same fused K|V layout as the staging slots (one copy per block)
        rk = torch.empty(cfg.B, 2, cfg.H_kv, n_calls * cfg.L_c, cfg.d, dtype=torch.bfloat16, device=dev)
        abl = {}
        for name, mode in (("stream_prefetch", ssb.SS_LAYERS_PREFETCH), ("stream_layerwise", ssb.SS_LAYERS_STREAM),
                           ("restore_then_verify", ssb.SS_LAYERS_RESTORE)):
            restore = (rk, None) if mode == ssb.SS_LAYERS_RESTORE else (None, None)
            ms_l = [w.ctx.ss_stream_layers(descs, mode, *restore).ms_device for _ in range(3)]
            abl[name + "_ms"] = min(ms_l)
        abl["layers"] = layers
        abl["prefetch_vs_layerwise"] = abl["stream_layerwise_ms"] / abl["stream_prefetch_ms"]
        abl["stream_vs_restore"] = abl["restore_then_verify_ms"] / abl["stream_layerwise_ms"]
        e2e["layers_ablation"] = abl
        del rk
    del host
    return e2e


def sustained_leg(w, sampler, warm_s=0.5, run_s=1.2):
    """The round repeated for `run_s` seconds after `warm_s` seconds of the same rounds, so that
    the SM clock has settled under the power cap; clocks sampled inside the timed window."""
    def burst(seconds):
        n, t0 = 0, time.time()
        while time.time() - t0 < seconds:
            for _ in range(50):
                w.round(n)
                n += 1
            torch.cuda.synchronize()   # keeps the launch queue short; costs one drain per 50 rounds
        return n
    burst(warm_s)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0 = time.time()
    e0.record()
    n, t_end = 0, time.time() + run_s
    while time.time() < t_end:
        for _ in range(50):
            w.round(n)
            n += 1
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    ms = e0.elapsed_time(e1) / n
    peak, peak_kind = peaks()
    val = w.nbytes / (ms * 1e-3) / 1e9
    return {"rounds": n, "seconds": (t1 - t0), "warmup_seconds": warm_s, "ms_per_round": ms,
            "kv_GBps": val, "rounds_per_s": 1e3 / ms, "pct_hbm_nominal_8TBps": 100.0 * val / 8000.0,
            "frac_of_measured_hbm": val / peak, "peak_kind": peak_kind,
            "clocks": sampler.summary(t0, t1)}


def secondary(ssb, name, dev, local_rank, flags, sampler, barrier, overlap):
    """One of the other workloads, briefly: resident rounds for about 0.4 s, the chunk kernel's
    roofline object, a clock sample; the streamed workload also through ss_stream_round."""
    cfg = inputs.CONFIGS[name]
    w = Workload(ssb, cfg, dev, local_rank, flags)
    for i in range(5):
        w.round(i)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(10):
        w.round(i)
    torch.cuda.synchronize()
    est = (time.perf_counter() - t0) / 10
    steps = int(max(50, min(5000, 0.4 / max(est, 1e-6))))
    ms_per_step, launches, window = timed_rounds(w, steps, 10, dev, barrier)
    value = w.nbytes / (ms_per_step * 1e-3) / 1e9
    out = {"config": w.config(overlap), "steps": steps, "kv_GBps": value, "ms_per_round": ms_per_step,
           "rounds_per_s": 1e3 / ms_per_step, "pct_hbm_nominal_8TBps": 100.0 * value / 8000.0,
           "gpu_launches": int(launches), "clocks": clocks_for(sampler, w, window),
           "roofline": chunk_roofline(w, min(steps, 50)),
           "single_call": w.single_call(min(steps, 2000))}
    if cfg.accept:
        out["streamed"] = streamed_leg(w, 3, barrier, local_rank, w.nbytes)
    w.close()
    del w
    torch.cuda.empty_cache()
    return out


def arg_parser():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_qwen3_8b", choices=sorted(inputs.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the other four workloads")
    ap.add_argument("--no-sustained", action="store_true", help="skip the sustained leg")
    ap.add_argument("--no-overlap", action="store_true", help="plain launches (no programmatic dependent launch)")
    ap.add_argument("--simt", action="store_true", help="force the CUDA-core chunk kernel")
    ap.add_argument("--flags", type=int, default=0, help="extra SS_FLAG_* bits for the context (A/B runs)")
    ap.add_argument("--layers", type=int, default=0,
                    help="also time N streamed layers back to back in the three pipeline modes "
                         "(cross-layer prefetch / layer by layer / restore-then-verify)")
    ap.add_argument("--shard", default="requests", choices=["requests", "chunks"],
                    help="how N ranks split the work: by request (every rank its own batch, no data-path "
                         "collective; weak scaling) or by history chunks of ONE batch (each rank reduces its "
                         "chunks, one all-gather of the (m, l, a) states, strong scaling)")
    ap.add_argument("--history-tokens", default="",
                    help="shrink every request's history to this many tokens, or to a seeded ragged range "
                         "LO:HI (small cases for profiler captures)")
    ap.add_argument("--chunk-calls", default="one", choices=["one", "separate"],
                    help="a round's history chunks in one ss_verify_chunks call (default) or one call per chunk")
    ap.add_argument("--page-size", type=int, default=0,
                    help="read the history through shuffled page tables of this many tokens per page "
                         "(ss_verify_chunk_paged; throughput only: the outputs are those of permuted tokens)")
    return ap


def run_chunk_sharded(args, cfg, ssb, rank, local_rank, world, dev, flags):
    """--shard chunks: ONE batch whose history chunks are dealt round-robin to the ranks.  Each
    round: every rank reduces its chunks (rank 0 also the local segment), the merged states are
    exchanged with one all-gather, imported and finalized; time = max over ranks, value = the
    batch's KV bytes per second (strong scaling).  Rank 0 checks sampled groups with the oracle."""
    lens = inputs.history_lengths(cfg)
    n_chunks = inputs.num_chunks(cfg, lens)
    plan = ssdist.chunk_shard_plan(cfg, n_chunks, rank, world)
    Q = inputs.make_q(cfg, dev)
    K_loc, V_loc = inputs.make_local(cfg, dev)
    bits = inputs.make_mask_bits(cfg, dev)
    mine = [inputs.make_history_chunk(cfg, j, lens, dev, fill=0.0) for j in plan.chunks]
    ctx = ssb.Context(cfg.B, cfg.H_q, cfg.H_kv, cfg.d, cfg.T_q, cfg.T_q, cfg.L_c,
                      max_chunks=len(mine) + world, device=local_rank, flags=flags)
    O = torch.empty(cfg.B, cfg.H_q, cfg.T_q, cfg.d, dtype=torch.bfloat16, device=dev)
    LSE = torch.empty(cfg.B, cfg.H_q, cfg.T_q, dtype=torch.float32, device=dev)
    ml, a = ssdist.state_buffers(plan, dev)

    def one_round():
        ssdist.chunk_sharded_round(ctx, ssb, cfg, Q, mine, K_loc, V_loc, bits, O, LSE, plan, ml, a)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        one_round()
    ssdist.barrier(cuda=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0, t0 = ctx.launch_count(), time.time()
    e0.record()
    for _ in range(args.steps):
        one_round()
    e1.record()
    ssdist.barrier(cuda=True)
    t1 = time.time()
    ms = ssdist.max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
    st, dev_bits = ctx.ss_poll_status()
    if st != 0:
        raise SystemExit(f"device status word set: {dev_bits}")
    nbytes = kv_bytes(cfg, lens)
    check = None
    if rank == 0 and not args.no_cpu_baseline:
        # the oracle needs the whole history of the sampled groups: regenerate those chunks here
        from tests import util
        full = [inputs.make_history_chunk(cfg, j, lens, dev, fill=0.0) for j in range(n_chunks)]
        groups = [(0, 0), (cfg.B - 1, cfg.H_kv - 1)]
        worst = util.compare(cfg, O, LSE, util.oracle_case(cfg, lens, Q, full, K_loc, V_loc, bits, groups=groups))
        check = {"groups": groups, "max_abs_O": float(worst["max_o"]), "max_abs_LSE": float(worst["lse"])}
        del full
    if rank == 0:
        sampler.stop()
        value = nbytes / (ms * 1e-3) / 1e9
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "shard": "chunks", "chunks_per_rank": len(plan.chunks),
                       "chunk_calls_per_round": n_chunks, "kv_bytes_per_round": nbytes,
                       "l2": "inputs larger than L2 (distinct chunk buffers)" if nbytes > 2 * L2_BYTES
                             else "history smaller than twice L2: not an HBM figure"},
            "collective": {"kind": "all_gather of the merged (m, l) and a[] states, fp32", "per_round": 2,
                           "bytes_per_rank_per_round": plan.state_bytes},
            "rounds_per_s": 1e3 / ms, "gpu_launches": int(ctx.launch_count() - launches0),
            "clocks": sampler.summary(t0, t1), "oracle_check": check,
        }))
    ctx.close()


def main():
    args = arg_parser().parse_args()
    args.warmup = max(args.warmup, 3)
    cfg = inputs.CONFIGS[args.workload]
    if args.history_tokens:
        lo, _, hi = args.history_tokens.partition(":")
        cfg = inputs.scaled(cfg, len_lo=int(lo), len_hi=int(hi or lo))

    rank, local_rank, world = ssdist.env_rank()
    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    from paper_2609_33184_b200 import binding as ssb
    from paper_2609_33184_b200 import build as ssbuild
    ssbuild.build()

    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    flags = 0 if args.no_overlap else ssb.SS_FLAG_OVERLAP_CHUNKS
    if args.simt:
        flags |= ssb.SS_FLAG_FORCE_SIMT
    flags |= args.flags
    if args.shard == "chunks":
        run_chunk_sharded(args, cfg, ssb, rank, local_rank, world, dev, flags)
        if dist is not None:
            dist.destroy_process_group()
        return
    # per-rank requests: same shapes, rank-specific seed (weak scaling, sharded by request)
    cfg = ssdist.rank_config(cfg, rank)
    w = Workload(ssb, cfg, dev, local_rank, flags, page_size=args.page_size, chunk_calls=args.chunk_calls)

    def barrier():
        ssdist.barrier(cuda=True)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()

    # ---- timed region: exactly K rounds, history resident in HBM -----------------------------
    ms_per_step, launches, window = timed_rounds(w, args.steps, args.warmup, dev, barrier)
    job_bytes = ssdist.sum_over_ranks(w.nbytes, dev)   # whole job: every rank's own requests
    value = job_bytes / (ms_per_step * 1e-3) / 1e9
    clocks = clocks_for(sampler, w, window) if rank == 0 else None

    roofline = chunk_roofline(w, min(args.steps, 50))
    round_stats = round_distribution(w, max(1, min(args.steps, 200)))
    probe = read_probe(w) if len(w.chunks) else None
    graph_info = graph_replay(w, max(10, min(args.steps, 200)))
    single = w.single_call(max(10, min(args.steps, 500))) if len(w.chunks) and not args.page_size else None

    # ---- end to end: history in pinned host memory, streamed through ss_stream_round ---------
    e2e = None
    if not args.no_e2e and len(w.chunks) and not args.page_size:
        e2e = streamed_leg(w, max(3, min(args.steps, 10)), barrier, local_rank, job_bytes,
                           layers=args.layers, rank=rank)

    sustained = None
    if rank == 0 and world == 1 and not args.no_sustained and not args.history_tokens and not args.page_size:
        sustained = sustained_leg(w, sampler)

    cpu = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu = cpu_baseline(cfg, w.lens, w.Q, w.chunks, w.K_loc, w.V_loc, w.bits)
    headline_config = w.config(not args.no_overlap)
    w.close()
    del w
    torch.cuda.empty_cache()

    # ---- the other workloads (one GPU only: they are reported beside the headline, not scaled)
    others = None
    if rank == 0 and world == 1 and not args.no_workloads and not args.history_tokens and not args.page_size:
        others = {}
        for name in sorted(inputs.CONFIGS):
            if name != cfg.name:
                others[name] = secondary(ssb, name, dev, local_rank, flags, sampler, barrier,
                                         not args.no_overlap)
    if rank == 0:
        sampler.stop()
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": headline_config,
            "rounds_per_s": world * 1e3 / ms_per_step,
            "pct_hbm_nominal_8TBps": 100.0 * value / world / 8000.0,
            "round_ms": round_stats, "hbm_read_probe": probe,
            "cuda_graph_replay": graph_info, "single_call": single,
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
            "roofline": roofline, "cpu_baseline": cpu,
            "sustained": sustained, "workloads": others,
        }
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
