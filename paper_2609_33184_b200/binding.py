"""ctypes binding of libspecstream: the same entry points as include/specstream.h.

Argument marshalling only - every step of the path runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  There is no fallback: if
the shared library is missing or the device is not sm_100, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libspecstream.so")

SS_OK = 0
STATUS_NAMES = ["SS_OK", "SS_ERR_ARG", "SS_ERR_SHAPE", "SS_ERR_ALIGN", "SS_ERR_STATE",
                "SS_ERR_CAPACITY", "SS_ERR_UNSUPPORTED", "SS_ERR_CUDA", "SS_ERR_DEVICE_FLAG",
                "SS_ERR_TIMEOUT"]
(SS_ERR_ARG, SS_ERR_SHAPE, SS_ERR_ALIGN, SS_ERR_STATE, SS_ERR_CAPACITY, SS_ERR_UNSUPPORTED,
 SS_ERR_CUDA, SS_ERR_DEVICE_FLAG, SS_ERR_TIMEOUT) = range(1, 10)
SS_DEV_BAD_VALID_LEN, SS_DEV_BAD_ACCEPT, SS_DEV_DST_OVERFLOW, SS_DEV_WAIT_EXPIRED, SS_DEV_BAD_PAGE = 1, 2, 4, 8, 16
SS_FLAG_FORCE_SIMT, SS_FLAG_OVERLAP_CHUNKS, SS_FLAG_ROWS_ON_M, SS_FLAG_KEYS_ON_M, SS_FLAG_STREAM_TIMING = 1, 2, 4, 8, 16
SS_MASK_CHAIN, SS_MASK_TREE_BITS = 0, 1

EXPORTS = ["ss_workspace_bytes", "ss_create", "ss_destroy", "ss_verify_begin", "ss_verify_chunk",
           "ss_verify_local", "ss_verify_finalize", "ss_commit_gather", "ss_poll_status",
           "ss_stream_round", "ss_strerror", "ss_sizeof_stream_desc", "ss_last_cuda_error", "ss_launch_count",
           "ss_last_chunk_kernel", "ss_trace_enable", "ss_trace_read", "ss_verify_round_static", "ss_verify_chunk_hinted", "ss_verify_export_state",
           "ss_verify_import_state", "ss_stream_layers", "ss_tier_create", "ss_tier_destroy",
           "ss_tier_reset", "ss_tier_get", "ss_tier_tail", "ss_tier_commit", "ss_tier_migrate", "ss_tier_poll",
           "ss_tier_d2h_bytes", "ss_verify_chunk_paged", "ss_width_create", "ss_width_destroy",
           "ss_width_observe", "ss_width_next", "ss_width_estimate", "ss_cohort_build", "ss_probe_read",
           "ss_selftest_wait_expiry", "ss_verify_abort", "ss_cta_log_set", "ss_get_stats", "ss_verify_round", "ss_verify_chunks",
           "ss_time_rounds"]


class ss_stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("launches", "rounds", "rows", "chunk_calls", "kv_bytes",
                                         "last_round_ns", "last_transfer_ns", "last_chunk_ns",
                                         "last_tail_ns", "last_wait_ns")]


class ss_config(C.Structure):
    _fields_ = [("max_B", C.c_int32), ("H_q", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32),
                ("max_Tq", C.c_int32), ("max_Tloc", C.c_int32), ("max_Lc", C.c_int32),
                ("max_chunks", C.c_int32), ("device", C.c_int32), ("flags", C.c_uint32)]


class ss_tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_b", C.c_int64), ("stride_h", C.c_int64),
                ("stride_t", C.c_int64)]


class ss_stream_desc(C.Structure):
    _fields_ = [("B", C.c_int32), ("T_q", C.c_int32), ("L_c", C.c_int32), ("scale", C.c_float),
                ("hist", C.POINTER(C.c_void_p)), ("hist_len", C.POINTER(C.c_int32)),
                ("batch_chunks", C.c_int32),
                ("stage_k", C.c_void_p * 2), ("stage_v", C.c_void_p * 2),
                ("scratch_fills", C.c_int32),
                ("valid_len_host", C.c_void_p), ("valid_len_dev", C.c_void_p),
                ("Q", ss_tensor), ("K_loc", ss_tensor), ("V_loc", ss_tensor),
                ("mask_kind", C.c_int), ("mask_bits", C.c_void_p),
                ("O", C.c_void_p), ("LSE", C.c_void_p),
                ("accept_idx", C.c_void_p), ("accept_cnt", C.c_void_p), ("zero_off", C.c_void_p),
                ("commit_k", C.c_void_p), ("commit_v", C.c_void_p),
                ("host_commit_k", C.c_void_p), ("host_commit_v", C.c_void_p),
                ("O_host", C.c_void_p), ("LSE_host", C.c_void_p),
                ("copy_only", C.c_int32),
                ("tail_K", ss_tensor), ("tail_V", ss_tensor), ("tail_Lc", C.c_int32),
                ("tail_len", C.c_void_p), ("commit_cap", C.c_int32), ("stage_fused", C.c_int32)]


class ss_tier_config(C.Structure):
    _fields_ = [("B", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32), ("L_c", C.c_int32),
                ("tail_target", C.c_int32), ("granularity", C.c_int32), ("tail_capacity", C.c_int32)]


class ss_task(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("layer", "width", "dtype", "n_kv", "d_h", "chunk_size",
                                         "request_id", "hist_len")]


class ss_width_config(C.Structure):
    _fields_ = [("n_widths", C.c_int32), ("widths", C.c_int32 * 8), ("sample_rounds", C.c_int32),
                ("switch_threshold", C.c_float), ("ema", C.c_float)]


class ss_width_obs(C.Structure):
    _fields_ = [("t_draft", C.c_float), ("t_transfer", C.c_float), ("t_compute", C.c_float),
                ("t_other", C.c_float), ("committed", C.c_int32)]


class ss_layers_desc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("layers", C.POINTER(ss_stream_desc)), ("mode", C.c_int32),
                ("restore_k", C.c_void_p), ("restore_v", C.c_void_p), ("restore_tokens", C.c_int64)]


SS_LAYERS_PREFETCH, SS_LAYERS_STREAM, SS_LAYERS_RESTORE = 0, 1, 2


class ss_chunk_desc(C.Structure):
    _fields_ = [("K", ss_tensor), ("V", ss_tensor), ("L_c", C.c_int32), ("valid_len", C.c_void_p),
                ("valid_len_host", C.POINTER(C.c_int32))]


class ss_static_round(C.Structure):
    _fields_ = [("B", C.c_int32), ("H_q", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32),
                ("T_q", C.c_int32), ("T_loc", C.c_int32), ("L_c", C.c_int32), ("scale", C.c_float),
                ("Q", ss_tensor), ("K", ss_tensor), ("V", ss_tensor), ("valid_len", C.c_void_p),
                ("K_loc", ss_tensor), ("V_loc", ss_tensor), ("mask_kind", C.c_int),
                ("mask_bits", C.c_void_p), ("O", C.c_void_p), ("LSE", C.c_void_p),
                ("status", C.c_void_p)]


SS_STATIC_SCRATCH_BYTES = 4 << 20


class ss_stream_stats(C.Structure):
    _fields_ = [("ms_total", C.c_double), ("ms_device", C.c_float), ("h2d_bytes", C.c_int64),
                ("d2h_bytes", C.c_int64), ("chunk_calls", C.c_int32), ("copies", C.c_int32)]


_lib = None


def load() -> C.CDLL:
    """Load the shared library (raises if it has not been built)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with "
                           "`python -m paper_2609_33184_b200.build` (there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, u32p = C.c_void_p, C.c_int32, C.POINTER(C.c_uint32)
    lib.ss_workspace_bytes.restype = C.c_size_t
    lib.ss_workspace_bytes.argtypes = [C.POINTER(ss_config)]
    lib.ss_create.restype = C.c_int
    lib.ss_create.argtypes = [C.POINTER(vp), C.POINTER(ss_config), vp, C.c_size_t]
    lib.ss_destroy.restype = C.c_int
    lib.ss_destroy.argtypes = [vp]
    lib.ss_verify_begin.restype = C.c_int
    lib.ss_verify_begin.argtypes = [vp, ss_tensor, i32, i32, C.c_float, vp]
    lib.ss_verify_chunk.restype = C.c_int
    lib.ss_verify_chunk.argtypes = [vp, ss_tensor, ss_tensor, i32, vp, vp]
    lib.ss_verify_chunk_hinted.restype = C.c_int
    lib.ss_verify_chunk_hinted.argtypes = [vp, ss_tensor, ss_tensor, i32, vp, C.POINTER(C.c_int32), vp]
    lib.ss_verify_chunk_paged.restype = C.c_int
    lib.ss_verify_chunk_paged.argtypes = [vp, ss_tensor, ss_tensor, i32, i32, vp, i32, vp, C.POINTER(C.c_int32), vp]
    lib.ss_verify_local.restype = C.c_int
    lib.ss_verify_local.argtypes = [vp, ss_tensor, ss_tensor, i32, C.c_int, vp, vp]
    lib.ss_verify_export_state.restype = C.c_int
    lib.ss_verify_export_state.argtypes = [vp, vp, vp, vp]
    lib.ss_verify_import_state.restype = C.c_int
    lib.ss_verify_import_state.argtypes = [vp, vp, vp, vp]
    lib.ss_verify_finalize.restype = C.c_int
    lib.ss_verify_finalize.argtypes = [vp, vp, vp, vp]
    lib.ss_verify_abort.restype = C.c_int
    lib.ss_verify_abort.argtypes = [vp]
    lib.ss_commit_gather.restype = C.c_int
    lib.ss_commit_gather.argtypes = [vp, ss_tensor, ss_tensor, i32, i32, vp, vp, ss_tensor,
                                     ss_tensor, i32, vp, vp]
    lib.ss_poll_status.restype = C.c_int
    lib.ss_poll_status.argtypes = [vp, vp, i32, u32p]
    lib.ss_stream_round.restype = C.c_int
    lib.ss_stream_round.argtypes = [vp, C.POINTER(ss_stream_desc), C.POINTER(ss_stream_stats)]
    lib.ss_stream_layers.restype = C.c_int
    lib.ss_stream_layers.argtypes = [vp, C.POINTER(ss_layers_desc), C.POINTER(ss_stream_stats)]
    i32p, i64p = C.POINTER(C.c_int32), C.POINTER(C.c_int64)
    lib.ss_tier_create.restype = C.c_int
    lib.ss_tier_create.argtypes = [C.POINTER(vp), C.POINTER(ss_tier_config), C.POINTER(vp), i64p, vp, vp, vp, vp,
                                   vp, vp]
    lib.ss_tier_destroy.restype = C.c_int
    lib.ss_tier_destroy.argtypes = [vp]
    lib.ss_tier_reset.restype = C.c_int
    lib.ss_tier_reset.argtypes = [vp, i32p, i32p, vp]
    lib.ss_tier_get.restype = C.c_int
    lib.ss_tier_get.argtypes = [vp, i32p, i32p, i32p, i32p]
    lib.ss_tier_tail.restype = C.c_int
    lib.ss_tier_tail.argtypes = [vp, C.POINTER(ss_tensor), C.POINTER(ss_tensor), C.POINTER(vp)]
    lib.ss_tier_commit.restype = C.c_int
    lib.ss_tier_commit.argtypes = [vp, i32p, vp]
    lib.ss_tier_migrate.restype = C.c_int
    lib.ss_tier_migrate.argtypes = [vp, vp, i32p]
    lib.ss_tier_poll.restype = C.c_int
    lib.ss_tier_poll.argtypes = [vp, i32, vp, i32p]
    lib.ss_tier_d2h_bytes.restype = C.c_int64
    lib.ss_tier_d2h_bytes.argtypes = [vp]
    lib.ss_width_create.restype = C.c_int
    lib.ss_width_create.argtypes = [C.POINTER(vp), C.POINTER(ss_width_config)]
    lib.ss_width_destroy.restype = C.c_int
    lib.ss_width_destroy.argtypes = [vp]
    lib.ss_width_observe.restype = C.c_int
    lib.ss_width_observe.argtypes = [vp, i32, C.POINTER(ss_width_obs)]
    lib.ss_width_next.restype = i32
    lib.ss_width_next.argtypes = [vp]
    lib.ss_width_estimate.restype = C.c_int
    lib.ss_width_estimate.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                      C.POINTER(C.c_double), C.POINTER(C.c_int32)]
    lib.ss_cohort_build.restype = i32
    lib.ss_cohort_build.argtypes = [C.POINTER(ss_task), i32, i32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.ss_strerror.restype = C.c_char_p
    lib.ss_strerror.argtypes = [C.c_int]
    lib.ss_sizeof_stream_desc.restype = C.c_size_t
    lib.ss_sizeof_stream_desc.argtypes = []
    lib.ss_last_cuda_error.restype = i32
    lib.ss_last_cuda_error.argtypes = [vp]
    lib.ss_trace_enable.restype = C.c_int
    lib.ss_trace_enable.argtypes = [vp, i32]
    lib.ss_verify_chunks.restype = C.c_int
    lib.ss_verify_chunks.argtypes = [vp, C.POINTER(ss_chunk_desc), i32, vp]
    lib.ss_verify_round.restype = C.c_int
    lib.ss_verify_round.argtypes = [vp, ss_tensor, i32, i32, C.c_float, C.POINTER(ss_chunk_desc), i32, ss_tensor,
                                    ss_tensor, i32, C.c_int, vp, vp, vp, vp]
    lib.ss_time_rounds.restype = C.c_int
    lib.ss_time_rounds.argtypes = [vp, ss_tensor, i32, i32, C.c_float, C.POINTER(ss_chunk_desc), i32, i32,
                                   ss_tensor, ss_tensor, i32, C.c_int, vp, vp, vp, vp, i32, i32,
                                   C.POINTER(C.c_float)]
    lib.ss_get_stats.restype = C.c_int
    lib.ss_get_stats.argtypes = [vp, C.POINTER(ss_stats)]
    lib.ss_cta_log_set.restype = C.c_int
    lib.ss_cta_log_set.argtypes = [vp, vp, i32]
    lib.ss_trace_read.restype = i32
    lib.ss_trace_read.argtypes = [vp, C.POINTER(C.c_uint64), i32]
    lib.ss_verify_round_static.restype = C.c_int
    lib.ss_verify_round_static.argtypes = [C.POINTER(ss_static_round), vp]
    lib.ss_launch_count.restype = C.c_int64
    lib.ss_launch_count.argtypes = [vp]
    lib.ss_last_chunk_kernel.restype = C.c_char_p
    lib.ss_last_chunk_kernel.argtypes = [vp]
    lib.ss_selftest_wait_expiry.restype = C.c_int
    lib.ss_selftest_wait_expiry.argtypes = [vp, i32, vp, vp]
    lib.ss_probe_read.restype = C.c_int
    lib.ss_probe_read.argtypes = [C.POINTER(vp), C.POINTER(C.c_size_t), i32, vp, vp]
    _lib = lib
    return lib


class SpecStreamError(RuntimeError):
    def __init__(self, status: int, where: str, cuda: int = 0):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        msg = f"{where}: {name} ({load().ss_strerror(status).decode()})"
        if cuda:
            msg += f" [cudaError {cuda}]"
        super().__init__(msg)


def as_ss_tensor(t: torch.Tensor) -> ss_tensor:
    """[B, H, T, d] bf16 torch tensor -> ss_tensor (strides in elements)."""
    assert t.dim() == 4 and t.dtype == torch.bfloat16 and t.stride(3) == 1, (t.shape, t.dtype, t.stride())
    return ss_tensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2))


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    """cudaStream_t of `stream`, or of torch's current stream on the current device (the raw
    getter costs 0.1 us per call against 3 us for building a torch.cuda.Stream object, which
    matters for rounds of a few small launches)."""
    if stream is not None:
        return stream.cuda_stream
    if _raw_stream is not None:
        return _raw_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


class Context:
    """Owns an ss_ctx and its torch-allocated workspace.  Methods mirror the C entry points."""

    def __init__(self, max_B: int, H_q: int, H_kv: int, d: int, max_Tq: int, max_Tloc: int,
                 max_Lc: int, max_chunks: int = 0, device: int = 0, flags: int = 0):
        self.lib = load()
        self.cfg = ss_config(max_B, H_q, H_kv, d, max_Tq, max_Tloc, max_Lc, max_chunks, device, flags)
        n = self.lib.ss_workspace_bytes(C.byref(self.cfg))
        if n == 0:
            raise SpecStreamError(SS_ERR_SHAPE, "ss_workspace_bytes")
        self.workspace = torch.empty(n, dtype=torch.uint8, device=f"cuda:{device}")
        self.handle = C.c_void_p()
        st = self.lib.ss_create(C.byref(self.handle), C.byref(self.cfg), self.workspace.data_ptr(), n)
        if st != SS_OK:
            raise SpecStreamError(st, "ss_create")
        self.H_q, self.H_kv, self.d = H_q, H_kv, d
        self._dev = device

    def _sp(self, stream) -> int:
        """cudaStream_t of `stream`, else torch's current stream on this context's device."""
        if stream is not None:
            return stream.cuda_stream
        if _raw_stream is not None:
            return _raw_stream(self._dev)
        return torch.cuda.current_stream(self._dev).cuda_stream

    def _check(self, st: int, where: str):
        if st != SS_OK:
            raise SpecStreamError(st, where, self.lib.ss_last_cuda_error(self.handle))

    def close(self):
        if self.handle:
            self.lib.ss_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- the five calls of the path -------------------------------------------------------
    def ss_verify_begin(self, Q: torch.Tensor, scale: float, stream=None):
        B, H_q, T_q, d = Q.shape
        assert H_q == self.H_q and d == self.d
        self._check(self.lib.ss_verify_begin(self.handle, as_ss_tensor(Q), B, T_q, scale,
                                             self._sp(stream)), "ss_verify_begin")

    def ss_verify_chunk(self, K: torch.Tensor, V: torch.Tensor, valid_len: Optional[torch.Tensor] = None,
                        stream=None):
        L_c = K.shape[2]
        if valid_len is not None:
            assert valid_len.dtype == torch.int32 and valid_len.is_cuda
        self._check(self.lib.ss_verify_chunk(self.handle, as_ss_tensor(K), as_ss_tensor(V), L_c,
                                             _ptr(valid_len), self._sp(stream)), "ss_verify_chunk")

    def ss_verify_chunk_hinted(self, K: torch.Tensor, V: torch.Tensor, valid_len: torch.Tensor,
                               valid_len_host, stream=None):
        """valid_len_host: a ctypes int32 array (or a list of ints) with the same values as valid_len."""
        L_c = K.shape[2]
        if not isinstance(valid_len_host, C.Array):
            valid_len_host = (C.c_int32 * len(valid_len_host))(*valid_len_host)
        self._check(self.lib.ss_verify_chunk_hinted(self.handle, as_ss_tensor(K), as_ss_tensor(V), L_c,
                                                    _ptr(valid_len), valid_len_host, self._sp(stream)),
                    "ss_verify_chunk_hinted")

    def ss_verify_chunk_paged(self, K_pool: torch.Tensor, V_pool: torch.Tensor, page_table: torch.Tensor,
                              valid_len: Optional[torch.Tensor] = None, valid_len_host=None, stream=None):
        """K_pool, V_pool [n_pages, H_kv, page_size, d]; page_table int32 [B, pages_per_req] on the device."""
        n_pages, _, page_size, _ = K_pool.shape
        assert page_table.dtype == torch.int32 and page_table.is_cuda and page_table.is_contiguous()
        if valid_len_host is not None and not isinstance(valid_len_host, C.Array):
            valid_len_host = (C.c_int32 * len(valid_len_host))(*valid_len_host)
        self._check(self.lib.ss_verify_chunk_paged(self.handle, as_ss_tensor(K_pool), as_ss_tensor(V_pool),
                                                   n_pages, page_size, page_table.data_ptr(),
                                                   page_table.shape[1], _ptr(valid_len), valid_len_host,
                                                   self._sp(stream)), "ss_verify_chunk_paged")

    def ss_verify_local(self, K_loc: torch.Tensor, V_loc: torch.Tensor, mask_kind: int = SS_MASK_CHAIN,
                        mask_bits: Optional[torch.Tensor] = None, stream=None):
        T_loc = K_loc.shape[2]
        if mask_bits is not None:
            assert mask_bits.dtype == torch.int64 and mask_bits.is_contiguous()
        self._check(self.lib.ss_verify_local(self.handle, as_ss_tensor(K_loc), as_ss_tensor(V_loc),
                                             T_loc, mask_kind, _ptr(mask_bits), self._sp(stream)),
                    "ss_verify_local")

    def ss_verify_export_state(self, ml: torch.Tensor, a: torch.Tensor, stream=None):
        assert ml.dtype == torch.float32 and a.dtype == torch.float32 and ml.is_contiguous() and a.is_contiguous()
        self._check(self.lib.ss_verify_export_state(self.handle, ml.data_ptr(), a.data_ptr(),
                                                    self._sp(stream)), "ss_verify_export_state")

    def ss_verify_import_state(self, ml: torch.Tensor, a: torch.Tensor, stream=None):
        assert ml.dtype == torch.float32 and a.dtype == torch.float32 and ml.is_contiguous() and a.is_contiguous()
        self._check(self.lib.ss_verify_import_state(self.handle, ml.data_ptr(), a.data_ptr(),
                                                    self._sp(stream)), "ss_verify_import_state")

    def ss_verify_finalize(self, O: torch.Tensor, LSE: Optional[torch.Tensor], stream=None):
        assert O.dtype == torch.bfloat16 and O.is_contiguous()
        if LSE is not None:
            assert LSE.dtype == torch.float32 and LSE.is_contiguous()
        self._check(self.lib.ss_verify_finalize(self.handle, O.data_ptr(), _ptr(LSE),
                                                self._sp(stream)), "ss_verify_finalize")

    def ss_verify_abort(self):
        self._check(self.lib.ss_verify_abort(self.handle), "ss_verify_abort")

    def ss_commit_gather(self, K_loc, V_loc, accept_idx, accept_cnt, K_dst, V_dst, dst_off, stream=None):
        B, _, T_loc, _ = K_loc.shape
        cap = K_dst.shape[2]
        for t in (accept_idx, accept_cnt, dst_off):
            assert t.dtype == torch.int32 and t.is_contiguous() and t.is_cuda
        self._check(self.lib.ss_commit_gather(self.handle, as_ss_tensor(K_loc), as_ss_tensor(V_loc), B,
                                              T_loc, accept_idx.data_ptr(), accept_cnt.data_ptr(),
                                              as_ss_tensor(K_dst), as_ss_tensor(V_dst), cap,
                                              dst_off.data_ptr(), self._sp(stream)), "ss_commit_gather")

    def ss_poll_status(self, stream=None, timeout_ms: int = 0):
        """Returns (status, device_bits)."""
        bits = C.c_uint32(0)
        st = self.lib.ss_poll_status(self.handle, self._sp(stream), timeout_ms, C.byref(bits))
        return st, bits.value

    def ss_stream_round(self, desc: ss_stream_desc) -> ss_stream_stats:
        stats = ss_stream_stats()
        self._check(self.lib.ss_stream_round(self.handle, C.byref(desc), C.byref(stats)), "ss_stream_round")
        return stats

    def ss_trace_enable(self, on: bool):
        self._check(self.lib.ss_trace_enable(self.handle, 1 if on else 0), "ss_trace_enable")

    @staticmethod
    def chunk_descs(chunk_sets, hints=None):
        """ctypes array of ss_chunk_desc for a list of chunk lists [(K, V, valid_len), ...] (all of
        the same length); hints: per chunk a ctypes int32 array with the host copy of valid_len."""
        n = len(chunk_sets[0])
        arr = (ss_chunk_desc * (n * len(chunk_sets)))()
        for s_, chunks in enumerate(chunk_sets):
            assert len(chunks) == n
            for j, (K, V, vl) in enumerate(chunks):
                d = arr[s_ * n + j]
                d.K, d.V, d.L_c = as_ss_tensor(K), as_ss_tensor(V), K.shape[2]
                d.valid_len = _ptr(vl)
                if hints is not None and vl is not None:
                    d.valid_len_host = C.cast(hints[j], C.POINTER(C.c_int32))
        arr._keep = (chunk_sets, hints)
        return arr

    def ss_verify_chunks(self, descs, n_chunks: int, stream=None):
        """Several chunks of the open round with one call; descs: a chunk_descs array."""
        self._check(self.lib.ss_verify_chunks(self.handle, descs, n_chunks, self._sp(stream)), "ss_verify_chunks")

    def ss_verify_round(self, Q, scale, chunks, K_loc, V_loc, mask_kind=SS_MASK_CHAIN, mask_bits=None,
                        O=None, LSE=None, hints=None, descs=None, stream=None):
        """One call for a whole round.  chunks: [(K, V, valid_len), ...]; descs: a prebuilt
        chunk_descs array for the same chunks (saves rebuilding it every round)."""
        if descs is None:
            descs = self.chunk_descs([chunks], hints) if chunks else None
        n = len(chunks)
        B, _, T_q, _ = Q.shape
        T_loc = K_loc.shape[2] if K_loc is not None else 0
        zero = ss_tensor(None, 0, 0, 0)
        self._check(self.lib.ss_verify_round(
            self.handle, as_ss_tensor(Q), B, T_q, scale, descs, n,
            as_ss_tensor(K_loc) if T_loc else zero, as_ss_tensor(V_loc) if T_loc else zero, T_loc, mask_kind,
            _ptr(mask_bits), O.data_ptr(), _ptr(LSE), self._sp(stream)), "ss_verify_round")

    def ss_time_rounds(self, Q, scale, descs, n_chunks, n_sets, K_loc, V_loc, mask_kind, mask_bits, O, LSE,
                       n_rounds, single_call, stream=None) -> float:
        """Device milliseconds of n_rounds rounds enqueued back to back from C."""
        B, _, T_q, _ = Q.shape
        ms = C.c_float(0.0)
        self._check(self.lib.ss_time_rounds(
            self.handle, as_ss_tensor(Q), B, T_q, scale, descs, n_chunks, n_sets, as_ss_tensor(K_loc),
            as_ss_tensor(V_loc), K_loc.shape[2], mask_kind, _ptr(mask_bits), O.data_ptr(), _ptr(LSE),
            self._sp(stream), n_rounds, 1 if single_call else 0, C.byref(ms)), "ss_time_rounds")
        return ms.value

    def ss_get_stats(self) -> ss_stats:
        st = ss_stats()
        self._check(self.lib.ss_get_stats(self.handle, C.byref(st)), "ss_get_stats")
        return st

    def ss_cta_log_set(self, log, capacity: int = 0):
        """log: zeroed device int64 tensor of 4 * (capacity + 1) words, or None to switch the log off."""
        self._check(self.lib.ss_cta_log_set(self.handle, _ptr(log), capacity if log is not None else 0),
                    "ss_cta_log_set")

    def ss_trace_read(self):
        """[3 roles][32 tiles][8 events] clock stamps of CTA (0,0,0) of the last traced chunk kernel."""
        n = 3 * 32 * 8
        buf = (C.c_uint64 * n)()
        got = self.lib.ss_trace_read(self.handle, buf, n)
        return [[[buf[(r * 32 + t) * 8 + e] for e in range(8)] for t in range(32)] for r in range(3)][:3] if got else None

    def ss_stream_layers(self, descs, mode: int = SS_LAYERS_PREFETCH, restore_k=None, restore_v=None) -> ss_stream_stats:
        """descs: list of ss_stream_desc, one per layer.  restore_k [B, H_kv, tokens, d] with
        restore_v of the same shape, or restore_k [B, 2, H_kv, tokens, d] alone (K and V fused)."""
        arr = (ss_stream_desc * len(descs))(*descs)
        ld = ss_layers_desc(len(descs), arr, mode, _ptr(restore_k), _ptr(restore_v),
                            restore_k.shape[-2] if restore_k is not None else 0)
        stats = ss_stream_stats()
        self._check(self.lib.ss_stream_layers(self.handle, C.byref(ld), C.byref(stats)), "ss_stream_layers")
        return stats

    def ss_selftest_wait_expiry(self, limit_ms: int, gave_up: torch.Tensor, stream=None):
        """gave_up: device int32[1], zeroed by the caller; counts the threads whose wait ran out."""
        assert gave_up.dtype == torch.int32 and gave_up.is_cuda
        self._check(self.lib.ss_selftest_wait_expiry(self.handle, limit_ms, gave_up.data_ptr(), self._sp(stream)),
                    "ss_selftest_wait_expiry")

    def launch_count(self) -> int:
        return int(self.lib.ss_launch_count(self.handle))

    def last_chunk_kernel(self) -> str:
        return self.lib.ss_last_chunk_kernel(self.handle).decode()


def ss_probe_read(srcs: Sequence[torch.Tensor], sink: torch.Tensor, stream=None) -> None:
    """Enqueue one streaming read of up to 64 contiguous device tensors; `sink` is a device int64[1]."""
    n = len(srcs)
    ptrs = (C.c_void_p * n)(*[t.data_ptr() for t in srcs])
    sizes = (C.c_size_t * n)(*[t.numel() * t.element_size() for t in srcs])
    st = load().ss_probe_read(ptrs, sizes, n, sink.data_ptr(), _stream_ptr(stream))
    if st != SS_OK:
        raise SpecStreamError(st, "ss_probe_read")


def verify_round(ctx: Context, Q, chunks: Sequence, K_loc, V_loc, scale: float, mask_kind=SS_MASK_CHAIN,
                 mask_bits=None, O=None, LSE=None, stream=None):
    """One full round through the five-call boundary.  ``chunks`` = [(K, V, valid_len|None), ...]."""
    B, H_q, T_q, d = Q.shape
    if O is None:
        O = torch.empty(B, H_q, T_q, d, dtype=torch.bfloat16, device=Q.device)
    if LSE is None:
        LSE = torch.empty(B, H_q, T_q, dtype=torch.float32, device=Q.device)
    ctx.ss_verify_begin(Q, scale, stream)
    for K, V, vl in chunks:
        ctx.ss_verify_chunk(K, V, vl, stream)
    if K_loc is not None:
        ctx.ss_verify_local(K_loc, V_loc, mask_kind, mask_bits, stream)
    ctx.ss_verify_finalize(O, LSE, stream)
    return O, LSE


class GraphRound:
    """A whole round (begin, chunk calls, local, finalize) recorded once into a CUDA graph.

    The library's calls only enqueue on the stream they are given, so a round can be captured
    and replayed; replay() then costs one graph launch instead of one host call per kernel,
    which matters for small rounds (the 1,024-token chain workload: 43 us per round driven call
    by call, 20 us replayed).  The graph reads and writes the SAME tensors on every replay:
    refresh Q, the chunks, valid lengths and the local KV in place, then replay().  The call
    sequence, shapes and split choices are frozen at capture time, so the number of chunk calls
    and every tensor's shape must stay what they were.  Results are bit-identical to the calls.
    """

    def __init__(self, ctx: "Context", Q, chunks: Sequence, K_loc, V_loc, scale: float,
                 mask_kind=SS_MASK_CHAIN, mask_bits=None):
        B, H_q, T_q, d = Q.shape
        self.O = torch.empty(B, H_q, T_q, d, dtype=torch.bfloat16, device=Q.device)
        self.LSE = torch.empty(B, H_q, T_q, dtype=torch.float32, device=Q.device)
        self._keep = (Q, list(chunks), K_loc, V_loc, mask_bits)   # the graph holds raw pointers
        # warm up outside the capture (first-use initialisation must not be recorded)
        verify_round(ctx, Q, chunks, K_loc, V_loc, scale, mask_kind, mask_bits, self.O, self.LSE)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            verify_round(ctx, Q, chunks, K_loc, V_loc, scale, mask_kind, mask_bits, self.O, self.LSE)

    def replay(self):
        """Enqueue the recorded round on the current stream; returns (O, LSE), valid once it ran."""
        self.graph.replay()
        return self.O, self.LSE


class Tier:
    """Owns an ss_tier: boundaries H <= C per request, tail buffers, offload of [H, E) (Eq. 9)."""

    def __init__(self, B, H_kv, d, L_c, tail_target, granularity, tail_capacity, host_hist, device="cuda:0"):
        self.lib = load()
        self.cfg = ss_tier_config(B, H_kv, d, L_c, tail_target, granularity, tail_capacity)
        self.host_hist = host_hist  # list of pinned tensors, chunk-block layout
        self.tail_k = [torch.zeros(B, H_kv, tail_capacity, d, dtype=torch.bfloat16, device=device) for _ in range(2)]
        self.tail_v = [torch.zeros(B, H_kv, tail_capacity, d, dtype=torch.bfloat16, device=device) for _ in range(2)]
        self.len_dev = torch.zeros(B, dtype=torch.int32, device=device)
        self.len_host = torch.zeros(4 * B, dtype=torch.int32).pin_memory()
        ptrs = (C.c_void_p * B)(*[h.data_ptr() for h in host_hist])
        caps = (C.c_int64 * B)(*[h.numel() // (2 * H_kv * d) for h in host_hist])
        self.handle = C.c_void_p()
        st = self.lib.ss_tier_create(C.byref(self.handle), C.byref(self.cfg), ptrs, caps,
                                     self.tail_k[0].data_ptr(), self.tail_v[0].data_ptr(),
                                     self.tail_k[1].data_ptr(), self.tail_v[1].data_ptr(),
                                     self.len_dev.data_ptr(), self.len_host.data_ptr())
        if st != SS_OK:
            raise SpecStreamError(st, "ss_tier_create")
        self.B = B

    def _arr(self, xs):
        return (C.c_int32 * self.B)(*[int(x) for x in xs])

    def _check(self, st, where):
        if st != SS_OK:
            raise SpecStreamError(st, where)

    def reset(self, H, Cc, stream=None):
        self._check(self.lib.ss_tier_reset(self.handle, self._arr(H), self._arr(Cc), _stream_ptr(stream)), "ss_tier_reset")

    def get(self):
        H, Cc, E = self._arr([0] * self.B), self._arr([0] * self.B), self._arr([0] * self.B)
        cur = C.c_int32(0)
        self._check(self.lib.ss_tier_get(self.handle, H, Cc, E, C.byref(cur)), "ss_tier_get")
        return list(H), list(Cc), list(E), cur.value

    def tail(self):
        K, V, p = ss_tensor(), ss_tensor(), C.c_void_p()
        self._check(self.lib.ss_tier_tail(self.handle, C.byref(K), C.byref(V), C.byref(p)), "ss_tier_tail")
        cur = self.get()[3]
        return self.tail_k[cur], self.tail_v[cur], K, V

    def commit(self, cnt, stream=None):
        self._check(self.lib.ss_tier_commit(self.handle, self._arr(cnt), _stream_ptr(stream)), "ss_tier_commit")

    def migrate(self, stream=None) -> int:
        n = C.c_int32(0)
        self._check(self.lib.ss_tier_migrate(self.handle, _stream_ptr(stream), C.byref(n)), "ss_tier_migrate")
        return n.value

    def poll(self, wait: bool, stream=None) -> bool:
        adv = C.c_int32(0)
        self._check(self.lib.ss_tier_poll(self.handle, 1 if wait else 0, _stream_ptr(stream), C.byref(adv)), "ss_tier_poll")
        return bool(adv.value)

    def d2h_bytes(self) -> int:
        return int(self.lib.ss_tier_d2h_bytes(self.handle))

    def close(self):
        if self.handle:
            self.lib.ss_tier_destroy(self.handle)
            self.handle = C.c_void_p()


class WidthController:
    """Owns an ss_width: the I/O-aware choice of the verification width q (Section 4.2)."""

    def __init__(self, widths: Sequence[int], sample_rounds: int = 2, switch_threshold: float = 0.05,
                 ema: float = 0.5):
        self.lib = load()
        cfg = ss_width_config(len(widths), (C.c_int32 * 8)(*widths), sample_rounds, switch_threshold, ema)
        self.handle = C.c_void_p()
        st = self.lib.ss_width_create(C.byref(self.handle), C.byref(cfg))
        if st != SS_OK:
            raise SpecStreamError(st, "ss_width_create")

    def observe(self, q: int, t_draft: float, t_transfer: float, t_compute: float, t_other: float,
                committed: int) -> None:
        obs = ss_width_obs(t_draft, t_transfer, t_compute, t_other, committed)
        st = self.lib.ss_width_observe(self.handle, q, C.byref(obs))
        if st != SS_OK:
            raise SpecStreamError(st, "ss_width_observe")

    def next(self) -> int:
        return int(self.lib.ss_width_next(self.handle))

    def estimate(self, q: int):
        """(T_round, committed, cost = T_round / committed, observations) of width q."""
        t, u, c, n = C.c_double(), C.c_double(), C.c_double(), C.c_int32()
        st = self.lib.ss_width_estimate(self.handle, q, C.byref(t), C.byref(u), C.byref(c), C.byref(n))
        if st != SS_OK:
            raise SpecStreamError(st, "ss_width_estimate")
        return t.value, u.value, c.value, n.value

    def close(self):
        if self.handle:
            self.lib.ss_width_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def cohort_build(tasks: Sequence[dict], max_batch: int):
    """Group the tasks of a scheduled batch into cohorts (ss_cohort_build).  Each task is a dict
    with layer, width, dtype, n_kv, d_h, chunk_size, hist_len; returns a list of lists of task
    indices, cohort by cohort, longest history first inside a cohort."""
    n = len(tasks)
    arr = (ss_task * max(1, n))(*[ss_task(t["layer"], t["width"], t["dtype"], t["n_kv"], t["d_h"],
                                         t["chunk_size"], i, t["hist_len"]) for i, t in enumerate(tasks)])
    order = (C.c_int32 * max(1, n))()
    start = (C.c_int32 * (n + 1))()
    k = load().ss_cohort_build(arr, n, max_batch, order, start)
    if k < 0:
        raise SpecStreamError(SS_ERR_ARG, "ss_cohort_build")
    return [list(order[start[c]:start[c + 1]]) for c in range(k)]
