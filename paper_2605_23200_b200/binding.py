"""ctypes binding of libams.so: argument marshalling only.

Every step of the compression path runs inside the library's CUDA kernels; this
module turns torch tensors into device pointers and owns the two buffers the
library asks the caller to allocate (EMA credit state and workspace).  If the
library is missing or fails to load, importing the functions raises: there is no
CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libams.so")

AMS_OK = 0
AMS_ERR_INVALID_ARG, AMS_ERR_UNSUPPORTED, AMS_ERR_CAPACITY = -1, -2, -3
AMS_ERR_CUDA, AMS_ERR_TIMEOUT, AMS_ERR_INTERNAL = -4, -5, -6
AMS_SCORER_TOVA, AMS_SCORER_KEYDIFF, AMS_SCORER_EXTERNAL, AMS_SCORER_EXPECTED = 0, 1, 2, 3

EXPORTS = ["ams_config_default", "ams_ema_state_bytes", "ams_workspace_bytes", "ams_segment_capacity",
           "ams_init_state", "ams_compress", "ams_get_status", "ams_last_launch_count", "ams_free",
           "ams_strerror", "ams_set_profiling", "ams_get_kernel_times", "ams_kernel_name", "ams_select_static",
           "ams_select_static_status", "ams_debug_expire_wait", "ams_set_query_stats"]
KERNEL_SLOTS = 10


class AmsConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "n_q_heads", "n_kv_heads", "head_dim", "page_size", "max_batch", "max_seq_len",
                 "max_window", "max_budget", "max_segments", "l_min", "l_max", "q_min", "n_sink", "n_last")] + \
               [("ema_lambda", ctypes.c_float), ("ema_beta", ctypes.c_float), ("eps", ctypes.c_float),
                ("causal_window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32), ("decoupled", ctypes.c_int32),
                ("fixed_segments", ctypes.c_int32), ("uniform_quotas", ctypes.c_int32), ("expected_scorer", ctypes.c_int32)]


class AmsDebugViews(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("scores", "usage", "mass", "n_segments", "seg_bounds", "quotas", "keep_idx", "prev_kept",
                                                "retained_iou")]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libams.so (must have been built: `python -m paper_2605_23200_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not built; run paper_2605_23200_b200/build.py (no CPU fallback exists)")
        L = ctypes.CDLL(LIB_PATH)
        L.ams_config_default.argtypes = [ctypes.POINTER(AmsConfig)]
        L.ams_config_default.restype = None
        for f in ("ams_ema_state_bytes", "ams_workspace_bytes"):
            getattr(L, f).argtypes = [ctypes.POINTER(AmsConfig)]
            getattr(L, f).restype = ctypes.c_size_t
        L.ams_segment_capacity.argtypes = [ctypes.POINTER(AmsConfig)]
        L.ams_segment_capacity.restype = ctypes.c_int32
        L.ams_init_state.argtypes = [ctypes.POINTER(AmsConfig), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                     ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)]
        L.ams_init_state.restype = ctypes.c_int
        L.ams_compress.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                   ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32,
                                   ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32,
                                   ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                   ctypes.POINTER(AmsDebugViews), ctypes.c_void_p]
        L.ams_compress.restype = ctypes.c_int
        L.ams_get_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)]
        L.ams_get_status.restype = ctypes.c_int
        L.ams_last_launch_count.argtypes = [ctypes.c_void_p]
        L.ams_last_launch_count.restype = ctypes.c_int32
        L.ams_free.argtypes = [ctypes.c_void_p]
        L.ams_free.restype = ctypes.c_int
        L.ams_set_profiling.argtypes = [ctypes.c_void_p, ctypes.c_int]
        L.ams_set_profiling.restype = ctypes.c_int
        L.ams_get_kernel_times.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_float)]
        L.ams_get_kernel_times.restype = ctypes.c_int
        L.ams_kernel_name.argtypes = [ctypes.c_int32]
        L.ams_kernel_name.restype = ctypes.c_char_p
        L.ams_select_static.argtypes = [ctypes.POINTER(AmsConfig), ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                        ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                        ctypes.c_void_p]
        L.ams_select_static.restype = ctypes.c_int
        L.ams_select_static_status.argtypes = [ctypes.POINTER(ctypes.c_int32), ctypes.c_void_p]
        L.ams_select_static_status.restype = ctypes.c_int
        L.ams_debug_expire_wait.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p]
        L.ams_debug_expire_wait.restype = ctypes.c_int
        L.ams_set_query_stats.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float]
        L.ams_set_query_stats.restype = ctypes.c_int
        L.ams_strerror.argtypes = [ctypes.c_int]
        L.ams_strerror.restype = ctypes.c_char_p
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().ams_strerror(code).decode()


class AmsError(RuntimeError):
    def __init__(self, code: int, where: str, detail=None):
        self.code = code
        self.detail = detail
        super().__init__(f"{where}: {strerror(code)} ({code})" + (f" detail={detail}" if detail else ""))


def default_config(**kw) -> AmsConfig:
    cfg = AmsConfig()
    lib().ams_config_default(ctypes.byref(cfg))
    for k, v in kw.items():
        if not hasattr(cfg, k):
            raise AttributeError(k)
        setattr(cfg, k, v)
    return cfg


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


@dataclass
class DebugViews:
    """Device tensors that receive the library's intermediate results."""
    scores: torch.Tensor
    usage: torch.Tensor
    mass: torch.Tensor
    n_segments: torch.Tensor
    seg_bounds: torch.Tensor
    quotas: torch.Tensor
    keep_idx: torch.Tensor
    prev_kept: torch.Tensor | None = None       # input: int32 [batch], previous event's retained count per sequence
    retained_iou: torch.Tensor | None = None    # output: float32 [L][batch][H]

    def c(self) -> AmsDebugViews:
        return AmsDebugViews(*(None if t is None else t.data_ptr() for t in
                               (self.scores, self.usage, self.mass, self.n_segments, self.seg_bounds, self.quotas,
                                self.keep_idx, self.prev_kept, self.retained_iou)))


class AmsCompressor:
    """Owns an `ams_state` handle together with the EMA credit and workspace tensors."""

    def __init__(self, cfg: AmsConfig, device="cuda:0", stream: torch.cuda.Stream | None = None):
        L = lib()
        self.cfg = cfg
        self.device = torch.device(device)
        ema_bytes = L.ams_ema_state_bytes(ctypes.byref(cfg))
        ws_bytes = L.ams_workspace_bytes(ctypes.byref(cfg))
        if ema_bytes == 0 or ws_bytes == 0:
            raise AmsError(AMS_ERR_INVALID_ARG, "ams_config")
        self.seg_cap = L.ams_segment_capacity(ctypes.byref(cfg))
        self.ema_state = torch.empty((cfg.n_layers, cfg.max_batch, cfg.n_kv_heads, cfg.max_seq_len),
                                     dtype=torch.float32, device=self.device)
        self.workspace = torch.empty(ws_bytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self._ws_ptr = self.workspace.data_ptr() + off
        self._ws_bytes = ws_bytes
        handle = ctypes.c_void_p()
        s = stream or torch.cuda.current_stream(self.device)
        rc = L.ams_init_state(ctypes.byref(cfg), _ptr(self.ema_state), ctypes.c_void_p(self._ws_ptr), ws_bytes,
                              ctypes.c_void_p(s.cuda_stream), ctypes.byref(handle))
        if rc != AMS_OK:
            raise AmsError(rc, "ams_init_state")
        self._h = handle

    def make_debug_views(self, batch: int, budget: int) -> DebugViews:
        c, dev = self.cfg, self.device
        U = (c.n_layers, batch, c.n_kv_heads)
        return DebugViews(torch.zeros(U + (c.max_seq_len,), dtype=torch.float32, device=dev),
                          torch.zeros(U + (c.max_seq_len,), dtype=torch.float32, device=dev),
                          torch.zeros(U + (c.max_seq_len,), dtype=torch.float32, device=dev),
                          torch.zeros(U, dtype=torch.int32, device=dev),
                          torch.zeros(U + (self.seg_cap + 1,), dtype=torch.int32, device=dev),
                          torch.zeros(U + (self.seg_cap,), dtype=torch.int32, device=dev),
                          torch.zeros(U + (budget,), dtype=torch.int32, device=dev))

    def compress(self, k_pages, v_pages, block_table, seq_lens, obs_queries, budget, n_segments, scorer_id,
                 dst_pages, *, ext_scores=None, ext_usage=None, dbg: DebugViews | None = None, ema_state=None,
                 stream: torch.cuda.Stream | None = None) -> None:
        """Enqueues one compression event on `stream` (default: torch's current stream)."""
        assert k_pages.is_contiguous() and v_pages.is_contiguous() and block_table.is_contiguous()
        assert k_pages.dtype == torch.bfloat16 and block_table.dtype == torch.int32 and seq_lens.dtype == torch.int32
        assert dst_pages.dtype == torch.int32 and dst_pages.is_contiguous()
        s = stream or torch.cuda.current_stream(self.device)
        window = 0 if obs_queries is None else obs_queries.shape[3]
        ema = self.ema_state if ema_state is None else ema_state
        views = dbg.c() if dbg is not None else None
        rc = lib().ams_compress(self._h, _ptr(k_pages), _ptr(v_pages), k_pages.shape[1], _ptr(block_table),
                                block_table.shape[1], _ptr(seq_lens), seq_lens.shape[0], _ptr(obs_queries), window,
                                _ptr(ema), budget, n_segments, scorer_id, _ptr(dst_pages), _ptr(ext_scores),
                                _ptr(ext_usage),
                                ctypes.byref(views) if views is not None else None, ctypes.c_void_p(s.cuda_stream))
        if rc != AMS_OK:
            raise AmsError(rc, "ams_compress")

    def set_query_stats(self, q_mean: torch.Tensor, q_cov: torch.Tensor, score_eps: float = 1e-2) -> None:
        """Mean (fp32 [L][batch][Hq][128]) and covariance (bf16 [L][batch][Hq][128][128]) of the future queries for
        AMS_SCORER_EXPECTED; the tensors are kept alive by this object until they are replaced."""
        assert q_mean.dtype == torch.float32 and q_mean.is_contiguous() and q_mean.shape[-1] == 128
        assert q_cov.dtype == torch.bfloat16 and q_cov.is_contiguous() and q_cov.shape == q_mean.shape + (128,)
        rc = lib().ams_set_query_stats(self._h, _ptr(q_mean), _ptr(q_cov), ctypes.c_float(score_eps))
        if rc != AMS_OK:
            raise AmsError(rc, "ams_set_query_stats")
        self._query_stats = (q_mean, q_cov)

    def status(self, stream: torch.cuda.Stream | None = None, check: bool = True):
        s = stream or torch.cuda.current_stream(self.device)
        detail = (ctypes.c_int32 * 4)()
        rc = lib().ams_get_status(self._h, ctypes.c_void_p(s.cuda_stream), detail)
        if check and rc != AMS_OK:
            raise AmsError(rc, "device status", list(detail))
        return rc, list(detail)

    def expire_wait(self, polls: int = 1000, stream: torch.cuda.Stream | None = None) -> None:
        """Failure-handling check: a bounded device wait that runs out after `polls` polls."""
        s = stream or torch.cuda.current_stream(self.device)
        rc = lib().ams_debug_expire_wait(self._h, polls, ctypes.c_void_p(s.cuda_stream))
        if rc != AMS_OK:
            raise AmsError(rc, "ams_debug_expire_wait")

    def set_profiling(self, enable: bool) -> None:
        rc = lib().ams_set_profiling(self._h, 1 if enable else 0)
        if rc != AMS_OK:
            raise AmsError(rc, "ams_set_profiling")

    def kernel_times_ms(self) -> dict:
        """Per-kernel durations of the last call (profiling must be on); waits for the call to finish."""
        buf = (ctypes.c_float * KERNEL_SLOTS)()
        rc = lib().ams_get_kernel_times(self._h, buf)
        if rc != AMS_OK:
            raise AmsError(rc, "ams_get_kernel_times")
        return {lib().ams_kernel_name(i).decode(): float(buf[i]) for i in range(KERNEL_SLOTS)}

    @property
    def last_launch_count(self) -> int:
        return lib().ams_last_launch_count(self._h)

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().ams_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def select_static(cfg: AmsConfig, scores: torch.Tensor, seq_len: int, budget: int, n_segments: int,
                  keep_idx: torch.Tensor, stream: torch.cuda.Stream | None = None) -> None:
    """Allocation-free selection for callers that cannot obtain device memory (stream capture in
    progress, a memory pool owned by the host framework): kept positions of each score row are
    written to `keep_idx` (int32 [n_units][budget]); the library's fixed scratch array is used, so
    calls must not overlap on the GPU.  `scores` is fp32 [n_units][stride], stride % 16 == 0."""
    assert scores.dtype == torch.float32 and scores.is_contiguous() and scores.dim() == 2
    assert keep_idx.dtype == torch.int32 and keep_idx.is_contiguous() and keep_idx.shape == (scores.shape[0], budget)
    s = stream or torch.cuda.current_stream(scores.device)
    rc = lib().ams_select_static(ctypes.byref(cfg), _ptr(scores), scores.shape[1], scores.shape[0], seq_len, budget,
                                 n_segments, _ptr(keep_idx), ctypes.c_void_p(s.cuda_stream))
    if rc != AMS_OK:
        raise AmsError(rc, "ams_select_static")


def select_static_status(stream: torch.cuda.Stream | None = None, device="cuda:0"):
    """(code, detail) of the allocation-free entry point's device status on the current device; clears it."""
    s = stream or torch.cuda.current_stream(torch.device(device))
    detail = (ctypes.c_int32 * 4)()
    rc = lib().ams_select_static_status(detail, ctypes.c_void_p(s.cuda_stream))
    return rc, list(detail)


def config_for(wl, **kw) -> AmsConfig:
    """Library configuration matching an `inputs.Workload`."""
    return default_config(n_layers=wl.layers_resident, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
                          max_batch=wl.batch, max_seq_len=wl.max_seq_len, max_window=max(wl.window, 0),
                          max_budget=wl.budget, max_segments=max(wl.n_segments, 1), l_min=wl.l_min, l_max=wl.l_max,
                          q_min=wl.q_min, n_sink=wl.n_sink, n_last=wl.n_last, ema_lambda=wl.ema_lambda,
                          ema_beta=wl.ema_beta, eps=wl.eps, pool_kernel=wl.pool_kernel, decoupled=int(wl.decoupled),
                          fixed_segments=int(wl.fixed_segments), uniform_quotas=int(wl.uniform_quotas),
                          **{"expected_scorer": int(wl.scorer_id == AMS_SCORER_EXPECTED), **kw})
