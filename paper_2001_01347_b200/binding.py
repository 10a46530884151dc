"""Thin ctypes binding of the ZipLine C ABI (include/zipline.h).

Argument marshalling only: every step of the search runs in the CUDA kernels
of ``libzipline.so``.  There is no CPU fallback; if the library cannot be
loaded the import of this module fails.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import torch

from . import build as _build

ZL_OK = 0
ZL_ERR_INVALID_ARG, ZL_ERR_UNSUPPORTED, ZL_ERR_NOMEM, ZL_ERR_CUDA, ZL_ERR_UNSORTED, ZL_ERR_TIMEOUT = range(1, 7)
ZL_OBJ_RANGE, ZL_OBJ_SUM = 0, 1
ZL_FLAG_CHECK_SORTED, ZL_FLAG_FULL_SWEEP, ZL_FLAG_PREDICTOR, ZL_FLAG_DEBUG_CHECKS, ZL_FLAG_FORCE_FILTER = 1, 2, 4, 8, 16

EXPORTS = ("zl_create", "zl_select_batched", "zl_select_batched_host", "zl_trace_batched", "zl_destroy",
           "zl_set_option", "zl_status_string", "zl_workspace_bytes", "zl_launches_per_call",
           "zl_segments_per_instance", "zl_max_workers", "zl_trace_max_elements", "zl_last_cuda_error",
           "zl_profile_begin", "zl_profile_read", "zl_profile_end",
           "zl_select_batched_noalloc", "zl_noalloc_max_batch", "zl_noalloc_scratch_bytes", "zl_filter_counts",
           "zl_predict_batched", "zl_predict_select_batched", "zl_gridscan_batched", "zl_route",
           "zl_probe_read_batched", "zl_debug_report", "zl_debug_stamps", "zl_check_canaries")


class zl_config(ctypes.Structure):
    _fields_ = [("n_workers", ctypes.c_int32), ("lookahead_R", ctypes.c_int32), ("max_batch", ctypes.c_int32),
                ("objective", ctypes.c_int32), ("device", ctypes.c_int32), ("flags", ctypes.c_int32)]


def _load() -> ctypes.CDLL:
    lib = ctypes.CDLL(_build.build())
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.zl_create.argtypes = [ctypes.POINTER(zl_config), ctypes.POINTER(vp)]
    lib.zl_select_batched.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
    lib.zl_select_batched_host.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.zl_trace_batched.argtypes = [vp, i32, i32, i32] + [vp] * 11 + [vp]
    lib.zl_destroy.argtypes = [vp]
    lib.zl_set_option.argtypes = [vp, ctypes.c_char_p, i32]
    lib.zl_status_string.argtypes = [ctypes.c_int]
    lib.zl_status_string.restype = ctypes.c_char_p
    lib.zl_workspace_bytes.argtypes = [vp]
    lib.zl_workspace_bytes.restype = ctypes.c_size_t
    lib.zl_launches_per_call.argtypes = [vp]
    lib.zl_segments_per_instance.argtypes = [vp, i32]
    lib.zl_route.argtypes = [vp]
    lib.zl_probe_read_batched.argtypes = [vp, vp, ctypes.c_int64, i32, vp, vp]
    lib.zl_probe_read_batched.restype = ctypes.c_int
    lib.zl_route.restype = ctypes.c_int
    lib.zl_last_cuda_error.argtypes = [vp]
    lib.zl_profile_begin.argtypes = [vp, i32]
    lib.zl_profile_read.argtypes = [vp, vp, vp]
    lib.zl_profile_end.argtypes = [vp]
    lib.zl_gridscan_batched.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.zl_gridscan_batched.restype = ctypes.c_int
    lib.zl_predict_batched.argtypes = [vp, vp, i32, i32, i32, vp, vp]
    lib.zl_predict_batched.restype = ctypes.c_int
    lib.zl_predict_select_batched.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp]
    lib.zl_predict_select_batched.restype = ctypes.c_int
    lib.zl_filter_counts.argtypes = [vp, i32, vp, vp, vp]
    lib.zl_filter_counts.restype = ctypes.c_int
    lib.zl_check_canaries.argtypes = [vp, vp, vp]
    lib.zl_check_canaries.restype = ctypes.c_int
    lib.zl_debug_report.argtypes = [vp, vp]
    lib.zl_debug_report.restype = ctypes.c_int
    lib.zl_debug_stamps.argtypes = [vp, i32, vp]
    lib.zl_debug_stamps.restype = ctypes.c_int
    lib.zl_select_batched_noalloc.argtypes = [i32, i32, i32, i32, vp, i32, vp, vp, vp, vp, vp]
    lib.zl_select_batched_noalloc.restype = ctypes.c_int
    lib.zl_noalloc_max_batch.restype = ctypes.c_int
    lib.zl_noalloc_scratch_bytes.restype = ctypes.c_size_t
    for name in ("zl_create", "zl_select_batched", "zl_select_batched_host", "zl_trace_batched", "zl_destroy",
                 "zl_set_option", "zl_launches_per_call", "zl_segments_per_instance", "zl_max_workers",
                 "zl_trace_max_elements", "zl_last_cuda_error", "zl_profile_begin", "zl_profile_read",
                 "zl_profile_end"):
        getattr(lib, name).restype = ctypes.c_int
    return lib


lib = _load()


class ZipLineError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib.zl_status_string(code).decode()} (status {code})")


def _check(code: int, where: str):
    if code != ZL_OK:
        raise ZipLineError(code, where)


def zl_status_string(code: int) -> str:
    return lib.zl_status_string(int(code)).decode()


def zl_max_workers() -> int:
    return lib.zl_max_workers()


def zl_trace_max_elements() -> int:
    return lib.zl_trace_max_elements()


def _dev_ptr(t: torch.Tensor | None, dtype, numel: int, name: str) -> int | None:
    if t is None:
        return None
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous() and t.numel() >= numel):
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of {dtype} with >= {numel} elements")
    return t.data_ptr()


@dataclass
class Selection:
    idx: torch.Tensor       # [B, n] int32
    barrier: torch.Tensor   # [B] int64
    wait: torch.Tensor      # [B] int64
    status: torch.Tensor    # [B] int32


class ZipLine:
    """Handle on the library's device scratch for one (n, R, max_batch, objective)."""

    def __init__(self, n_workers: int, lookahead_R: int, max_batch: int, objective: int = ZL_OBJ_RANGE,
                 device: int = 0, flags: int = 0):
        self.n, self.R, self.max_batch, self.objective, self.device = n_workers, lookahead_R, max_batch, objective, device
        cfg = zl_config(n_workers, lookahead_R, max_batch, objective, device, flags)
        h = ctypes.c_void_p()
        _check(lib.zl_create(ctypes.byref(cfg), ctypes.byref(h)), "zl_create")
        self._h = h

    # -- zl_select_batched ---------------------------------------------------------------
    def select_batched(self, ts: torch.Tensor, out: Selection | None = None, stream: torch.cuda.Stream | None = None) -> Selection:
        """ts: CUDA int64 [B, n, R].  Enqueues on ``stream`` (default: the current stream)."""
        if ts.dim() != 3 or ts.shape[1] != self.n or ts.shape[2] != self.R:
            raise ValueError(f"ts must be [B, {self.n}, {self.R}]")
        B = ts.shape[0]
        if out is None:
            dev = ts.device
            out = Selection(torch.empty((B, self.n), dtype=torch.int32, device=dev),
                            torch.empty(B, dtype=torch.int64, device=dev),
                            torch.empty(B, dtype=torch.int64, device=dev),
                            torch.empty(B, dtype=torch.int32, device=dev))
        s = stream if stream is not None else torch.cuda.current_stream(ts.device)
        rc = lib.zl_select_batched(self._h, _dev_ptr(ts, torch.int64, B * self.n * self.R, "ts"), B,
                                   _dev_ptr(out.idx, torch.int32, B * self.n, "idx"),
                                   _dev_ptr(out.barrier, torch.int64, B, "barrier"),
                                   _dev_ptr(out.wait, torch.int64, B, "wait"),
                                   _dev_ptr(out.status, torch.int32, B, "status"), s.cuda_stream)
        _check(rc, "zl_select_batched")
        return out

    # -- zl_predict_select_batched -------------------------------------------------------
    def predict_select_batched(self, last: torch.Tensor, interval: torch.Tensor, out: Selection | None = None,
                               stream: torch.cuda.Stream | None = None) -> Selection:
        """last, interval: CUDA int64 [B, n].  Needs a handle created with ZL_FLAG_PREDICTOR."""
        B = last.shape[0]
        if last.shape != (B, self.n) or interval.shape != (B, self.n):
            raise ValueError(f"last and interval must be [B, {self.n}]")
        if out is None:
            dev = last.device
            out = Selection(torch.empty((B, self.n), dtype=torch.int32, device=dev),
                            torch.empty(B, dtype=torch.int64, device=dev),
                            torch.empty(B, dtype=torch.int64, device=dev),
                            torch.empty(B, dtype=torch.int32, device=dev))
        s = stream if stream is not None else torch.cuda.current_stream(last.device)
        rc = lib.zl_predict_select_batched(self._h, _dev_ptr(last, torch.int64, B * self.n, "last"),
                                           _dev_ptr(interval, torch.int64, B * self.n, "interval"), B,
                                           _dev_ptr(out.idx, torch.int32, B * self.n, "idx"),
                                           _dev_ptr(out.barrier, torch.int64, B, "barrier"),
                                           _dev_ptr(out.wait, torch.int64, B, "wait"),
                                           _dev_ptr(out.status, torch.int32, B, "status"), s.cuda_stream)
        _check(rc, "zl_predict_select_batched")
        return out

    # -- zl_select_batched_host ----------------------------------------------------------
    def select_batched_host(self, ts: torch.Tensor, out: Selection | None = None) -> Selection:
        """ts: host int64 [B, n, R] (pinned for speed).  Returns host tensors; synchronous."""
        if ts.is_cuda or ts.dtype != torch.int64 or not ts.is_contiguous() or ts.dim() != 3 \
                or ts.shape[1] != self.n or ts.shape[2] != self.R:
            raise ValueError(f"ts must be a contiguous host int64 tensor [B, {self.n}, {self.R}]")
        B = ts.shape[0]
        if out is None:
            out = Selection(torch.empty((B, self.n), dtype=torch.int32), torch.empty(B, dtype=torch.int64),
                            torch.empty(B, dtype=torch.int64), torch.empty(B, dtype=torch.int32))
        rc = lib.zl_select_batched_host(self._h, ts.data_ptr(), B, out.idx.data_ptr(), out.barrier.data_ptr(),
                                        out.wait.data_ptr(), out.status.data_ptr())
        _check(rc, "zl_select_batched_host")
        return out

    def profile_begin(self, max_calls: int):
        _check(lib.zl_profile_begin(self._h, int(max_calls)), "zl_profile_begin")

    def profile_read(self) -> dict:
        calls = ctypes.c_int32()
        ms = (ctypes.c_float * 4)()
        _check(lib.zl_profile_read(self._h, ctypes.addressof(calls), ctypes.addressof(ms)), "zl_profile_read")
        return {"calls": calls.value, "ms_prologue": ms[0], "ms_filter": ms[1], "ms_sweep": ms[2], "ms_finalize": ms[3]}

    def profile_end(self):
        _check(lib.zl_profile_end(self._h), "zl_profile_end")

    def filter_counts(self, B: int):
        """(filter-pass survivors, refined survivors, overflow flags) per instance of the last call.  Synchronises."""
        f, r, o = (ctypes.c_uint32 * B)(), (ctypes.c_uint32 * B)(), (ctypes.c_uint32 * B)()
        _check(lib.zl_filter_counts(self._h, B, ctypes.addressof(f), ctypes.addressof(r), ctypes.addressof(o)),
               "zl_filter_counts")
        return list(f), list(r), list(o)

    def check_canaries(self):
        """(buffers, damaged): scratch buffers of a ZL_FLAG_DEBUG_CHECKS handle that end in canary bytes, and how
        many of those have been written over.  Synchronises."""
        nb, bad = ctypes.c_int32(0), ctypes.c_int32(0)
        _check(lib.zl_check_canaries(self._h, ctypes.addressof(nb), ctypes.addressof(bad)), "zl_check_canaries")
        return int(nb.value), int(bad.value)

    def debug_report(self):
        """(code, cta, index) of the first index violation since the last report, (0, 0, 0) if none.  Synchronises."""
        rec = (ctypes.c_uint32 * 4)()
        _check(lib.zl_debug_report(self._h, ctypes.addressof(rec)), "zl_debug_report")
        return int(rec[0]), int(rec[1]), int(rec[2]) | (int(rec[3]) << 32)

    def debug_stamps(self, ctas: int):
        """[ctas, 16] uint64 nanosecond stamps of the RANGE filter route's phase boundaries in the last call (numpy)."""
        import numpy as np
        out = np.zeros((ctas, 16), dtype=np.uint64)
        _check(lib.zl_debug_stamps(self._h, ctas, out.ctypes.data), "zl_debug_stamps")
        return out

    def set_option(self, key: str, value: int):
        _check(lib.zl_set_option(self._h, key.encode(), int(value)), f"zl_set_option({key})")

    @property
    def workspace_bytes(self) -> int:
        return lib.zl_workspace_bytes(self._h)

    @property
    def launches_per_call(self) -> int:
        return lib.zl_launches_per_call(self._h)

    @property
    def route(self) -> int:
        """0: segment sweep only, 1: RANGE filter route, 2: bucket route."""
        return lib.zl_route(self._h)

    def segments_per_instance(self, B: int) -> int:
        return lib.zl_segments_per_instance(self._h, B)

    @property
    def last_cuda_error(self) -> int:
        return lib.zl_last_cuda_error(self._h)

    def destroy(self):
        if getattr(self, "_h", None):
            lib.zl_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def zl_predict_batched(last: torch.Tensor, interval: torch.Tensor, R: int,
                       stream: torch.cuda.Stream | None = None) -> torch.Tensor:
    """Phase 1 of ZipLine: CUDA int64 [B, n] last end timestamps and intervals -> [B, n, R] predictions."""
    B, n = last.shape
    out = torch.empty((B, n, R), dtype=torch.int64, device=last.device)
    s = stream if stream is not None else torch.cuda.current_stream(last.device)
    rc = lib.zl_predict_batched(_dev_ptr(last, torch.int64, B * n, "last"), _dev_ptr(interval, torch.int64, B * n, "interval"),
                                B, n, R, out.data_ptr(), s.cuda_stream)
    _check(rc, "zl_predict_batched")
    return out


def zl_gridscan_batched(ts: torch.Tensor, full: bool = False, stream: torch.cuda.Stream | None = None):
    """The paper's heuristic baselines (Algorithm 1): GridScan, or FullGridScan with full=True.
    ts: CUDA int64 [B, n, R] -> (idx [B, n] int32, barrier [B], wait [B])."""
    B, n, R = ts.shape
    dev = ts.device
    scratch = torch.empty(B * (n * R if full else R), dtype=torch.int64, device=dev)
    idx = torch.empty((B, n), dtype=torch.int32, device=dev)
    barrier = torch.empty(B, dtype=torch.int64, device=dev)
    wait = torch.empty(B, dtype=torch.int64, device=dev)
    s = stream if stream is not None else torch.cuda.current_stream(dev)
    rc = lib.zl_gridscan_batched(_dev_ptr(ts, torch.int64, B * n * R, "ts"), B, n, R, int(bool(full)),
                                 scratch.data_ptr(), idx.data_ptr(), barrier.data_ptr(), wait.data_ptr(), s.cuda_stream)
    _check(rc, "zl_gridscan_batched")
    return idx, barrier, wait


def zl_probe_read_batched(ts: torch.Tensor, count: torch.Tensor, sink: torch.Tensor,
                          stream: torch.cuda.Stream | None = None) -> None:
    """Measurement aid: only load the first count[row] timestamps of every row.
    ts: CUDA int64 [..., R]; count: CUDA int32, one per row; sink: CUDA int64/uint64 scalar."""
    R = ts.shape[-1]
    rows = ts.numel() // R
    s = stream if stream is not None else torch.cuda.current_stream(ts.device)
    rc = lib.zl_probe_read_batched(_dev_ptr(ts, torch.int64, rows * R, "ts"), _dev_ptr(count, torch.int32, rows, "count"),
                                   rows, R, sink.data_ptr(), s.cuda_stream)
    _check(rc, "zl_probe_read_batched")


def zl_noalloc_max_batch() -> int:
    return lib.zl_noalloc_max_batch()


def zl_noalloc_scratch_bytes() -> int:
    return lib.zl_noalloc_scratch_bytes()


def zl_select_batched_noalloc(ts: torch.Tensor, out: Selection, objective: int = ZL_OBJ_RANGE, flags: int = 0,
                              stream: torch.cuda.Stream | None = None) -> Selection:
    """The search through the entry point that allocates nothing: no handle, scratch in the library's
    fixed device array.  ``ts`` is CUDA int64 [B, n, R] on the current device and ``out`` holds the
    caller's result tensors (this wrapper allocates nothing either).  Calls that overlap on the GPU
    race on the shared array; keep them on one stream."""
    B, n, R = ts.shape
    s = stream if stream is not None else torch.cuda.current_stream(ts.device)
    rc = lib.zl_select_batched_noalloc(n, R, objective, flags, _dev_ptr(ts, torch.int64, B * n * R, "ts"), B,
                                       _dev_ptr(out.idx, torch.int32, B * n, "idx"),
                                       _dev_ptr(out.barrier, torch.int64, B, "barrier"),
                                       _dev_ptr(out.wait, torch.int64, B, "wait"),
                                       _dev_ptr(out.status, torch.int32, B, "status"), s.cuda_stream)
    _check(rc, "zl_select_batched_noalloc")
    return out


TRACE_FIELDS = (("om_t", torch.int64), ("om_p", torch.int32), ("om_i", torch.int32), ("delta", torch.int64),
                ("first", torch.int32), ("S", torch.int64), ("cnt", torch.int32), ("next", torch.int64),
                ("PM", torch.int64), ("d_range", torch.int64), ("w_sum", torch.int64))


def zl_trace_batched(ts: torch.Tensor, stream: torch.cuda.Stream | None = None) -> dict:
    """Per-position intermediates of the sweep for small instances; ts: CUDA int64 [B, n, R]."""
    B, n, R = ts.shape
    out = {k: torch.empty((B, n * R), dtype=dt, device=ts.device) for k, dt in TRACE_FIELDS}
    s = stream if stream is not None else torch.cuda.current_stream(ts.device)
    rc = lib.zl_trace_batched(_dev_ptr(ts, torch.int64, B * n * R, "ts"), B, n, R,
                              *[out[k].data_ptr() for k, _ in TRACE_FIELDS], s.cuda_stream)
    _check(rc, "zl_trace_batched")
    return out
