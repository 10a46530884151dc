"""CPU oracle for the ZipLine barrier-selection search.

Test infrastructure only: the tests, the smoke check and the CPU-baseline leg
of the benchmark use it; the CUDA library never does, and the two share no
code.  The arithmetic lives in ``zl_oracle.c`` (plain C, compiled with gcc);
this module marshals numpy arrays to it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

RANGE = 0   # d_Z = max(Z) - min(Z), the paper's objective function (Section III)
SUM = 1     # d_Z = sum_p (max(Z) - z_p)

INF = np.iinfo(np.int64).max

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zl_oracle.c")
_LIB = os.path.join(_HERE, "libzl_oracle.so")
_ERR = {-1: "bad argument", -2: "a row is not non-decreasing",
        -3: "objective does not fit int64", -4: "out of memory"}


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, ci = ctypes.c_void_p, ctypes.c_int
        for name in ("zlo_enumerate", "zlo_sweep", "zlo_sweep_window"):
            f = getattr(lib, name)
            f.argtypes = [vp, ci, ci, ci, vp, vp, vp]
            f.restype = ci
        lib.zlo_alg2.argtypes = [vp, ci, ci, vp, vp, vp]
        lib.zlo_alg2.restype = ci
        lib.zlo_trace.argtypes = [vp, ci, ci] + [vp] * 11
        lib.zlo_trace.restype = ci
        lib.zlo_gridscan.argtypes = [vp, ci, ci, ci, vp, vp, vp]
        lib.zlo_gridscan.restype = ci
        lib.zlo_predict.argtypes = [vp, vp, ci, ci, vp]
        lib.zlo_predict.restype = ci
        _lib = lib
    return _lib


def _matrix(M) -> np.ndarray:
    M = np.ascontiguousarray(M, dtype=np.int64)
    if M.ndim != 2 or M.shape[0] < 1 or M.shape[1] < 1:
        raise ValueError("expected an [n, R] matrix")
    return M


def _check(rc: int):
    if rc != 0:
        raise ValueError(f"oracle: {_ERR.get(rc, rc)}")


def _select(fn_name: str, M, objective: int):
    M = _matrix(M)
    n, R = M.shape
    wait, barrier = ctypes.c_int64(), ctypes.c_int64()
    idx = np.empty(n, dtype=np.int32)
    rc = getattr(_load(), fn_name)(M.ctypes.data, n, R, int(objective),
                                   ctypes.addressof(wait), ctypes.addressof(barrier), idx.ctypes.data)
    _check(rc)
    return int(wait.value), int(barrier.value), idx


def enumerate_all(M, objective: int = RANGE):
    """Minimum over all R^n combinations (Section IV, naive search) -> (wait, barrier, idx[n])."""
    return _select("zlo_enumerate", M, objective)


def sweep(M, objective: int = RANGE):
    """One pass over sorted Omega with an O(n) evaluation per position (Section IV, ZipLine)."""
    return _select("zlo_sweep", M, objective)


def sweep_window(M, objective: int = RANGE):
    """The same pass with min(Z) / sum(Z) kept incrementally; for large n."""
    return _select("zlo_sweep_window", M, objective)


def alg2(M):
    """Algorithm 2 step by step -> (wait, barrier, idx of Z* itself). RANGE only."""
    M = _matrix(M)
    n, R = M.shape
    wait, barrier = ctypes.c_int64(), ctypes.c_int64()
    idx = np.empty(n, dtype=np.int32)
    _check(_load().zlo_alg2(M.ctypes.data, n, R, ctypes.addressof(wait),
                            ctypes.addressof(barrier), idx.ctypes.data))
    return int(wait.value), int(barrier.value), idx


TRACE_FIELDS = (("om_t", np.int64), ("om_p", np.int32), ("om_i", np.int32), ("delta", np.int64),
                ("first", np.int32), ("S", np.int64), ("cnt", np.int32), ("next", np.int64),
                ("PM", np.int64), ("d_range", np.int64), ("w_sum", np.int64))


def trace(M) -> dict:
    """Per-position intermediates of the pass over Omega (order: time, worker, iteration)."""
    M = _matrix(M)
    n, R = M.shape
    out = {k: np.empty(n * R, dtype=dt) for k, dt in TRACE_FIELDS}
    _check(_load().zlo_trace(M.ctypes.data, n, R, *[out[k].ctypes.data for k, _ in TRACE_FIELDS]))
    return out


def gridscan(M, full: bool = False):
    """Algorithm 1 (GridScan), or FullGridScan with full=True -> (wait, barrier, idx of Z*). Heuristic baselines."""
    M = _matrix(M)
    n, R = M.shape
    wait, barrier = ctypes.c_int64(), ctypes.c_int64()
    idx = np.empty(n, dtype=np.int32)
    _check(_load().zlo_gridscan(M.ctypes.data, n, R, int(bool(full)), ctypes.addressof(wait),
                                ctypes.addressof(barrier), idx.ctypes.data))
    return int(wait.value), int(barrier.value), idx


def predict(last, interval, R: int) -> np.ndarray:
    """Phase 1 of ZipLine: [n, R] future end timestamps, e_i = last + i * interval (i = 1..R)."""
    last = np.ascontiguousarray(last, dtype=np.int64)
    interval = np.ascontiguousarray(interval, dtype=np.int64)
    if last.ndim != 1 or last.shape != interval.shape or R < 1:
        raise ValueError("expected last[n], interval[n], R >= 1")
    out = np.empty((last.shape[0], R), dtype=np.int64)
    _check(_load().zlo_predict(last.ctypes.data, interval.ctypes.data, last.shape[0], int(R), out.ctypes.data))
    return out


def select_batched(ts, objective: int = RANGE, fn=sweep_window):
    """Apply ``fn`` to every instance of ``ts[B, n, R]`` -> (idx[B, n], barrier[B], wait[B])."""
    ts = np.ascontiguousarray(ts, dtype=np.int64)
    B, n, _ = ts.shape
    idx = np.empty((B, n), dtype=np.int32)
    barrier = np.empty(B, dtype=np.int64)
    wait = np.empty(B, dtype=np.int64)
    for b in range(B):
        wait[b], barrier[b], idx[b] = fn(ts[b], objective)
    return idx, barrier, wait
