"""Seeded synthetic inputs for the ZipLine barrier-selection search.

Holds input generation only (no search arithmetic).  ``generate`` fills a
``[B, n, R]`` int64 array of per-worker predicted iteration end timestamps in
microseconds; ``CONFIGS`` names the five heterogeneous-cluster workloads and
the six shapes of the paper's Table II.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libzl_inputs.so")


class _CWorkload(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_int32), ("R", ctypes.c_int32), ("B", ctypes.c_int32),
        ("mean_kind", ctypes.c_int32),
        ("mean_us", ctypes.c_double), ("sigma", ctypes.c_double), ("mean2_us", ctypes.c_double),
        ("jitter", ctypes.c_double),
        ("straggler_frac", ctypes.c_double), ("straggler_mult", ctypes.c_double),
        ("spike_prob", ctypes.c_double), ("spike_mult", ctypes.c_double),
        ("offset_max_us", ctypes.c_double),
        ("base_seed", ctypes.c_int64), ("epoch_us", ctypes.c_int64),
    ]


@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    R: int
    B: int
    mean_kind: int = 0          # 0 lognormal(ln mean_us, sigma), 1 bimodal halves
    mean_us: float = 200_000.0
    sigma: float = 0.3
    mean2_us: float = 0.0
    jitter: float = 0.05
    straggler_frac: float = 0.0
    straggler_mult: float = 1.0
    spike_prob: float = 0.0
    spike_mult: float = 1.0
    offset_max_us: float = 0.0
    base_seed: int = 0
    epoch_us: int = 0

    @property
    def timestamps(self) -> int:
        return self.n * self.R * self.B

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


CONFIGS = {
    "c1": Workload("c1", n=4, R=8, B=1),
    "c2": Workload("c2", n=16, R=64, B=4096),
    "c3": Workload("c3", n=128, R=256, B=1024, mean_us=150_000.0, sigma=0.2, jitter=0.10,
                   straggler_frac=0.10, straggler_mult=3.0),
    "c4": Workload("c4", n=1024, R=1024, B=64, mean_us=100_000.0, sigma=0.5, jitter=0.08,
                   spike_prob=0.01, spike_mult=5.0),
    "c5": Workload("c5", n=4096, R=4096, B=8, mean_kind=1, mean_us=80_000.0, mean2_us=240_000.0,
                   jitter=0.05, offset_max_us=1_000_000.0),
}
# Shapes of the paper's Table II (its data were generated and never published).
for _n in (10, 100, 1000):
    for _R in (15, 150):
        CONFIGS[f"t2_n{_n}_R{_R}"] = Workload(f"t2_n{_n}_R{_R}", n=_n, R=_R, B=1)


def build(force: bool = False) -> str:
    """Compile the generator with gcc (OpenMP) when missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.zl_generate.argtypes = [ctypes.POINTER(_CWorkload), ctypes.c_void_p]
        _lib.zl_generate.restype = ctypes.c_int
    return _lib


def generate(w: Workload, B: int | None = None, first_instance: int = 0,
             out: np.ndarray | None = None) -> np.ndarray:
    """Return ``[B, n, R]`` int64 timestamps for instances first_instance .. first_instance+B-1."""
    B = w.B if B is None else int(B)
    cw = _CWorkload(w.n, w.R, B, w.mean_kind, w.mean_us, w.sigma, w.mean2_us, w.jitter,
                    w.straggler_frac, w.straggler_mult, w.spike_prob, w.spike_mult,
                    w.offset_max_us, w.base_seed + first_instance, w.epoch_us)
    if out is None:
        out = np.empty((B, w.n, w.R), dtype=np.int64)
    assert out.dtype == np.int64 and out.flags.c_contiguous and out.size == B * w.n * w.R
    rc = _load().zl_generate(ctypes.byref(cw), out.ctypes.data)
    if rc != 0:
        raise ValueError("zl_generate rejected the workload")
    return out
