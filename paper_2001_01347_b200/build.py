"""Compile the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libzipline.so")
SOURCES = [os.path.join(CSRC, "zipline.cu")]
DEPS = SOURCES + [os.path.join(CSRC, "zl_device.cuh"),
                  os.path.join(os.path.dirname(_HERE), "include", "zipline.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the ZipLine CUDA library cannot be built")


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Build ``libzipline.so`` next to this file when missing or older than its sources."""
    if force or is_stale():
        tmp = LIB + f".tmp{os.getpid()}"
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
        subprocess.run(cmd, check=True, cwd=CSRC)
        os.replace(tmp, LIB)
    return LIB
