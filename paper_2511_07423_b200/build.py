"""Compile the CUDA library for sm_100a into this package directory (in-tree, no JIT cache)."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsynera.so")
SOURCES = ["synera.cu", "scheduler.cpp"]
HEADERS = ["ptx.cuh", "gemm.cuh", "gemm2.cuh", "attention.cuh", "attention2.cuh", "sampling.cuh", os.path.join("..", "..", "include", "synera.h"),
           os.path.join("..", "..", "include", "synera_sched.h")]


def _nvcc() -> str:
    return shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"


def _stale(out: str) -> bool:
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, extra=(), out: str = LIB) -> str:
    if not force and not _stale(out):
        return out
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC", "-o", out, *extra,
           *[os.path.join(CSRC, s) for s in SOURCES]]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return out


PROBE = os.path.join(HERE, "probe_mma_rate")


def build_probe(force: bool = False) -> str:
    """The stand-alone tcgen05.mma issue-rate measurement (csrc/probe_mma_rate.cu), built beside the library."""
    src = os.path.join(CSRC, "probe_mma_rate.cu")
    if not force and os.path.exists(PROBE) and os.path.getmtime(PROBE) >= max(os.path.getmtime(src), os.path.getmtime(os.path.join(CSRC, "ptx.cuh"))):
        return PROBE
    subprocess.check_call([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-o", PROBE, src])
    return PROBE


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
