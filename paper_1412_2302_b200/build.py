"""Compile the CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libalexnet_b200.so")
LIB_TIMELINE = os.path.join(HERE, "libalexnet_b200_timeline.so")      # the same sources with -DALEXNET_TIMELINE
SOURCES = ["alexnet_api.cu", "loader.cpp"]
HEADERS = ["tc_gemm.cuh", "kernels.cuh", os.path.join("..", "..", "include", "alexnet.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, timeline: bool = False) -> str:
    """timeline=True builds the instrumented variant (per-role timers inside conv_kernel) as a second library."""
    lib = LIB_TIMELINE if timeline else LIB
    if not force and not timeline and not _stale():
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-Xcompiler", "-fPIC", "-Xcompiler", "-pthread", "-shared", "-o", lib] + [os.path.join(CSRC, s) for s in SOURCES]
    if timeline:
        cmd.insert(1, "-DALEXNET_TIMELINE")
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="--quiet" not in sys.argv, timeline="--timeline" in sys.argv))
