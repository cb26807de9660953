"""Builds libvosti.so in-tree with nvcc for sm_100a (no JIT cache involved)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libvosti.so")
SOURCES = ["vosti.cu", "vosti_noalloc.cu", "vosti_linear.cu", "prefix_cache.cpp"]
HEADERS = ["attn_split.cuh", "attn_tile.cuh", "aux_kernels.cuh", "device_plan.cuh", "tile_math.cuh", "meta.cuh", "nc_math.cuh", "ptx.cuh", "tcgen05.cuh", os.path.join("..", "..", "include", "vosti.h"),
           os.path.join("..", "..", "include", "vosti_cache.h"),
           os.path.join("..", "..", "include", "vosti_linear.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > built for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or _stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-O2", "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
