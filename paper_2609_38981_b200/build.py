"""Builds the two shared libraries in-tree with nvcc for sm_100a (no JIT cache involved):
libvosti.so (attention, KV append, prefix-cache manager) and libvosti_linear.so (the linear
layer and RMS normalisation, which the attention path does not need)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libvosti.so")
LIB_LINEAR = os.path.join(HERE, "libvosti_linear.so")
_INC = os.path.join("..", "..", "include")
TARGETS = {
    LIB: (["vosti.cu", "vosti_noalloc.cu", "prefix_cache.cpp"],
          ["attn_split.cuh", "attn_tile.cuh", "aux_kernels.cuh", "device_plan.cuh", "tile_math.cuh", "meta.cuh",
           "nc_math.cuh", "ptx.cuh", "tcgen05.cuh", "selftest_mma.cuh", os.path.join(_INC, "vosti.h"), os.path.join(_INC, "vosti_cache.h")]),
    LIB_LINEAR: (["vosti_linear.cu"],
                 ["ptx.cuh", "tcgen05.cuh", os.path.join(_INC, "vosti.h"), os.path.join(_INC, "vosti_linear.h")]),
}


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    built = os.path.getmtime(lib)
    sources, headers = TARGETS[lib]
    return any(os.path.getmtime(os.path.join(CSRC, f)) > built for f in sources + headers)


def build(force: bool = False, verbose: bool = False) -> str:
    """Builds what is stale (or everything); returns the path of libvosti.so."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    for lib, (sources, _) in TARGETS.items():
        if not (force or _stale(lib)):
            continue
        if not all(os.path.exists(os.path.join(CSRC, f)) for f in sources):
            continue    # a source tree without the linear layer still builds the attention library
        tmp = lib + f".tmp{os.getpid()}"
        cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
               "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-O2", "-o", tmp] + \
              [os.path.join(CSRC, f) for f in sources]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        subprocess.run(cmd, check=True)
        os.replace(tmp, lib)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
