"""Build libconef.so in-tree with nvcc for sm_100a (no JIT cache involved)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libconef.so")
SOURCES = ["conef_api.cu", "conef_noalloc.cu"]
HEADERS = ["conef_internal.h", "conef_kernels.cuh", "conef_hash.cuh", "conef_fast.cuh", "conef_gs.cuh", "conef_rowsketch.cuh", "conef_apply.cuh", "conef_flatvec.cuh", "conef_chunksketch.cuh", "conef_rowsp1.cuh", "conef_rowsp3.cuh", os.path.join("..", "..", "include", "conef.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-shared", "-Xcompiler", "-fPIC"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc, *NVCC_FLAGS] + (["-Xptxas", "-v"] if verbose else []) + \
              ["-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
        subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
