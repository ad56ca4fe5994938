"""Build the CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsailor_b200.so")
SOURCES = [os.path.join(CSRC, "sailor_lib.cu")]
DEPS = SOURCES + [os.path.join(CSRC, f) for f in ("sailor_tables.cuh", "sailor_plan_kernels.cuh", "sailor_dp.cuh", "sailor_dp_budget.cuh", "sailor_batch.cuh", "sailor_mixed.cuh", "sailor_mixed_search.cuh", "sailor_peaks.cuh")] + [
    os.path.join(os.path.dirname(HERE), "include", "sailor.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-shared", "-Xcompiler", "-fPIC"]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libsailor_b200.so next to this file; returns its path."""
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
