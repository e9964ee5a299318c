"""Build the CUDA library in-tree for sm_100a (no GPU needed: nvcc cross-compiles)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libecq.so")
SOURCES = ["ecq_api.cu"]
HEADERS = ["ecq_common.cuh", "ecq_encode.cuh", "ecq_decode.cuh", "ecq_decode_ring.cuh", "ecq_stats.cuh", "ecq_entropy.cuh"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    # every fp32 operation of the codec is an explicit round-to-nearest intrinsic;
    # contraction is also switched off globally so nothing can be fused behind them
    "-fmad=false", "-shared", "-Xcompiler", "-fPIC",
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(os.path.dirname(_HERE), "include", "ecq.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile ``libecq.so`` next to this file if it is missing or out of date."""
    if force or _stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = LIB + ".tmp.%d" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
              ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
        subprocess.check_call(cmd)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
