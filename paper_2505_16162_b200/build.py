"""Builds libknnssd.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libknnssd.so")
SOURCES = ["knnssd.cu"]
HEADERS = ["kernels.cuh", "linear_stream.cuh", "linear_presplit.cuh", "pass_kernel.cuh", "prefill.cuh", "prefill_host.cuh", "anchors.cuh", "linear_tc.cuh", "sampling.cuh", os.path.join("..", "..", "include", "knnssd.h")]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "--use_fast_math=false"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
        if verbose:
            flags += ["-Xptxas", "-v"]
        cmd = [nvcc] + flags + ["-o", LIB] + [os.path.join(CSRC, f) for f in SOURCES]
        subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
