"""Compiles the CUDA library in-tree for sm_100a with nvcc (no GPU needed: nvcc cross-compiles)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libwkv.so")
SOURCES = ["wkv_api.cu"]
DEPS = SOURCES + ["wkv_kernels.cuh", "wkv_prefill.cuh", "wkv_block.cuh", os.path.join("..", "..", "include", "wkv.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > built for d in DEPS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        extra = os.environ.get("WKV_NVCC_EXTRA", "").split()      # build-time tuning macros, e.g. -DWKV_RING_BYTES=49152
        cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB + ".tmp"] + SOURCES
        subprocess.run(cmd, check=True, cwd=CSRC)
        os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
