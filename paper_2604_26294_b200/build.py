"""Compile the CUDA library in-tree for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = [os.path.join(HERE, "csrc", "tsp_mlp.cu")]
HEADERS = [os.path.join(HERE, "csrc", n) for n in ("ptx.cuh", "gemm_core.cuh", "fwd_kernels.cuh", "bwd_kernels.cuh", "dyn_kernels.cuh", "skew_kernels.cuh",
                                                   "pair_kernels.cuh", "attn_kernels.cuh", "tsp_attn_host.cuh")]
HEADERS += [os.path.join(os.path.dirname(HERE), "include", n) for n in ("tsp_mlp.h", "tsp_attn.h")]
LIB = os.path.join(HERE, "libtsp_mlp.so")


def _nvcc() -> str:
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return nvcc


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Build libtsp_mlp.so next to this file; returns its path."""
    if not force and not is_stale():
        return LIB
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xptxas", "-v", "-shared", "-Xcompiler", "-fPIC", "-o", LIB] + SOURCES + ["-lcudart"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        print(res.stdout)
        print(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libtsp_mlp.so")
    return LIB


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
