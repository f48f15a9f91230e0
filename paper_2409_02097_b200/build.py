"""Compile the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "liblinfusion_attn.so")
_SOURCES = ["linfusion_attn.cu"]
_HEADERS = ["common.cuh", "split_kernels.cuh", "stream_kernels.cuh", "fused_kernels.cuh"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(_CSRC, f) for f in _SOURCES + _HEADERS]
    paths.append(os.path.join(os.path.dirname(_PKG), "include", "linfusion_attn.h"))
    return max(os.path.getmtime(p) for p in paths)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Build ``liblinfusion_attn.so`` next to this file if it is missing or stale."""
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-o", LIB_PATH]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(_CSRC, f) for f in _SOURCES]
    subprocess.run(cmd, check=True)
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
