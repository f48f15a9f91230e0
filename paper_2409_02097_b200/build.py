"""Compile the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "liblinfusion_attn.so")
_SOURCES = ["linfusion_attn.cu"]
_HEADERS = ["common.cuh", "split_kernels.cuh", "stream_kernels.cuh", "fused_kernels.cuh", "producer_kernels.cuh",
            "padded_kernels.cuh"]
CHECKED_LIB_PATH = os.path.join(_PKG, "liblinfusion_attn_checked.so")


def _newest_source_mtime() -> float:
    paths = [os.path.join(_CSRC, f) for f in _SOURCES + _HEADERS]
    paths.append(os.path.join(os.path.dirname(_PKG), "include", "linfusion_attn.h"))
    return max(os.path.getmtime(p) for p in paths)


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Build ``liblinfusion_attn.so`` next to this file if it is missing or stale.  ``checked=True``
    builds ``liblinfusion_attn_checked.so`` instead: the same sources with -DLF_CHECKED, in which every
    global-memory address the split / cluster kernels compute is compared with the buffers of the
    call and an access outside them is counted and skipped (a debugging build, slower)."""
    out = CHECKED_LIB_PATH if checked else LIB_PATH
    if not force and os.path.exists(out) and os.path.getmtime(out) >= _newest_source_mtime():
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-o", out]
    if checked:
        cmd += ["-DLF_CHECKED"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(_CSRC, f) for f in _SOURCES]
    subprocess.run(cmd, check=True)
    return out


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
