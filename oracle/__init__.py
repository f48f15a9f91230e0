"""fp64 CPU oracle for normalized non-causal linear attention — TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``linfusion_oracle.c`` (plain C, fp64, sums in index
order).  Nothing here is on the product path and nothing here imports the CUDA
package: only the tests, the smoke check and the benchmark's CPU-baseline leg
use this module.  The arithmetic lives in the C file, which states which passage
of the paper each routine follows (Prop. 2 for the state, Eq. 5 for the
normalizer, Sec. 2.2 for the non-negative activation).

Every routine is pinned by ``tests/test_oracle_pins.py`` against closed forms,
hand-worked rational examples, a library mean, and invariants that the paper
fixes (row sums of one, non-causality, resolution invariance, shard additivity).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "linfusion_oracle.c")
_LIB = os.path.join(_HERE, "liblinfusion_oracle.so")

PHI_ELU_PLUS_ONE = 0
PHI_IDENTITY = 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math: sums keep their written order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.oracle_phi.restype = ctypes.c_double
        lib.oracle_phi.argtypes = [ctypes.c_double, ctypes.c_int]
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_state.restype = None
        lib.oracle_state.argtypes = [dp, dp, ctypes.c_long, ctypes.c_long, ctypes.c_int,
                                     ctypes.c_int, dp, dp]
        lib.oracle_apply.restype = None
        lib.oracle_apply.argtypes = [dp, dp, dp, ctypes.c_long, ctypes.c_long, ctypes.c_int,
                                     ctypes.c_double, ctypes.c_int, dp]
        lib.oracle_apply_unnormalized.restype = None
        lib.oracle_apply_unnormalized.argtypes = [dp, dp, ctypes.c_long, ctypes.c_long, ctypes.c_int,
                                                  ctypes.c_int, dp]
        lib.oracle_linear.restype = ctypes.c_int
        lib.oracle_linear.argtypes = [dp, dp, dp, ctypes.c_long, ctypes.c_long, ctypes.c_int,
                                      ctypes.c_double, ctypes.c_int, dp]
        lib.oracle_quadratic.restype = None
        lib.oracle_quadratic.argtypes = [dp, dp, dp, ctypes.c_long, ctypes.c_long, ctypes.c_int,
                                         ctypes.c_double, ctypes.c_int, dp, dp]
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _slabs_n_d(a: np.ndarray):
    if a.ndim < 2:
        raise ValueError("expected [..., n, d]")
    n, d = a.shape[-2], a.shape[-1]
    slabs = int(np.prod(a.shape[:-2], dtype=np.int64)) if a.ndim > 2 else 1
    return slabs, n, d


def num_threads() -> int:
    """Threads the C routines will use (OpenMP's maximum for this process)."""
    return int(_load().oracle_num_threads())


def phi(x, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """Elementwise non-negative activation (Sec. 2.2); reading: elu(x) + 1."""
    lib = _load()
    x = _f64(x)
    out = np.empty_like(x)
    flat_in, flat_out = x.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = lib.oracle_phi(float(flat_in[i]), phi_kind)
    return out


def state(k, v, phi_kind: int = PHI_ELU_PLUS_ONE):
    """S = phi(K)^T V  [..., d, d] and z = sum_j phi(K_j)  [..., d]   (Prop. 2, Eq. 5)."""
    k, v = _f64(k), _f64(v)
    if k.shape != v.shape:
        raise ValueError("k and v must have the same shape")
    slabs, n, d = _slabs_n_d(k)
    S = np.empty(k.shape[:-2] + (d, d), dtype=np.float64)
    z = np.empty(k.shape[:-2] + (d,), dtype=np.float64)
    _load().oracle_state(_ptr(k), _ptr(v), slabs, n, d, phi_kind, _ptr(S), _ptr(z))
    return S, z


def apply(q, S, z, eps: float, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """Y_i = phi(Q_i) S / (phi(Q_i) . z + eps)."""
    q, S, z = _f64(q), _f64(S), _f64(z)
    slabs, n, d = _slabs_n_d(q)
    if S.shape != q.shape[:-2] + (d, d) or z.shape != q.shape[:-2] + (d,):
        raise ValueError("S / z do not match q")
    y = np.empty_like(q)
    _load().oracle_apply(_ptr(q), _ptr(S), _ptr(z), slabs, n, d, float(eps), phi_kind, _ptr(y))
    return y


def apply_unnormalized(q, S, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """Y_i = phi(Q_i) S: Prop. 2 without Eq. 5's division (the Tab. 2 ablation)."""
    q, S = _f64(q), _f64(S)
    slabs, n, d = _slabs_n_d(q)
    if S.shape != q.shape[:-2] + (d, d):
        raise ValueError("S does not match q")
    y = np.empty_like(q)
    _load().oracle_apply_unnormalized(_ptr(q), _ptr(S), slabs, n, d, phi_kind, _ptr(y))
    return y


def linear_unnormalized(q, k, v, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """State, then the apply without the normalizer."""
    S, _ = state(k, v, phi_kind)
    return apply_unnormalized(q, S, phi_kind)


def linear(q, k, v, eps: float, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """The whole path, linear form: state then apply.  Inputs [..., n, d]; fp64 output."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    if not (q.shape == k.shape == v.shape):
        raise ValueError("q, k, v must have the same shape")
    slabs, n, d = _slabs_n_d(q)
    y = np.empty_like(q)
    rc = _load().oracle_linear(_ptr(q), _ptr(k), _ptr(v), slabs, n, d, float(eps), phi_kind,
                               _ptr(y))
    if rc != 0:
        raise MemoryError("oracle_linear could not allocate its state")
    return y


def quadratic(q, k, v, eps: float, phi_kind: int = PHI_ELU_PLUS_ONE, return_weights=False):
    """The attention-matrix form, O(n^2 d): Y = M V with row-normalized M.  Tiny n only."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    if not (q.shape == k.shape == v.shape):
        raise ValueError("q, k, v must have the same shape")
    slabs, n, d = _slabs_n_d(q)
    if n > 4096:
        raise ValueError("quadratic oracle is for tiny n")
    y = np.empty_like(q)
    m = np.empty(q.shape[:-2] + (n, n), dtype=np.float64) if return_weights else None
    _load().oracle_quadratic(_ptr(q), _ptr(k), _ptr(v), slabs, n, d, float(eps), phi_kind,
                             _ptr(y), _ptr(m) if m is not None else None)
    return (y, m) if return_weights else y
