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
        cl, ci, cd = ctypes.c_long, ctypes.c_int, ctypes.c_double
        lib.oracle_state.restype = None
        lib.oracle_state.argtypes = [dp, dp, cl, cl, ci, ci, ci, dp, dp]
        lib.oracle_apply.restype = None
        lib.oracle_apply.argtypes = [dp, dp, dp, cl, cl, ci, ci, cd, ci, dp]
        lib.oracle_apply_unnormalized.restype = None
        lib.oracle_apply_unnormalized.argtypes = [dp, dp, cl, cl, ci, ci, ci, dp]
        lib.oracle_linear.restype = ci
        lib.oracle_linear.argtypes = [dp, dp, dp, cl, cl, ci, ci, cd, ci, dp]
        lib.oracle_quadratic.restype = None
        lib.oracle_quadratic.argtypes = [dp, dp, dp, cl, cl, ci, ci, cd, ci, dp, dp]
        lib.oracle_linear_map.restype = None
        lib.oracle_linear_map.argtypes = [dp, dp, dp, cl, ci, ci, dp]
        lib.oracle_layernorm.restype = None
        lib.oracle_layernorm.argtypes = [dp, dp, dp, cd, cl, ci, dp]
        lib.oracle_leaky_relu.restype = cd
        lib.oracle_leaky_relu.argtypes = [cd, cd]
        lib.oracle_mlp_producer.restype = ci
        lib.oracle_mlp_producer.argtypes = [dp, dp, dp, dp, dp, dp, cd, cd, cl, ci, ci, dp]
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


def _widths(qk: np.ndarray, v: np.ndarray):
    """(slabs, n, dk, dv) of a feature tensor [..., n, dk] and a value tensor [..., n, dv]."""
    if qk.shape[:-1] != v.shape[:-1]:
        raise ValueError("feature and value tensors must agree in every axis but the last")
    slabs, n, dk = _slabs_n_d(qk)
    return slabs, n, dk, v.shape[-1]


def state(k, v, phi_kind: int = PHI_ELU_PLUS_ONE):
    """S = phi(K)^T V  [..., dk, dv] and z = sum_j phi(K_j)  [..., dk]   (Prop. 2, Eq. 5; K may be
    wider or narrower than V, Prop. 3)."""
    k, v = _f64(k), _f64(v)
    slabs, n, dk, dv = _widths(k, v)
    S = np.empty(k.shape[:-2] + (dk, dv), dtype=np.float64)
    z = np.empty(k.shape[:-2] + (dk,), dtype=np.float64)
    _load().oracle_state(_ptr(k), _ptr(v), slabs, n, dk, dv, phi_kind, _ptr(S), _ptr(z))
    return S, z


def apply(q, S, z, eps: float, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """Y_i = phi(Q_i) S / (phi(Q_i) . z + eps);  q [..., n, dk], S [..., dk, dv] -> [..., n, dv]."""
    q, S, z = _f64(q), _f64(S), _f64(z)
    slabs, n, dk = _slabs_n_d(q)
    dv = S.shape[-1]
    if S.shape != q.shape[:-2] + (dk, dv) or z.shape != q.shape[:-2] + (dk,):
        raise ValueError("S / z do not match q")
    y = np.empty(q.shape[:-1] + (dv,), dtype=np.float64)
    _load().oracle_apply(_ptr(q), _ptr(S), _ptr(z), slabs, n, dk, dv, float(eps), phi_kind, _ptr(y))
    return y


def apply_unnormalized(q, S, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """Y_i = phi(Q_i) S: Prop. 2 without Eq. 5's division (the Tab. 2 ablation)."""
    q, S = _f64(q), _f64(S)
    slabs, n, dk = _slabs_n_d(q)
    dv = S.shape[-1]
    if S.shape != q.shape[:-2] + (dk, dv):
        raise ValueError("S does not match q")
    y = np.empty(q.shape[:-1] + (dv,), dtype=np.float64)
    _load().oracle_apply_unnormalized(_ptr(q), _ptr(S), slabs, n, dk, dv, phi_kind, _ptr(y))
    return y


def linear_unnormalized(q, k, v, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """State, then the apply without the normalizer."""
    S, _ = state(k, v, phi_kind)
    return apply_unnormalized(q, S, phi_kind)


def linear(q, k, v, eps: float, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """The whole path, linear form: state then apply.  q, k [..., n, dk]; v [..., n, dv]; fp64 output
    [..., n, dv]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    if q.shape != k.shape:
        raise ValueError("q and k must have the same shape")
    slabs, n, dk, dv = _widths(q, v)
    y = np.empty_like(v)
    rc = _load().oracle_linear(_ptr(q), _ptr(k), _ptr(v), slabs, n, dk, dv, float(eps), phi_kind,
                               _ptr(y))
    if rc != 0:
        raise MemoryError("oracle_linear could not allocate its state")
    return y


def quadratic(q, k, v, eps: float, phi_kind: int = PHI_ELU_PLUS_ONE, return_weights=False):
    """The attention-matrix form, O(n^2 d): Y = M V with row-normalized M.  Tiny n only."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    if q.shape != k.shape:
        raise ValueError("q and k must have the same shape")
    slabs, n, dk, dv = _widths(q, v)
    if n > 4096:
        raise ValueError("quadratic oracle is for tiny n")
    y = np.empty_like(v)
    m = np.empty(q.shape[:-2] + (n, n), dtype=np.float64) if return_weights else None
    _load().oracle_quadratic(_ptr(q), _ptr(k), _ptr(v), slabs, n, dk, dv, float(eps), phi_kind,
                             _ptr(y), _ptr(m) if m is not None else None)
    return (y, m) if return_weights else y


# ---- producers of Q, K, V from the layer input X (Sec. 3.1, implementation details; Eq. 2) ----

LN_EPS = 1e-5          # LayerNorm's epsilon (the paper gives none; the common default)
LEAKY_SLOPE = 0.01     # LeakyReLU's negative slope (likewise)


def linear_map(x, w, bias=None) -> np.ndarray:
    """X W (+ bias): x [..., c_in], w [c_in, c_out]."""
    x, w = _f64(x), _f64(w)
    c_in, c_out = w.shape
    if x.shape[-1] != c_in:
        raise ValueError("x and w do not match")
    n = int(np.prod(x.shape[:-1], dtype=np.int64))
    out = np.empty(x.shape[:-1] + (c_out,), dtype=np.float64)
    b = _f64(bias) if bias is not None else None
    _load().oracle_linear_map(_ptr(x), _ptr(w), _ptr(b) if b is not None else None, n, c_in, c_out, _ptr(out))
    return out


def layernorm(p, gamma, beta, ln_eps: float = LN_EPS) -> np.ndarray:
    """Row-wise LayerNorm over the last axis with scale gamma and shift beta."""
    p, gamma, beta = _f64(p), _f64(gamma), _f64(beta)
    c = p.shape[-1]
    n = int(np.prod(p.shape[:-1], dtype=np.int64))
    out = np.empty_like(p)
    _load().oracle_layernorm(_ptr(p), _ptr(gamma), _ptr(beta), float(ln_eps), n, c, _ptr(out))
    return out


def leaky_relu(x: float, slope: float = LEAKY_SLOPE) -> float:
    return float(_load().oracle_leaky_relu(float(x), float(slope)))


def mlp_producer(x, w_lin, w_1, b_1, gamma, beta, ln_eps: float = LN_EPS,
                 slope: float = LEAKY_SLOPE) -> np.ndarray:
    """f'(X) or g'(X): X W_lin + LeakyReLU(LayerNorm(X W_1 + b_1)); x [..., c_in] -> [..., c_out]."""
    x, w_lin, w_1, b_1, gamma, beta = (_f64(a) for a in (x, w_lin, w_1, b_1, gamma, beta))
    c_in, c_out = w_lin.shape
    if w_1.shape != (c_in, c_out) or x.shape[-1] != c_in:
        raise ValueError("weights do not match")
    n = int(np.prod(x.shape[:-1], dtype=np.int64))
    out = np.empty(x.shape[:-1] + (c_out,), dtype=np.float64)
    rc = _load().oracle_mlp_producer(_ptr(x), _ptr(w_lin), _ptr(w_1), _ptr(b_1), _ptr(gamma), _ptr(beta),
                                     float(ln_eps), float(slope), n, c_in, c_out, _ptr(out))
    if rc != 0:
        raise MemoryError("oracle_mlp_producer could not allocate its scratch")
    return out


def split_heads(t: np.ndarray, heads: int) -> np.ndarray:
    """[B, N, H*d] -> [B, H, N, d] (pure re-indexing)."""
    B, N, C = t.shape
    return np.ascontiguousarray(t.reshape(B, N, heads, C // heads).transpose(0, 2, 1, 3))


def linfusion_from_x(x, weights: dict, heads: int, eps: float, ln_eps: float = LN_EPS,
                     slope: float = LEAKY_SLOPE, phi_kind: int = PHI_ELU_PLUS_ONE) -> np.ndarray:
    """The whole module from the layer input: Q = f'(X), K = g'(X), V = X W_V, heads split, then the
    normalized linear attention; x [B, N, C] -> Y [B, N, H*d] (heads merged back).  `weights` holds
    q_lin, q_w1, q_b1, q_gamma, q_beta, k_lin, k_w1, k_b1, k_gamma, k_beta, v."""
    w = weights
    q = mlp_producer(x, w["q_lin"], w["q_w1"], w["q_b1"], w["q_gamma"], w["q_beta"], ln_eps, slope)
    k = mlp_producer(x, w["k_lin"], w["k_w1"], w["k_b1"], w["k_gamma"], w["k_beta"], ln_eps, slope)
    v = linear_map(x, w["v"])
    y = linear(split_heads(q, heads), split_heads(k, heads), split_heads(v, heads), eps, phi_kind)
    B, H, N, d = y.shape
    return np.ascontiguousarray(y.transpose(0, 2, 1, 3).reshape(B, N, H * d))
