"""Helpers shared by the GPU parity tests: run the CUDA library, run the oracle, compare."""
import numpy as np
import torch

import oracle

# Gate on the bf16 outputs against the fp64 oracle.  The relative-Frobenius companion catches
# what the absolute gate cannot at large N, where |Y| ~ 1/sqrt(N) (an all-zero output would pass
# the absolute gate there); bf16 output rounding alone contributes about 2e-3 to it.
MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3
REL_FRO_TOL = 1e-2
# Element-wise gate that scales with the output: per (batch, head) slab,
# max|Y_gpu - Y_oracle| <= SCALED_MAX_UNITS * 2^-8 * max|Y_oracle|.  2^-8 is the unit roundoff of
# the 16-bit output (8 significant bits): rounding the largest element alone may cost one unit.
# The 16-bit operands phi(Q), phi(K), S | z add an error that is Gaussian-like over the slab with
# a standard deviation of about 1.5e-3 of rms|Y|; over 3e7 elements its maximum is near 6 sigma,
# i.e. about 1e-2 rms|Y|, which is 2^-8 * 2.3 rms|Y| and at most about one unit of max|Y|
# (max|Y| / rms|Y| is between 1.0 for V ~ N(1,1) and 5.7 for V ~ N(0,1)).  Measured on B200 over
# the ten smaller workload shapes with every kernel variant, V ~ N(0,1) and V ~ N(1,1), and the
# edge list (131 runs): 1.44 units at worst (N = 4096, d = 40, V ~ N(1,1)), 1.1 - 1.3 typically.
# The gate is twice the measured maximum, rounded: it was set from runs that were green under the
# other gates and before any test depended on it.
SCALED_MAX_UNITS = 3.0
UNIT_ROUNDOFF_16 = 2.0 ** -8
EPS = 1e-6


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_y(q, k, v, eps=EPS, phi_kind=oracle.PHI_ELU_PLUS_ONE) -> np.ndarray:
    return oracle.linear(to_f64(q), to_f64(k), to_f64(v), eps, phi_kind)


def error_metrics(y_gpu: torch.Tensor, y_ref: np.ndarray):
    diff = to_f64(y_gpu) - y_ref
    max_abs = float(np.abs(diff).max()) if diff.size else 0.0
    mean_abs = float(np.abs(diff).mean()) if diff.size else 0.0
    ref_norm = float(np.linalg.norm(y_ref.ravel()))
    rel_fro = float(np.linalg.norm(diff.ravel()) / ref_norm) if ref_norm > 0 else 0.0
    return max_abs, mean_abs, rel_fro


def scaled_max_units(y_gpu, y_ref: np.ndarray, y_scale: np.ndarray = None) -> float:
    """Largest per-slab max|Y_gpu - Y_ref| in units of 2^-8 * max|Y| of that slab.  Arrays are
    [..., n, d]; everything before the last two axes indexes slabs.  ``y_scale`` (same leading
    axes) supplies the slabs' max|Y| when ``y_ref`` holds only some rows of each slab."""
    diff = np.abs(to_f64(y_gpu) - y_ref)
    if diff.size == 0:
        return 0.0
    lead = diff.shape[:-2]
    d_max = diff.reshape(lead + (-1,)).max(axis=-1)
    scale = np.abs(y_ref).reshape(lead + (-1,)).max(axis=-1) if y_scale is None else np.asarray(y_scale)
    scale = np.maximum(scale, np.finfo(np.float64).tiny)
    return float((d_max / (UNIT_ROUNDOFF_16 * scale)).max())


def assert_parity(y_gpu, y_ref, what="", rel_fro_tol=REL_FRO_TOL, mean_abs_tol=MEAN_ABS_TOL,
                  scaled_units=SCALED_MAX_UNITS, y_scale=None):
    assert torch.isfinite(y_gpu.float()).all(), f"{what}: non-finite output"
    max_abs, mean_abs, rel_fro = error_metrics(y_gpu, y_ref)
    units = scaled_max_units(y_gpu, y_ref, y_scale)
    msg = (f"{what}: max_abs={max_abs:.3e} mean_abs={mean_abs:.3e} rel_fro={rel_fro:.3e} "
           f"scaled_max={units:.2f} units of 2^-8 max|Y|")
    assert max_abs <= MAX_ABS_TOL, msg
    assert mean_abs <= mean_abs_tol, msg
    assert rel_fro <= rel_fro_tol, msg
    if scaled_units is not None:
        assert units <= scaled_units, msg
    return max_abs, mean_abs, rel_fro
