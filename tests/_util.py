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


def assert_parity(y_gpu, y_ref, what="", rel_fro_tol=REL_FRO_TOL, mean_abs_tol=MEAN_ABS_TOL):
    assert torch.isfinite(y_gpu.float()).all(), f"{what}: non-finite output"
    max_abs, mean_abs, rel_fro = error_metrics(y_gpu, y_ref)
    msg = f"{what}: max_abs={max_abs:.3e} mean_abs={mean_abs:.3e} rel_fro={rel_fro:.3e}"
    assert max_abs <= MAX_ABS_TOL, msg
    assert mean_abs <= mean_abs_tol, msg
    assert rel_fro <= rel_fro_tol, msg
    return max_abs, mean_abs, rel_fro
