"""GPU parity of the operator without its normalizer, Y_i = phi(Q_i) S (Prop. 2 before Eq. 5's
division; the "without normalization" rows of Tab. 2), against the fp64 oracle.  |Y| grows with
N here, so the gates are relative: the absolute gates of the normalized operator scaled by
max|Y_oracle|, and the relative Frobenius error as it is."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_02097_b200 import attn, workloads as wl

from _util import MAX_ABS_TOL, MEAN_ABS_TOL, REL_FRO_TOL, error_metrics, to_f64

pytestmark = pytest.mark.gpu


def run_unnormalized(q, k, v, variant, layout="head_major"):
    B, H, N, d = q.shape
    op = attn.LinFusionAttention(B, H, N, d, device=q.device.index or 0, variant=variant, normalize=False)
    y = op.forward(q, k, v)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    return y, op


def assert_relative_parity(y, ref, what):
    assert torch.isfinite(y.float()).all(), what
    scale = float(np.abs(ref).max())
    max_abs, mean_abs, rel_fro = error_metrics(y, ref)
    msg = f"{what}: max_abs/scale={max_abs / scale:.3e} mean_abs/scale={mean_abs / scale:.3e} rel_fro={rel_fro:.3e}"
    assert max_abs <= MAX_ABS_TOL * scale, msg
    assert mean_abs <= MEAN_ABS_TOL * scale, msg
    assert rel_fro <= REL_FRO_TOL, msg


CASES = [
    # (B, H, N, d, variants): several tiles and a ragged tail for every kernel family
    (2, 3, 1000, 64, ("split", "stream", "cluster")),
    (1, 2, 333, 40, ("split", "cluster")),
    (1, 4, 2500, 160, ("split",)),
    (2, 20, 144, 64, ("auto", "stream")),
    (1, 10, 40000, 64, ("auto", "stream", "split")),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "x".join(map(str, c[:4])))
def test_unnormalized_matches_oracle(case):
    B, H, N, d, variants = case
    q, k, v = wl.make_small(B, H, N, d, seed=41, device="cuda")
    ref = oracle.linear_unnormalized(to_f64(q), to_f64(k), to_f64(v))
    for variant in variants:
        y, op = run_unnormalized(q, k, v, variant)
        assert_relative_parity(y, ref, f"{case[:4]}/{variant}->{op.variant}")
        op.close()


def test_unnormalized_is_the_normalized_output_times_its_denominator():
    """Same handle shape, both operators: Y_un = Y_norm * (phi(Q) . z + eps) row by row (to bf16 rounding)."""
    B, H, N, d = 1, 2, 3000, 64
    q, k, v = wl.make_small(B, H, N, d, seed=43, device="cuda")
    op_n = attn.LinFusionAttention(B, H, N, d, variant="stream")
    op_u = attn.LinFusionAttention(B, H, N, d, variant="stream", normalize=False)
    y_n, y_u = op_n.forward(q, k, v), op_u.forward(q, k, v)
    torch.cuda.synchronize()
    _, z = op_n.read_state()
    den = oracle.phi(to_f64(q)) @ z[..., None]                       # [B, H, N, 1]
    got, want = to_f64(y_u), to_f64(y_n) * den
    assert np.linalg.norm(got - want) <= 1e-2 * np.linalg.norm(want)
    op_n.close()
    op_u.close()


def test_unnormalized_host_buffers_and_no_alloc_entry_point():
    B, H, N, d = 1, 3, 700, 64
    q, k, v = wl.make_small(B, H, N, d, seed=44, device="cuda")
    ref = oracle.linear_unnormalized(to_f64(q), to_f64(k), to_f64(v))
    op = attn.LinFusionAttention(B, H, N, d, normalize=False)
    qh, kh, vh = q.cpu(), k.cpu(), v.cpu()
    y_host = torch.empty_like(qh)
    op.forward_host(qh, kh, vh, y_host)
    torch.cuda.synchronize()
    assert_relative_parity(y_host, ref, "forward_host")
    op.close()
    y = torch.empty_like(q)
    desc = attn.make_desc(B, H, N, d, normalize=False)
    attn.linfusion_attn_forward_noalloc(desc, q.data_ptr(), k.data_ptr(), v.data_ptr(), y.data_ptr(),
                                        torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert_relative_parity(y, ref, "forward_noalloc")
