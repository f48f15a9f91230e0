"""The attention fed from the layer input X (Sec. 3.1 implementation details, Eq. 2): projections
fused into the state and apply kernels, against the fp64 oracle's producers + attention on the same
seeded 16-bit inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_02097_b200 import attn, workloads as wl

from _util import EPS, assert_parity, to_f64

pytestmark = pytest.mark.gpu

# (B, H, N): C = 64 H.  One tile, ragged tails, several tiles per CTA, many heads.
SHAPES = [(1, 2, 1), (2, 2, 129), (1, 3, 300), (2, 10, 1000), (1, 20, 520)]


def _x_and_weights(B, H, N, seed, names, device="cuda"):
    """X ~ N(0,1) [B,N,C]; every weight [C,C] ~ N(0, 1/C) so that the projections are ~ N(0,1); all bf16."""
    return wl.make_producer_inputs(B, H, N, 64, seed=seed, names=names, device=device)


def _state_oracle(x, w_k, w_v, H, t_k=None):
    k = oracle.linear_map(to_f64(x), to_f64(w_k))
    if t_k is not None:
        k = k + to_f64(t_k)
    v = oracle.linear_map(to_f64(x), to_f64(w_v))
    return oracle.state(oracle.split_heads(k, H), oracle.split_heads(v, H))


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_state_from_x_matches_the_oracle(shape):
    B, H, N = shape
    x, w = _x_and_weights(B, H, N, seed=91, names=("k", "v", "tk"))
    op = attn.LinFusionAttention(B, H, N, 64, eps=EPS, variant="stream", layout="token_major")
    for t_k in (None, w["tk"]):
        S_ref, z_ref = _state_oracle(x, w["k"], w["v"], H, t_k)
        op.state_x(x, w["k"], w["v"], t_k)
        torch.cuda.synchronize()
        assert op.status() == attn.OK
        S, z = op.read_state()
        # 16-bit operands phi(K), V (unit roundoff 2^-8 each) bound the error for any N; the tight
        # gates hold once many tokens average the roundings out
        z_tol, s_tol = (2e-3, 5e-3) if N >= 256 else (2.0 ** -8, 2.0 ** -7)
        assert np.abs(z - z_ref).max() <= z_tol * np.abs(z_ref).max(), (shape, t_k is not None)
        assert np.linalg.norm(S - S_ref) <= s_tol * np.linalg.norm(S_ref), (shape, t_k is not None)
        S2, z2 = (a.copy() for a in (S, z))
        op.state_x(x, w["k"], w["v"], t_k)
        S, z = op.read_state()
        assert np.array_equal(S, S2) and np.array_equal(z, z2), "not bit-reproducible"
    op.close()


def _module_oracle(x, w, H, t_q=None, t_k=None):
    """Q = X W_q (+ T_q), K = X W_k (+ T_k), V = X W_v, heads split, attention, heads merged: [B, N, C]."""
    xf = to_f64(x)
    q = oracle.linear_map(xf, to_f64(w["q"])) + (to_f64(t_q) if t_q is not None else 0.0)
    k = oracle.linear_map(xf, to_f64(w["k"])) + (to_f64(t_k) if t_k is not None else 0.0)
    v = oracle.linear_map(xf, to_f64(w["v"]))
    y = oracle.linear(oracle.split_heads(q, H), oracle.split_heads(k, H), oracle.split_heads(v, H), EPS)
    return y  # [B, H, N, d]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
def test_state_then_apply_from_x_matches_the_oracle(shape):
    B, H, N = shape
    for x_mean in (0.0, 0.5):
        x, w = wl.make_producer_inputs(B, H, N, 64, seed=93, names=("q", "k", "v", "tq", "tk"), device="cuda",
                                       x_mean=x_mean)
        op = attn.LinFusionAttention(B, H, N, 64, eps=EPS, variant="stream", layout="token_major")
        for t_q, t_k in ((None, None), (w["tq"], w["tk"])):
            ref = _module_oracle(x, w, H, t_q, t_k)
            op.state_x(x, w["k"], w["v"], t_k)
            y = op.apply_x(x, w["q"], t_q)
            torch.cuda.synchronize()
            assert op.status() == attn.OK
            y_bhnd = y.view(B, N, H, 64).permute(0, 2, 1, 3)
            assert_parity(y_bhnd, ref, f"{shape} x_mean={x_mean} branches={t_q is not None}")
            y2 = op.apply_x(x, w["q"], t_q)
            torch.cuda.synchronize()
            assert torch.equal(y, y2), "not bit-reproducible"
        op.close()
