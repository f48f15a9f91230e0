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


MODULE_NAMES = ("q_lin", "q_w1", "b_q", "g_q", "e_q", "k_lin", "k_w1", "b_k", "g_k", "e_k", "v")


def _module_weights(B, H, N, seed, x_mean=0.0):
    x, w = wl.make_producer_inputs(B, H, N, 64, seed=seed, names=MODULE_NAMES, device="cuda", x_mean=x_mean)
    w = dict(w)
    for side in ("q", "k"):
        w[f"{side}_b1"], w[f"{side}_gamma"], w[f"{side}_beta"] = w.pop(f"b_{side}"), w.pop(f"g_{side}"), w.pop(f"e_{side}")
    return x, w


@pytest.mark.parametrize("shape", [(1, 2, 1), (2, 3, 129), (1, 5, 300), (2, 10, 520)], ids=lambda s: "x".join(map(str, s)))
def test_non_linear_branch_matches_the_oracle(shape):
    """T = LeakyReLU(LayerNorm(X W_1 + b_1)): C = 128 (one column block), 192 (an odd half block), 320, 640."""
    B, H, N = shape
    x, w = _module_weights(B, H, N, seed=95, x_mean=0.25)
    op = attn.LinFusionAttention(B, H, N, 64, eps=EPS, variant="stream", layout="token_major")
    f = to_f64
    for slope in (0.01, 0.5):
        pre = oracle.linear_map(f(x), f(w["k_w1"]), f(w["k_b1"]))
        nrm = oracle.layernorm(pre, f(w["k_gamma"]), f(w["k_beta"]), oracle.LN_EPS)
        ref = np.where(nrm >= 0.0, nrm, slope * nrm)
        t = op.branch_x(x, w["k_w1"], w["k_b1"], w["k_gamma"], w["k_beta"], oracle.LN_EPS, slope)
        torch.cuda.synchronize()
        assert op.status() == attn.OK
        diff = np.abs(f(t) - ref)
        # U is rounded to 16 bits before it is normalized and T after: two unit roundoffs of 2^-8 on values of
        # order 1 (|T| <= ~4), plus the fp32 statistics
        assert diff.max() <= 3e-2 and diff.mean() <= 3e-3, (shape, slope, diff.max(), diff.mean())
        assert np.linalg.norm(diff) <= 6e-3 * np.linalg.norm(ref), (shape, slope)
    # no bias
    ref0 = oracle.layernorm(oracle.linear_map(f(x), f(w["k_w1"])), f(w["k_gamma"]), f(w["k_beta"]), oracle.LN_EPS)
    ref0 = np.where(ref0 >= 0.0, ref0, 0.01 * ref0)
    t0 = op.branch_x(x, w["k_w1"], None, w["k_gamma"], w["k_beta"], oracle.LN_EPS, 0.01)
    torch.cuda.synchronize()
    assert np.linalg.norm(f(t0) - ref0) <= 6e-3 * np.linalg.norm(ref0)
    op.close()


@pytest.mark.parametrize("shape", [(2, 2, 129), (1, 5, 300), (2, 10, 1000)], ids=lambda s: "x".join(map(str, s)))
def test_whole_module_from_x_matches_the_oracle(shape):
    B, H, N = shape
    x, w = _module_weights(B, H, N, seed=97, x_mean=0.25)
    ref = oracle.linfusion_from_x(to_f64(x), {k: to_f64(v) for k, v in w.items()}, H, EPS)   # [B, N, C]
    ref = oracle.split_heads(ref, H)
    op = attn.LinFusionAttention(B, H, N, 64, eps=EPS, variant="stream", layout="token_major")
    y = op.forward_x(x, w, oracle.LN_EPS, oracle.LEAKY_SLOPE)
    torch.cuda.synchronize()
    assert op.status() == attn.OK
    assert_parity(y.view(B, N, H, 64).permute(0, 2, 1, 3), ref, f"module {shape}")
    y2 = op.forward_x(x, w, oracle.LN_EPS, oracle.LEAKY_SLOPE)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)
    # the paper's initialization: zero scale and shift => the module is the plain projections
    w0 = dict(w)
    for side in ("q", "k"):
        w0[f"{side}_gamma"] = torch.zeros_like(w[f"{side}_gamma"])
        w0[f"{side}_beta"] = torch.zeros_like(w[f"{side}_beta"])
    y0 = op.forward_x(x, w0, oracle.LN_EPS, oracle.LEAKY_SLOPE)
    w_lin_only = {"q_lin": w["q_lin"], "k_lin": w["k_lin"], "v": w["v"]}
    y_lin = op.forward_x(x, w_lin_only)
    torch.cuda.synchronize()
    assert torch.equal(y0, y_lin)
    op.close()
