"""Pins for the oracle routines added for Prop. 3 (feature width d' != value width d) and for the
producers of Q, K, V (Sec. 3.1, implementation details; Eq. 2): hand-worked values, library
cross-checks with independently written formulas, and invariants the definitions fix."""
import json
import math
import os

import numpy as np
import pytest

import oracle

EPS = 1e-6


def _ev(expr):
    return eval(expr, {"__builtins__": {}}, {"e": math.e, "sqrt": math.sqrt})


def _arr(exprs):
    return np.array([[_ev(x) for x in row] for row in exprs], dtype=np.float64)


@pytest.fixture(scope="module")
def cases(golden_dir):
    with open(os.path.join(golden_dir, "rectangular_and_producer_cases.json")) as f:
        return json.load(f)


# ---------------------------------------------------------------- Prop. 3: d' != d
def test_rectangular_state_hand_worked(cases):
    c = cases["rect_state"]
    S, z = oracle.state(np.array(c["k"], float), np.array(c["v"], float))
    assert S.shape == (3, 2) and z.shape == (3,)
    np.testing.assert_allclose(S, _arr(c["S_expr"]), rtol=1e-14)
    np.testing.assert_allclose(z, [_ev(x) for x in c["z_expr"]], rtol=1e-14)


def test_rectangular_apply_hand_worked(cases):
    c, a = cases["rect_state"], cases["rect_apply"]
    k, v, q = (np.array(t, float) for t in (c["k"], c["v"], a["q"]))
    want = _arr(a["y_expr"])
    np.testing.assert_allclose(oracle.linear(q, k, v, 0.0), want, rtol=1e-14)
    np.testing.assert_allclose(oracle.quadratic(q, k, v, 0.0), want, rtol=1e-14)
    S, z = oracle.state(k, v)
    np.testing.assert_allclose(oracle.apply(q, S, z, 0.0), want, rtol=1e-14)
    den = oracle.phi(q) @ z
    np.testing.assert_allclose(oracle.apply_unnormalized(q, S), want * den[:, None], rtol=1e-14)


@pytest.mark.parametrize("dk,dv", [(3, 2), (128, 64), (80, 40), (32, 64), (8, 24)])
@pytest.mark.parametrize("n", [1, 7, 130])
def test_rectangular_linear_equals_attention_matrix_form(dk, dv, n):
    rng = np.random.default_rng(dk * 1000 + dv + n)
    q, k = rng.standard_normal((2, 2, n, dk))
    v = rng.standard_normal((2, n, dv))
    y_lin = oracle.linear(q, k, v, EPS)
    y_quad, m = oracle.quadratic(q, k, v, EPS, return_weights=True)
    assert y_lin.shape == (2, n, dv)
    np.testing.assert_allclose(y_lin, y_quad, rtol=1e-11, atol=1e-13)
    assert (m >= 0).all()
    np.testing.assert_allclose(m.sum(-1), 1.0, atol=1e-6)            # rows normalized (Sec. 2.2)
    # an independent numpy statement of S and z
    S, z = oracle.state(k, v)
    pk = np.where(k > 0, k + 1, np.exp(k))
    np.testing.assert_allclose(S, np.einsum("snc,sne->sce", pk, v), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(z, pk.sum(1), rtol=1e-12)


def test_zero_features_add_nothing_under_the_identity_activation():
    """With non-negative features taken as they are, padding Q and K with zero features (a wider
    d') leaves Y unchanged: the added products are zero."""
    rng = np.random.default_rng(5)
    q, k = np.abs(rng.standard_normal((2, 50, 8)))
    v = rng.standard_normal((50, 5))
    y = oracle.linear(q, k, v, EPS, oracle.PHI_IDENTITY)
    pad = np.zeros((50, 4))
    y_wide = oracle.linear(np.hstack([q, pad]), np.hstack([k, pad]), v, EPS, oracle.PHI_IDENTITY)
    np.testing.assert_allclose(y_wide, y, rtol=1e-13)


def test_value_channels_are_independent_and_square_case_is_unchanged():
    rng = np.random.default_rng(6)
    q, k = rng.standard_normal((2, 40, 16))
    v = rng.standard_normal((40, 12))
    y = oracle.linear(q, k, v, EPS)
    np.testing.assert_allclose(oracle.linear(q, k, v[:, 3:7], EPS), y[:, 3:7], rtol=1e-13)
    v16 = rng.standard_normal((40, 16))                                # dk == dv: the released model's case
    S, z = oracle.state(k, v16)
    assert S.shape == (16, 16)
    np.testing.assert_allclose(oracle.linear(q, k, v16, EPS), oracle.apply(q, S, z, EPS), rtol=1e-14)


# ---------------------------------------------------------------- producers
def test_linear_map_hand_worked_and_against_matmul(cases):
    c = cases["linear_map"]
    x, w = np.array(c["x"], float), np.array(c["w"], float)
    np.testing.assert_array_equal(oracle.linear_map(x, w), np.array(c["out"], float))
    np.testing.assert_array_equal(oracle.linear_map(x, w, c["bias"]), np.array(c["out_with_bias"], float))
    rng = np.random.default_rng(1)
    x, w, b = rng.standard_normal((3, 17, 24)), rng.standard_normal((24, 40)), rng.standard_normal(40)
    np.testing.assert_allclose(oracle.linear_map(x, w, b), x @ w + b, rtol=1e-12, atol=1e-12)


def test_layernorm_hand_worked_and_invariants(cases):
    c = cases["layernorm"]
    ones2, zeros2 = np.ones(2), np.zeros(2)
    np.testing.assert_allclose(oracle.layernorm(c["rows2"], ones2, zeros2, 0.0), _arr(c["plain2_expr"]), rtol=1e-15)
    np.testing.assert_allclose(oracle.layernorm(c["rows2"], c["gamma2"], c["beta2"], 0.0), _arr(c["affine2_expr"]), rtol=1e-15)
    np.testing.assert_allclose(oracle.layernorm(c["rows4"], np.ones(4), np.zeros(4), 0.0), _arr(c["plain4_expr"]), rtol=1e-15)
    rng = np.random.default_rng(2)
    p = rng.standard_normal((5, 9, 64)) * 3 + 1.5
    out = oracle.layernorm(p, np.ones(64), np.zeros(64), 0.0)
    np.testing.assert_allclose(out.mean(-1), 0.0, atol=1e-13)          # rows have mean 0 ...
    np.testing.assert_allclose(out.var(-1), 1.0, rtol=1e-12)           # ... and variance 1
    np.testing.assert_allclose(oracle.layernorm(4.0 * p - 7.0, np.ones(64), np.zeros(64), 0.0), out, rtol=1e-10, atol=1e-12)
    g, b = rng.standard_normal(64), rng.standard_normal(64)
    want = (p - p.mean(-1, keepdims=True)) / np.sqrt(p.var(-1, keepdims=True) + 1e-5) * g + b
    np.testing.assert_allclose(oracle.layernorm(p, g, b, 1e-5), want, rtol=1e-12, atol=1e-13)
    # the epsilon sits inside the root: a constant row maps to beta exactly, not to NaN
    np.testing.assert_allclose(oracle.layernorm(np.full((1, 64), 3.0), g, b, 1e-5), b[None], atol=1e-15)


def test_leaky_relu_spot_values():
    assert oracle.leaky_relu(2.0) == 2.0 and oracle.leaky_relu(0.0) == 0.0
    assert oracle.leaky_relu(-2.0) == -0.02 and oracle.leaky_relu(-2.0, 0.5) == -1.0
    assert oracle.LEAKY_SLOPE == 0.01 and oracle.LN_EPS == 1e-5


def test_mlp_producer_hand_worked(cases):
    c = cases["mlp_producer"]
    eye, x = np.eye(2), np.array(c["x"], float)
    out = oracle.mlp_producer(x, eye, eye, np.zeros(2), np.ones(2), np.zeros(2), 0.0, c["slope"])
    np.testing.assert_allclose(out, np.array(c["out"]), rtol=1e-15)
    out = oracle.mlp_producer(x, eye, eye, np.array([0.0, 2.0]), np.ones(2), np.zeros(2), 0.0, c["slope"])
    np.testing.assert_allclose(out, np.array(c["out"]), rtol=1e-15)


def _random_weights(rng, c, c_qk):
    w = {}
    for name in ("q", "k"):
        w[f"{name}_lin"] = rng.standard_normal((c, c_qk)) / np.sqrt(c)
        w[f"{name}_w1"] = rng.standard_normal((c, c_qk)) / np.sqrt(c)
        w[f"{name}_b1"] = rng.standard_normal(c_qk) * 0.1
        w[f"{name}_gamma"] = 1.0 + 0.1 * rng.standard_normal(c_qk)
        w[f"{name}_beta"] = 0.1 * rng.standard_normal(c_qk)
    w["v"] = rng.standard_normal((c, c)) / np.sqrt(c)
    return w


def test_mlp_producer_at_the_papers_initialization_is_the_plain_projection():
    """Non-linear branch's output initialized to zero (Sec. 3.1): LayerNorm's scale and shift are
    zero, LeakyReLU(0) = 0, and f'(X) = X W_Q exactly."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((2, 33, 24))
    w = _random_weights(rng, 24, 24)
    out = oracle.mlp_producer(x, w["q_lin"], w["q_w1"], w["q_b1"], np.zeros(24), np.zeros(24))
    np.testing.assert_allclose(out, x @ w["q_lin"], rtol=1e-12, atol=1e-13)


def test_mlp_producer_against_an_independent_numpy_statement():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((3, 20, 16))
    w = _random_weights(rng, 16, 32)                                   # widened features (Prop. 3)
    out = oracle.mlp_producer(x, w["k_lin"], w["k_w1"], w["k_b1"], w["k_gamma"], w["k_beta"])
    pre = np.einsum("bnc,co->bno", x, w["k_w1"]) + w["k_b1"]
    mu = pre.mean(-1, keepdims=True)
    nrm = (pre - mu) / np.sqrt(((pre - mu) ** 2).mean(-1, keepdims=True) + oracle.LN_EPS) * w["k_gamma"] + w["k_beta"]
    want = np.einsum("bnc,co->bno", x, w["k_lin"]) + np.where(nrm >= 0, nrm, oracle.LEAKY_SLOPE * nrm)
    assert out.shape == (3, 20, 32)
    np.testing.assert_allclose(out, want, rtol=1e-12, atol=1e-13)
    # the non-linear branch matters: it is not the plain projection
    assert np.abs(out - x @ w["k_lin"]).max() > 0.1


def test_split_heads_is_a_pure_reindexing():
    B, N, H, d = 2, 3, 4, 5
    t = np.arange(B * N * H * d, dtype=float).reshape(B, N, H * d)
    s = oracle.split_heads(t, H)
    assert s.shape == (B, H, N, d)
    for b in range(B):
        for h in range(H):
            for n in range(N):
                np.testing.assert_array_equal(s[b, h, n], t[b, n, h * d:(h + 1) * d])


def test_whole_module_from_x_is_the_composition_of_its_parts():
    rng = np.random.default_rng(7)
    B, N, C, H = 2, 37, 24, 3
    x = rng.standard_normal((B, N, C))
    w = _random_weights(rng, C, C)
    y = oracle.linfusion_from_x(x, w, H, EPS)
    q = oracle.mlp_producer(x, w["q_lin"], w["q_w1"], w["q_b1"], w["q_gamma"], w["q_beta"])
    k = oracle.mlp_producer(x, w["k_lin"], w["k_w1"], w["k_b1"], w["k_gamma"], w["k_beta"])
    v = x @ w["v"]
    sh = lambda t: oracle.split_heads(t, H)
    want = oracle.quadratic(sh(q), sh(k), sh(v), EPS)                  # the attention-matrix form, per head
    want = want.transpose(0, 2, 1, 3).reshape(B, N, C)
    np.testing.assert_allclose(y, want, rtol=1e-10, atol=1e-12)
    # at the paper's initialization the module is the linear attention of the plain projections
    w0 = dict(w, q_gamma=np.zeros(C), q_beta=np.zeros(C), k_gamma=np.zeros(C), k_beta=np.zeros(C))
    y0 = oracle.linfusion_from_x(x, w0, H, EPS)
    want0 = oracle.linear(sh(x @ w["q_lin"]), sh(x @ w["k_lin"]), sh(v), EPS).transpose(0, 2, 1, 3).reshape(B, N, C)
    np.testing.assert_allclose(y0, want0, rtol=1e-11, atol=1e-13)
    # widened features: H * d' != C for Q and K, V keeps C
    w2 = _random_weights(rng, C, 2 * C)
    y2 = oracle.linfusion_from_x(x, w2, H, EPS)
    assert y2.shape == (B, N, C)
