"""Pins for the fp64 CPU oracle: closed forms, hand-worked values, a library mean, brute force
and the invariants the paper fixes.  None of these re-type the oracle's own formula."""
import json
import math
import os

import numpy as np
import pytest

import oracle

EPS = 1e-6


def _rand(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


# ---- phi: spot values and shape (Sec. 2.2: a non-negative activation; reading elu + 1) -------

def test_phi_spot_values():
    assert oracle.phi([0.0])[0] == 1.0
    assert oracle.phi([1.0])[0] == 2.0
    assert oracle.phi([2.5])[0] == 3.5
    assert oracle.phi([-1.0])[0] == pytest.approx(1.0 / math.e, rel=1e-15)
    assert oracle.phi([-3.0])[0] == pytest.approx(math.e ** -3, rel=1e-15)
    assert oracle.phi([-800.0])[0] == 0.0
    assert oracle.phi([1e30])[0] == 1e30


def test_phi_positive_monotone_c1():
    x = np.linspace(-20, 20, 4001)
    p = oracle.phi(x)
    assert np.all(p > 0)
    assert np.all(np.diff(p) > 0)
    h = 1e-7
    left = (oracle.phi([0.0])[0] - oracle.phi([-h])[0]) / h
    right = (oracle.phi([h])[0] - oracle.phi([0.0])[0]) / h
    assert left == pytest.approx(1.0, abs=1e-6) and right == pytest.approx(1.0, abs=1e-6)


def test_phi_identity_kind():
    x = np.array([-2.0, 0.0, 3.0])
    assert np.array_equal(oracle.phi(x, oracle.PHI_IDENTITY), x)


# ---- hand-worked values (tests/golden) ----------------------------------------------------------

def _golden_cases(golden_dir):
    with open(os.path.join(golden_dir, "hand_worked_cases.json")) as f:
        return json.load(f)["cases"]


def test_hand_worked_cases(golden_dir):
    env = {"e": math.e, "__builtins__": {}}
    cases = _golden_cases(golden_dir)
    assert len(cases) >= 4
    for case in cases:
        q, k, v = (np.array(case[n], dtype=np.float64) for n in ("q", "k", "v"))
        want = np.array([[eval(x, env) for x in row] for row in case["y_expr"]])
        for fn in (oracle.linear, oracle.quadratic):
            got = fn(q, k, v, 0.0)
            np.testing.assert_allclose(got, want, rtol=1e-14, atol=0, err_msg=case["name"])


def test_hand_worked_state(golden_dir):
    case = [c for c in _golden_cases(golden_dir) if c["name"] == "asymmetric_state_d2_n3"][0]
    S, z = oracle.state(np.array(case["k"], float), np.array(case["v"], float))
    assert np.array_equal(S, np.array([[5.0, 5.0], [6.0, 0.0]]))
    assert np.array_equal(z, np.array([5.0, 4.0]))


# ---- brute force: linear form == attention-matrix form (Prop. 2, associativity) -----------------

@pytest.mark.parametrize("n", [1, 2, 7, 64, 256])
@pytest.mark.parametrize("d", [8, 40, 64, 160])
def test_linear_equals_quadratic(n, d):
    q, k, v = _rand((2, n, d), 1), _rand((2, n, d), 2), _rand((2, n, d), 3)
    yl = oracle.linear(q, k, v, EPS)
    yq = oracle.quadratic(q, k, v, EPS)
    scale = np.abs(yq).max()
    assert np.abs(yl - yq).max() <= 1e-12 * max(scale, 1.0)


def test_quadratic_weights_nonnegative_rowsum_one():
    n, d = 33, 16
    q, k, v = _rand((n, d), 4), _rand((n, d), 5), _rand((n, d), 6)
    y, m = oracle.quadratic(q, k, v, EPS, return_weights=True)
    assert np.all(m >= 0)
    # row sums are 1 - eps/(den + eps): strictly below one, by less than eps / min(den)
    rs = m.sum(axis=-1)
    assert np.all(rs < 1.0) and np.all(rs > 1.0 - 1e-6)
    np.testing.assert_allclose(m @ v, y, rtol=1e-13, atol=1e-15)
    y0, m0 = oracle.quadratic(q, k, v, 0.0, return_weights=True)
    np.testing.assert_allclose(m0.sum(axis=-1), 1.0, rtol=1e-14)


# ---- normalization (Sec. 2.2, Prop. 1): sum_k M_ik = 1 ------------------------------------------

def test_constant_v_gives_constant_y():
    n, d = 300, 40
    q, k = _rand((3, n, d), 7), _rand((3, n, d), 8)
    row = _rand((d,), 9)
    v = np.broadcast_to(row, (3, n, d)).copy()
    y = oracle.linear(q, k, v, 0.0)
    np.testing.assert_allclose(y, np.broadcast_to(row, y.shape), rtol=1e-12, atol=1e-13)
    ones = oracle.linear(q, k, np.ones((3, n, d)), 0.0)
    np.testing.assert_allclose(ones, 1.0, rtol=1e-13)


def test_eps_shrinks_rows_by_den_over_den_plus_eps():
    n, d = 5, 8
    q, k = _rand((n, d), 10, 3.0) - 4.0, _rand((n, d), 11, 3.0) - 4.0   # small phi: eps matters
    eps = 0.25
    y1 = oracle.linear(q, k, np.ones((n, d)), eps)
    _, m0 = oracle.quadratic(q, k, np.ones((n, d)), 0.0, return_weights=True)
    # den_i from an independent route: K-side column sums times phi(Q_i), via numpy
    pk = np.where(k > 0, k + 1, np.exp(k)).sum(axis=0)
    pq = np.where(q > 0, q + 1, np.exp(q))
    den = pq @ pk
    np.testing.assert_allclose(y1, np.repeat((den / (den + eps))[:, None], d, 1), rtol=1e-13)
    assert np.all(y1 < 1.0) and np.all(y1 > 0.0)


# ---- textbook special case: uniform weights -> column mean (library mean) -----------------------

def test_zero_qk_gives_column_mean():
    n, d = 257, 24
    v = _rand((2, n, d), 12)
    zeros = np.zeros((2, n, d))
    y = oracle.linear(zeros, zeros, v, 0.0)
    want = np.broadcast_to(v.mean(axis=1, keepdims=True), v.shape)
    np.testing.assert_allclose(y, want, rtol=1e-12, atol=1e-14)


def test_equal_k_rows_give_column_mean():
    n, d = 100, 16
    q, v = _rand((n, d), 13), _rand((n, d), 14)
    k = np.broadcast_to(_rand((d,), 15), (n, d)).copy()
    y = oracle.linear(q, k, v, 0.0)
    np.testing.assert_allclose(y, np.broadcast_to(v.mean(axis=0), v.shape), rtol=1e-12, atol=1e-14)


def test_single_token():
    d = 40
    q, k, v = _rand((1, d), 16), _rand((1, d), 17), _rand((1, d), 18)
    np.testing.assert_allclose(oracle.linear(q, k, v, 0.0), v, rtol=1e-14)


# ---- non-causality (Sec. 2.3): every token sees every token -------------------------------------

def test_kv_permutation_invariance_and_q_equivariance():
    n, d = 129, 40
    q, k, v = _rand((n, d), 19), _rand((n, d), 20), _rand((n, d), 21)
    y = oracle.linear(q, k, v, EPS)
    perm = np.random.default_rng(22).permutation(n)
    y_kv = oracle.linear(q, k[perm], v[perm], EPS)
    assert np.abs(y_kv - y).max() <= 1e-12
    y_q = oracle.linear(q[perm], k, v, EPS)
    assert np.array_equal(y_q, y[perm])


def test_not_causal_last_token_influences_first():
    n, d = 16, 8
    q, k, v = _rand((n, d), 23), _rand((n, d), 24), _rand((n, d), 25)
    y = oracle.linear(q, k, v, EPS)
    v2 = v.copy()
    v2[-1] += 10.0
    assert np.abs(oracle.linear(q, k, v2, EPS)[0] - y[0]).max() > 1e-3


# ---- resolution invariance (Sec. 2.2): duplicating the K/V tokens leaves Y unchanged ------------

def test_token_duplication_invariance():
    n, d = 64, 16
    q, k, v = _rand((n, d), 26), _rand((n, d), 27), _rand((n, d), 28)
    y = oracle.linear(q, k, v, 0.0)
    q2 = np.concatenate([q, q]); k2 = np.concatenate([k, k]); v2 = np.concatenate([v, v])
    y2 = oracle.linear(q2, k2, v2, 0.0)
    np.testing.assert_allclose(y2[:n], y, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(y2[n:], y, rtol=1e-12, atol=1e-14)


# ---- convex hull (non-negative weights) ---------------------------------------------------------

def test_rows_in_convex_hull_bounds():
    n, d = 500, 64
    q, k, v = _rand((2, n, d), 29), _rand((2, n, d), 30), _rand((2, n, d), 31)
    y = oracle.linear(q, k, v, EPS)
    lo = np.minimum(v.min(axis=1, keepdims=True), 0.0)   # hull of {V_j} and 0 (the eps shrink)
    hi = np.maximum(v.max(axis=1, keepdims=True), 0.0)
    assert np.all(y >= lo - 1e-12) and np.all(y <= hi + 1e-12)


# ---- linearity in V, shard additivity of the state ----------------------------------------------

def test_linear_in_v():
    n, d = 77, 40
    q, k = _rand((n, d), 32), _rand((n, d), 33)
    v1, v2 = _rand((n, d), 34), _rand((n, d), 35)
    lhs = oracle.linear(q, k, 2.0 * v1 - 3.0 * v2, EPS)
    rhs = 2.0 * oracle.linear(q, k, v1, EPS) - 3.0 * oracle.linear(q, k, v2, EPS)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-11, atol=1e-13)


def test_state_is_additive_over_token_shards():
    n, d = 200, 64
    q, k, v = _rand((n, d), 36), _rand((n, d), 37), _rand((n, d), 38)
    cuts = [0, 13, 64, 150, n]
    S = np.zeros((d, d)); z = np.zeros(d)
    for a, b in zip(cuts[:-1], cuts[1:]):
        Sp, zp = oracle.state(k[a:b], v[a:b])
        S += Sp; z += zp
    y_shard = oracle.apply(q, S, z, EPS)
    np.testing.assert_allclose(y_shard, oracle.linear(q, k, v, EPS), rtol=1e-12, atol=1e-14)


def test_state_against_numpy_matmul():
    n, d = 300, 40
    k, v = _rand((2, n, d), 39), _rand((2, n, d), 40)
    S, z = oracle.state(k, v, oracle.PHI_IDENTITY)        # phi = id: plain K^T V, library matmul
    np.testing.assert_allclose(S, np.swapaxes(k, -1, -2) @ v, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(z, k.sum(axis=1), rtol=1e-12, atol=1e-12)


def test_identity_phi_row_scale_invariance():
    n, d = 50, 16
    q, k, v = np.abs(_rand((n, d), 41)), np.abs(_rand((n, d), 42)), _rand((n, d), 43)
    y = oracle.linear(q, k, v, 0.0, oracle.PHI_IDENTITY)
    q2 = q.copy(); q2[3] *= 7.5
    np.testing.assert_allclose(oracle.linear(q2, k, v, 0.0, oracle.PHI_IDENTITY), y, rtol=1e-12)


def test_slabs_are_independent():
    n, d = 40, 8
    q, k, v = _rand((2, 3, n, d), 44), _rand((2, 3, n, d), 45), _rand((2, 3, n, d), 46)
    y = oracle.linear(q, k, v, EPS)
    assert y.shape == (2, 3, n, d)
    for b in range(2):
        for h in range(3):
            assert np.array_equal(y[b, h], oracle.linear(q[b, h], k[b, h], v[b, h], EPS))


def test_threads_reported():
    assert oracle.num_threads() >= 1


# ---- the un-normalized operator (Prop. 2 without Eq. 5's division; Tab. 2 ablation) -------------

def _phi_closed_form(x):
    return np.where(x > 0, x + 1.0, np.exp(np.minimum(x, 0.0)))


def test_unnormalized_hand_worked_case(golden_dir):
    env = {"e": math.e, "__builtins__": {}}
    with open(os.path.join(golden_dir, "hand_worked_cases.json")) as f:
        cases = json.load(f)["unnormalized_cases"]
    assert cases
    for case in cases:
        q, k, v = (np.array(case[n], dtype=np.float64) for n in ("q", "k", "v"))
        want = np.array([[eval(x, env) for x in row] for row in case["y_expr"]])
        np.testing.assert_allclose(oracle.linear_unnormalized(q, k, v), want, rtol=1e-14, atol=0)


def test_unnormalized_equals_attention_matrix_form():
    """Y = (phi(Q) phi(K)^T) V with the n x n weights written out (Eq. 4 with the mask dropped)."""
    rng = np.random.default_rng(77)
    q, k, v = (rng.standard_normal((3, 37, 5)) for _ in range(3))
    w = _phi_closed_form(q) @ np.swapaxes(_phi_closed_form(k), -1, -2)   # [3, 37, 37]
    np.testing.assert_allclose(oracle.linear_unnormalized(q, k, v), w @ v, rtol=1e-12, atol=1e-12)


def test_unnormalized_times_reciprocal_denominator_is_the_normalized_output():
    rng = np.random.default_rng(78)
    q, k, v = (rng.standard_normal((2, 50, 8)) for _ in range(3))
    eps = 1e-3
    S, z = oracle.state(k, v)
    den = _phi_closed_form(q) @ z[..., None] + eps                          # [2, 50, 1]
    np.testing.assert_allclose(oracle.apply_unnormalized(q, S) / den, oracle.apply(q, S, z, eps),
                               rtol=1e-12, atol=1e-14)


def test_unnormalized_is_not_the_normalized_operator():
    """A plausible mistake (dividing anyway) must fail: with V = const the rows are not V."""
    rng = np.random.default_rng(79)
    q, k = (rng.standard_normal((1, 20, 4)) for _ in range(2))
    v = np.ones((1, 20, 4))
    y = oracle.linear_unnormalized(q, k, v)
    w = _phi_closed_form(q) @ np.swapaxes(_phi_closed_form(k), -1, -2)
    np.testing.assert_allclose(y[..., 0], w.sum(-1), rtol=1e-12)            # row sums of the weights
    assert np.abs(y - 1.0).min() > 1.0
