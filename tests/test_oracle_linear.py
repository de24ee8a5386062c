"""Pins for the Linear + bias + tanh-GELU oracle (CPU only)."""
import math

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(7)


def test_gelu_closed_forms_and_invariants():
    assert oracle.gelu_tanh(0.0) == 0.0
    for z in [0.1, 0.5, 1.0, 2.0, 3.3, 7.0]:
        # odd tanh => gelu(z) - gelu(-z) = z
        assert abs(oracle.gelu_tanh(z) - oracle.gelu_tanh(-z) - z) < 1e-15 * max(1.0, z)
    assert abs(oracle.gelu_tanh(30.0) - 30.0) < 1e-12       # saturates to identity
    assert abs(oracle.gelu_tanh(-30.0)) < 1e-12             # and to zero
    # the minimum of tanh-GELU is about -0.17 near z = -0.75; it is negative only for z < 0
    assert -0.171 < oracle.gelu_tanh(-0.75) < -0.169


def test_gelu_is_the_tanh_form_not_erf():
    """tanh-GELU(1) = 0.841192; the erf form gives 0.841345, 1.5e-4 away."""
    erf_form = 0.5 * (1.0 + math.erf(1.0 / math.sqrt(2.0)))
    assert abs(oracle.gelu_tanh(1.0) - 0.841192) < 5e-7
    assert abs(oracle.gelu_tanh(1.0) - erf_form) > 1e-4


def test_gelu_against_torch_library():
    z = np.concatenate([np.linspace(-8, 8, 2001), RNG.standard_normal(1000) * 3])
    ref = torch.nn.functional.gelu(torch.from_numpy(z), approximate="tanh").numpy()
    got = np.array([oracle.gelu_tanh(t) for t in z])
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-15)


def _gelu_np(z):
    return torch.nn.functional.gelu(torch.from_numpy(np.asarray(z, dtype=np.float64)), approximate="tanh").numpy()


def test_linear_k1_outer_product():
    x = RNG.standard_normal((5, 1)); w = RNG.standard_normal((1, 7)); b = RNG.standard_normal(7)
    np.testing.assert_allclose(oracle.linear_bias_gelu(x, w, b), _gelu_np(x * w + b), rtol=0, atol=1e-15)


def test_linear_identity_weight():
    n = 6
    x = RNG.standard_normal((n, n)); b = RNG.standard_normal(n)
    np.testing.assert_allclose(oracle.linear_bias_gelu(x, np.eye(n), b), _gelu_np(x + b), rtol=0, atol=1e-15)


def test_linear_all_ones():
    M, N, K = 3, 4, 9
    b = np.array([0.0, -9.0, 0.5, -8.0])
    y = oracle.linear_bias_gelu(np.ones((M, K)), np.ones((K, N)), b)
    np.testing.assert_allclose(y, np.broadcast_to(_gelu_np(K + b), (M, N)), rtol=0, atol=1e-14)
    assert (y[:, 1] == 0.0).all()  # K + b = 0 exactly


def test_linear_layout_is_x_times_w_kn():
    """Non-square, asymmetric operands: a transposed or [N,K]-indexed W would fail."""
    M, N, K = 4, 3, 5
    x = RNG.standard_normal((M, K)); w = RNG.standard_normal((K, N)); b = RNG.standard_normal(N)
    y = oracle.linear_bias_gelu(x, w, b)
    np.testing.assert_allclose(y, _gelu_np(x @ w + b), rtol=0, atol=1e-14)
    # other loop order, accumulated column by column
    z = np.zeros((M, N))
    for n in range(N):
        for k in range(K):
            for m in range(M):
                z[m, n] += x[m, k] * w[k, n]
    np.testing.assert_allclose(y, _gelu_np(z + b[None, :]), rtol=0, atol=1e-14)


def test_linear_against_torch_library():
    M, N, K = 33, 17, 29
    x = RNG.standard_normal((M, K)); w = RNG.standard_normal((K, N)) * 0.2; b = RNG.standard_normal(N)
    ref = torch.nn.functional.gelu(
        torch.nn.functional.linear(torch.from_numpy(x), torch.from_numpy(w).t(), torch.from_numpy(b)),
        approximate="tanh").numpy()
    np.testing.assert_allclose(oracle.linear_bias_gelu(x, w, b), ref, rtol=0, atol=1e-13)


def test_linear_invalid_arguments():
    with pytest.raises((ValueError, AssertionError)):
        oracle.linear_bias_gelu(np.zeros((2, 3)), np.zeros((4, 2)), np.zeros(2))


# ---- the other operator-fusion patterns: linear+relu, linear+silu, erf-GELU, mm+add, [N,K] weights
ACTS = {
    oracle.ACT_GELU_TANH: lambda t: torch.nn.functional.gelu(t, approximate="tanh"),
    oracle.ACT_GELU_ERF: lambda t: torch.nn.functional.gelu(t),
    oracle.ACT_RELU: torch.relu,
    oracle.ACT_SILU: torch.nn.functional.silu,
    oracle.ACT_NONE: lambda t: t,
}


@pytest.mark.parametrize("act", sorted(ACTS))
@pytest.mark.parametrize("w_layout", [0, 1])
def test_linear_act_against_torch_library(act, w_layout):
    M, N, K = 9, 7, 11
    x = RNG.standard_normal((M, K)); w = RNG.standard_normal((K, N)) * 0.5
    b = RNG.standard_normal(N); r = RNG.standard_normal((M, N))
    ws = w if w_layout == 0 else np.ascontiguousarray(w.T)
    want = ACTS[act](torch.from_numpy(x @ w + b)).numpy() + r
    np.testing.assert_allclose(oracle.linear_act(x, ws, b, r, act, w_layout), want, rtol=0, atol=1e-13)
    # optional operands really are optional
    np.testing.assert_allclose(oracle.linear_act(x, ws, None, None, act, w_layout),
                               ACTS[act](torch.from_numpy(x @ w)).numpy(), rtol=0, atol=1e-13)


def test_linear_act_closed_forms():
    one = np.ones((1, 1))
    f = lambda z, act: oracle.linear_act(np.array([[z]]), one, None, None, act)[0, 0]
    assert f(-2.0, oracle.ACT_RELU) == 0.0 and f(2.5, oracle.ACT_RELU) == 2.5
    assert f(0.0, oracle.ACT_SILU) == 0.0
    for z in (0.3, 1.0, 4.0):   # z sigma(z) + z sigma(-z) = z
        assert abs(f(z, oracle.ACT_SILU) - f(-z, oracle.ACT_SILU) - z) < 1e-15 * max(1, z)
        assert abs(f(z, oracle.ACT_GELU_ERF) - f(-z, oracle.ACT_GELU_ERF) - z) < 1e-15 * max(1, z)
    assert abs(f(1.0, oracle.ACT_SILU) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16
    assert abs(f(1.0, oracle.ACT_GELU_ERF) - 0.8413447460685429) < 1e-15     # Phi(1)
    assert abs(f(1.0, oracle.ACT_GELU_ERF) - f(1.0, oracle.ACT_GELU_TANH)) > 1e-4


def test_linear_act_matches_the_gelu_entry_and_mm_add():
    M, N, K = 6, 5, 4
    x = RNG.standard_normal((M, K)); w = RNG.standard_normal((K, N)); b = RNG.standard_normal(N)
    r = RNG.standard_normal((M, N))
    np.testing.assert_array_equal(oracle.linear_act(x, w, b), oracle.linear_bias_gelu(x, w, b))
    np.testing.assert_allclose(oracle.linear_act(x, w, None, r, oracle.ACT_NONE), x @ w + r, rtol=0, atol=1e-14)
    with pytest.raises(ValueError):
        oracle.linear_act(x, w, b, None, 9)


# ---- gated form: silu(x Wg) * (x Wu)
def test_swiglu_hand_values_and_closed_forms():
    """K = 1: y = silu(x wg) * x wu.  silu(ln 3) = ln 3 / (1 + 1/3) = 0.75 ln 3; silu(0) = 0; wu = 0 gives 0."""
    import math
    x = np.array([[1.0], [2.0]]); wg = np.array([[math.log(3), 0.0]]); wu = np.array([[2.0, 5.0]])
    y = oracle.linear_swiglu(x, wg, wu)
    np.testing.assert_allclose(y[0], [0.75 * math.log(3) * 2.0, 0.0], atol=1e-15)
    # row 1: gate = 2 ln 3 = ln 9: silu = ln 9 * 0.9; up = 4
    np.testing.assert_allclose(y[1], [0.9 * math.log(9) * 4.0, 0.0], atol=1e-14)
    assert np.all(oracle.linear_swiglu(RNG.standard_normal((3, 4)), RNG.standard_normal((4, 5)), np.zeros((4, 5))) == 0)
    # the gate is the activated branch: swapping the weights changes the result
    a = RNG.standard_normal((3, 4)); g = RNG.standard_normal((4, 5)); u = RNG.standard_normal((4, 5))
    assert np.abs(oracle.linear_swiglu(a, g, u) - oracle.linear_swiglu(a, u, g)).max() > 1e-3
    # silu(z) - silu(-z) = z: with the up projection fixed to ones, y(x) - y(-x)... uses gate only
    ones = np.ones((4, 5))
    up = a @ ones
    d = oracle.linear_swiglu(a, g, ones) / up + oracle.linear_swiglu(-a, g, ones) / up   # silu(z) - silu(-z)
    np.testing.assert_allclose(d, a @ g, atol=1e-12)


@pytest.mark.parametrize("w_layout", [0, 1])
def test_swiglu_against_torch_cpu(w_layout):
    x = RNG.standard_normal((7, 9)); g = RNG.standard_normal((9, 6)); u = RNG.standard_normal((9, 6))
    want = (torch.nn.functional.silu(torch.from_numpy(x @ g)) * torch.from_numpy(x @ u)).numpy()
    gg, uu = (g, u) if w_layout == 0 else (np.ascontiguousarray(g.T), np.ascontiguousarray(u.T))
    np.testing.assert_allclose(oracle.linear_swiglu(x, gg, uu, w_layout), want, atol=1e-13)
    # equals the already pinned linear+silu pattern times a plain matrix product
    np.testing.assert_allclose(oracle.linear_swiglu(x, g, u),
                               oracle.linear_act(x, g, None, None, oracle.ACT_SILU) * (x @ u), atol=1e-13)


# ---- weight-only int8: y = act(scale[n] * (x Wq^T) + b) + r
def test_w8_hand_value_and_reduction_to_the_dense_linear():
    """One output channel, integers (3, -2), scale 0.5, x = (2, 5): 0.5 * (6 - 10) = -2, plus bias 3 = 1; relu
    keeps 1, a negative pre-activation gives 0.  And: the quantised linear is the dense one on the
    dequantised weights (exactly representable here), which is pinned above."""
    x = np.array([[2.0, 5.0]]); wq = np.array([[3.0, -2.0], [1.0, 1.0]]); sc = np.array([0.5, -1.0])
    y = oracle.linear_w8(x, wq, sc, np.array([3.0, 0.0]), None, oracle.ACT_RELU)
    np.testing.assert_array_equal(y, [[1.0, 0.0]])
    np.testing.assert_array_equal(oracle.linear_w8(x, wq, sc, None, np.array([[10.0, 20.0]]), oracle.ACT_NONE), [[8.0, 13.0]])
    x = RNG.standard_normal((6, 8)); wq = RNG.integers(-128, 128, size=(5, 8)).astype(np.float64)
    sc = 2.0 ** RNG.integers(-6, -2, size=5).astype(np.float64)   # powers of two: dequantisation is exact
    b = RNG.standard_normal(5); r = RNG.standard_normal((6, 5))
    for act in (oracle.ACT_GELU_TANH, oracle.ACT_SILU, oracle.ACT_NONE):
        np.testing.assert_allclose(oracle.linear_w8(x, wq, sc, b, r, act),
                                   oracle.linear_act(x, wq * sc[:, None], b, r, act, 1), atol=1e-13)
    with pytest.raises(AssertionError):
        oracle.linear_w8(x, wq + 0.5, sc)
