"""GPU parity of the fused linear's activation (Eq. 11), at a resolution that tells the forms apart.

tanh-GELU and erf-GELU differ by at most 4.7e-4, far below the bf16 tolerance of the GEMM parity
tests, so those tests cannot see which form the epilogue computes.  Two checks close that gap:

  1. forge_activation_f32 runs the epilogue's own device function element-wise in fp32; with the
     accurate library routines and as the kernels run it (special-function-unit exponential and
     reciprocal) it must match the oracle's activation to 1e-6 for all five activations;
  2. through forge_linear_act with identity weights, pre-activations in [-3.25, -2.5] (where the two
     GELU forms differ by 3e-4 .. 4.7e-4 and the bf16 rounding of the output is below 3.1e-5) must land on
     the right form and off the wrong one, in both directions.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding
from util import to_f64

pytestmark = pytest.mark.gpu

ACTS = [oracle.ACT_GELU_TANH, oracle.ACT_GELU_ERF, oracle.ACT_RELU, oracle.ACT_SILU, oracle.ACT_NONE]


def _oracle_act(z64, act):
    """act(z) from the oracle: a K = 1 linear with weight 1 and no bias."""
    z = np.asarray(z64, dtype=np.float64).reshape(-1, 1)
    return oracle.linear_act(z, np.ones((1, 1)), None, None, act, 0).reshape(-1)


def _grid():
    z = np.concatenate([np.linspace(-9.0, 9.0, 7201), [0.0, -0.0, 1.0, -1.0, 3.0, 1e-6, -1e-6, 20.0, -20.0]])
    return z.astype(np.float32)


@pytest.mark.parametrize("act", ACTS)
@pytest.mark.parametrize("exact", [True, False])
def test_formula_matches_the_oracle_at_fp32_resolution(act, exact):
    """exact: the formulas with the accurate library routines; not exact: what the GEMM epilogues run
    (ex2.approx / rcp.approx in place of expf and the division).  1e-6 absolute, relative above 1."""
    z = _grid()
    got = to_f64(binding.activation_f32(torch.from_numpy(z).cuda(), act, exact=exact))
    ref = _oracle_act(z.astype(np.float64), act)
    assert np.all(np.abs(got - ref) <= 1e-6 * np.maximum(1.0, np.abs(ref)))


@pytest.mark.parametrize("act", [oracle.ACT_GELU_TANH, oracle.ACT_SILU])
def test_production_variant_keeps_relative_accuracy_in_the_negative_tail(act):
    """z sigmoid(.) rather than 0.5 z (1 + tanh(.)): no cancellation where the result is tiny."""
    z = np.linspace(-6.0, 6.0, 2401).astype(np.float32)
    got = to_f64(binding.activation_f32(torch.from_numpy(z).cuda(), act, exact=False))
    ref = _oracle_act(z.astype(np.float64), act)
    assert np.all(np.abs(got - ref) <= 5e-5 * np.abs(ref))


def test_elementwise_entry_separates_the_two_gelu_forms():
    z = np.linspace(-3.25, -2.25, 301).astype(np.float32)
    zt = torch.from_numpy(z).cuda()
    tanh_ref = _oracle_act(z.astype(np.float64), oracle.ACT_GELU_TANH)
    erf_ref = _oracle_act(z.astype(np.float64), oracle.ACT_GELU_ERF)
    assert np.abs(tanh_ref - erf_ref).min() > 3e-4  # the forms are far apart here ...
    for exact in (True, False):
        got_t = to_f64(binding.activation_f32(zt, oracle.ACT_GELU_TANH, exact=exact))
        got_e = to_f64(binding.activation_f32(zt, oracle.ACT_GELU_ERF, exact=exact))
        assert np.abs(got_t - tanh_ref).max() <= 1e-6 and np.abs(got_t - erf_ref).min() > 2e-4
        assert np.abs(got_e - erf_ref).max() <= 1e-6 and np.abs(got_e - tanh_ref).min() > 2e-4


def test_fused_linear_lands_on_the_right_gelu_form():
    """Identity weights, no bias: y = act(x) rounded to bf16 once.  |y| < 2^-6 on this range, so a bf16
    ulp is at most 2^-14 = 6.1e-5 and the rounding error at most 3.1e-5; the forms differ by > 3e-4."""
    n = 256
    rng = np.random.default_rng(11)
    x = torch.from_numpy(rng.uniform(-3.25, -2.5, (n, n)).astype(np.float32)).to(torch.bfloat16).cuda()
    z = to_f64(x)  # the bf16 values the kernel reads; x @ I = x exactly
    eye = torch.eye(n, dtype=torch.bfloat16, device="cuda")
    tanh_ref = _oracle_act(z.reshape(-1), oracle.ACT_GELU_TANH).reshape(n, n)
    erf_ref = _oracle_act(z.reshape(-1), oracle.ACT_GELU_ERF).reshape(n, n)
    assert np.abs(tanh_ref - erf_ref).min() > 3e-4
    tau = 4e-5
    y_t = to_f64(binding.linear_act(x, eye, None, None, binding.ACT_GELU_TANH))
    y_e = to_f64(binding.linear_act(x, eye, None, None, binding.ACT_GELU_ERF))
    y_d = to_f64(binding.linear_bias_gelu(x, eye, torch.zeros(n, dtype=torch.bfloat16, device="cuda")))
    assert np.abs(y_t - tanh_ref).max() <= tau and np.abs(y_t - erf_ref).min() > tau
    assert np.abs(y_e - erf_ref).max() <= tau and np.abs(y_e - tanh_ref).min() > tau
    assert np.array_equal(y_d, y_t)  # forge_linear_bias_gelu is the tanh form
