"""GPU parity of the fused linear's activation (Eq. 11), at a resolution that tells the forms apart.

tanh-GELU and erf-GELU differ by at most 4.7e-4, far below the bf16 tolerance of the GEMM parity
tests, so those tests cannot see which form the epilogue computes.  These checks close that gap:

  1. forge_activation_f32 runs the epilogue's own device function element-wise in fp32.  With the
     accurate library routines (exact = 1) it must match the oracle's activation to 1e-6 for all five
     activations, which settles the formulas; there the two GELU forms are told apart in both
     directions.  As the kernels run it (exact = 0: one tanh.approx per element, relative error 2^-11
     of the tanh) it must stay within 3e-4 max(1, |z|) of the oracle;
  2. through forge_linear_act with identity weights, pre-activations in [-3.25, -2.5] (where the two
     GELU forms differ by 3e-4 .. 4.7e-4 and the bf16 rounding of the output is below 3.1e-5): the
     erf form, which uses no approximation, must land on the erf oracle and off the tanh oracle; the
     tanh form must stay within its approximation's bound of the tanh oracle.
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
def test_formula_matches_the_oracle_at_fp32_resolution(act):
    """The epilogue's formulas with the accurate library routines: 1e-6 absolute, relative above 1."""
    z = _grid()
    got = to_f64(binding.activation_f32(torch.from_numpy(z).cuda(), act, exact=True))
    ref = _oracle_act(z.astype(np.float64), act)
    assert np.all(np.abs(got - ref) <= 1e-6 * np.maximum(1.0, np.abs(ref)))


@pytest.mark.parametrize("act", ACTS)
def test_production_variant_stays_within_its_approximation(act):
    """What the GEMM epilogues run: tanh.approx (relative error 2^-11 of the tanh) in the tanh-GELU and in the
    sigmoid of SiLU, i.e. at most 0.5 |z| 2^-11 = 2.5e-4 |z| on the activation; the others are unchanged."""
    z = _grid()
    got = to_f64(binding.activation_f32(torch.from_numpy(z).cuda(), act, exact=False))
    ref = _oracle_act(z.astype(np.float64), act)
    approx = act in (oracle.ACT_GELU_TANH, oracle.ACT_SILU)
    tol = 3e-4 * np.maximum(1.0, np.abs(z.astype(np.float64))) if approx else 1e-6 * np.maximum(1.0, np.abs(ref))
    assert np.all(np.abs(got - ref) <= tol)


def test_elementwise_entry_separates_the_two_gelu_forms():
    z = np.linspace(-3.25, -2.25, 301).astype(np.float32)
    zt = torch.from_numpy(z).cuda()
    tanh_ref = _oracle_act(z.astype(np.float64), oracle.ACT_GELU_TANH)
    erf_ref = _oracle_act(z.astype(np.float64), oracle.ACT_GELU_ERF)
    assert np.abs(tanh_ref - erf_ref).min() > 3e-4  # the forms are far apart here ...
    got_t = to_f64(binding.activation_f32(zt, oracle.ACT_GELU_TANH, exact=True))
    got_e = to_f64(binding.activation_f32(zt, oracle.ACT_GELU_ERF, exact=True))
    assert np.abs(got_t - tanh_ref).max() <= 1e-6 and np.abs(got_t - erf_ref).min() > 2e-4
    assert np.abs(got_e - erf_ref).max() <= 1e-6 and np.abs(got_e - tanh_ref).min() > 2e-4
    # the erf form is the same in the kernels' variant
    got_e = to_f64(binding.activation_f32(zt, oracle.ACT_GELU_ERF, exact=False))
    assert np.abs(got_e - erf_ref).max() <= 1e-6


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
    assert np.abs(y_e - erf_ref).max() <= tau and np.abs(y_e - tanh_ref).min() > tau
    # the tanh form with the hardware tanh: within 0.5 |z| 2^-11 + rounding of the tanh oracle
    assert np.abs(y_t - tanh_ref).max() <= 0.5 * 3.25 * 2.0 ** -11 + tau
    assert np.array_equal(y_d, y_t)  # forge_linear_bias_gelu is the same epilogue
