"""GPU parity: forge_linear_act (the other operator-fusion epilogues) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device, to_f64

pytestmark = pytest.mark.gpu


def _case(M, N, K, seed=51):
    w = wl.linear_workload("t", seed, M, N, K, w_std=1.0 / np.sqrt(K), b_std=0.5)
    r = wl.normal_tensor(wl.seed_for(seed, "q"), (M, N), "bf16")
    return w, r


@pytest.mark.parametrize("act", [binding.ACT_GELU_TANH, binding.ACT_GELU_ERF, binding.ACT_RELU, binding.ACT_SILU,
                                 binding.ACT_NONE])
@pytest.mark.parametrize("w_layout", [binding.W_KN, binding.W_NK])
def test_activations_and_weight_layouts(act, w_layout):
    M, N, K = 300, 456, 200          # ragged in every dimension, several tiles
    w, r = _case(M, N, K)
    wdev = to_device(w.w) if w_layout == binding.W_KN else to_device(w.w).t().contiguous()
    wref = w.w.values if w_layout == binding.W_KN else np.ascontiguousarray(w.w.values.T)
    y = binding.linear_act(to_device(w.x), wdev, to_device(w.b), to_device(r), act, w_layout)
    binding.check_status()
    ref = oracle.linear_act(w.x.values, wref, w.b.values, r.values, act, w_layout)
    assert_close_bf16(y, ref)


def test_mm_add_pattern_without_bias():
    """Residual addition after a raw matrix multiply."""
    M, N, K = 256, 384, 128
    w, r = _case(M, N, K, seed=52)
    y = binding.linear_act(to_device(w.x), to_device(w.w), None, to_device(r), binding.ACT_NONE)
    assert_close_bf16(y, oracle.linear_act(w.x.values, w.w.values, None, r.values, oracle.ACT_NONE))


def test_linear_layout_nk_at_benchmark_size_sampled_rows():
    w = wl.cfg2_linear()
    wt = to_device(w.w).t().contiguous()
    y = binding.linear_act(to_device(w.x), wt, to_device(w.b), None, binding.ACT_SILU, binding.W_NK)
    binding.check_status()
    rows = np.array([0, 127, 128, 4097, 8191])
    ref = oracle.linear_act(w.x.values[rows], w.w.values, w.b.values, None, oracle.ACT_SILU)
    assert_close_bf16(y[torch.from_numpy(rows).cuda()], ref)
    assert np.isfinite(to_f64(y)).all()


def test_gelu_entry_point_is_the_same_kernel():
    w, _ = _case(256, 192, 64, seed=53)
    x, ww, b = to_device(w.x), to_device(w.w), to_device(w.b)
    assert torch.equal(binding.linear_bias_gelu(x, ww, b), binding.linear_act(x, ww, b))


def test_argument_validation():
    w, _ = _case(16, 16, 16, seed=54)
    x, ww = to_device(w.x), to_device(w.w)
    with pytest.raises(binding.ForgeError) as e:
        binding.linear_act(x, ww, None, None, 7)
    assert e.value.status == binding.ERR_INVALID_ARG


@pytest.mark.parametrize("shape", [(16, 4104, 2112), (100, 14344, 640)])
@pytest.mark.parametrize("w_layout", [binding.W_KN, binding.W_NK])
def test_single_row_tile_with_a_large_weight(shape, w_layout):
    """M <= 128 and a weight of 17-18 MB: the narrow tiles (64 and 128 columns) that spread the weight stream over
    more SMs; the last column tile is ragged."""
    M, N, K = shape
    w, r = _case(M, N, K, seed=55)
    wdev = to_device(w.w) if w_layout == binding.W_KN else to_device(w.w).t().contiguous()
    wref = w.w.values if w_layout == binding.W_KN else np.ascontiguousarray(w.w.values.T)
    y = binding.linear_act(to_device(w.x), wdev, to_device(w.b), to_device(r), binding.ACT_GELU_TANH, w_layout)
    binding.check_status()
    assert_close_bf16(y, oracle.linear_act(w.x.values, wref, w.b.values, r.values, oracle.ACT_GELU_TANH, w_layout))
