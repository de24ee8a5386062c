"""GPU parity: forge_linear_swiglu (gated MLP input, silu(x Wg) * (x Wu) in one kernel) against the fp64
oracle.  Tolerance: the product of two unit-variance pre-activations is not bounded like they are (values
near 10 occur), so the single rounding of the output to bf16 (half an ulp = 2^-9 relative) is allowed for on
top of the common bound: |err| <= 2e-2 + 2^-8 |ref| element-wise, and mean-abs <= 2e-3."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import BF16_MAX_ABS, BF16_MEAN_ABS, to_device, to_f64

pytestmark = pytest.mark.gpu


def assert_close_bf16(got, ref):
    g = to_f64(got)
    assert np.isfinite(g).all()
    err = np.abs(g - ref)
    excess = err - 2.0 ** -8 * np.abs(ref)
    assert excess.max() <= BF16_MAX_ABS, f"max excess {excess.max():.3e} > {BF16_MAX_ABS}"
    assert err.mean() <= BF16_MEAN_ABS, f"mean-abs {err.mean():.3e} > {BF16_MEAN_ABS}"


def _weights(seed, M, N, K):
    x = wl.normal_tensor(wl.seed_for(seed, "x"), (M, K), "bf16")
    wg = wl.normal_tensor(wl.seed_for(seed, "w"), (K, N), "bf16", std=1.0 / np.sqrt(K))
    wu = wl.normal_tensor(wl.seed_for(seed, "b"), (K, N), "bf16", std=1.0 / np.sqrt(K))
    return x, wg, wu


@pytest.mark.parametrize("w_layout", [binding.W_KN, binding.W_NK])
@pytest.mark.parametrize("shape", [(128, 128, 64), (300, 456, 200), (130, 72, 1024)])
def test_shapes_and_weight_layouts(shape, w_layout):
    M, N, K = shape  # ragged in every dimension, one to several tiles, 1 to 16 k-blocks
    x, wg, wu = _weights(53, M, N, K)
    if w_layout == binding.W_KN:
        y = binding.linear_swiglu(to_device(x), to_device(wg), to_device(wu), w_layout)
        ref = oracle.linear_swiglu(x.values, wg.values, wu.values, 0)
    else:
        y = binding.linear_swiglu(to_device(x), to_device(wg).t().contiguous(), to_device(wu).t().contiguous(), w_layout)
        ref = oracle.linear_swiglu(x.values, np.ascontiguousarray(wg.values.T), np.ascontiguousarray(wu.values.T), 1)
    binding.check_status()
    assert_close_bf16(y, ref)


def test_decoder_mlp_shape_sampled_rows():
    """1B-class decoder MLP input (hidden 2048, intermediate 8192) on 4096 tokens, [N,K] weights as the
    models store them; the oracle checks 48 sampled rows."""
    M, N, K = 4096, 8192, 2048
    x, wg, wu = _weights(54, M, N, K)
    y = binding.linear_swiglu(to_device(x), to_device(wg).t().contiguous(), to_device(wu).t().contiguous(), binding.W_NK)
    binding.check_status()
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], (wl.splitmix64(5401, 44) % np.uint64(M)).astype(np.int64)]))
    ref = oracle.linear_swiglu(x.values[rows], wg.values, wu.values, 0)
    assert_close_bf16(y[torch.from_numpy(rows).cuda()], ref)


def test_zero_up_weights_give_zero_and_argument_checks():
    x, wg, wu = _weights(55, 128, 128, 64)
    y = binding.linear_swiglu(to_device(x), to_device(wg), torch.zeros((64, 128), dtype=torch.bfloat16, device="cuda"))
    assert torch.all(y == 0)
    with pytest.raises(ValueError):
        binding.linear_swiglu(to_device(x), to_device(wg), to_device(wu).t().contiguous())
    with pytest.raises(binding.ForgeError) as e:
        binding.linear_swiglu(torch.zeros((8, 12), dtype=torch.bfloat16, device="cuda"),
                              torch.zeros((12, 16), dtype=torch.bfloat16, device="cuda"),
                              torch.zeros((12, 16), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == binding.ERR_UNSUPPORTED
