"""GPU parity: forge_linear_act_w8a16 (fp16 activations, int8 weights with a per-channel scale, widened to
fp16 inside the kernel) against the fp64 oracle.  Tolerances of the 16-bit paths (max-abs <= 2e-2, mean-abs
<= 2e-3 on unit-variance pre-activations).  Weights are seeded: integers uniform on [-127, 127], scales
chosen so that the pre-activations have unit variance."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device

pytestmark = pytest.mark.gpu


def _case(seed, M, N, K):
    x = wl.normal_tensor(wl.seed_for(seed, "x"), (M, K), "f16")
    wq = (wl.uniform_int(wl.seed_for(seed, "w"), N * K, -127, 127)).reshape(N, K).astype(np.int8)
    # std of a uniform integer on [-127, 127] is 73.6: unit-variance pre-activations, scales varying per channel
    scale = ((0.5 + wl.splitmix64(wl.seed_for(seed, "lens"), N) % np.uint64(1000) / 1000.0) / (73.6 * np.sqrt(K))).astype(np.float32)
    b = wl.normal_tensor(wl.seed_for(seed, "b"), (N,), "f16", std=0.5)
    r = wl.normal_tensor(wl.seed_for(seed, "q"), (M, N), "f16")
    return x, wq, scale, b, r


@pytest.mark.parametrize("act", [binding.ACT_GELU_TANH, binding.ACT_SILU, binding.ACT_NONE])
@pytest.mark.parametrize("shape", [(128, 192, 64), (300, 456, 208), (130, 72, 1024)])
def test_shapes_and_activations(shape, act):
    M, N, K = shape
    x, wq, scale, b, r = _case(71, M, N, K)
    y = binding.linear_act_w8a16(to_device(x), torch.from_numpy(wq).cuda(), torch.from_numpy(scale).cuda(),
                                 to_device(b), to_device(r), act)
    binding.check_status()
    ref = oracle.linear_w8(x.values, wq.astype(np.float64), scale.astype(np.float64), b.values, r.values, act)
    assert_close_bf16(y, ref)


@pytest.mark.parametrize("M", [128, 384])  # one row tile (one-CTA kernel) and several (CTA pairs)
def test_extreme_weights_are_widened_exactly(M):
    """-128, 127 and 0 only, identity-like activations: the result is an exact small integer combination."""
    N, K = 64, 64
    x = torch.zeros((M, K), dtype=torch.float16, device="cuda"); x[:, 0] = 1.0; x[:, 1] = 2.0
    wq = torch.zeros((N, K), dtype=torch.int8, device="cuda"); wq[:, 0] = -128; wq[:, 1] = 127; wq[5, 1] = -128
    y = binding.linear_act_w8a16(x, wq, torch.ones(N, device="cuda"), None, None, binding.ACT_NONE)
    want = torch.full((M, N), 126.0, device="cuda"); want[:, 5] = -384.0
    assert torch.equal(y.float(), want)


def test_layer_shape_sampled_rows_without_bias():
    M, N, K = 4096, 4096, 4096
    x, wq, scale, _, _ = _case(72, M, N, K)
    y = binding.linear_act_w8a16(to_device(x), torch.from_numpy(wq).cuda(), torch.from_numpy(scale).cuda(), None, None,
                                 binding.ACT_SILU)
    binding.check_status()
    rows = np.unique((wl.splitmix64(7201, 48) % np.uint64(M)).astype(np.int64))
    ref = oracle.linear_w8(x.values[rows], wq.astype(np.float64), scale.astype(np.float64), None, None, oracle.ACT_SILU)
    assert_close_bf16(y[torch.from_numpy(rows).cuda()], ref)


def test_argument_checks():
    x = torch.zeros((8, 24), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.ForgeError) as e:  # K not a multiple of 16
        binding.linear_act_w8a16(x, torch.zeros((16, 24), dtype=torch.int8, device="cuda"), torch.ones(16, device="cuda"))
    assert e.value.status == binding.ERR_UNSUPPORTED
