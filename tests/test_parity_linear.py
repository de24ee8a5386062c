"""GPU parity: forge_linear_bias_gelu against the fp64 oracle (bf16 tolerances)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device, to_pinned, to_f64

pytestmark = pytest.mark.gpu


def _run(w):
    y = binding.linear_bias_gelu(to_device(w.x), to_device(w.w), to_device(w.b))
    binding.check_status()
    return y


@pytest.mark.parametrize("M,N,K", [
    (128, 192, 64),      # exactly one tile, one K block
    (128, 192, 256),     # one tile, several K blocks
    (256, 384, 128),     # 2 x 2 tiles
    (200, 200, 72),      # ragged in M, N and K
    (1, 8, 8),           # smallest legal problem
    (1000, 3072, 768),   # more tiles than one wave of the persistent grid at the benchmark's N and K
])
def test_shapes(M, N, K):
    # unit-variance pre-activations: std(w) = 1/sqrt(K)
    w = wl.linear_workload("t", 31, M, N, K, w_std=1.0 / np.sqrt(K), b_std=0.5)
    y = _run(w)
    ref = oracle.linear_bias_gelu(w.x.values, w.w.values, w.b.values)
    assert_close_bf16(y, ref)


def test_cfg2b_full_size():
    """Benchmark shape and launch configuration, every output element against the oracle."""
    w = wl.cfg2_linear()
    y = _run(w)
    assert_close_bf16(y, oracle.linear_bias_gelu(w.x.values, w.w.values, w.b.values))


def test_identity_weight_gives_gelu_of_x_plus_b():
    n = 256
    x = wl.normal_tensor(77, (n, n), "bf16")
    b = wl.normal_tensor(78, (n,), "bf16")
    eye = torch.eye(n, dtype=torch.bfloat16, device="cuda")
    y = binding.linear_bias_gelu(to_device(x), eye, to_device(b))
    ref = oracle.linear_bias_gelu(x.values, np.eye(n), b.values)
    assert_close_bf16(y, ref)


def test_run_to_run_bitwise_identical():
    w = wl.linear_workload("t", 32, 512, 768, 256, w_std=1.0 / 16)
    x, ww, b = to_device(w.x), to_device(w.w), to_device(w.b)
    assert torch.equal(binding.linear_bias_gelu(x, ww, b), binding.linear_bias_gelu(x, ww, b))


def test_host_buffer_variant():
    w = wl.linear_workload("t", 33, 300, 256, 128, w_std=1.0 / np.sqrt(128))
    x, ww, b = to_pinned(w.x), to_pinned(w.w), to_pinned(w.b)
    y = torch.empty((300, 256), dtype=torch.bfloat16).pin_memory()
    scratch = torch.empty(binding.linear_host_scratch_bytes(300, 256, 128), dtype=torch.uint8, device="cuda")
    binding.linear_bias_gelu_host(x, ww, b, y, scratch)
    binding.check_status()
    assert_close_bf16(y, oracle.linear_bias_gelu(w.x.values, w.w.values, w.b.values))
