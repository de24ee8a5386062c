"""GPU parity of the fp16 variants of the decode step and of the fused linear (the paper's inference
precision) against the fp64 oracle on the same fp16-rounded inputs.  Tolerances of the bf16 paths."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", [  # B, Hq, Hkv, Smax, D, splits, lens range
    (2, 8, 2, 300, 128, 4, (1, 300)),
    (3, 4, 4, 200, 64, 7, (1, 200)),
    (4, 16, 2, 1024, 128, 16, (100, 1024)),
])
def test_decode_f16(cfg):
    B, Hq, Hkv, Smax, D, ns, lr = cfg
    d = wl.decode_workload("t", 61, B, Hq, Hkv, Smax, D, ns, D ** -0.5, lr, dtype="f16")
    out = binding.attn_decode_splitkv(to_device(d.q), to_device(d.k_cache), to_device(d.v_cache),
                                      torch.from_numpy(d.lens).cuda(), ns, d.scale)
    binding.check_status()
    assert out.dtype == torch.float16
    assert_close_bf16(out, oracle.attn_decode(d.q.values, d.k_cache.values, d.v_cache.values, d.lens, d.scale))


@pytest.mark.parametrize("act", [binding.ACT_GELU_TANH, binding.ACT_SILU, binding.ACT_NONE])
@pytest.mark.parametrize("w_layout", [binding.W_KN, binding.W_NK])
def test_linear_act_f16(act, w_layout):
    M, N, K = 300, 456, 200
    w = wl.linear_workload("t", 62, M, N, K, w_std=1.0 / np.sqrt(K), b_std=0.5, dtype="f16")
    r = wl.normal_tensor(wl.seed_for(62, "q"), (M, N), "f16")
    wdev = to_device(w.w) if w_layout == binding.W_KN else to_device(w.w).t().contiguous()
    wref = w.w.values if w_layout == binding.W_KN else np.ascontiguousarray(w.w.values.T)
    y = binding.linear_act(to_device(w.x), wdev, to_device(w.b), to_device(r), act, w_layout)
    binding.check_status()
    assert y.dtype == torch.float16
    assert_close_bf16(y, oracle.linear_act(w.x.values, wref, w.b.values, r.values, act, w_layout))


def test_linear_gelu_f16_layer_shape_sampled_rows():
    """Config-2 GEMM shape in fp16, 64 sampled rows against the oracle."""
    w = wl.linear_workload("cfg2b in fp16", 2, 8192, 3072, 768, dtype="f16")
    y = binding.linear_act(to_device(w.x), to_device(w.w), to_device(w.b), None, binding.ACT_GELU_TANH)
    rows = np.unique((wl.splitmix64(6201, 64) % np.uint64(8192)).astype(np.int64))
    ref = oracle.linear_bias_gelu(w.x.values[rows], w.w.values, w.b.values)
    assert_close_bf16(y[torch.from_numpy(rows).cuda()], ref)
