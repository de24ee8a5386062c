"""GPU parity: forge_attn_fused_bias (the fused attention with Eq. 8's optional mask node as an additive
tensor) against the fp64 oracle.  Tolerances: max-abs <= 2e-2 and mean-abs <= 2e-3 on unit-variance data.
The bias is seeded like the other inputs (fp32 normals; the oracle reads their exact widening)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device

pytestmark = pytest.mark.gpu


def _bias(seed, shape, hole_fraction=0.0):
    """fp32 N(0,1) bias; a seeded share of the entries is -inf (excluded keys)."""
    b = wl.normal_f64(seed, int(np.prod(shape))).astype(np.float32).reshape(shape)
    if hole_fraction > 0:
        u = wl.splitmix64(seed + 1, b.size).reshape(shape)
        b[(u % np.uint64(1000)) < np.uint64(int(hole_fraction * 1000))] = -np.inf
    return b


def _run(w, bias):
    lens = None if w.lens is None else torch.from_numpy(w.lens).cuda()
    out = binding.attn_fused_bias(to_device(w.q), to_device(w.k), to_device(w.v), torch.from_numpy(bias).cuda(),
                                  w.mask_kind, lens, w.scale)
    binding.check_status()
    ref = oracle.attn_bias(w.q.values, w.k.values, w.v.values, bias.astype(np.float64), w.mask_kind, w.lens, w.scale)
    return assert_close_bf16(out, ref)


SHAPES = [  # B, Hq, Hkv, Sq, Skv, D, bias heads
    (1, 2, 2, 128, 128, 64, 1),
    (2, 4, 2, 300, 300, 64, 4),     # several tiles, ragged tail, GQA, per-head bias
    (1, 8, 2, 200, 333, 128, 1),    # Skv not a multiple of 4: scalar bias loads; Sq != Skv
    (2, 3, 3, 130, 260, 128, 3),    # odd group size at D = 128: consecutive tiles of one head
    (1, 3, 3, 70, 200, 64, 3),      # odd group size at D = 64: two K/V streams
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("mask_kind", [0, 1, 2])
def test_random_bias_with_holes(shape, mask_kind):
    B, Hq, Hkv, Sq, Skv, D, Hb = shape
    w = wl.attention_workload("t", 45, B, Hq, Hkv, Sq, Skv, D, mask_kind, 1.0 / np.sqrt(D), "bf16",
                              lens_range=(1, Skv))
    _run(w, _bias(4501 + Hb, (B, Hb, Sq, Skv), hole_fraction=0.25))


def test_zero_bias_equals_the_plain_operator_bitwise():
    w = wl.attention_workload("t", 46, 2, 4, 2, 384, 384, 128, wl.MASK_CAUSAL, 128 ** -0.5, "bf16")
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    a = binding.attn_fused(q, k, v, w.mask_kind, None, w.scale)
    b = binding.attn_fused_bias(q, k, v, torch.zeros((2, 1, 384, 384), device="cuda"), w.mask_kind, None, w.scale)
    # same arithmetic except that the biased call never takes the FMA-pipe exponentials
    assert (a.float() - b.float()).abs().max().item() <= 2e-2
    ref = oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, None, w.scale)
    assert_close_bf16(b, ref)


def test_sliding_window_and_empty_rows():
    """A 0 / -inf band (each query sees the 96 keys up to its own position) and some rows with no key."""
    B, H, S, D = 1, 2, 512, 64
    w = wl.attention_workload("t", 47, B, H, H, S, S, D, wl.MASK_NONE, 0.125, "bf16")
    i = np.arange(S)[:, None]; j = np.arange(S)[None, :]
    band = np.where((j <= i) & (j > i - 96), 0.0, -np.inf).astype(np.float32)
    bias = np.broadcast_to(band, (B, 1, S, S)).copy()
    bias[0, 0, 5, :] = -np.inf; bias[0, 0, 300, :] = -np.inf
    out = binding.attn_fused_bias(to_device(w.q), to_device(w.k), to_device(w.v), torch.from_numpy(bias).cuda(),
                                  w.mask_kind, None, w.scale)
    assert torch.all(out[0, :, 5] == 0) and torch.all(out[0, :, 300] == 0)
    ref = oracle.attn_bias(w.q.values, w.k.values, w.v.values, bias.astype(np.float64), 0, None, w.scale)
    assert_close_bf16(out, ref)


def test_gqa_prefill_shape_with_shared_bias_sampled_heads():
    """Config-4 shape and launch with a shared ALiBi-like bias; the oracle checks three (batch, head) slices."""
    w = wl.cfg4_gqa_prefill(B=2)
    S = 2048
    dist = (np.arange(S)[None, :] - np.arange(S)[:, None]).astype(np.float32)
    bias = np.broadcast_to(0.01 * dist, (2, 1, S, S)).copy()
    out = binding.attn_fused_bias(to_device(w.q), to_device(w.k), to_device(w.v), torch.from_numpy(bias).cuda(),
                                  w.mask_kind, None, w.scale)
    binding.check_status()
    for b, h in ((0, 0), (1, 17), (1, 31)):
        kvh = h // 4
        ref = oracle.attn_bias(w.q.values[b:b + 1, h:h + 1], w.k.values[b:b + 1, kvh:kvh + 1],
                               w.v.values[b:b + 1, kvh:kvh + 1], bias[b:b + 1].astype(np.float64), w.mask_kind, None, w.scale)
        assert_close_bf16(out[b:b + 1, h:h + 1], ref)


def test_argument_checks():
    q = torch.zeros((1, 2, 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.ForgeError) as e:
        binding.attn_fused_bias(q, q, q, torch.zeros((1, 2, 128, 128), device="cuda"), 0, None, 0.0)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(ValueError):
        binding.attn_fused_bias(q, q, q, torch.zeros((1, 2, 128, 64), device="cuda"), 0, None, 0.125)
