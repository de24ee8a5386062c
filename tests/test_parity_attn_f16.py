"""GPU parity: forge_attn_fused_f16 (the tcgen05 attention kernel with fp16 operands, the inference
precision of the paper's evaluation) against the fp64 oracle on the same fp16-rounded inputs.
Tolerances: those of the bf16 path (max-abs <= 2e-2, mean-abs <= 2e-3 on unit-variance data); fp16
carries three more mantissa bits, so the observed errors are several times smaller."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device

pytestmark = pytest.mark.gpu


def _run(w):
    lens = None if w.lens is None else torch.from_numpy(w.lens).cuda()
    out = binding.attn_fused_f16(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, lens, w.scale)
    binding.check_status()
    assert out.dtype == torch.float16
    ref = oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, w.lens, w.scale)
    return assert_close_bf16(out, ref)


SHAPES = [  # B, Hq, Hkv, Sq, Skv, D
    (1, 2, 2, 128, 128, 64),
    (2, 4, 2, 300, 300, 64),    # several tiles and a ragged tail, GQA
    (1, 8, 2, 200, 333, 128),   # Sq != Skv, group 4
    (2, 2, 1, 260, 100, 128),   # Sq > Skv: with a causal mask the first rows see no key
    (1, 3, 3, 1, 500, 128),     # a single query row, odd group size
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
def test_shapes_and_masks(shape, mask_kind):
    B, Hq, Hkv, Sq, Skv, D = shape
    w = wl.attention_workload("t", 43, B, Hq, Hkv, Sq, Skv, D, mask_kind, 1.0 / np.sqrt(D), "f16",
                              lens_range=(1, Skv))
    _run(w)


def test_gpt2_layer_shape_and_tighter_error():
    """Config-2 attention shape in fp16: within the common tolerance, and (three more mantissa bits than
    bf16 in P and in the output) well inside a quarter of it."""
    w = wl.attention_workload("cfg2a in fp16", 2, 2, 12, 12, 1024, 1024, 64, wl.MASK_CAUSAL, 0.125, "f16")
    mx, mean = _run(w)
    assert mx <= 5e-3 and mean <= 5e-4


def test_gqa_prefill_shape_sampled_heads():
    """Config-4 shape and launch in fp16; the oracle checks four whole (batch, head) slices."""
    w = wl.attention_workload("cfg4 in fp16", 4, 4, 32, 8, 2048, 2048, 128, wl.MASK_CAUSAL, 128 ** -0.5, "f16")
    out = binding.attn_fused_f16(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, None, w.scale)
    binding.check_status()
    for b, h in ((0, 0), (1, 13), (2, 22), (3, 31)):
        kvh = h // 4
        ref = oracle.attn(w.q.values[b:b + 1, h:h + 1], w.k.values[b:b + 1, kvh:kvh + 1],
                          w.v.values[b:b + 1, kvh:kvh + 1], w.mask_kind, None, w.scale)
        assert_close_bf16(out[b:b + 1, h:h + 1], ref)


def test_zero_scale_and_constant_v():
    """scale = 0 gives the causal prefix mean of V; constant V rows come back unchanged."""
    w = wl.attention_workload("t", 44, 1, 2, 2, 256, 256, 64, wl.MASK_CAUSAL, 0.0, "f16")
    out = binding.attn_fused_f16(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, None, 0.0)
    ref = np.cumsum(w.v.values, axis=2) / np.arange(1, 257)[None, None, :, None]
    assert_close_bf16(out, ref)
    v = torch.full((1, 2, 256, 64), 0.75, dtype=torch.float16, device="cuda")
    out = binding.attn_fused_f16(to_device(w.q), to_device(w.k), v, wl.MASK_CAUSAL, None, 0.125)
    assert torch.all(out == 0.75)
