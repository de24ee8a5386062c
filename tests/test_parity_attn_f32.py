"""GPU parity: forge_attn_fused_f32 against the fp64 oracle (max-abs <= 1e-4)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_f32, to_device, to_pinned

pytestmark = pytest.mark.gpu


def _run(w):
    lens = None if w.lens is None else torch.from_numpy(w.lens).cuda()
    out = binding.attn_fused_f32(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, lens, w.scale)
    ref = oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, w.lens, w.scale)
    assert_close_f32(out, ref)
    return out


def test_cfg1_gpt2_small_causal():
    out = _run(wl.cfg1_gpt2_f32())
    assert out.shape == (1, 12, 128, 64)


SHAPES = [  # B, Hq, Hkv, Sq, Skv, D
    (2, 4, 2, 70, 70, 64),     # ragged tail in both tile directions
    (1, 8, 2, 33, 130, 64),    # Sq != Skv, GQA group 4
    (2, 2, 2, 150, 45, 128),   # Sq > Skv, D = 128
    (1, 3, 1, 1, 200, 64),     # single query row, group 3
    (1, 2, 2, 17, 1, 128),     # single key
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
def test_shapes_and_masks(shape, mask_kind):
    B, Hq, Hkv, Sq, Skv, D = shape
    w = wl.attention_workload("t", 11, B, Hq, Hkv, Sq, Skv, D, mask_kind, 1.0 / np.sqrt(D), "f32",
                              lens_range=(1, Skv))
    _run(w)


def test_degenerate_lengths():
    """lens = 0 gives zeros; lens beyond Skv is clamped."""
    w = wl.attention_workload("t", 12, 3, 2, 2, 20, 40, 64, wl.MASK_PADDING, 0.125, "f32", lens_range=(1, 40))
    w.lens = np.array([0, 1000, 7], dtype=np.int32)
    out = _run(w)
    assert (out[0] == 0).all()


def test_run_to_run_bitwise_identical():
    w = wl.cfg1_gpt2_f32()
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    a = binding.attn_fused_f32(q, k, v, w.mask_kind, None, w.scale)
    b = binding.attn_fused_f32(q, k, v, w.mask_kind, None, w.scale)
    assert torch.equal(a, b)


def test_host_buffer_variant():
    w = wl.cfg1_gpt2_f32()
    q, k, v = to_pinned(w.q), to_pinned(w.k), to_pinned(w.v)
    out = torch.empty_like(q).pin_memory()
    scratch = torch.empty(binding.attn_host_scratch_bytes(1, 12, 12, 128, 128, 64, 4), dtype=torch.uint8,
                          device="cuda")
    binding.attn_fused_host(q, k, v, out, scratch, w.mask_kind, None, w.scale)
    binding.check_status()
    ref = oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, None, w.scale)
    assert_close_f32(out, ref)
