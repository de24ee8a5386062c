"""GPU parity: head sizes above 128 (the one-tile-per-CTA kernel) against the fp64 oracle.
Tolerances: max-abs <= 2e-2 and mean-abs <= 2e-3 on unit-variance data."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import Guarded, assert_close_bf16, to_device

pytestmark = pytest.mark.gpu


def _run(w, fn=binding.attn_fused, guarded=True):
    lens = None if w.lens is None else torch.from_numpy(w.lens).cuda()
    g = Guarded((w.B, w.Hq, w.Sq, w.D), torch.float16 if w.dtype == "f16" else torch.bfloat16)
    fn(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, lens, w.scale, out=g.tensor)
    binding.check_status()
    assert_close_bf16(g.tensor, oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, w.lens, w.scale))
    g.assert_intact()
    return g.tensor


SHAPES = [  # B, Hq, Hkv, Sq, Skv
    (1, 1, 1, 128, 128),     # exactly one tile, two key steps
    (2, 4, 2, 300, 300),     # several tiles and a ragged tail, GQA
    (1, 8, 2, 200, 333),     # Sq != Skv, group 4
    (2, 2, 1, 260, 100),     # Sq > Skv: with a causal mask the first rows see no key
    (1, 3, 3, 1, 500),       # a single query row
    (1, 2, 2, 77, 1),        # a single key
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
def test_shapes_and_masks_d256(shape, mask_kind):
    B, Hq, Hkv, Sq, Skv = shape
    _run(wl.attention_workload("t", 61, B, Hq, Hkv, Sq, Skv, 256, mask_kind, 1.0 / 16, "bf16", lens_range=(1, Skv)))


@pytest.mark.parametrize("D", [136, 160, 192, 248])
@pytest.mark.parametrize("mask_kind", [1, 2])
def test_other_wide_head_dimensions(D, mask_kind):
    _run(wl.attention_workload("t", 62, 2, 4, 2, 200, 333, D, mask_kind, 1.0 / np.sqrt(D), "bf16", lens_range=(1, 333)))


def test_many_items_per_cta_and_long_rows():
    """More work items than SMs (several rounds of the persistent schedule) and 32 key steps per row."""
    _run(wl.attention_workload("t", 63, 2, 24, 8, 1024, 2048, 256, wl.MASK_CAUSAL, 1.0 / 16, "bf16"))


def test_fp16_tensors():
    w = wl.attention_workload("t", 64, 2, 4, 2, 300, 300, 256, wl.MASK_CAUSAL, 1.0 / 16, "f16")
    _run(w, fn=binding.attn_fused_f16)


def test_padded_rows_never_reach_the_result():
    B, Hq, Hkv, S, D = 4, 6, 2, 333, 192
    w = wl.attention_workload("t", 65, B, Hq, Hkv, S, S, D, wl.MASK_CAUSAL_PADDING, 1.0 / np.sqrt(D), "bf16", lens_range=(1, S))
    w.lens = np.array([37, 333, 129, 200], dtype=np.int32)
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    for b in range(B):
        k[b, :, int(w.lens[b]):] = float("nan")
        v[b, :, int(w.lens[b]):] = float("inf")
    out = binding.attn_fused(q, k, v, w.mask_kind, torch.from_numpy(w.lens).cuda(), w.scale)
    binding.check_status()
    assert_close_bf16(out, oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, w.lens, w.scale))


def test_large_scores_and_degenerate_lengths():
    w = wl.attention_workload("t", 66, 3, 2, 2, 140, 140, 256, wl.MASK_PADDING, 0.5, "bf16", lens_range=(1, 140))
    w.lens = np.array([0, 1000, 1], dtype=np.int32)
    out = _run(w)
    assert (out[0] == 0).all()


def test_run_to_run_bitwise_identical():
    w = wl.attention_workload("t", 67, 2, 4, 2, 384, 384, 256, wl.MASK_CAUSAL, 1.0 / 16, "bf16")
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    assert torch.equal(binding.attn_fused(q, k, v, 1, None, w.scale), binding.attn_fused(q, k, v, 1, None, w.scale))


def test_strided_views_d256():
    B, Hq, Hkv, S, D = 2, 4, 2, 200, 256
    w = wl.attention_workload("t", 68, B, Hq, Hkv, S, S, D, wl.MASK_CAUSAL, 1.0 / 16, "bf16")
    n_tot = (Hq + 2 * Hkv) * D
    qkv = torch.empty((B, S, n_tot), dtype=torch.bfloat16, device="cuda")
    qkv[:, :, :Hq * D] = to_device(w.q).permute(0, 2, 1, 3).reshape(B, S, Hq * D)
    qkv[:, :, Hq * D:(Hq + Hkv) * D] = to_device(w.k).permute(0, 2, 1, 3).reshape(B, S, Hkv * D)
    qkv[:, :, (Hq + Hkv) * D:] = to_device(w.v).permute(0, 2, 1, 3).reshape(B, S, Hkv * D)
    q = qkv[:, :, :Hq * D].view(B, S, Hq, D).permute(0, 2, 1, 3)
    k = qkv[:, :, Hq * D:(Hq + Hkv) * D].view(B, S, Hkv, D).permute(0, 2, 1, 3)
    v = qkv[:, :, (Hq + Hkv) * D:].view(B, S, Hkv, D).permute(0, 2, 1, 3)
    out = torch.empty((B, S, Hq * D), dtype=torch.bfloat16, device="cuda")
    binding.attn_fused_strided(q, k, v, out.view(B, S, Hq, D).permute(0, 2, 1, 3), 1, None, w.scale)
    binding.check_status()
    assert_close_bf16(out.view(B, S, Hq, D).permute(0, 2, 1, 3).contiguous(),
                      oracle.attn(w.q.values, w.k.values, w.v.values, 1, None, w.scale))
