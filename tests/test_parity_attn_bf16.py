"""GPU parity: forge_attn_fused (tcgen05 path) against the fp64 oracle.
Tolerances: max-abs <= 2e-2 and mean-abs <= 2e-3 on unit-variance data."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import assert_close_bf16, to_device, to_pinned, to_f64

pytestmark = pytest.mark.gpu


def _gpu(w):
    lens = None if w.lens is None else torch.from_numpy(w.lens).cuda()
    out = binding.attn_fused(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, lens, w.scale)
    binding.check_status()
    return out


def _run(w):
    out = _gpu(w)
    ref = oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, w.lens, w.scale)
    assert_close_bf16(out, ref)
    return out


SHAPES = [  # B, Hq, Hkv, Sq, Skv, D
    (1, 1, 1, 128, 128, 64),    # exactly one tile
    (1, 2, 2, 128, 128, 128),
    (2, 4, 2, 300, 300, 64),    # several tiles and a ragged tail, GQA
    (1, 8, 2, 200, 333, 128),   # Sq != Skv, group 4
    (2, 2, 1, 260, 100, 64),    # Sq > Skv: with a causal mask the first rows see no key
    (1, 3, 3, 1, 500, 128),     # a single query row
    (1, 2, 2, 77, 1, 64),       # a single key
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
def test_shapes_and_masks(shape, mask_kind):
    B, Hq, Hkv, Sq, Skv, D = shape
    w = wl.attention_workload("t", 41, B, Hq, Hkv, Sq, Skv, D, mask_kind, 1.0 / np.sqrt(D), "bf16",
                              lens_range=(1, Skv))
    _run(w)


@pytest.mark.parametrize("D", [8, 32, 40, 80, 96, 120])
@pytest.mark.parametrize("mask_kind", [1, 2])
def test_other_head_dimensions(D, mask_kind):
    """Head dimensions other than 64 and 128 (multiples of 8): the kernel pads them with the TMA unit's
    zero fill; nothing is read or written beyond the rows."""
    w = wl.attention_workload("t", 48, 2, 4, 2, 200, 333, D, mask_kind, 1.0 / np.sqrt(D), "bf16", lens_range=(1, 333))
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    dense = binding.attn_fused(q, k, v, mask_kind, torch.from_numpy(w.lens).cuda(), w.scale)
    assert_close_bf16(dense, oracle.attn(w.q.values, w.k.values, w.v.values, mask_kind, w.lens, w.scale))


def test_cfg2a_gpt2_layer_full():
    _run(wl.cfg2_attention())


def test_cfg3_encoder_padding_full():
    w = wl.cfg3_encoder()
    assert w.lens.min() >= 16 and w.lens.max() <= 128
    _run(w)


def test_cfg4_gqa_prefill_full():
    """Full benchmark shape and launch, every output element against the oracle."""
    _run(wl.cfg4_gqa_prefill())


@pytest.mark.parametrize("D", [64, 128, 40])
@pytest.mark.parametrize("mask_kind", [wl.MASK_PADDING, wl.MASK_CAUSAL_PADDING])
def test_padded_rows_never_reach_the_result(D, mask_kind):
    """K and V rows at and beyond lens[b] hold NaN and Inf (a caller's uninitialised padding).  Masked keys
    contribute exactly 0 (Eq. 8's mask node), so the result is finite and equals the oracle's, which never
    looks at them.  The lengths are not multiples of 64: the boundary falls inside a key tile."""
    B, Hq, Hkv, S = 4, 6, 2, 333
    w = wl.attention_workload("t", 49, B, Hq, Hkv, S, S, D, mask_kind, 1.0 / np.sqrt(D), "bf16", lens_range=(1, S))
    w.lens = np.array([37, 333, 129, 200], dtype=np.int32)
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    for b in range(B):
        k[b, :, int(w.lens[b]):] = float("nan")
        v[b, :, int(w.lens[b]):] = float("inf")
    if B > 1:
        v[2, :, int(w.lens[2]):] = float("nan")
    out = binding.attn_fused(q, k, v, mask_kind, torch.from_numpy(w.lens).cuda(), w.scale)
    binding.check_status()
    assert_close_bf16(out, oracle.attn(w.q.values, w.k.values, w.v.values, mask_kind, w.lens, w.scale))


def test_degenerate_lengths():
    """lens = 0 gives zeros; lens beyond Skv is clamped; lens = 1 returns V[0]."""
    w = wl.attention_workload("t", 42, 3, 2, 2, 140, 140, 64, wl.MASK_PADDING, 0.125, "bf16", lens_range=(1, 140))
    w.lens = np.array([0, 1000, 1], dtype=np.int32)
    out = _run(w)
    assert (out[0] == 0).all()
    assert torch.equal(out[2], to_device(w.v)[2, :, :1, :].expand(-1, 140, -1))


def test_invariants_at_size():
    """Properties that hold at any size: constant V rows give that row back; zero scale gives
    causal prefix means."""
    B, H, S, D = 2, 4, 512, 64
    w = wl.attention_workload("t", 43, B, H, H, S, S, D, wl.MASK_CAUSAL, 0.125, "bf16")
    q, k = to_device(w.q), to_device(w.k)
    c = to_device(w.v)[:, :, :1, :].expand(-1, -1, S, -1).contiguous()
    out = binding.attn_fused(q, k, c, wl.MASK_CAUSAL, None, 0.125)
    assert (to_f64(out) - to_f64(c)).__abs__().max() <= 2e-2
    v = to_device(w.v)
    out0 = binding.attn_fused(q, k, v, wl.MASK_CAUSAL, None, 0.0)
    prefix = np.cumsum(w.v.values, axis=2) / np.arange(1, S + 1)[None, None, :, None]
    assert_close_bf16(out0, prefix)


def test_large_scores_stay_finite():
    """A sharp softmax (large scale) must pick the arg-max value without overflow."""
    w = wl.attention_workload("t", 44, 1, 2, 2, 256, 256, 64, wl.MASK_NONE, 4.0, "bf16")
    _run(w)


def test_run_to_run_bitwise_identical():
    w = wl.attention_workload("t", 45, 2, 4, 2, 384, 384, 128, wl.MASK_CAUSAL, 0.088, "bf16")
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    a = binding.attn_fused(q, k, v, w.mask_kind, None, w.scale)
    b = binding.attn_fused(q, k, v, w.mask_kind, None, w.scale)
    assert torch.equal(a, b)


def test_negative_scale_is_refused():
    w = wl.attention_workload("t", 46, 1, 1, 1, 128, 128, 64, wl.MASK_NONE, 0.125, "bf16")
    with pytest.raises(binding.ForgeError) as e:
        binding.attn_fused(to_device(w.q), to_device(w.k), to_device(w.v), 0, None, -1.0)
    assert e.value.status == binding.ERR_UNSUPPORTED


def test_host_buffer_variant():
    w = wl.attention_workload("t", 47, 2, 4, 2, 200, 200, 64, wl.MASK_CAUSAL_PADDING, 0.125, "bf16",
                              lens_range=(50, 200))
    q, k, v = to_pinned(w.q), to_pinned(w.k), to_pinned(w.v)
    out = torch.empty_like(q).pin_memory()
    scratch = torch.empty(binding.attn_host_scratch_bytes(2, 4, 2, 200, 200, 64, 2), dtype=torch.uint8,
                          device="cuda")
    binding.attn_fused_host(q, k, v, out, scratch, w.mask_kind, torch.from_numpy(w.lens), w.scale)
    binding.check_status()
    assert_close_bf16(out, oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, w.lens, w.scale))


def test_host_buffer_variant_is_ordered_on_the_callers_stream():
    """Three batch entries (the entry-by-entry path): work given to the stream after the call sees the result, and
    the device scratch may be reused by the next call without a synchronisation in between."""
    w = wl.attention_workload("t", 48, 3, 4, 2, 300, 300, 128, wl.MASK_CAUSAL, 128 ** -0.5, "bf16")
    q, k, v = to_pinned(w.q), to_pinned(w.k), to_pinned(w.v)
    out1 = torch.empty_like(q).pin_memory()
    out2 = torch.empty_like(q).pin_memory()
    scratch = torch.empty(binding.attn_host_scratch_bytes(3, 4, 2, 300, 300, 128, 2), dtype=torch.uint8, device="cuda")
    binding.attn_fused_host(q, k, v, out1, scratch, w.mask_kind, None, w.scale)
    back = torch.empty(out1.shape, dtype=out1.dtype, device="cuda")
    back.copy_(out1, non_blocking=True)  # same stream, right behind the call
    binding.attn_fused_host(q, k, v, out2, scratch, w.mask_kind, None, w.scale)
    binding.check_status()
    ref = oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, None, w.scale)
    assert_close_bf16(back.cpu(), ref)
    assert torch.equal(out1, out2)
