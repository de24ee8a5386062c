"""Nothing is written outside `out`, `y` or the decode workspace.

The kernels lean on the TMA unit's clipping for ragged row counts, ragged N and head sizes below
the kernel's own (64 or 128), and on plain stores for rows that see no key.  Each case here gives the
kernel an output (and workspace) that sits between two sentinel-filled guard regions, checks the
result against the oracle (so every element inside was written: the buffer starts as NaN) and then
checks that both guards are untouched.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import Guarded, assert_close_bf16, assert_close_f32, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Skv,D,mask_kind", [
    (2, 4, 2, 300, 300, 64, 1),     # ragged last query tile
    (1, 2, 2, 77, 1, 64, 0),        # fewer rows than one store box, a single key
    (2, 4, 2, 200, 333, 8, 2),      # head sizes below the kernel's: columns clipped on store
    (2, 4, 2, 200, 333, 40, 3),
    (1, 8, 2, 130, 130, 120, 1),
    (2, 2, 1, 260, 100, 64, 1),     # Sq > Skv with a causal mask: rows without a visible key (plain stores)
    (1, 3, 3, 1, 500, 128, 0),      # a single query row
])
def test_attention_output_stays_inside(B, Hq, Hkv, Sq, Skv, D, mask_kind):
    w = wl.attention_workload("t", 51, B, Hq, Hkv, Sq, Skv, D, mask_kind, 1.0 / np.sqrt(D), "bf16", lens_range=(1, Skv))
    lens = None if w.lens is None else torch.from_numpy(w.lens).cuda()
    g = Guarded((B, Hq, Sq, D), torch.bfloat16)
    binding.attn_fused(to_device(w.q), to_device(w.k), to_device(w.v), mask_kind, lens, w.scale, out=g.tensor)
    binding.check_status()
    assert_close_bf16(g.tensor, oracle.attn(w.q.values, w.k.values, w.v.values, mask_kind, w.lens, w.scale))
    g.assert_intact()


def test_attention_rows_with_no_key_stay_inside():
    """lens = 0 for a whole sequence: its rows are written as zeros with plain stores."""
    w = wl.attention_workload("t", 52, 3, 2, 2, 140, 140, 40, wl.MASK_PADDING, 0.125, "bf16", lens_range=(1, 140))
    w.lens = np.array([0, 1000, 1], dtype=np.int32)
    g = Guarded((3, 2, 140, 40), torch.bfloat16)
    binding.attn_fused(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, torch.from_numpy(w.lens).cuda(),
                       w.scale, out=g.tensor)
    binding.check_status()
    assert_close_bf16(g.tensor, oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, w.lens, w.scale))
    assert (g.tensor[0] == 0).all()
    g.assert_intact()


def test_attention_f32_output_stays_inside():
    w = wl.attention_workload("t", 53, 1, 3, 3, 77, 90, 64, wl.MASK_CAUSAL, 0.125, "f32")
    g = Guarded((1, 3, 77, 64), torch.float32)
    binding.attn_fused_f32(to_device(w.q), to_device(w.k), to_device(w.v), w.mask_kind, None, w.scale, out=g.tensor)
    binding.check_status()
    assert_close_f32(g.tensor, oracle.attn(w.q.values, w.k.values, w.v.values, w.mask_kind, None, w.scale))
    g.assert_intact()


@pytest.mark.parametrize("M,N,K", [(200, 200, 72), (1, 8, 8), (129, 264, 64), (300, 3080, 128)])
def test_linear_output_stays_inside(M, N, K):
    w = wl.linear_workload("t", 54, M, N, K, w_std=1.0 / np.sqrt(K), b_std=0.5)
    g = Guarded((M, N), torch.bfloat16)
    binding.linear_bias_gelu(to_device(w.x), to_device(w.w), to_device(w.b), out=g.tensor)
    binding.check_status()
    assert_close_bf16(g.tensor, oracle.linear_bias_gelu(w.x.values, w.w.values, w.b.values))
    g.assert_intact()


def test_swiglu_output_stays_inside():
    M, N, K = 200, 136, 72
    x = wl.normal_tensor(55, (M, K), "bf16")
    wg = wl.normal_tensor(56, (K, N), "bf16", std=1.0 / np.sqrt(K))
    wu = wl.normal_tensor(57, (K, N), "bf16", std=1.0 / np.sqrt(K))
    g = Guarded((M, N), torch.bfloat16)
    binding.linear_swiglu(to_device(x), to_device(wg), to_device(wu), out=g.tensor)
    binding.check_status()
    ref = oracle.linear_swiglu(x.values, wg.values, wu.values)
    err = np.abs(g.tensor.float().cpu().double().numpy() - ref)
    assert np.all(err <= 2e-2 + 2.0 ** -8 * np.abs(ref))
    g.assert_intact()


@pytest.mark.parametrize("D,Hq,Hkv,splits,lens", [
    (96, 8, 2, 5, [1, 300, 17]),
    (128, 8, 2, 16, [1, 3, 0, 64, 1000]),   # empty splits, a sequence of zero rows, lens beyond Smax
    (64, 6, 2, 7, [64, 33]),
    (40, 4, 4, 3, [5, 64, 31]),
])
def test_decode_output_and_workspace_stay_inside(D, Hq, Hkv, splits, lens):
    B, Smax = len(lens), 64 if max(lens) <= 64 or max(lens) == 1000 else 300
    w = wl.decode_workload("t", 58, B, Hq, Hkv, Smax, D, splits, 1.0 / np.sqrt(D), (1, Smax))
    w.lens = np.array(lens, dtype=np.int32)
    out = Guarded((B, Hq, D), torch.bfloat16)
    ws = Guarded((binding.attn_decode_workspace_bytes(B, Hq, D, splits),), torch.uint8)
    binding.attn_decode_workspace_init(ws.tensor)
    binding.attn_decode_splitkv(to_device(w.q), to_device(w.k_cache), to_device(w.v_cache),
                                torch.from_numpy(w.lens).cuda(), splits, w.scale, out=out.tensor, workspace=ws.tensor)
    binding.check_status()
    assert_close_bf16(out.tensor, oracle.attn_decode(w.q.values, w.k_cache.values, w.v_cache.values, w.lens, w.scale))
    out.assert_intact()
    ws.assert_intact()
