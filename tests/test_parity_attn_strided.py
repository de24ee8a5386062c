"""GPU parity: forge_attn_fused_strided (views of a fused QKV projection, token-major output) against the
fp64 oracle on the same values in dense layout."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16498_b200 import binding, workloads as wl
from util import Guarded, assert_close_bf16, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,Hq,Hkv,S,D,mask_kind", [
    (2, 8, 2, 300, 128, wl.MASK_CAUSAL),
    (3, 12, 12, 200, 64, wl.MASK_PADDING),
    (2, 6, 2, 130, 40, wl.MASK_CAUSAL_PADDING),
    (1, 4, 4, 77, 96, wl.MASK_NONE),
])
def test_views_of_a_fused_qkv_buffer(B, Hq, Hkv, S, D, mask_kind):
    """q, k, v are column slices of one [B*S, (Hq + 2 Hkv) D] buffer seen as [B, heads, S, D]; the output goes
    to a [B*S, Hq D] buffer seen the same way."""
    w = wl.attention_workload("t", 71, B, Hq, Hkv, S, S, D, mask_kind, 1.0 / np.sqrt(D), "bf16", lens_range=(1, S))
    n_tot = (Hq + 2 * Hkv) * D
    qkv = torch.empty((B, S, n_tot), dtype=torch.bfloat16, device="cuda")
    qkv[:, :, :Hq * D] = to_device(w.q).permute(0, 2, 1, 3).reshape(B, S, Hq * D)
    qkv[:, :, Hq * D:(Hq + Hkv) * D] = to_device(w.k).permute(0, 2, 1, 3).reshape(B, S, Hkv * D)
    qkv[:, :, (Hq + Hkv) * D:] = to_device(w.v).permute(0, 2, 1, 3).reshape(B, S, Hkv * D)
    q = qkv[:, :, :Hq * D].view(B, S, Hq, D).permute(0, 2, 1, 3)
    k = qkv[:, :, Hq * D:(Hq + Hkv) * D].view(B, S, Hkv, D).permute(0, 2, 1, 3)
    v = qkv[:, :, (Hq + Hkv) * D:].view(B, S, Hkv, D).permute(0, 2, 1, 3)
    g = Guarded((B, S, Hq * D), torch.bfloat16)
    out = g.tensor.view(B, S, Hq, D).permute(0, 2, 1, 3)
    lens = None if w.lens is None else torch.from_numpy(w.lens).cuda()
    binding.attn_fused_strided(q, k, v, out, mask_kind, lens, w.scale)
    binding.check_status()
    ref = oracle.attn(w.q.values, w.k.values, w.v.values, mask_kind, w.lens, w.scale)
    assert_close_bf16(out.contiguous(), ref)
    g.assert_intact()


def test_dense_strides_give_the_dense_entry_points_result():
    w = wl.attention_workload("t", 72, 2, 4, 2, 260, 260, 64, wl.MASK_CAUSAL, 0.125, "bf16")
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    a = binding.attn_fused(q, k, v, w.mask_kind, None, w.scale)
    b = torch.empty_like(q)
    binding.attn_fused_strided(q, k, v, b, w.mask_kind, None, w.scale)
    assert torch.equal(a, b)


def test_bad_strides_are_refused():
    w = wl.attention_workload("t", 73, 1, 2, 2, 64, 64, 64, 0, 0.125, "bf16")
    q, k, v = to_device(w.q), to_device(w.k), to_device(w.v)
    out = torch.empty_like(q)
    lib = binding.load()
    import ctypes
    ok = (ctypes.c_int64 * 3)(2 * 64 * 64, 64 * 64, 64)
    bad_row = (ctypes.c_int64 * 3)(2 * 64 * 64, 64 * 64, 60)     # rows would overlap
    odd = (ctypes.c_int64 * 3)(2 * 64 * 64 + 4, 64 * 64, 64)     # not a multiple of 8 elements
    call = lambda sq: lib.forge_attn_fused_strided(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), 1, 2, 2, 64, 64,
                                                    64, sq, ok, ok, ok, 0, None, 0.125, None)
    assert call(bad_row) == binding.ERR_INVALID_ARG
    assert call(odd) == binding.ERR_UNSUPPORTED
    assert call(None) == binding.ERR_INVALID_ARG
