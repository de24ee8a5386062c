"""CPU oracle for the decoder layer built from the fused operators.  Test infrastructure only.

The layer is a fixed composition of the already defined operators (fused linear, fused attention, gated
or GELU MLP input, mm+add), each taken from this package's fp64 oracle.  The tensors that pass from one
operator to the next are 16-bit tensors by the operators' interfaces, so each intermediate is rounded to
bf16 (round to nearest even) before the next operator reads it, exactly where the interface puts a bf16
tensor.
"""
from __future__ import annotations

import numpy as np

from . import ref

MLP_SWIGLU, MLP_GELU = 0, 1


def round_bf16(a):
    """fp64 -> nearest bf16 (ties to even), returned as fp64."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32)
    r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)) << np.uint32(16)
    return r.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


def decoder_layer(x, w, B, S, Hq, Hkv, D, F, mlp_kind=MLP_SWIGLU, w_layout=0, mask_kind=1, scale=None, lens=None):
    """x [B*S, Hq*D]; w: dict with w_qkv, w_o, w_up, w_down, w_gate (gated form) and optional biases, as fp64
    arrays holding bf16 values, weights [in, out] (w_layout 0) or [out, in] (w_layout 1)."""
    scale = D ** -0.5 if scale is None else scale
    T, H = B * S, Hq * D
    qkv = round_bf16(ref.linear_act(x, w["w_qkv"], w.get("b_qkv"), None, ref.ACT_NONE, w_layout))
    q = qkv[:, :H].reshape(B, S, Hq, D).transpose(0, 2, 1, 3)
    k = qkv[:, H:H + Hkv * D].reshape(B, S, Hkv, D).transpose(0, 2, 1, 3)
    v = qkv[:, H + Hkv * D:].reshape(B, S, Hkv, D).transpose(0, 2, 1, 3)
    a = ref.attn(q, k, v, mask_kind, lens, scale)                       # [B, Hq, S, D]
    attn = round_bf16(a.transpose(0, 2, 1, 3).reshape(T, H))
    h1 = round_bf16(ref.linear_act(attn, w["w_o"], w.get("b_o"), x, ref.ACT_NONE, w_layout))
    if mlp_kind == MLP_SWIGLU:
        g = round_bf16(ref.linear_swiglu(h1, w["w_gate"], w["w_up"], w_layout))
    else:
        g = round_bf16(ref.linear_act(h1, w["w_up"], w.get("b_up"), None, ref.ACT_GELU_TANH, w_layout))
    return ref.linear_act(g, w["w_down"], w.get("b_down"), h1, ref.ACT_NONE, w_layout)
