"""Pin of the decoder-layer oracle (oracle/layer.py): an independent restatement with torch CPU fp64 routines
(matmul, softmax, silu, gelu) and torch's own bf16 rounding at the same places, on small shapes."""
import numpy as np
import pytest
import torch

from oracle import layer as olayer
from paper_2604_16498_b200 import workloads as wl


def _bf(t):
    return t.to(torch.bfloat16).to(torch.float64)


def _torch_layer(x, w, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, scale, lens):
    x = torch.from_numpy(x)
    W = {k: torch.from_numpy(v) for k, v in w.items() if v is not None}
    mm = (lambda a, m: a @ m) if w_layout == 0 else (lambda a, m: a @ m.T)
    bias = lambda n: W[n] if n in W else 0.0
    T, H, G = B * S, Hq * D, Hq // Hkv
    qkv = _bf(mm(x, W["w_qkv"]) + bias("b_qkv"))
    q = qkv[:, :H].reshape(B, S, Hq, D).permute(0, 2, 1, 3)
    k = qkv[:, H:H + Hkv * D].reshape(B, S, Hkv, D).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    v = qkv[:, H + Hkv * D:].reshape(B, S, Hkv, D).permute(0, 2, 1, 3).repeat_interleave(G, dim=1)
    s = scale * (q @ k.transpose(-1, -2))
    allowed = torch.ones(B, 1, S, S, dtype=torch.bool)
    if mask_kind & 1:
        allowed &= torch.tril(torch.ones(S, S, dtype=torch.bool))
    if mask_kind & 2:
        allowed &= (torch.arange(S)[None, :] < torch.from_numpy(lens)[:, None])[:, None, None, :]
    p = torch.softmax(s.masked_fill(~allowed, float("-inf")), dim=-1)
    attn = _bf((p @ v).permute(0, 2, 1, 3).reshape(T, H))
    h1 = _bf(mm(attn, W["w_o"]) + bias("b_o") + x)
    if mlp_kind == olayer.MLP_SWIGLU:
        g = _bf(torch.nn.functional.silu(mm(h1, W["w_gate"])) * mm(h1, W["w_up"]))
    else:
        g = _bf(torch.nn.functional.gelu(mm(h1, W["w_up"]) + bias("b_up"), approximate="tanh"))
    return (mm(g, W["w_down"]) + bias("b_down") + h1).numpy()


def _weights(seed, H, Nqkv, F, mlp_kind, w_layout, biases):
    shape = (lambda k, n: (k, n)) if w_layout == 0 else (lambda k, n: (n, k))
    w = {"w_qkv": wl.normal_tensor(seed, shape(H, Nqkv), "bf16", H ** -0.5).values,
         "w_o": wl.normal_tensor(seed + 1, shape(H, H), "bf16", H ** -0.5).values,
         "w_up": wl.normal_tensor(seed + 2, shape(H, F), "bf16", H ** -0.5).values,
         "w_down": wl.normal_tensor(seed + 3, shape(F, H), "bf16", F ** -0.5).values}
    if mlp_kind == olayer.MLP_SWIGLU:
        w["w_gate"] = wl.normal_tensor(seed + 4, shape(H, F), "bf16", H ** -0.5).values
    if biases:
        w["b_qkv"] = wl.normal_tensor(seed + 5, (Nqkv,), "bf16", 0.1).values
        w["b_o"] = wl.normal_tensor(seed + 6, (H,), "bf16", 0.1).values
        w["b_down"] = wl.normal_tensor(seed + 7, (H,), "bf16", 0.1).values
        if mlp_kind == olayer.MLP_GELU:
            w["b_up"] = wl.normal_tensor(seed + 8, (F,), "bf16", 0.1).values
    return w


@pytest.mark.parametrize("mlp_kind,w_layout,mask_kind,biases", [
    (olayer.MLP_SWIGLU, 0, 1, False), (olayer.MLP_SWIGLU, 1, 3, False), (olayer.MLP_GELU, 0, 1, True), (olayer.MLP_GELU, 1, 2, True)])
def test_layer_oracle_against_torch_cpu(mlp_kind, w_layout, mask_kind, biases):
    B, S, Hq, Hkv, D, F = 2, 24, 4, 2, 16, 96
    H, Nqkv = Hq * D, (Hq + 2 * Hkv) * D
    x = wl.normal_tensor(900, (B * S, H), "bf16").values
    w = _weights(901, H, Nqkv, F, mlp_kind, w_layout, biases)
    lens = np.array([24, 7], dtype=np.int32) if mask_kind & 2 else None
    got = olayer.decoder_layer(x, w, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, 0.25, lens)
    want = _torch_layer(x, w, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, 0.25, lens)
    # identical rounding points; a rare intermediate may round the other way when the two fp64 evaluations
    # straddle a bf16 tie, which moves a few outputs by a fraction of a bf16 ulp of an input
    assert np.abs(got - want).max() <= 2e-3
    assert np.abs(got - want).mean() <= 1e-5


def test_rounding_helper_is_round_to_nearest_even():
    a = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -9, -3.14159, 0.0])
    want = torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(olayer.round_bf16(a), want)
