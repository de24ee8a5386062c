"""GPU parity: forge_decoder_layer (fused QKV projection, strided attention, mm+add, gated or GELU MLP, mm+add in
planned buffers) against the layer oracle, on a GPT-2-small-shaped and an 8B-class-shaped layer."""
import numpy as np
import pytest
import torch

from oracle import layer as olayer
from paper_2604_16498_b200 import binding, workloads as wl
from util import Guarded, to_f64

pytestmark = pytest.mark.gpu


def _draw(gen, shape, std):
    """bf16 values drawn on the CPU from a seeded torch generator; (fp64 numpy for the oracle, CUDA bf16 tensor)."""
    t = (torch.randn(shape, generator=gen, dtype=torch.float32) * std).to(torch.bfloat16)
    return t.to(torch.float64).numpy(), t.cuda()


def _layer_case(seed, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, biases):
    gen = torch.Generator().manual_seed(seed)
    H, Nqkv = Hq * D, (Hq + 2 * Hkv) * D
    shape = (lambda k, n: (k, n)) if w_layout == binding.W_KN else (lambda k, n: (n, k))
    host, dev = {}, {}
    specs = [("w_qkv", shape(H, Nqkv), H ** -0.5), ("w_o", shape(H, H), H ** -0.5), ("w_up", shape(H, F), H ** -0.5),
             ("w_down", shape(F, H), F ** -0.5)]
    if mlp_kind == binding.MLP_SWIGLU:
        specs.append(("w_gate", shape(H, F), H ** -0.5))
    if biases:
        specs += [("b_qkv", (Nqkv,), 0.1), ("b_o", (H,), 0.1), ("b_down", (H,), 0.1)]
        if mlp_kind == binding.MLP_GELU:
            specs.append(("b_up", (F,), 0.1))
    for name, shp, std in specs:
        host[name], dev[name] = _draw(gen, shp, std)
    x_host, x_dev = _draw(gen, (B * S, H), 1.0)
    return x_host, x_dev, host, dev


def _check(y, ref):
    got = to_f64(y)
    assert np.isfinite(got).all()
    err = np.abs(got - ref)
    # The bf16 tolerances (max-abs 2e-2, mean-abs 2e-3) are stated for unit-variance data.  The layer's output
    # carries two residual additions, has a root mean square r above 1 and reaches |y| = 7, where one bf16 ulp is
    # 0.031.  Five operators with four bf16 tensors between them: an intermediate that rounds the other way on the
    # GPU moves an output by up to one ulp of the output, on top of the output's own half ulp.  So the bounds
    # scale: 1.5 ulp (ulp <= 2^-7 |y|) on top of the absolute 2e-2, and r times the mean.
    rms = max(1.0, float(np.sqrt(np.mean(ref ** 2))))
    assert np.all(err <= 2e-2 + 1.5 * 2.0 ** -7 * np.abs(ref)), f"max-abs {err.max():.3e}"
    assert err.mean() <= 2e-3 * rms, f"mean-abs {err.mean():.3e} (rms of the reference {rms:.2f})"


@pytest.mark.parametrize("name,B,S,Hq,Hkv,D,F,mlp_kind,w_layout,mask_kind,biases", [
    ("gpt2_small", 2, 300, 12, 12, 64, 3072, binding.MLP_GELU, binding.W_KN, wl.MASK_CAUSAL, True),
    ("8b_class", 2, 160, 32, 8, 128, 14336, binding.MLP_SWIGLU, binding.W_NK, wl.MASK_CAUSAL, False),
    ("padded_small", 3, 100, 8, 2, 40, 264, binding.MLP_SWIGLU, binding.W_KN, wl.MASK_CAUSAL_PADDING, False),
])
def test_layer_matches_the_oracle(name, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, biases):
    x_host, x_dev, host, dev = _layer_case(1234, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, biases)
    lens_np = np.array([S, max(1, S // 3), 1], dtype=np.int32)[:B] if mask_kind & wl.MASK_PADDING else None
    lens = None if lens_np is None else torch.from_numpy(lens_np).cuda()
    plan = binding.decoder_layer_plan(B, S, Hq, Hkv, D, F, mlp_kind)
    ws = Guarded((plan.workspace_bytes,), torch.uint8)
    out = Guarded((B * S, Hq * D), torch.bfloat16)
    binding.decoder_layer(x_dev, dev, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, D ** -0.5, lens,
                          out=out.tensor, workspace=ws.tensor)
    binding.check_status()
    ref = olayer.decoder_layer(x_host, host, B, S, Hq, Hkv, D, F, mlp_kind, w_layout, mask_kind, D ** -0.5, lens_np)
    _check(out.tensor, ref)
    out.assert_intact()
    ws.assert_intact()   # the planned buffers are all the layer touches
    assert plan.num_bufs == 2 and plan.workspace_bytes < plan.unplanned_bytes


def test_two_runs_are_bitwise_identical_and_the_workspace_can_be_reused():
    B, S, Hq, Hkv, D, F = 1, 256, 8, 2, 128, 1024
    x_host, x_dev, host, dev = _layer_case(77, B, S, Hq, Hkv, D, F, binding.MLP_SWIGLU, binding.W_KN, False)
    ws = torch.empty(binding.decoder_layer_plan(B, S, Hq, Hkv, D, F).workspace_bytes, dtype=torch.uint8, device="cuda")
    a = binding.decoder_layer(x_dev, dev, B, S, Hq, Hkv, D, F, workspace=ws)
    b = binding.decoder_layer(x_dev, dev, B, S, Hq, Hkv, D, F, workspace=ws)
    assert torch.equal(a, b)


def test_workspace_too_small_is_refused():
    B, S, Hq, Hkv, D, F = 1, 128, 4, 4, 64, 512
    x_host, x_dev, host, dev = _layer_case(78, B, S, Hq, Hkv, D, F, binding.MLP_SWIGLU, binding.W_KN, False)
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.ForgeError) as e:
        binding.decoder_layer(x_dev, dev, B, S, Hq, Hkv, D, F, workspace=ws)
    assert e.value.status == binding.ERR_WORKSPACE
