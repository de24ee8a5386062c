"""Do the pins have teeth?  Each case plants one plausible mistake in a copy of the oracle's C source
(on the CPU, never in the product), builds it, and runs a compact set of the pins against it: at least
one pin must fail.  The unmodified source must pass the same set."""
import math
import os
import subprocess

import numpy as np
import pytest
import torch

import oracle
from oracle import ref

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "forge_ref.c")
RNG = np.random.default_rng(99)

MUTANTS = {
    "sign of the exponent": ("p[j] = exp(p[j] - m);", "p[j] = exp(m - p[j]);"),
    "scale dropped": ("        s *= scale;\n", ""),
    "causal off by one": ("j > i + (Skv - Sq)", "j >= i + (Skv - Sq)"),
    "causal aligned top-left": ("j > i + (Skv - Sq)", "j > i"),
    "interleaved GQA mapping": ("const int kvh = h / G;", "const int kvh = h % Hkv;"),
    "lens ignored": ("    if (mask_kind & 2) {\n        n = lens[b];", "    if (0) {\n        n = lens[b];"),
    "K used for V": ("const double *vmat = v + ", "const double *vmat = k + "),
    "no normalisation": ("        p[j] /= denom;\n", ""),
    "K indexed transposed": ("kmat[(size_t)j * D + d]", "kmat[(size_t)d * Skv + j]"),
    "max not subtracted": ("if (!any || s > m) m = s;", "m = 0.0;"),
    "GELU cubic coefficient": ("0.044715 * z * z * z", "0.44715 * z * z * z"),
    "GELU erf form": ("0.5 * z * (1.0 + tanh(c * (z + 0.044715 * z * z * z)))", "0.5 * z * (1.0 + erf(z / sqrt(2.0)))"),
    "GELU missing half": ("return 0.5 * z *", "return z *"),
    "W indexed [N,K]": ("w[(size_t)kk * N + n]", "w[(size_t)n * K + kk]"),
    "bias dropped": ("forge_ref_gelu_tanh(acc + b[n])", "forge_ref_gelu_tanh(acc)"),
    "bias indexed by row": ("forge_ref_gelu_tanh(acc + b[n])", "forge_ref_gelu_tanh(acc + b[m % N])"),
    "swiglu gate and up swapped": ("y[(size_t)m * N + n] = gate / (1.0 + exp(-gate)) * up;", "y[(size_t)m * N + n] = up / (1.0 + exp(-up)) * gate;"),
    "swiglu product dropped": ("gate / (1.0 + exp(-gate)) * up;", "gate / (1.0 + exp(-gate));"),
    "swiglu sigmoid instead of silu": ("gate / (1.0 + exp(-gate)) * up;", "1.0 / (1.0 + exp(-gate)) * up;"),
    "swiglu up weights transposed": ("up += x[(size_t)m * K + kk] * wu[wi];", "up += x[(size_t)m * K + kk] * wu[w_layout == 0 ? (size_t)n * K + kk : (size_t)kk * N + n];"),
    "w8 scale dropped": ("            z *= scale[n];\n", ""),
    "w8 scale after the bias": ("            z *= scale[n];\n            if (b) z += b[n];", "            if (b) z += b[n];\n            z *= scale[n];"),
    "w8 scale indexed by row": ("z *= scale[n];", "z *= scale[m % N];"),
    "w8 weights read as [K,N]": ("wq[(size_t)n * K + kk]", "wq[(size_t)kk * N + n]"),
    "attention bias dropped": ("        if (bias_row) s += bias_row[j];\n", ""),
    "attention bias scaled": ("        s *= scale;\n        if (bias_row) s += bias_row[j];", "        if (bias_row) s += bias_row[j];\n        s *= scale;"),
    "attention bias subtracted": ("if (bias_row) s += bias_row[j];", "if (bias_row) s -= bias_row[j];"),
    "attention bias of another head": ("(Hb == 1 ? 0 : h)) * (size_t)Sq + i)", "(Hb == 1 ? 0 : (h + 1) % Hq)) * (size_t)Sq + i)"),
    "attention bias transposed": ("(Hb == 1 ? 0 : h)) * (size_t)Sq + i) * (size_t)Skv", "(Hb == 1 ? 0 : h)) * (size_t)Sq) * (size_t)Skv + i"),
}


def _pins():
    """A compact version of the pins in test_oracle_attention.py / test_oracle_linear.py."""
    ln = math.log
    # hand examples (exact rational weights)
    q = np.array([[[[1.0, 2.0]]]]); k = np.array([[[[0.0, 0.0], [ln(3), 0.0]]]]); v = np.array([[[[1.0, 2.0], [5.0, -2.0]]]])
    np.testing.assert_allclose(oracle.attn(q, k, v, 0, None, 1.0), [[[[4.0, -1.0]]]], atol=1e-14)
    q = np.array([[[[2.0]]]]); k = np.array([[[[0.0], [ln(3)]]]]); v = np.array([[[[8.0], [0.0]]]])
    np.testing.assert_allclose(oracle.attn(q, k, v, 0, None, 0.5), [[[[2.0]]]], atol=1e-14)
    q = np.ones((1, 1, 2, 1)); k = np.array([[[[0.0], [ln(3)], [ln(4)]]]]); v = np.array([[[[1.0], [5.0], [9.0]]]])
    np.testing.assert_allclose(oracle.attn(q, k, v, 1, None, 1.0), [[[[4.0], [6.5]]]], atol=1e-14)
    # padding and clamping
    q = RNG.standard_normal((2, 2, 3, 4)); k = RNG.standard_normal((2, 2, 5, 4)); v = RNG.standard_normal((2, 2, 5, 4))
    out = oracle.attn(q, k, v, 2, np.array([1, 99], dtype=np.int32), 0.7)
    np.testing.assert_allclose(out[0], np.broadcast_to(v[0, :, :1], out[0].shape), atol=1e-14)
    np.testing.assert_allclose(out[1], oracle.attn(q[1:], k[1:], v[1:], 0, None, 0.7)[0], atol=1e-14)
    # large scores stay finite and select the arg-max value
    big = oracle.attn(q, k, v, 0, None, 1e4)
    assert np.isfinite(big).all()
    best = np.einsum("bhid,bhjd->bhij", q, k).argmax(-1)
    np.testing.assert_allclose(big[0, 0, 0], v[0, 0, best[0, 0, 0]], atol=1e-9)
    # GQA grouping = MHA on repeated KV
    q8 = RNG.standard_normal((1, 4, 3, 4)); k2 = RNG.standard_normal((1, 2, 3, 4)); v2 = RNG.standard_normal((1, 2, 3, 4))
    np.testing.assert_allclose(oracle.attn(q8, k2, v2, 0, None, 0.5),
                               oracle.attn(q8, np.repeat(k2, 2, 1), np.repeat(v2, 2, 1), 0, None, 0.5), atol=1e-14)
    # library second opinion
    tq, tk, tv = (torch.from_numpy(a) for a in (q, k, v))
    ref_out = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=0.4).numpy()
    np.testing.assert_allclose(oracle.attn(q, k, v, 0, None, 0.4), ref_out, atol=1e-13)
    # additive bias tensor: exact hand weights, unscaled, per head, -inf excludes (also a whole row)
    q0 = np.zeros((1, 2, 2, 2)); kb = RNG.standard_normal((1, 1, 3, 2)); vb = np.array([[[[8.0, 0.0], [0.0, 8.0], [16.0, 16.0]]]])
    bias = np.zeros((1, 2, 2, 3)); bias[0, 1, 1] = [0.0, ln(2), ln(5)]; bias[0, 0, 1] = [0.0, -np.inf, -np.inf]
    bias[0, 1, 0] = -np.inf
    ob = oracle.attn_bias(q0, kb, vb, bias, 0, None, 0.37)
    np.testing.assert_allclose(ob[0, 1, 1], [11.0, 12.0], atol=1e-14)
    np.testing.assert_allclose(ob[0, 0, 1], [8.0, 0.0], atol=1e-14)
    np.testing.assert_allclose(ob[0, 0, 0], [8.0, 8.0], atol=1e-14)
    assert np.all(ob[0, 1, 0] == 0.0)
    q1 = np.array([[[[1.0]]]]); k1 = np.array([[[[0.0], [2 * ln(3)]]]]); v1 = np.array([[[[10.0], [0.0]]]])
    np.testing.assert_allclose(oracle.attn_bias(q1, k1, v1, np.array([[[[ln(2), 0.0]]]]), 0, None, 0.5), [[[[4.0]]]], atol=1e-14)
    # gated MLP input: hand values (silu(ln 3) = 0.75 ln 3) and torch's silu on non-square weights
    np.testing.assert_allclose(oracle.linear_swiglu(np.array([[1.0]]), np.array([[ln(3), 0.0]]), np.array([[2.0, 5.0]])),
                               [[1.5 * ln(3), 0.0]], atol=1e-15)
    xs = RNG.standard_normal((4, 5)); gs = RNG.standard_normal((5, 3)); us = RNG.standard_normal((5, 3))
    np.testing.assert_allclose(oracle.linear_swiglu(xs, gs, us),
                               (torch.nn.functional.silu(torch.from_numpy(xs @ gs)) * torch.from_numpy(xs @ us)).numpy(), atol=1e-13)
    # weight-only int8: hand value, and the dense linear on the dequantised weights (non-square)
    np.testing.assert_array_equal(oracle.linear_w8(np.array([[2.0, 5.0]]), np.array([[3.0, -2.0], [1.0, 1.0]]),
                                                   np.array([0.5, -1.0]), np.array([3.0, 0.0]), None, oracle.ACT_RELU), [[1.0, 0.0]])
    xq = RNG.standard_normal((4, 6)); wq = RNG.integers(-128, 128, size=(3, 6)).astype(np.float64); sq = np.array([0.25, 0.5, 0.125])
    np.testing.assert_allclose(oracle.linear_w8(xq, wq, sq, np.ones(3), None, oracle.ACT_NONE),
                               xq @ (wq * sq[:, None]).T + 1.0, atol=1e-13)
    # GELU and linear
    assert abs(oracle.gelu_tanh(1.0) - 0.841192) < 5e-7
    assert abs(oracle.gelu_tanh(3.0) - oracle.gelu_tanh(-3.0) - 3.0) < 1e-14
    x = RNG.standard_normal((4, 5)); w = RNG.standard_normal((5, 3)); b = RNG.standard_normal(3)
    want = torch.nn.functional.gelu(torch.from_numpy(x @ w + b), approximate="tanh").numpy()
    np.testing.assert_allclose(oracle.linear_bias_gelu(x, w, b), want, atol=1e-13)


def _build(tmp_path, name, source):
    c = tmp_path / f"{name}.c"
    so = tmp_path / f"{name}.so"
    c.write_text(source)
    subprocess.run(["gcc", "-O1", "-shared", "-fPIC", "-o", str(so), str(c), "-lm"], check=True)
    return str(so)


def test_unmodified_oracle_passes_the_compact_pins(tmp_path):
    try:
        ref.use_library(_build(tmp_path, "clean", open(SRC).read()))
        _pins()
    finally:
        ref.use_library(None)
    _pins()


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(tmp_path, name):
    old, new = MUTANTS[name]
    source = open(SRC).read()
    assert source.count(old) >= 1, f"pattern for '{name}' no longer in the oracle source"
    so = _build(tmp_path, "mutant", source.replace(old, new, 1))
    try:
        ref.use_library(so)
        with pytest.raises((AssertionError, ValueError)):
            _pins()
    finally:
        ref.use_library(None)
