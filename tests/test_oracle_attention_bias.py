"""Pins for the oracle's attention with an additive bias tensor (the optional mask node of Eq. 8 as a
tensor): s = scale * q.k + bias, -inf excludes a key.  None of these retypes the oracle's formula: they
are exact hand values, reductions to the already pinned mask kinds, an independent library routine
(torch CPU fp64 SDPA with attn_mask) and invariants."""
import math

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(7)


def _rand(B=2, Hq=4, Hkv=2, Sq=5, Skv=7, D=3):
    return (RNG.standard_normal((B, Hq, Sq, D)), RNG.standard_normal((B, Hkv, Skv, D)),
            RNG.standard_normal((B, Hkv, Skv, D)))


def test_hand_example_weights_are_exp_of_bias():
    """q = 0: the weights are softmax(bias).  bias = (ln 1, ln 2, ln 5) gives 1/8, 2/8, 5/8."""
    q = np.zeros((1, 1, 1, 2)); k = RNG.standard_normal((1, 1, 3, 2))
    v = np.array([[[[8.0, 0.0], [0.0, 8.0], [16.0, 16.0]]]])
    bias = np.array([[[[0.0, math.log(2), math.log(5)]]]])
    out, probs = oracle.attn_bias(q, k, v, bias, 0, None, 0.37, return_probs=True)
    np.testing.assert_allclose(probs[0, 0, 0], [0.125, 0.25, 0.625], atol=1e-15)
    np.testing.assert_allclose(out[0, 0, 0], [11.0, 12.0], atol=1e-14)


def test_hand_example_bias_adds_to_scaled_score():
    """q.k = ln 3 for key 1 (scale 1), bias ln 2 on key 0: weights 2 : 3."""
    q = np.array([[[[1.0]]]]); k = np.array([[[[0.0], [math.log(3)]]]]); v = np.array([[[[10.0], [0.0]]]])
    bias = np.array([[[[math.log(2), 0.0]]]])
    np.testing.assert_allclose(oracle.attn_bias(q, k, v, bias, 0, None, 1.0), [[[[4.0]]]], atol=1e-14)
    # the bias is not scaled: with scale 0.5 and q.k = 2 ln 3 the result is the same
    k2 = np.array([[[[0.0], [2 * math.log(3)]]]])
    np.testing.assert_allclose(oracle.attn_bias(q, k2, v, bias, 0, None, 0.5), [[[[4.0]]]], atol=1e-14)


def test_zero_bias_is_no_bias():
    q, k, v = _rand()
    for mk, lens in ((0, None), (1, None), (2, np.array([3, 7], dtype=np.int32))):
        np.testing.assert_array_equal(oracle.attn_bias(q, k, v, np.zeros((2, 1, 5, 7)), mk, lens, 0.6),
                                      oracle.attn(q, k, v, mk, lens, 0.6))


def test_minus_inf_bias_reproduces_the_mask_kinds():
    """A causal (bottom-right aligned) or key-padding pattern written as a 0 / -inf tensor gives exactly
    what the corresponding mask kind gives (those are pinned in test_oracle_attention.py)."""
    q, k, v = _rand()
    i = np.arange(5)[:, None]; j = np.arange(7)[None, :]
    causal = np.where(j <= i + 2, 0.0, -np.inf)[None, None].repeat(2, axis=0)
    np.testing.assert_array_equal(oracle.attn_bias(q, k, v, causal, 0, None, 0.6), oracle.attn(q, k, v, 1, None, 0.6))
    lens = np.array([3, 6], dtype=np.int32)
    pad = np.where(j < lens[:, None, None, None], 0.0, -np.inf) + np.zeros((2, 1, 5, 7))
    np.testing.assert_array_equal(oracle.attn_bias(q, k, v, pad, 0, None, 0.6), oracle.attn(q, k, v, 2, lens, 0.6))
    # and the kinds still apply on top of a bias
    np.testing.assert_array_equal(oracle.attn_bias(q, k, v, pad, 1, None, 0.6), oracle.attn(q, k, v, 3, lens, 0.6))


def test_row_without_visible_key_gives_zeros():
    q, k, v = _rand()
    bias = np.zeros((2, 4, 5, 7)); bias[1, 2, 3, :] = -np.inf
    out, probs = oracle.attn_bias(q, k, v, bias, 0, None, 1.0, return_probs=True)
    assert np.all(out[1, 2, 3] == 0.0) and np.all(probs[1, 2, 3] == 0.0)
    assert np.isfinite(out).all()
    np.testing.assert_allclose(probs.sum(-1)[0], 1.0, atol=1e-14)


@pytest.mark.parametrize("Hb", [1, 4])
def test_against_torch_cpu_sdpa_with_attn_mask(Hb):
    """Independent library routine: torch's CPU fp64 scaled_dot_product_attention with a float attn_mask."""
    q, k, v = _rand(B=2, Hq=4, Hkv=2, Sq=6, Skv=9, D=8)
    bias = RNG.standard_normal((2, Hb, 6, 9))
    bias[RNG.random(bias.shape) < 0.2] = -np.inf
    bias[..., 0] = 0.0  # keep every row alive (torch gives NaN for an empty row)
    kt = torch.from_numpy(k).repeat_interleave(2, dim=1); vt = torch.from_numpy(v).repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q), kt, vt,
                                                           attn_mask=torch.from_numpy(bias), scale=0.45)
    np.testing.assert_allclose(oracle.attn_bias(q, k, v, bias, 0, None, 0.45), ref.numpy(), atol=1e-13)


def test_per_row_constant_leaves_the_result_unchanged_and_heads_are_not_mixed_up():
    q, k, v = _rand()
    bias = RNG.standard_normal((2, 4, 5, 7))
    base = oracle.attn_bias(q, k, v, bias, 0, None, 0.8)
    shifted = bias + RNG.standard_normal((2, 4, 5, 1))
    np.testing.assert_allclose(oracle.attn_bias(q, k, v, shifted, 0, None, 0.8), base, atol=1e-13)
    # a bias that differs between heads must change only that head, that batch entry, that row
    b2 = bias.copy(); b2[1, 3, 2, 4] += 1.5
    out2 = oracle.attn_bias(q, k, v, b2, 0, None, 0.8)
    changed = np.abs(out2 - base).max(-1) > 1e-12
    expect = np.zeros_like(changed); expect[1, 3, 2] = True
    assert np.array_equal(changed, expect)
    # per-key bias shared by all heads (Hb = 1) equals the same bias repeated per head
    shared = RNG.standard_normal((2, 1, 5, 7))
    np.testing.assert_array_equal(oracle.attn_bias(q, k, v, shared, 0, None, 0.8),
                                  oracle.attn_bias(q, k, v, np.repeat(shared, 4, axis=1), 0, None, 0.8))
