"""Pins for the attention oracle (CPU only).

The oracle is checked against things other than itself: hand-derived closed
forms (tests/golden/attn_hand_examples.txt), a dense brute-force evaluation
written a different way, algebraic invariants of Eq. 9, and torch's CPU fp64
scaled_dot_product_attention as an independent library routine.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "attn_hand_examples.txt")
RNG = np.random.default_rng(20260416)


def _num(tok):
    return math.log(float(tok[2:])) if tok.startswith("ln") else float(tok)


def _hand_examples():
    cases = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, mask, dims, scale, lens, q, k, v, exp = [s.strip() for s in line.split("|")]
            B, Hq, Hkv, Sq, Skv, D = map(int, dims.split())
            arr = lambda s, shape: np.array([_num(t) for t in s.split()], dtype=np.float64).reshape(shape)
            cases.append(pytest.param(
                int(mask), float(scale), None if lens == "-" else np.array(lens.split(), dtype=np.int32),
                arr(q, (B, Hq, Sq, D)), arr(k, (B, Hkv, Skv, D)), arr(v, (B, Hkv, Skv, D)),
                arr(exp, (B, Hq, Sq, D)), id=name))
    return cases


@pytest.mark.parametrize("mask,scale,lens,q,k,v,expected", _hand_examples())
def test_hand_examples(mask, scale, lens, q, k, v, expected):
    out = oracle.attn(q, k, v, mask, lens, scale)
    np.testing.assert_allclose(out, expected, rtol=0, atol=1e-14)


def _dense(q, k, v, mask_kind, lens, scale):
    """Brute force the other way round: materialise S with -inf, P, then matmul."""
    B, Hq, Sq, D = q.shape
    Hkv, Skv = k.shape[1], k.shape[2]
    G = Hq // Hkv
    out = np.zeros_like(q)
    probs = np.zeros((B, Hq, Sq, Skv))
    for b in range(B):
        for h in range(Hq):
            S = scale * (q[b, h] @ k[b, h // G].T)
            M = np.zeros((Sq, Skv), dtype=bool)
            if mask_kind & 1:
                M |= np.arange(Skv)[None, :] > (np.arange(Sq)[:, None] + Skv - Sq)
            if mask_kind & 2:
                M |= np.arange(Skv)[None, :] >= min(max(int(lens[b]), 0), Skv)
            S = np.where(M, -np.inf, S)
            rowmax = S.max(axis=1, keepdims=True)
            dead = ~np.isfinite(rowmax)
            E = np.exp(S - np.where(dead, 0.0, rowmax))
            E = np.where(M, 0.0, E)
            denom = E.sum(axis=1, keepdims=True)
            P = np.where(dead, 0.0, E / np.where(dead, 1.0, denom))
            probs[b, h] = P
            out[b, h] = P @ v[b, h // G]
    return out, probs


SHAPES = [  # B, Hq, Hkv, Sq, Skv, D
    (1, 1, 1, 1, 1, 1), (2, 4, 2, 8, 8, 4), (1, 4, 1, 5, 7, 3), (2, 2, 2, 7, 5, 4), (1, 6, 3, 3, 8, 2),
]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
def test_against_dense_brute_force(shape, mask_kind):
    B, Hq, Hkv, Sq, Skv, D = shape
    q = RNG.standard_normal((B, Hq, Sq, D))
    k = RNG.standard_normal((B, Hkv, Skv, D))
    v = RNG.standard_normal((B, Hkv, Skv, D))
    lens = RNG.integers(1, Skv + 1, size=B).astype(np.int32)
    out, probs = oracle.attn_probs(q, k, v, mask_kind, lens, 0.7)
    ref_out, ref_probs = _dense(q, k, v, mask_kind, lens, 0.7)
    np.testing.assert_allclose(out, ref_out, rtol=0, atol=1e-13)
    np.testing.assert_allclose(probs, ref_probs, rtol=0, atol=1e-14)
    np.testing.assert_array_equal(oracle.attn(q, k, v, mask_kind, lens, 0.7), out)


@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
def test_rows_sum_to_one_and_masked_are_exact_zero(mask_kind):
    B, Hq, Hkv, Sq, Skv, D = 2, 4, 2, 9, 12, 8
    q = RNG.standard_normal((B, Hq, Sq, D))
    k = RNG.standard_normal((B, Hkv, Skv, D))
    v = RNG.standard_normal((B, Hkv, Skv, D))
    lens = np.array([5, 12], dtype=np.int32)
    _, probs = oracle.attn_probs(q, k, v, mask_kind, lens, 0.35)
    np.testing.assert_allclose(probs.sum(-1), 1.0, rtol=0, atol=1e-15 * Skv)
    assert (probs >= 0).all()
    for b in range(B):
        for i in range(Sq):
            for j in range(Skv):
                masked = ((mask_kind & 1) and j > i + Skv - Sq) or ((mask_kind & 2) and j >= lens[b])
                if masked:
                    assert (probs[b, :, i, j] == 0.0).all()
                else:
                    assert (probs[b, :, i, j] > 0.0).all()


@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
def test_constant_v_rows_give_that_row(mask_kind):
    B, Hq, Hkv, Sq, Skv, D = 2, 4, 2, 6, 6, 5
    q = RNG.standard_normal((B, Hq, Sq, D))
    k = RNG.standard_normal((B, Hkv, Skv, D))
    c = RNG.standard_normal((B, Hkv, 1, D))
    v = np.broadcast_to(c, (B, Hkv, Skv, D)).copy()
    lens = np.array([3, 6], dtype=np.int32)
    out = oracle.attn(q, k, v, mask_kind, lens, 1.3)
    expect = np.repeat(c, Hq // Hkv, axis=1)
    np.testing.assert_allclose(out, np.broadcast_to(expect, out.shape), rtol=0, atol=1e-14)


@pytest.mark.parametrize("zero", ["q", "scale"])
def test_zero_scores_give_prefix_means(zero):
    B, H, S, D = 2, 3, 10, 4
    q = RNG.standard_normal((B, H, S, D))
    k = RNG.standard_normal((B, H, S, D))
    v = RNG.standard_normal((B, H, S, D))
    scale = 1.0
    if zero == "q":
        q = np.zeros_like(q)
    else:
        scale = 0.0
    out = oracle.attn(q, k, v, 1, None, scale)  # causal -> mean of V[0..i]
    prefix = np.cumsum(v, axis=2) / np.arange(1, S + 1)[None, None, :, None]
    np.testing.assert_allclose(out, prefix, rtol=0, atol=1e-14)
    lens = np.array([4, 10], dtype=np.int32)
    out = oracle.attn(q, k, v, 2, lens, scale)  # padding -> mean of V[0..len-1] for every row
    for b in range(B):
        m = v[b, :, :lens[b]].mean(axis=1, keepdims=True)
        np.testing.assert_allclose(out[b], np.broadcast_to(m, out[b].shape), rtol=0, atol=1e-14)


def test_shift_and_permutation_invariance():
    B, H, Sq, Skv, D = 1, 2, 5, 9, 6
    q = RNG.standard_normal((B, H, Sq, D))
    k = RNG.standard_normal((B, H, Skv, D))
    v = RNG.standard_normal((B, H, Skv, D))
    base = oracle.attn(q, k, v, 0, None, 0.5)
    u = RNG.standard_normal((1, 1, 1, D))
    np.testing.assert_allclose(oracle.attn(q, k + u, v, 0, None, 0.5), base, rtol=0, atol=1e-12)
    perm = RNG.permutation(Skv)
    np.testing.assert_allclose(oracle.attn(q, k[:, :, perm], v[:, :, perm], 0, None, 0.5), base,
                               rtol=0, atol=1e-13)
    # permuting keys without permuting values must change the result (guards a k/v mix-up)
    assert np.abs(oracle.attn(q, k[:, :, perm], v, 0, None, 0.5) - base).max() > 1e-3


def test_sharp_limit_selects_argmax_value():
    B, H, Sq, Skv, D = 1, 2, 4, 7, 3
    q = RNG.standard_normal((B, H, Sq, D))
    k = RNG.standard_normal((B, H, Skv, D))
    v = RNG.standard_normal((B, H, Skv, D))
    out = oracle.attn(q, k, v, 0, None, 1e4)
    best = np.einsum("bhid,bhjd->bhij", q, k).argmax(-1)
    for h in range(H):
        for i in range(Sq):
            np.testing.assert_allclose(out[0, h, i], v[0, h, best[0, h, i]], rtol=0, atol=1e-9)


def test_gqa_equals_mha_on_repeated_kv():
    B, Hq, Hkv, S, D = 2, 8, 2, 6, 4
    q = RNG.standard_normal((B, Hq, S, D))
    k = RNG.standard_normal((B, Hkv, S, D))
    v = RNG.standard_normal((B, Hkv, S, D))
    lens = np.array([6, 2], dtype=np.int32)
    gqa = oracle.attn(q, k, v, 3, lens, 0.5)
    mha = oracle.attn(q, np.repeat(k, Hq // Hkv, axis=1), np.repeat(v, Hq // Hkv, axis=1), 3, lens, 0.5)
    np.testing.assert_array_equal(gqa, mha)
    # the interleaved (h % Hkv) mapping is a different function: make sure we do not compute it
    wrong = oracle.attn(q, np.tile(k, (1, Hq // Hkv, 1, 1)), np.tile(v, (1, Hq // Hkv, 1, 1)), 3, lens, 0.5)
    assert np.abs(gqa - wrong).max() > 1e-3


@pytest.mark.parametrize("mask_kind", [0, 1, 2, 3])
@pytest.mark.parametrize("Sq,Skv", [(16, 16), (5, 16)])
def test_against_torch_cpu_sdpa(mask_kind, Sq, Skv):
    """Library second opinion: torch CPU fp64 SDPA with an explicit boolean mask."""
    B, Hq, Hkv, D = 2, 4, 2, 8
    q = RNG.standard_normal((B, Hq, Sq, D))
    k = RNG.standard_normal((B, Hkv, Skv, D))
    v = RNG.standard_normal((B, Hkv, Skv, D))
    lens = np.array([Skv, 3], dtype=np.int32)
    keep = torch.ones(B, 1, Sq, Skv, dtype=torch.bool)
    if mask_kind & 1:
        keep &= torch.ones(Sq, Skv, dtype=torch.bool).tril(diagonal=Skv - Sq)
    if mask_kind & 2:
        keep &= (torch.arange(Skv)[None, :] < torch.from_numpy(lens.astype(np.int64))[:, None])[:, None, None, :]
    tq, tk, tv = (torch.from_numpy(a) for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, tk.repeat_interleave(Hq // Hkv, dim=1), tv.repeat_interleave(Hq // Hkv, dim=1),
        attn_mask=keep, scale=0.4)
    out = oracle.attn(q, k, v, mask_kind, lens, 0.4)
    np.testing.assert_allclose(out, ref.numpy(), rtol=0, atol=1e-13)


def test_decode_is_last_row_of_causal_prefill():
    B, Hq, Hkv, Smax, D = 3, 4, 2, 12, 8
    kc = RNG.standard_normal((B, Hkv, Smax, D))
    vc = RNG.standard_normal((B, Hkv, Smax, D))
    qd = RNG.standard_normal((B, Hq, D))
    lens = np.array([12, 1, 7], dtype=np.int32)
    out = oracle.attn_decode(qd, kc, vc, lens, 0.3)
    for b in range(B):
        L = int(lens[b])
        qfull = RNG.standard_normal((1, Hq, L, D))
        qfull[0, :, L - 1] = qd[b]
        pre = oracle.attn(qfull, kc[b:b + 1, :, :L], vc[b:b + 1, :, :L], 1, None, 0.3)
        np.testing.assert_allclose(out[b], pre[0, :, L - 1], rtol=0, atol=1e-14)
    # rows beyond lens[b] must not matter
    kc2, vc2 = kc.copy(), vc.copy()
    for b in range(B):
        kc2[b, :, lens[b]:] = 1e6
        vc2[b, :, lens[b]:] = np.nan
    np.testing.assert_array_equal(oracle.attn_decode(qd, kc2, vc2, lens, 0.3), out)


def test_lens_clamped_and_empty_rows_zero():
    q = RNG.standard_normal((2, 1, 3, 4))
    k = RNG.standard_normal((2, 1, 5, 4))
    v = RNG.standard_normal((2, 1, 5, 4))
    out = oracle.attn(q, k, v, 2, np.array([0, 99], dtype=np.int32), 1.0)
    assert (out[0] == 0.0).all()
    np.testing.assert_array_equal(out[1:], oracle.attn(q[1:], k[1:], v[1:], 0, None, 1.0))
    # Sq > Skv with causal: leading rows see no key
    out = oracle.attn(RNG.standard_normal((1, 1, 4, 2)), k[:1, :, :2, :2], v[:1, :, :2, :2], 1, None, 1.0)
    assert (out[0, 0, :2] == 0.0).all() and np.abs(out[0, 0, 2:]).min() > 0


def test_invalid_arguments_rejected():
    q = np.zeros((1, 3, 2, 2)); k = np.zeros((1, 2, 2, 2))
    with pytest.raises(ValueError):
        oracle.attn(q, k, k, 0, None, 1.0)       # Hq % Hkv != 0
    q = np.zeros((1, 2, 2, 2))
    with pytest.raises(ValueError):
        oracle.attn(q, k, k, 2, None, 1.0)       # padding mask without lens
    with pytest.raises(ValueError):
        oracle.attn(q, k, k, 7, None, 1.0)       # unknown mask kind
