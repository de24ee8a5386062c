"""Seeded synthetic inputs for the fused-attention / fused-MLP workloads.

This module only draws numbers and describes shapes.  It holds none of the
method's arithmetic (no dot products, softmax, GELU), so both the CPU oracle's
tests and the CUDA path's tests can feed from it without sharing any compute.

Generator: a counter-based splitmix64 stream (element ``i`` of stream ``seed``
is ``mix(seed + (i + 1) * 0x9E3779B97F4A7C15)``), turned into standard normals
by the Box-Muller transform.  Everything is numpy; values are bit-reproducible
on any host.

bf16 (and fp16) tensors are produced as fp64 -> fp32 -> 16 bits (round to nearest
even) and returned both as raw 16-bit patterns (what the GPU consumes) and as the
exact fp64 widening of those patterns (what the oracle consumes).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

BASE_SEED = 20260416
# tensor_index used in seed = BASE_SEED + 1000 * config + tensor_index
TENSOR_INDEX = {"q": 0, "k": 1, "v": 2, "x": 3, "w": 4, "b": 5, "lens": 6}

MASK_NONE, MASK_CAUSAL, MASK_PADDING, MASK_CAUSAL_PADDING = 0, 1, 2, 3


def seed_for(config: int, tensor: str) -> int:
    return BASE_SEED + 1000 * config + TENSOR_INDEX[tensor]


def splitmix64(seed: int, n: int, start: int = 0) -> np.ndarray:
    """Elements ``start .. start+n-1`` of the splitmix64 stream ``seed`` (uint64)."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + n + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def normal_f64(seed: int, n: int, std: float = 1.0) -> np.ndarray:
    """``n`` i.i.d. N(0, std^2) draws in fp64 (Box-Muller on pairs of stream elements)."""
    pairs = (n + 1) // 2
    out = np.empty(2 * pairs, dtype=np.float64)
    chunk = 1 << 22
    for p0 in range(0, pairs, chunk):
        p1 = min(pairs, p0 + chunk)
        u = splitmix64(seed, 2 * (p1 - p0), start=2 * p0)
        # u1 in (0, 1], u2 in [0, 1): 53-bit mantissas
        u1 = ((u[0::2] >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
        u2 = (u[1::2] >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
        r = np.sqrt(-2.0 * np.log(u1))
        t = 2.0 * np.pi * u2
        out[2 * p0:2 * p1:2] = r * np.cos(t)
        out[2 * p0 + 1:2 * p1:2] = r * np.sin(t)
    out = out[:n]
    if std != 1.0:
        out *= std
    return out


def uniform_int(seed: int, n: int, lo: int, hi: int) -> np.ndarray:
    """``n`` integers uniform on the inclusive range [lo, hi] as int32."""
    u = splitmix64(seed, n)
    return (lo + (u % np.uint64(hi - lo + 1)).astype(np.int64)).astype(np.int32)


def f32_to_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 with round-to-nearest-even; returns the uint16 patterns."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 patterns to fp64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


@dataclass
class Tensor:
    """One synthetic tensor: ``values`` is what the oracle reads (fp64, exactly the
    numbers the GPU sees), ``device_bits`` is what the GPU reads (uint16 bf16
    patterns, or float32 for the fp32 workload)."""
    values: np.ndarray
    device_bits: np.ndarray
    dtype: str  # "bf16" | "f16" | "f32"


def normal_tensor(seed: int, shape, dtype: str, std: float = 1.0) -> Tensor:
    n = int(np.prod(shape))
    x32 = normal_f64(seed, n, std).astype(np.float32)
    if dtype == "f32":
        return Tensor(x32.astype(np.float64).reshape(shape), x32.reshape(shape), "f32")
    if dtype == "bf16":
        bits = f32_to_bf16_bits(x32)
        return Tensor(bf16_bits_to_f64(bits).reshape(shape), bits.reshape(shape), "bf16")
    if dtype == "f16":  # numpy rounds fp32 -> fp16 to nearest even
        h = x32.astype(np.float16)
        return Tensor(h.astype(np.float64).reshape(shape), h.view(np.uint16).reshape(shape), "f16")
    raise ValueError(dtype)


@dataclass
class AttentionWorkload:
    name: str
    B: int
    Hq: int
    Hkv: int
    Sq: int
    Skv: int
    D: int
    mask_kind: int
    scale: float
    dtype: str
    q: Tensor
    k: Tensor
    v: Tensor
    lens: np.ndarray | None = None

    def unmasked_pairs(self) -> int:
        """(query, key) pairs that are not masked, summed over batch and query heads."""
        total = 0
        for b in range(self.B):
            kv = self.Skv
            if self.mask_kind & MASK_PADDING:
                kv = int(min(max(int(self.lens[b]), 0), self.Skv))
            if self.mask_kind & MASK_CAUSAL:
                off = self.Skv - self.Sq
                i = np.arange(self.Sq)
                total += int(np.clip(np.minimum(i + off + 1, kv), 0, None).sum())
            else:
                total += self.Sq * kv
        return total * self.Hq

    def flops(self) -> int:
        return 4 * self.D * self.unmasked_pairs()

    def bytes(self) -> int:
        es = 4 if self.dtype == "f32" else 2
        qo = 2 * self.B * self.Hq * self.Sq * self.D * es
        if self.mask_kind & MASK_PADDING:
            rows = int(np.clip(self.lens, 0, self.Skv).sum())
        else:
            rows = self.B * self.Skv
        return qo + 2 * rows * self.Hkv * self.D * es


@dataclass
class DecodeWorkload:
    name: str
    B: int
    Hq: int
    Hkv: int
    Smax: int
    D: int
    num_splits: int
    scale: float
    q: Tensor          # [B, Hq, D]
    k_cache: Tensor    # [B, Hkv, Smax, D]
    v_cache: Tensor
    lens: np.ndarray   # int32 [B]

    def flops(self) -> int:
        return 4 * self.D * self.Hq * int(self.lens.sum())

    def bytes(self) -> int:
        return 2 * 2 * self.Hkv * self.D * int(self.lens.sum()) + 2 * 2 * self.B * self.Hq * self.D


@dataclass
class LinearWorkload:
    name: str
    M: int
    N: int
    K: int
    x: Tensor  # [M, K]
    w: Tensor  # [K, N]
    b: Tensor  # [N]

    def flops(self) -> int:
        return 2 * self.M * self.N * self.K

    def bytes(self) -> int:
        return 2 * (self.M * self.K + self.K * self.N + self.N + self.M * self.N)


def attention_workload(name, config, B, Hq, Hkv, Sq, Skv, D, mask_kind, scale, dtype,
                       lens_range=None) -> AttentionWorkload:
    q = normal_tensor(seed_for(config, "q"), (B, Hq, Sq, D), dtype)
    k = normal_tensor(seed_for(config, "k"), (B, Hkv, Skv, D), dtype)
    v = normal_tensor(seed_for(config, "v"), (B, Hkv, Skv, D), dtype)
    lens = None
    if lens_range is not None:
        lens = uniform_int(seed_for(config, "lens"), B, lens_range[0], lens_range[1])
    return AttentionWorkload(name, B, Hq, Hkv, Sq, Skv, D, mask_kind, scale, dtype, q, k, v, lens)


def decode_workload(name, config, B, Hq, Hkv, Smax, D, num_splits, scale, lens_range, dtype="bf16") -> DecodeWorkload:
    q = normal_tensor(seed_for(config, "q"), (B, Hq, D), dtype)
    k = normal_tensor(seed_for(config, "k"), (B, Hkv, Smax, D), dtype)
    v = normal_tensor(seed_for(config, "v"), (B, Hkv, Smax, D), dtype)
    lens = uniform_int(seed_for(config, "lens"), B, lens_range[0], lens_range[1])
    return DecodeWorkload(name, B, Hq, Hkv, Smax, D, num_splits, scale, q, k, v, lens)


def linear_workload(name, config, M, N, K, w_std=0.02, b_std=0.02, dtype="bf16") -> LinearWorkload:
    x = normal_tensor(seed_for(config, "x"), (M, K), dtype)
    w = normal_tensor(seed_for(config, "w"), (K, N), dtype, std=w_std)
    b = normal_tensor(seed_for(config, "b"), (N,), dtype, std=b_std)
    return LinearWorkload(name, M, N, K, x, w, b)


# The five benchmark configurations (shapes of 125M- to 8B-class models).
def cfg1_gpt2_f32() -> AttentionWorkload:
    return attention_workload("cfg1: fp32 causal B1 H12 S128 D64", 1, 1, 12, 12, 128, 128, 64,
                              MASK_CAUSAL, 0.125, "f32")


def cfg2_attention(B: int = 8) -> AttentionWorkload:
    return attention_workload(f"cfg2a: bf16 causal B{B} H12 S1024 D64", 2, B, 12, 12, 1024, 1024, 64,
                              MASK_CAUSAL, 0.125, "bf16")


def cfg2_linear(M: int = 8192) -> LinearWorkload:
    return linear_workload(f"cfg2b: bf16 GEMM {M}x3072x768 + bias + tanh-GELU", 2, M, 3072, 768)


def cfg3_encoder(B: int = 32) -> AttentionWorkload:
    return attention_workload(f"cfg3: bf16 key-padding B{B} H12 S128 D64 lens U[16,128]", 3, B, 12, 12,
                              128, 128, 64, MASK_PADDING, 0.125, "bf16", lens_range=(16, 128))


def cfg4_gqa_prefill(B: int = 4, S: int = 2048) -> AttentionWorkload:
    return attention_workload(f"cfg4: bf16 causal GQA B{B} 32/8 S{S} D128", 4, B, 32, 8, S, S, 128,
                              MASK_CAUSAL, 1.0 / np.sqrt(128.0), "bf16")


def cfg5_gqa_decode(B: int = 16, Smax: int = 4096, lens_range=(1024, 4096)) -> DecodeWorkload:
    return decode_workload(f"cfg5: bf16 GQA decode B{B} 32/8 D128 lens U{list(lens_range)} 16 splits", 5,
                           B, 32, 8, Smax, 128, 16, 1.0 / np.sqrt(128.0), lens_range)
