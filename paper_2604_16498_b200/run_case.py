"""Runs one operator of the library a few times on a seeded synthetic case (for profilers).

    python -m paper_2604_16498_b200.run_case attention --B 8 --Hq 12 --Hkv 12 --S 1024 --D 64 --mask 1
    python -m paper_2604_16498_b200.run_case linear --M 8192 --N 3072 --K 768
    python -m paper_2604_16498_b200.run_case decode --B 16 --Hq 32 --Hkv 8 --S 4096 --D 128 --splits 16
    python -m paper_2604_16498_b200.run_case attention_f32 --B 1 --Hq 12 --Hkv 12 --S 128 --D 64 --mask 1

Prints the mean device time per call (CUDA events) after the warm-up calls.
"""
from __future__ import annotations

import argparse

import torch

from . import binding


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["attention", "attention_f32", "linear", "linear_w8", "decode"])
    ap.add_argument("--B", type=int, default=8)
    ap.add_argument("--Hq", type=int, default=12)
    ap.add_argument("--Hkv", type=int, default=12)
    ap.add_argument("--S", type=int, default=1024, help="sequence length (Sq = Skv; cache length for decode)")
    ap.add_argument("--D", type=int, default=64)
    ap.add_argument("--mask", type=int, default=1)
    ap.add_argument("--min-len", type=int, default=0, help="lens uniform in [min-len, S] (padding masks, decode)")
    ap.add_argument("--splits", type=int, default=16)
    ap.add_argument("--M", type=int, default=8192)
    ap.add_argument("--N", type=int, default=3072)
    ap.add_argument("--K", type=int, default=768)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    a = ap.parse_args()

    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev)
    g.manual_seed(20260416)

    def randn(shape, dtype=torch.bfloat16, std=1.0):
        return (torch.randn(shape, generator=g, device=dev) * std).to(dtype)

    lens = None
    lo = a.min_len if a.min_len > 0 else max(1, a.S // 4)
    if a.op == "decode" or (a.mask & 2):
        lens = torch.randint(lo, a.S + 1, (a.B,), generator=g, device=dev, dtype=torch.int32)

    if a.op in ("attention", "attention_f32"):
        dt = torch.float32 if a.op == "attention_f32" else torch.bfloat16
        q = randn((a.B, a.Hq, a.S, a.D), dt)
        k = randn((a.B, a.Hkv, a.S, a.D), dt)
        v = randn((a.B, a.Hkv, a.S, a.D), dt)
        out = torch.empty_like(q)
        fn = binding.attn_fused_f32 if a.op == "attention_f32" else binding.attn_fused
        call = lambda: fn(q, k, v, a.mask, lens, a.D ** -0.5, out=out)
    elif a.op == "linear":
        x, w, b = randn((a.M, a.K)), randn((a.K, a.N), std=0.02), randn((a.N,), std=0.02)
        y = torch.empty((a.M, a.N), dtype=torch.bfloat16, device=dev)
        call = lambda: binding.linear_bias_gelu(x, w, b, out=y)
    elif a.op == "linear_w8":
        x = randn((a.M, a.K), torch.float16)
        wq = torch.randint(-127, 128, (a.N, a.K), generator=g, device=dev, dtype=torch.int8)
        sc = torch.rand((a.N,), generator=g, device=dev) * 0.01
        y = torch.empty((a.M, a.N), dtype=torch.float16, device=dev)
        call = lambda: binding.linear_act_w8a16(x, wq, sc, None, None, binding.ACT_GELU_TANH, out=y)
    else:
        q = randn((a.B, a.Hq, a.D))
        kc = randn((a.B, a.Hkv, a.S, a.D))
        vc = randn((a.B, a.Hkv, a.S, a.D))
        out = torch.empty_like(q)
        ws = torch.empty(binding.attn_decode_workspace_bytes(a.B, a.Hq, a.D, a.splits), dtype=torch.uint8, device=dev)
        binding.attn_decode_workspace_init(ws)
        call = lambda: binding.attn_decode_splitkv(q, kc, vc, lens, a.splits, a.D ** -0.5, out=out, workspace=ws)

    for _ in range(a.warmup):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        call()
    e1.record()
    torch.cuda.synchronize()
    binding.check_status()
    print(f"{a.op}: {e0.elapsed_time(e1) / a.iters * 1e3:.2f} us per call over {a.iters} calls")


if __name__ == "__main__":
    main()
