#!/usr/bin/env python
"""Benchmark of the fused-operator hot path on B200.

One step = one pass of the whole path over one batch of synthetic input:
  1. fused c_fc GEMM + bias + tanh-GELU               (8192 x 3072 x 768, bf16)
  2. fused causal attention, GPT-2-small layer shape  (B8 H12 S1024 D64, bf16)
  3. split-KV GQA decode over a KV cache              (B16 32/8 heads D128, lens U[1024,4096], 16 splits)
The headline value is the step's algorithmic FLOPs per second; the per-kernel numbers
(TFLOP/s or GB/s and the fraction of the measured peak) are in "kernels" and "roofline".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 (torchrun, one rank per GPU) every rank runs the same step on its own data:
the path shards by batch with no exchange, so scaling is weak and no collective is timed.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same step.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_16498_b200 import workloads as wl  # noqa: E402

METRIC = "fused attention TFLOP/s (% bf16 TC peak); split-KV decode HBM GB/s (% peak)"
WORKLOAD = ("GPT-2-small layer (causal attention B8 H12 S1024 D64 + c_fc GEMM 8192x3072x768 with bias and "
            "tanh-GELU) followed by 8B-class GQA split-KV decode (B16 32/8 heads D128, cached lengths "
            "U[1024,4096], 16 splits)")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (None once the kernel has changed since the capture).
NCU_TRAFFIC_BYTES = {"attention": 37918464, "linear": 18876928, "decode": 151960000}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _loop(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = get_reasons(self._h)
                for name, bit in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self._period)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs):
    """One pass of the step on the CPU oracle over a sample: the first n_heads (batch 0.., head)
    slices of the attention, the first n_rows rows of the GEMM, the first n_seqs decode sequences.
    Returns the algorithmic FLOPs it performed."""
    import oracle
    H = att.Hq
    flops = 0
    done = 0
    b = 0
    while done < n_heads:
        take = min(H, n_heads - done)
        oracle.attn(att.q.values[b:b + 1, :take], att.k.values[b:b + 1, :take], att.v.values[b:b + 1, :take],
                    att.mask_kind, None, att.scale)
        done += take
        b += 1
    flops += att.flops() // (att.B * H) * n_heads
    oracle.linear_bias_gelu(lin.x.values[:n_rows], lin.w.values, lin.b.values)
    flops += 2 * n_rows * lin.N * lin.K
    oracle.attn_decode(dec.q.values[:n_seqs], dec.k_cache.values[:n_seqs], dec.v_cache.values[:n_seqs],
                       dec.lens[:n_seqs], dec.scale)
    flops += 4 * dec.D * dec.Hq * int(dec.lens[:n_seqs].sum())
    return flops


def make_host_workloads(decode_B=16):
    att = wl.cfg2_attention()
    lin = wl.cfg2_linear()
    dec = wl.cfg5_gqa_decode(B=decode_B)
    return att, lin, dec


def cpu_baseline(att, lin, dec):
    """The oracle as it stands, on a bounded sample of the step (about 10-30 s of CPU work)."""
    import oracle
    n_heads, n_rows, n_seqs = 48, 4096, min(16, dec.B)
    oracle_sample_step(att, lin, dec, 1, 16, 1)  # loads the library, spins up the threads
    t0 = time.perf_counter()
    flops = oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs)
    dt = time.perf_counter() - t0
    return {"value": flops / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one pass: {n_heads} of {att.B * att.Hq} attention (batch, head) slices, {n_rows} of "
                      f"{lin.M} GEMM rows, {n_seqs} of {dec.B} decode sequences; {dt:.1f} s",
            "seconds": dt}


def run_reference(args):
    """`--impl reference`: the fp64 CPU oracle timed on the host cores, K steps of a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    att, lin, dec = make_host_workloads(decode_B=4)
    # calibrate on the smallest sample, then size the per-step sample for ~90 s in total
    oracle_sample_step(att, lin, dec, 1, 16, 1)
    t0 = time.perf_counter()
    f_small = oracle_sample_step(att, lin, dec, 2, 32, 1)
    t_small = time.perf_counter() - t0
    budget = 90.0 / max(1, args.steps + args.warmup)
    scale = max(1.0, min(48.0, budget / max(t_small, 1e-4)))
    n_heads = int(min(att.B * att.Hq, max(1, round(2 * scale))))
    n_rows = int(min(lin.M, max(16, round(32 * scale))))
    n_seqs = int(min(dec.B, max(1, round(scale / 8))))
    for _ in range(args.warmup):
        oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs)
    t0 = time.perf_counter()
    flops = 0
    for _ in range(args.steps):
        flops += oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs)
    dt = time.perf_counter() - t0
    value = flops / dt / 1e12
    sample = (f"per step: {n_heads} of {att.B * att.Hq} attention (batch, head) slices, {n_rows} of {lin.M} GEMM "
              f"rows, {n_seqs} of 16 decode sequences")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- multi-rank helpers
def max_over_ranks(ms: float, device=None, distributed: bool = False) -> float:
    """The slowest rank's time: every rank passes its own device time, all get the maximum."""
    if not distributed:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, units_per_rank: float, ms: float) -> float:
    """Units all ranks processed per second (every rank does `units_per_rank`; weak scaling)."""
    return world * units_per_rank / (ms * 1e-3)


# ----------------------------------------------------------------------------- GPU arm
def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2604_16498_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    distributed = world > 1

    # The CPU baseline runs first, before any CUDA call (rank 0, single GPU only).
    att, lin, dec = make_host_workloads()
    base = cpu_baseline(att, lin, dec) if (rank == 0 and world == 1 and not args.no_cpu_baseline) else None

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if distributed:
        dist.init_process_group("nccl", device_id=dev)
    binding.load()
    peaks, peak_src = load_peaks()

    def dev_bf16(t):
        return torch.from_numpy(np.ascontiguousarray(t.device_bits).view(np.int16)).view(torch.bfloat16).to(dev)

    # Input set 0 is the seeded workload (also used for the spot check); the other sets are seeded
    # device draws of the same shapes and distributions, rotated so that no input is L2-resident.
    nsets = 3
    gen = torch.Generator(device=dev)
    gen.manual_seed(20260416 + rank)

    def randn(shape, std=1.0):
        return (torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)

    lens_dev = torch.from_numpy(dec.lens).to(dev)
    sets = []
    for i in range(nsets):
        if i == 0:
            s = dict(q=dev_bf16(att.q), k=dev_bf16(att.k), v=dev_bf16(att.v),
                     x=dev_bf16(lin.x), w=dev_bf16(lin.w), b=dev_bf16(lin.b),
                     dq=dev_bf16(dec.q), kc=dev_bf16(dec.k_cache), vc=dev_bf16(dec.v_cache))
        else:
            s = dict(q=randn(att.q.values.shape), k=randn(att.k.values.shape), v=randn(att.v.values.shape),
                     x=randn((lin.M, lin.K)), w=randn((lin.K, lin.N), 0.02), b=randn((lin.N,), 0.02),
                     dq=randn(dec.q.values.shape), kc=randn(dec.k_cache.values.shape),
                     vc=randn(dec.v_cache.values.shape))
        s["o"] = torch.empty_like(s["q"])
        s["y"] = torch.empty((lin.M, lin.N), dtype=torch.bfloat16, device=dev)
        s["do"] = torch.empty_like(s["dq"])
        s["ws"] = torch.empty(binding.attn_decode_workspace_bytes(dec.B, dec.Hq, dec.D, dec.num_splits),
                              dtype=torch.uint8, device=dev)
        binding.attn_decode_workspace_init(s["ws"])
        sets.append(s)
    set_bytes = sum(t.numel() * t.element_size() for t in sets[0].values())

    def step(s, ev=None):
        if ev is not None:
            ev[0].record()
        # GEMM first: its 50 MB of output drain from L2 under the compute-bound attention, not under the
        # bandwidth-bound decode
        binding.linear_bias_gelu(s["x"], s["w"], s["b"], out=s["y"])
        if ev is not None:
            ev[1].record()
        binding.attn_fused(s["q"], s["k"], s["v"], att.mask_kind, None, att.scale, out=s["o"])
        if ev is not None:
            ev[2].record()
        binding.attn_decode_splitkv(s["dq"], s["kc"], s["vc"], lens_dev, dec.num_splits, dec.scale,
                                    out=s["do"], workspace=s["ws"])
        if ev is not None:
            ev[3].record()

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(sets[i % nsets])
    binding.check_status()

    # ---- timed region: K steps back to back, device events around the region only (the library launches
    # its kernels with programmatic stream serialisation, so consecutive launches overlap their heads and
    # tails; an event between two kernels would take that away)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    barrier()
    launches0 = binding.launch_count()
    sampler.start()
    t_wall0 = time.perf_counter()
    ev0.record()
    for i in range(args.steps):
        step(sets[i % nsets])
    ev1.record()
    barrier()
    wall = time.perf_counter() - t_wall0
    launches = binding.launch_count() - launches0
    binding.check_status()
    dev_ms = ev0.elapsed_time(ev1)

    # ---- the same K steps again with events around every kernel: per-kernel launch durations (each
    # event separates the kernels, so these add up to a little more than the step above)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    for i in range(args.steps):
        step(sets[i % nsets], evs[i])
    barrier()
    clocks = sampler.stop()
    binding.check_status()
    k_ms = [float(np.mean([e[i].elapsed_time(e[i + 1]) for e in evs])) for i in range(3)]
    split_ms = evs[0][0].elapsed_time(evs[-1][3]) / args.steps

    dev_ms = max_over_ranks(dev_ms, dev, distributed)
    ms_per_step = dev_ms / args.steps

    step_flops = att.flops() + lin.flops() + dec.flops()
    value = whole_job_rate(world, step_flops, ms_per_step) / 1e12

    # ---- per-kernel numbers and the roofline of the dominant one
    sustained = dev_ms >= 1000.0
    tensor_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    kern = {
        "attention": {"ms": k_ms[1], "tflops": att.flops() / k_ms[1] / 1e9, "gbs": att.bytes() / k_ms[1] / 1e6,
                      "bound": "tensor", "flops": att.flops(), "bytes": att.bytes()},
        "linear": {"ms": k_ms[0], "tflops": lin.flops() / k_ms[0] / 1e9, "gbs": lin.bytes() / k_ms[0] / 1e6,
                   "bound": "tensor", "flops": lin.flops(), "bytes": lin.bytes()},
        "decode": {"ms": k_ms[2], "tflops": dec.flops() / k_ms[2] / 1e9, "gbs": dec.bytes() / k_ms[2] / 1e6,
                   "bound": "hbm", "flops": dec.flops(), "bytes": dec.bytes()},
    }
    for name, k in kern.items():
        k["frac"] = k["tflops"] / tensor_peak if k["bound"] == "tensor" else k["gbs"] / peaks["hbm_gbs"]
    dom = max(kern, key=lambda n: kern[n]["ms"])
    d = kern[dom]
    roofline = {
        "kernel": dom, "bound": d["bound"],
        "achieved": d["tflops"] if d["bound"] == "tensor" else d["gbs"],
        "peak": tensor_peak if d["bound"] == "tensor" else peaks["hbm_gbs"],
        "unit": "TFLOP/s" if d["bound"] == "tensor" else "GB/s",
        "frac": d["frac"], "traffic": NCU_TRAFFIC_BYTES[dom],
        "peak_source": f"{peak_src} ({'sustained' if sustained and d['bound'] == 'tensor' else 'burst'})",
    }

    # ---- the other configurations, each timed on its own after the step loop (not part of `value`):
    # 8B-class GQA prefill (the shape where the tensor-core target applies), the padded encoder batch and
    # the fp32 GPT-2-small case (latency).  Device-drawn inputs of the workloads' shapes and distributions.
    other = None
    if rank == 0 and not args.no_other_configs:
        def timed(fn, iters):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(iters):
                fn()
            b_.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b_) / iters

        other = {}
        B4, Hq4, Hkv4, S4, D4 = 4, 32, 8, 2048, 128
        q4, k4, v4 = randn((B4, Hq4, S4, D4)), randn((B4, Hkv4, S4, D4)), randn((B4, Hkv4, S4, D4))
        o4 = torch.empty_like(q4)
        ms = timed(lambda: binding.attn_fused(q4, k4, v4, wl.MASK_CAUSAL, None, D4 ** -0.5, out=o4), 20)
        fl = 4 * D4 * B4 * Hq4 * (S4 * (S4 + 1) // 2)
        other["cfg4_gqa_prefill_B4_32/8_S2048_D128"] = {
            "ms": ms, "tflops": fl / ms / 1e9, "frac_of_bf16_peak": fl / ms / 1e9 / peaks["bf16_tflops"],
            "flops": fl, "l2": "warm (inputs 101 MB, reused across calls)"}
        del q4, k4, v4, o4
        B3, H3, S3, D3 = 32, 12, 128, 64
        lens3 = torch.from_numpy(wl.cfg3_encoder().lens).to(dev)
        q3, k3, v3 = randn((B3, H3, S3, D3)), randn((B3, H3, S3, D3)), randn((B3, H3, S3, D3))
        o3 = torch.empty_like(q3)
        ms = timed(lambda: binding.attn_fused(q3, k3, v3, wl.MASK_PADDING, lens3, 0.125, out=o3), 50)
        sl = int(lens3.sum().item())
        other["cfg3_encoder_padding_B32_H12_S128_D64"] = {
            "ms": ms, "tflops": 393216 * sl / ms / 1e9, "gbs": (12582912 + 3072 * sl) / ms / 1e6, "sum_lens": sl,
            "l2": "warm"}
        q1 = torch.randn((1, 12, 128, 64), generator=gen, device=dev)
        k1, v1 = torch.randn_like(q1), torch.randn_like(q1)
        o1 = torch.empty_like(q1)
        ms = timed(lambda: binding.attn_fused_f32(q1, k1, v1, wl.MASK_CAUSAL, None, 0.125, out=o1), 50)
        other["cfg1_gpt2_fp32_B1_H12_S128_D64"] = {"latency_us": ms * 1e3, "l2": "warm"}

    # ---- spot check of set 0 against values the oracle computes one by one (not timed)
    spot = None
    if rank == 0 and base is not None:
        import oracle
        s = sets[0]
        step(s)
        torch.cuda.synchronize()
        ref = oracle.attn(att.q.values[7:8, 11:12], att.k.values[7:8, 11:12], att.v.values[7:8, 11:12],
                          att.mask_kind, None, att.scale)
        e_att = float(np.abs(s["o"][7:8, 11:12].float().cpu().double().numpy() - ref).max())
        rows = [0, 4097, 8191]
        ref = oracle.linear_bias_gelu(lin.x.values[rows], lin.w.values, lin.b.values)
        e_lin = float(np.abs(s["y"][rows].float().cpu().double().numpy() - ref).max())
        ref = oracle.attn_decode(dec.q.values[:2], dec.k_cache.values[:2], dec.v_cache.values[:2], dec.lens[:2],
                                 dec.scale)
        e_dec = float(np.abs(s["do"][:2].float().cpu().double().numpy() - ref).max())
        spot = {"attention_max_abs": e_att, "linear_max_abs": e_lin, "decode_max_abs": e_dec,
                "ok": bool(max(e_att, e_lin, e_dec) <= 2e-2)}

    # ---- end to end: the same step through the host-buffer entry points, pinned host memory,
    # host->device and device->host copies inside the timed region
    e2e = None
    if not args.no_e2e:
        s0 = sets[0]
        pin = {k: s0[k].cpu().pin_memory() for k in ("q", "k", "v", "x", "w", "b", "dq", "kc", "vc")}
        outs = {"o": torch.empty_like(pin["q"]).pin_memory(),
                "y": torch.empty((lin.M, lin.N), dtype=torch.bfloat16).pin_memory(),
                "do": torch.empty_like(pin["dq"]).pin_memory()}
        lens_host = torch.from_numpy(dec.lens)
        sc_a = torch.empty(binding.attn_host_scratch_bytes(att.B, att.Hq, att.Hkv, att.Sq, att.Skv, att.D, 2),
                           dtype=torch.uint8, device=dev)
        sc_l = torch.empty(binding.linear_host_scratch_bytes(lin.M, lin.N, lin.K), dtype=torch.uint8, device=dev)
        sc_d = torch.empty(binding.attn_decode_host_scratch_bytes(dec.B, dec.Hq, dec.Hkv, dec.Smax, dec.D,
                                                                  dec.num_splits), dtype=torch.uint8, device=dev)

        def host_step():
            binding.attn_fused_host(pin["q"], pin["k"], pin["v"], outs["o"], sc_a, att.mask_kind, None, att.scale)
            binding.linear_bias_gelu_host(pin["x"], pin["w"], pin["b"], outs["y"], sc_l)
            binding.attn_decode_splitkv_host(pin["dq"], pin["kc"], pin["vc"], lens_host, dec.num_splits,
                                             outs["do"], sc_d, dec.scale)

        e_steps = max(1, min(args.steps, 10))
        for _ in range(2):
            host_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e_steps):
            host_step()
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), dev, distributed)
        h2d = sum(pin[k].numel() * 2 for k in pin) + dec.B * 4
        d2h = sum(outs[k].numel() * 2 for k in outs)
        e2e = {"value": world * step_flops / (e2e_ms / e_steps * 1e-3) / 1e12, "unit": "TFLOP/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e_steps,
               "ms_per_step": e2e_ms / e_steps}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD,
                       "l2": f"rotating {nsets} input sets of {set_bytes / 1e6:.0f} MB each (a step streams "
                             f"more than the 126 MB L2 between two uses of any buffer)",
                       "sum_lens": int(dec.lens.sum())},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": base, "kernels": kern, "other_configs": other,
            "decode_hbm": {"value": kern["decode"]["gbs"], "unit": "GB/s", "frac_of_measured_peak": kern["decode"]["frac"]},
            "wall_ms_per_step": wall / args.steps * 1e3, "ms_per_step_with_kernel_events": split_ms,
            "spot_check": spot,
        }
        print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="forge", choices=["forge", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
