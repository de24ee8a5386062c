#!/usr/bin/env python
"""Benchmark of the fused-operator hot path on B200.

One step = one pass of the whole path over one batch of synthetic input:
  1. fused c_fc GEMM + bias + tanh-GELU                        (8192 x 3072 x 768, bf16)
  2. fused causal GQA prefill attention, 8B-class shape        (B4 32/8 heads S2048 D128, bf16)
  3. split-KV GQA decode over a KV cache                       (B16 32/8 heads D128, lens U[1024,4096], 16 splits)
on three rotating input sets, so that no buffer is L2-resident when it is used again.

The metric has two halves.  `value` is the first: fused-attention TFLOP/s (algorithmic FLOPs of the
prefill attention / its average launch duration); the second, split-KV decode GB/s, is in `decode_hbm`.
`ms_per_step` is the whole step.  `kernels` holds every kernel's duration, rate and fraction of the
measured peak; `roofline` repeats that for the kernel with the longest duration.

Kernel durations: the library launches with programmatic stream serialisation, so an event between two
kernels changes what it measures.  Each kernel is therefore timed on its own, K calls back to back on the
rotating cold inputs with events around the K calls (`ms`); the step loop is timed the same way
(`ms_per_step`); and a third pass puts events around every kernel inside the step (`ms_in_step`, an upper
bound: the events take the overlap of neighbouring launches away).  Every timed region is repeated
`--repeats` times; medians are reported with the extremes beside them.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With N > 1 every rank runs the same step on its own data: the path shards by batch with no exchange, so
scaling is weak and no collective is timed.  Started without a launcher (`WORLD_SIZE` unset), `--gpus N`
starts the N ranks itself through torch.distributed.run.  `--impl reference` times the fp64 CPU oracle on
a bounded sample of the same step.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_16498_b200 import workloads as wl  # noqa: E402

METRIC = "fused attention TFLOP/s (% bf16 TC peak); split-KV decode HBM GB/s (% peak)"
WORKLOAD = ("8B-class causal GQA prefill attention (B4 32/8 heads S2048 D128) + GPT-2-small c_fc GEMM 8192x3072x768 "
            "with bias and tanh-GELU + 8B-class GQA split-KV decode (B16 32/8 heads D128, cached lengths "
            "U[1024,4096], 16 splits)")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (None once the kernel has changed since the capture).
NCU_TRAFFIC_BYTES = {"attention": 136300000, "linear": 19230000, "decode": 147200000}


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
    """Samples SM clock and throttle reasons through NVML while the timed regions run."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.samples, self.reasons = [], set()
        self.active = True  # samples are kept only while this is set
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
                if self.active:
                    mhz = nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)
                    mask = get_reasons(self._h)
                    if self.active:
                        self.samples.append(mhz)
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
def make_host_workloads(decode_B=16):
    att = wl.cfg4_gqa_prefill()
    lin = wl.cfg2_linear()
    dec = wl.cfg5_gqa_decode(B=decode_B)
    return att, lin, dec


def oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs):
    """One pass of the step on the CPU oracle over a sample: the first n_heads (batch, query head) slices of
    the attention, the first n_rows rows of the GEMM, the first n_seqs decode sequences.  Returns the seconds
    and algorithmic FLOPs of the attention part and of the whole pass."""
    import oracle
    G = att.Hq // att.Hkv
    t0 = time.perf_counter()
    done = 0
    while done < n_heads:
        b, h0 = divmod(done, att.Hq)
        take = min(att.Hq - h0, n_heads - done)
        h1 = h0 + take
        if h0 % G == 0 and h1 % G == 0:  # whole KV groups in one call
            oracle.attn(att.q.values[b:b + 1, h0:h1], att.k.values[b:b + 1, h0 // G:h1 // G],
                        att.v.values[b:b + 1, h0 // G:h1 // G], att.mask_kind, None, att.scale)
        else:                            # a partial group: head by head, each with its one KV head
            for h in range(h0, h1):
                oracle.attn(att.q.values[b:b + 1, h:h + 1], att.k.values[b:b + 1, h // G:h // G + 1],
                            att.v.values[b:b + 1, h // G:h // G + 1], att.mask_kind, None, att.scale)
        done += take
    t_att = time.perf_counter() - t0
    f_att = att.flops() // (att.B * att.Hq) * n_heads
    oracle.linear_bias_gelu(lin.x.values[:n_rows], lin.w.values, lin.b.values)
    oracle.attn_decode(dec.q.values[:n_seqs], dec.k_cache.values[:n_seqs], dec.v_cache.values[:n_seqs],
                       dec.lens[:n_seqs], dec.scale)
    t_all = time.perf_counter() - t0
    f_all = f_att + 2 * n_rows * lin.N * lin.K + 4 * dec.D * dec.Hq * int(dec.lens[:n_seqs].sum())
    return t_att, f_att, t_all, f_all


def cpu_baseline(att, lin, dec):
    """The oracle as it stands, on a bounded sample of the step (about 10-30 s of CPU work)."""
    import oracle
    n_heads, n_rows, n_seqs = 64, 4096, min(16, dec.B)
    oracle_sample_step(att, lin, dec, 1, 16, 1)  # loads the library, spins up the threads
    t_att, f_att, t_all, f_all = oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs)
    return {"value": f_att / t_att / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one pass: {n_heads} of {att.B * att.Hq} attention (batch, head) slices ({t_att:.1f} s, the "
                      f"rate reported), then {n_rows} of {lin.M} GEMM rows and {n_seqs} of {dec.B} decode "
                      f"sequences ({t_all:.1f} s in all)",
            "seconds": t_all, "step_tflops": f_all / t_all / 1e12}


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
    oracle_sample_step(att, lin, dec, 2, 32, 1)
    t_small = time.perf_counter() - t0
    budget = 90.0 / max(1, args.steps + args.warmup)
    scale = max(1.0, min(32.0, budget / max(t_small, 1e-4)))
    n_heads = int(min(att.B * att.Hq, max(1, round(2 * scale))))
    n_rows = int(min(lin.M, max(16, round(32 * scale))))
    n_seqs = int(min(dec.B, max(1, round(scale / 8))))
    for _ in range(args.warmup):
        oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs)
    t_att = f_att = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ta, fa, _, _ = oracle_sample_step(att, lin, dec, n_heads, n_rows, n_seqs)
        t_att += ta
        f_att += fa
    dt = time.perf_counter() - t0
    value = f_att / t_att / 1e12
    sample = (f"per step: {n_heads} of {att.B * att.Hq} attention (batch, head) slices (the rate reported), "
              f"{n_rows} of {lin.M} GEMM rows, {n_seqs} of 16 decode sequences")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample,
                   "value_is": "fused-attention TFLOP/s of the oracle on the sampled slices"},
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


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launcher_command(argv, gpus: int, port: int):
    """The command that starts `gpus` ranks of this script on one node (one per GPU, rendezvous on 127.0.0.1)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def maybe_relaunch(args, argv):
    """`--gpus N` (N > 1) without a launcher around it: start the N replicas and pass their output through.
    Returns the launcher's exit code, or None when this process is itself a rank (or N = 1)."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ or args.impl == "reference":
        return None
    return subprocess.run(launcher_command(argv, args.gpus, free_port())).returncode


def run_dry(args):
    """`--dry-run-cpu`: the rank plumbing of the GPU arm (process group, barrier, maximum over ranks, rank 0's
    JSON line) on CPU with the gloo backend and a made-up per-rank time, for tests without a GPU."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    distributed = world > 1
    if distributed:
        dist.init_process_group("gloo")
        dist.barrier()
    my_ms = 10.0 + 5.0 * rank
    ms = max_over_ranks(my_ms, torch.device("cpu"), distributed)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": whole_job_rate(world, 1.0, ms), "unit": "dry-run units/s",
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "scaling": "weak", "dry_run": True}))
    if distributed:
        dist.destroy_process_group()
    return 0


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

    def randn(shape, std=1.0, dtype=torch.bfloat16):
        return (torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * std).to(dtype)

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

    def k_linear(s):
        binding.linear_bias_gelu(s["x"], s["w"], s["b"], out=s["y"])

    def k_attention(s):
        binding.attn_fused(s["q"], s["k"], s["v"], att.mask_kind, None, att.scale, out=s["o"])

    def k_decode(s):
        binding.attn_decode_splitkv(s["dq"], s["kc"], s["vc"], lens_dev, dec.num_splits, dec.scale,
                                    out=s["do"], workspace=s["ws"])

    KERNELS = (("linear", k_linear), ("attention", k_attention), ("decode", k_decode))

    def step(s, ev=None):
        # GEMM first: its 50 MB of output drain from L2 under the compute-bound attention, not under the
        # bandwidth-bound decode
        for i, (_, fn) in enumerate(KERNELS):
            if ev is not None:
                ev[i].record()
            fn(s)
        if ev is not None:
            ev[len(KERNELS)].record()

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(sets[i % nsets])
    binding.check_status()

    def timed_region(fn, iters):
        """K back-to-back calls of fn(set) on the rotating sets, device events around the region only.  The
        GPU idles for `--cooldown` seconds first: back-to-back regions of the tensor-core kernels run into the
        board's power cap within tens of milliseconds and the clock drops, which the burst peaks they are
        compared with did not see.  Three untimed calls bring the clocks back up from idle before the region
        starts.  The clock sampler only looks while a region runs."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        time.sleep(args.cooldown)
        for i in range(3):  # the clocks come back up from idle during a few untimed calls
            fn(sets[(iters + i) % nsets])
        sampler.active = True
        e0.record()
        for i in range(iters):
            fn(sets[i % nsets])
        e1.record()
        barrier()
        sampler.active = False
        return e0.elapsed_time(e1)

    def stats(ms_list, iters):
        per = [max_over_ranks(m, dev, distributed) / iters for m in ms_list]
        return {"median": float(np.median(per)), "min": float(min(per)), "max": float(max(per)), "repeats": len(per)}

    reps = max(1, args.repeats)
    sampler = ClockSampler(local_rank)
    sampler.active = False
    launches0 = binding.launch_count()
    sampler.start()
    t_wall0 = time.perf_counter()
    # ---- timed region 1: K whole steps back to back, repeated
    step_ms = [timed_region(step, args.steps) for _ in range(reps)]
    wall = time.perf_counter() - t_wall0
    launches = binding.launch_count() - launches0
    # ---- timed region 2: each kernel on its own, K calls back to back on the rotating sets, repeated
    kernel_ms = {name: [timed_region(fn, args.steps) for _ in range(reps)] for name, fn in KERNELS}
    # ---- pass 3: events around every kernel inside the step (upper bounds)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(KERNELS) + 1)] for _ in range(args.steps)]
    barrier()
    time.sleep(args.cooldown)
    sampler.active = True
    for i in range(args.steps):
        step(sets[i % nsets], evs[i])
    barrier()
    clocks = sampler.stop()
    binding.check_status()
    per_call = [np.array([e[i].elapsed_time(e[i + 1]) for e in evs]) for i in range(len(KERNELS))]
    in_step_ms = [float(np.median(pc)) for pc in per_call]
    # the same samples as a distribution (one call each, events on both sides: launch gaps included)
    in_step_dist = [{"mean": float(pc.mean() * 1e3), "p50": float(np.percentile(pc, 50) * 1e3),
                     "p90": float(np.percentile(pc, 90) * 1e3), "p99": float(np.percentile(pc, 99) * 1e3),
                     "best": float(pc.min() * 1e3), "calls": int(pc.size)} for pc in per_call]

    st = stats(step_ms, args.steps)
    ms_per_step = st["median"]
    sustained = sum(step_ms) >= 1000.0
    tensor_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    work = {"linear": lin, "attention": att, "decode": dec}
    bound = {"linear": "tensor", "attention": "tensor", "decode": "hbm"}
    kern = {}
    for i, (name, _) in enumerate(KERNELS):
        ks = stats(kernel_ms[name], args.steps)
        w = work[name]
        ms = ks["median"]
        k = {"ms": ms, "ms_min": ks["min"], "ms_max": ks["max"], "ms_in_step": in_step_ms[i],
             "in_step_us": in_step_dist[i],
             "tflops": w.flops() / ms / 1e9, "gbs": w.bytes() / ms / 1e6, "bound": bound[name],
             "flops": w.flops(), "bytes": w.bytes()}
        if bound[name] == "tensor":
            k["frac"] = k["tflops"] / tensor_peak
            k["frac_of_nominal"] = k["tflops"] / NOMINAL_PEAKS["bf16_tflops"]
        else:
            k["frac"] = k["gbs"] / peaks["hbm_gbs"]
            k["frac_of_nominal"] = k["gbs"] / NOMINAL_PEAKS["hbm_gbs"]
        kern[name] = k
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
    # the metric's first half: fused-attention TFLOP/s, whole job (every rank runs its own replica)
    value = whole_job_rate(world, att.flops(), kern["attention"]["ms"]) / 1e12
    step_flops = att.flops() + lin.flops() + dec.flops()

    # ---- the other configurations, each timed on its own after the step loop (not part of `value`)
    other = None
    if rank == 0 and not args.no_other_configs:
        other = other_configs(torch, binding, dev, gen, randn, peaks, args)

    # ---- spot check of set 0 against values the oracle computes one by one (not timed)
    spot = None
    if rank == 0 and base is not None:
        import oracle
        s = sets[0]
        step(s)
        torch.cuda.synchronize()
        G = att.Hq // att.Hkv
        b_, h_ = 3, 29
        ref = oracle.attn(att.q.values[b_:b_ + 1, h_:h_ + 1], att.k.values[b_:b_ + 1, h_ // G:h_ // G + 1],
                          att.v.values[b_:b_ + 1, h_ // G:h_ // G + 1], att.mask_kind, None, att.scale)
        e_att = float(np.abs(s["o"][b_:b_ + 1, h_:h_ + 1].float().cpu().double().numpy() - ref).max())
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
        e_steps = max(1, min(args.steps, 10))
        ea = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(e_steps)]

        def host_step(ev=None):
            if ev:
                ev[0].record()
            binding.linear_bias_gelu_host(pin["x"], pin["w"], pin["b"], outs["y"], sc_l)
            if ev:
                ev[1].record()
            binding.attn_fused_host(pin["q"], pin["k"], pin["v"], outs["o"], sc_a, att.mask_kind, None, att.scale)
            if ev:
                ev[2].record()
            binding.attn_decode_splitkv_host(pin["dq"], pin["kc"], pin["vc"], lens_host, dec.num_splits,
                                             outs["do"], sc_d, dec.scale)
            if ev:
                ev[3].record()

        for _ in range(2):
            host_step()
        barrier()
        for i in range(e_steps):
            host_step(ea[i])
        barrier()
        att_ms = max_over_ranks(float(np.median([e[1].elapsed_time(e[2]) for e in ea])), dev, distributed)
        all_ms = max_over_ranks(float(np.median([e[0].elapsed_time(e[3]) for e in ea])), dev, distributed)
        h2d = sum(pin[k].numel() * 2 for k in pin) + dec.B * 4
        d2h = sum(outs[k].numel() * 2 for k in outs)
        e2e = {"value": whole_job_rate(world, att.flops(), att_ms) / 1e12, "unit": "TFLOP/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e_steps,
               "ms_per_step": all_ms, "attention_ms": att_ms,
               "attention_h2d_bytes": int(sum(pin[k].numel() * 2 for k in ("q", "k", "v"))),
               "attention_d2h_bytes": int(outs["o"].numel() * 2),
               "note": "value = attention FLOPs / duration of forge_attn_fused_host (copies included); "
                       "ms_per_step is the whole host step"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD,
                       "value_is": "fused-attention TFLOP/s: FLOPs of the prefill attention / its median launch "
                                   "duration (K calls back to back on rotating inputs); decode GB/s is in decode_hbm",
                       "l2": f"rotating {nsets} input sets of {set_bytes / 1e6:.0f} MB each (more than the 126 MB L2 "
                             f"is streamed between two uses of any buffer)",
                       "sum_lens": int(dec.lens.sum()), "repeats": reps, "cooldown_s": args.cooldown},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": base, "kernels": kern, "other_configs": other,
            "decode_hbm": {"value": kern["decode"]["gbs"], "unit": "GB/s",
                           "frac_of_measured_peak": kern["decode"]["frac"],
                           "frac_of_nominal_8tbs": kern["decode"]["frac_of_nominal"]},
            "step": {"ms_median": st["median"], "ms_min": st["min"], "ms_max": st["max"], "repeats": st["repeats"],
                     "tflops": whole_job_rate(world, step_flops, ms_per_step) / 1e12,
                     "sum_of_kernel_ms": sum(k["ms"] for k in kern.values())},
            "wall_ms_per_step": wall / (args.steps * reps) * 1e3,
            "spot_check": spot,
        }
        print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()
    return 0


def other_configs(torch, binding, dev, gen, randn, peaks, args):
    """The remaining configurations and the other fused patterns, each K calls back to back on two rotating
    input sets.  Device-drawn inputs of the workloads' shapes and distributions."""
    iters = max(5, min(args.steps, 50))
    bf, h = torch.bfloat16, torch.float16

    def empty(shape, dtype=bf):
        return torch.empty(shape, dtype=dtype, device=dev)

    def timed(make, call, nset=2):
        data = [make() for _ in range(nset)]
        for d in data:
            call(d)
        torch.cuda.synchronize()
        per = []
        for _ in range(3):
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(iters):
                call(data[i % nset])
            b_.record()
            torch.cuda.synchronize()
            per.append(a.elapsed_time(b_) / iters)
        return float(np.median(per))

    other = {}
    pk = peaks["bf16_tflops"]
    # cfg 2a: GPT-2-small layer attention (the D = 64 shape, bound by the exponentials)
    B, H, S, D = 8, 12, 1024, 64
    ms = timed(lambda: (randn((B, H, S, D)), randn((B, H, S, D)), randn((B, H, S, D)), empty((B, H, S, D))),
               lambda d: binding.attn_fused(d[0], d[1], d[2], wl.MASK_CAUSAL, None, 0.125, out=d[3]))
    fl = 4 * D * B * H * (S * (S + 1) // 2)
    other["cfg2a_gpt2_attention_B8_H12_S1024_D64"] = {"ms": ms, "tflops": fl / ms / 1e9,
                                                      "frac_of_bf16_peak": fl / ms / 1e9 / pk, "flops": fl}
    # cfg 3: padded encoder batch
    B3, H3, S3, D3 = 32, 12, 128, 64
    lens3 = torch.from_numpy(wl.cfg3_encoder().lens).to(dev)
    sl = int(lens3.sum().item())
    mk3 = lambda: (randn((B3, H3, S3, D3)), randn((B3, H3, S3, D3)), randn((B3, H3, S3, D3)), empty((B3, H3, S3, D3)))
    call3 = lambda d: binding.attn_fused(d[0], d[1], d[2], wl.MASK_PADDING, lens3, 0.125, out=d[3])
    ms = timed(mk3, call3, nset=20)   # 20 sets of 25 MB: four times the L2, every input comes from HBM
    ms_warm = timed(mk3, call3, nset=2)
    b3 = 12582912 + 3072 * sl
    other["cfg3_encoder_padding_B32_H12_S128_D64"] = {"ms": ms, "tflops": 393216 * sl / ms / 1e9,
                                                      "gbs": b3 / ms / 1e6, "frac_of_hbm_peak": b3 / ms / 1e6 / peaks["hbm_gbs"],
                                                      "sum_lens": sl, "l2": "cold (20 rotating sets of 25 MB)",
                                                      "ms_warm_l2": ms_warm, "gbs_warm_l2": b3 / ms_warm / 1e6}
    # cfg 1: fp32 GPT-2-small attention (latency)
    def f32(shape):
        return torch.randn(shape, generator=gen, device=dev)
    s1 = (1, 12, 128, 64)
    ms = timed(lambda: (f32(s1), f32(s1), f32(s1), empty(s1, torch.float32)),
               lambda d: binding.attn_fused_f32(d[0], d[1], d[2], wl.MASK_CAUSAL, None, 0.125, out=d[3]))
    other["cfg1_gpt2_fp32_B1_H12_S128_D64"] = {"latency_us": ms * 1e3, "l2": "warm"}
    # the other fused patterns at the 8B-class prefill shape
    B4, Hq4, Hkv4, S4, D4 = 4, 32, 8, 2048, 128
    fl4 = 4 * D4 * B4 * Hq4 * (S4 * (S4 + 1) // 2)
    ms = timed(lambda: (randn((B4, Hq4, S4, D4), dtype=h), randn((B4, Hkv4, S4, D4), dtype=h),
                        randn((B4, Hkv4, S4, D4), dtype=h), empty((B4, Hq4, S4, D4), h)),
               lambda d: binding.attn_fused_f16(d[0], d[1], d[2], wl.MASK_CAUSAL, None, D4 ** -0.5, out=d[3]))
    other["attention_fp16_cfg4_shape"] = {"ms": ms, "tflops": fl4 / ms / 1e9, "frac_of_bf16_peak": fl4 / ms / 1e9 / pk}
    Bw, Hqw, Hkvw, Sw, Dw = 4, 16, 4, 2048, 256  # head size 256: the one-tile-per-CTA kernel
    flw = 4 * Dw * Bw * Hqw * (Sw * (Sw + 1) // 2)
    ms = timed(lambda: (randn((Bw, Hqw, Sw, Dw)), randn((Bw, Hkvw, Sw, Dw)), randn((Bw, Hkvw, Sw, Dw)), empty((Bw, Hqw, Sw, Dw))),
               lambda d: binding.attn_fused(d[0], d[1], d[2], wl.MASK_CAUSAL, None, Dw ** -0.5, out=d[3]))
    other["attention_D256_B4_16/4_S2048"] = {"ms": ms, "tflops": flw / ms / 1e9, "frac_of_bf16_peak": flw / ms / 1e9 / pk}
    bias = torch.zeros((B4, 1, S4, S4), device=dev)
    ms = timed(lambda: (randn((B4, Hq4, S4, D4)), randn((B4, Hkv4, S4, D4)), randn((B4, Hkv4, S4, D4)),
                        empty((B4, Hq4, S4, D4))),
               lambda d: binding.attn_fused_bias(d[0], d[1], d[2], bias, wl.MASK_CAUSAL, None, D4 ** -0.5, out=d[3]))
    other["attention_additive_bias_cfg4_shape"] = {"ms": ms, "tflops": fl4 / ms / 1e9,
                                                    "frac_of_bf16_peak": fl4 / ms / 1e9 / pk,
                                                    "bias_bytes": int(bias.numel() * 4)}
    del bias
    M, N, K = 8192, 8192, 2048
    ms = timed(lambda: (randn((M, K)), randn((K, N), 0.02), randn((K, N), 0.02), empty((M, N))),
               lambda d: binding.linear_swiglu(d[0], d[1], d[2], out=d[3]))
    fl = 4 * M * N * K
    other["linear_swiglu_8192x8192x2048"] = {"ms": ms, "tflops": fl / ms / 1e9, "frac_of_bf16_peak": fl / ms / 1e9 / pk}
    M, N, K = 8192, 8192, 4096
    ms = timed(lambda: (randn((M, K), dtype=h), torch.randint(-127, 128, (N, K), generator=gen, device=dev, dtype=torch.int8),
                        torch.rand((N,), generator=gen, device=dev) * 0.01, empty((M, N), h)),
               lambda d: binding.linear_act_w8a16(d[0], d[1], d[2], None, None, binding.ACT_GELU_TANH, out=d[3]))
    fl = 2 * M * N * K
    other["linear_w8a16_8192x8192x4096"] = {"ms": ms, "tflops": fl / ms / 1e9, "frac_of_fp16_peak": fl / ms / 1e9 / pk}
    # split-KV decode of a single long sequence (the small-batch case the splits exist for): 128 pieces per
    # sequence keep every worker warp busy, and groups of sixteen pieces are merged in two levels
    B1, Hq1, Hkv1, S1, D1, splits1 = 1, 32, 8, 32768, 128, 128
    lens1 = torch.full((B1,), S1, dtype=torch.int32, device=dev)
    ws1 = torch.empty(binding.attn_decode_workspace_bytes(B1, Hq1, D1, splits1), dtype=torch.uint8, device=dev)
    binding.attn_decode_workspace_init(ws1)
    ms = timed(lambda: (randn((B1, Hq1, D1)), randn((B1, Hkv1, S1, D1)), randn((B1, Hkv1, S1, D1)), empty((B1, Hq1, D1))),
               lambda d: binding.attn_decode_splitkv(d[0], d[1], d[2], lens1, splits1, D1 ** -0.5, out=d[3], workspace=ws1),
               nset=5)  # 5 x 134 MB
    by = 4 * Hkv1 * D1 * S1 + 4 * B1 * Hq1 * D1
    other["decode_B1_32k_context_128_splits"] = {"ms": ms, "gbs": by / ms / 1e6, "frac_of_hbm_peak": by / ms / 1e6 / peaks["hbm_gbs"],
                                                 "bytes": by}
    del ws1
    # a whole decoder layer of the 8B-class shape (QKV projection, causal GQA attention, output projection with
    # residual, SwiGLU MLP, down projection with residual) into its two planned buffers; one set of weights
    # (436 MB, larger than L2), rotating activations
    B, S, Hq, Hkv, D, F = 4, 2048, 32, 8, 128, 14336
    Hd, Nqkv, T = Hq * D, (Hq + 2 * Hkv) * D, B * S
    weights = {"w_qkv": randn((Hd, Nqkv), 0.02), "w_o": randn((Hd, Hd), 0.02), "w_gate": randn((Hd, F), 0.02),
               "w_up": randn((Hd, F), 0.02), "w_down": randn((F, Hd), 0.02)}
    plan = binding.decoder_layer_plan(B, S, Hq, Hkv, D, F)
    ws = torch.empty(max(int(plan.workspace_bytes), 256), dtype=torch.uint8, device=dev)
    ms = timed(lambda: (randn((T, Hd)), empty((T, Hd))),
               lambda d: binding.decoder_layer(d[0], weights, B, S, Hq, Hkv, D, F, out=d[1], workspace=ws))
    fl = 2 * T * Hd * (Nqkv + Hd + 3 * F) + 4 * D * B * Hq * (S * (S + 1) // 2)
    other["decoder_layer_8b_shape_B4_S2048"] = {
        "ms": ms, "tflops": fl / ms / 1e9, "frac_of_bf16_peak_sustained": fl / ms / 1e9 / peaks.get("bf16_tflops_sustained", pk),
        "flops": fl, "launches": 5, "intermediates": int(plan.num_regs), "buffers": int(plan.num_bufs), "rho_buf": float(plan.rho_buf),
        "workspace_bytes": int(plan.workspace_bytes), "unplanned_bytes": int(plan.unplanned_bytes)}
    del weights, ws
    return other


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=5, help="how often every K-step timed region is repeated")
    ap.add_argument("--cooldown", type=float, default=0.2, help="idle seconds before every timed region")
    ap.add_argument("--impl", default="forge", choices=["forge", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true")
    ap.add_argument("--dry-run-cpu", action="store_true", help="rank plumbing only, on CPU with gloo (for tests)")
    args = ap.parse_args(argv)
    rc = maybe_relaunch(args, argv)
    if rc is not None:
        return rc
    if args.dry_run_cpu:
        return run_dry(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
