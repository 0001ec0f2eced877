#!/usr/bin/env python
"""Benchmark of the BiGLA forward hot path (gate preparation + bidirectional GLA scan) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole path over one batch of the workload: gate preparation
(log alpha = logsigmoid(g)/tau for both directions) and the bidirectional scan, as the one call
vig_bigla_fwd_gates_bf16 through the C ABI with device buffers; the un-fused pair of calls
(vig_gate_prep_bf16, vig_bigla_fwd_bf16) and the scan call alone are timed beside it.  Inputs are
seeded synthetic tensors of the workload's shape that are resident in HBM before the timed region;
several buffer sets are rotated so that the bytes touched between two uses of a set exceed twice the
L2 capacity.  The K-step timed region is repeated (at least five times, at least 50 ms in all) and
the median is reported.  Prints ONE JSON line, which also carries shorter runs of the other bf16
workloads.

Under torchrun (N > 1) every rank runs the same workload on its own GPU (the (batch, head) units
are independent, so the path shards by batch with no collective: weak scaling); the timed region is
bracketed by a barrier + synchronize and the reported time is the maximum over ranks.

`--impl reference` times the fp64 CPU oracle (plain recurrence, as it stands) on the host cores
on a bounded sample of the same workload; it is a deliberately slow program and only a reported
baseline.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0
DEFAULT_WORKLOAD = "vig_b_224"

def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Polls SM clock, power and throttle reasons through NVML (read-only) while the benchmark runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period, self.samples, self._stop_evt = index, period_s, [], threading.Event()
        self.max_mhz = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                self.samples.append((time.perf_counter(),
                                     nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM),
                                     nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h),
                                     nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0))
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()

    def summary(self, t0: float, t1: float) -> dict:
        if self.nv is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        nv = self.nv
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = None
        if len(inside) < 3:   # a very short timed region: use every sample taken under load (warm-up included)
            inside, note = [s for s in self.samples if s[0] <= t1] or self.samples, "timed region shorter than the sampling period: warm-up samples included"
        names = {
            "hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
            "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
            "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
            "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap,
            "hw_power_brake": nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown,
        }
        mask = 0
        for s in inside:
            mask |= s[2]
        out = {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": self.max_mhz,
               "reasons": sorted(n for n, bit in names.items() if mask & bit),
               "power_w_max": max(s[3] for s in inside), "samples": len(inside)}
        if note:
            out["note"] = note
        return out


def _oracle_sample_units(cfg, budget_units=None):
    """Units of the workload the CPU legs run: a prefix of the (b, h) units, whole heads of whole images."""
    if budget_units is None:
        budget_units = cfg.units
    return max(cfg.H, min(cfg.units, budget_units) // cfg.H * cfg.H)


def _time_oracle(cfg, n_units, threads, passes=1):
    """`passes` oracle passes (gate preparation + Eq. 6 recurrence) over the first n_units units.
    Returns (seconds per pass, threads used)."""
    import oracle
    from paper_2405_18425_b200 import synth

    x = synth.make_inputs(cfg, units=slice(0, n_units))
    f = {n: synth.stored_to_f64(a, cfg.dtype) for n, a in x.items()}
    used = threads
    t0 = time.perf_counter()
    for _ in range(passes):
        la_f = oracle.gate_prep(f["g_fwd"], cfg.tau)
        la_b = oracle.gate_prep(f["g_bwd"], cfg.tau)
        _, _, _, used = oracle.bigla_fwd_directions(f["q"], f["k"], f["v"], la_f, la_b, nthreads=threads)
    return (time.perf_counter() - t0) / passes, used


def _cpu_baseline(cfg, threads, target_core_seconds=16.0):
    """The oracle, as it stands, on a bounded sample: whole passes over the workload until about
    `target_core_seconds` of CPU work (threads x wall time) have been spent."""
    n_units = _oracle_sample_units(cfg)
    probe, used = _time_oracle(cfg, n_units, threads, passes=1)
    passes = int(max(1, min(50, round(target_core_seconds / max(probe * used, 1e-3)))))
    secs, used = _time_oracle(cfg, n_units, threads, passes=passes)
    return {"value": (n_units // cfg.H * cfg.L) / secs, "unit": "tokens/s", "cores": used, "kind": "oracle",
            "seconds": secs * passes,
            "sample": f"{passes} passes over all {n_units} (b,h) units of the workload (about {secs * passes * used:.0f} core-seconds)"}


def run_reference(args, cfg):
    """The reference arm: the fp64 oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle

    oracle.build_oracle()
    threads = max(1, min(os.cpu_count() or 1, 64))
    n_units = _oracle_sample_units(cfg, budget_units=max(cfg.H, cfg.units // 8))
    steps, warmup = max(1, min(args.steps, 5)), max(1, min(args.warmup, 1))
    for _ in range(warmup):
        _time_oracle(cfg, n_units, threads)
    secs, used = [], threads
    for _ in range(steps):
        s, used = _time_oracle(cfg, n_units, threads)
        secs.append(s)
    tokens = n_units // cfg.H * cfg.L
    value = tokens / (sum(secs) / len(secs))
    sample = f"first {n_units} of {cfg.units} (b,h) units ({n_units // cfg.H} images) per step"
    line = {
        "impl": "reference", "metric": "bigla_fwd_tokens_per_s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * sum(secs) / len(secs),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "L": cfg.L, "dk": cfg.dk, "dv": cfg.dv,
                   "storage": cfg.dtype, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def _ncu_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per call of vig_bigla_fwd_bf16, per workload, from the table that is
    rewritten whenever the ncu captures under profiles/ are re-taken (workload, kernel, bytes, commit of the kernels)."""
    out = {}
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.txt")) as fh:
            for ln in fh:
                f = ln.split()
                if len(f) >= 4 and not ln.startswith("#"):
                    out[f[0]] = {"bytes": int(f[2]), "kernel": f[1], "kernels_at_commit": f[3]}
    except OSError:
        pass
    return out


class _Workload:
    """Rotating device buffer sets of one configuration and the three timed call sequences over them."""

    def __init__(self, cfg, lib, torch, stream):
        from paper_2405_18425_b200 import synth

        self.cfg, self.lib, self.torch, self.stream = cfg, lib, torch, stream
        self.set_bytes = cfg.algorithmic_bytes + 2 * cfg.units * cfg.L * cfg.dk * cfg.elem_bytes   # + the two g tensors
        self.n_sets = max(3, int(np.ceil(2.0 * L2_BYTES / self.set_bytes)) + 1)
        self.host = synth.make_inputs(cfg)
        base = {n: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16) for n, a in self.host.items()}
        self.sets = []
        for s in range(self.n_sets):
            d = {}
            for n, t in base.items():
                # a cheap re-draw for the extra sets: a rotation of the flattened tensor keeps the value
                # distribution and the [B,H,L,d] structure-free i.i.d. statistics of the generator
                d[n] = t if s == 0 else torch.roll(t.flatten(), 7919 * s).view_as(t).contiguous()
            if s == 0:
                loc = synth.make_locality_inputs(cfg)
                d["o_local"], d["z2d"] = (torch.from_numpy(loc[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("o_local", "z2d"))
            else:   # the blend's two extra inputs of the other sets: rotations of set 0's, like the other tensors
                d["o_local"] = torch.roll(self.sets[0]["o_local"].flatten(), 7919 * s).view_as(d["v"]).contiguous()
                d["z2d"] = torch.roll(self.sets[0]["z2d"].flatten(), 7919 * s).view_as(d["v"]).contiguous()
            # the gradient call: d_out in (stream 7 of the generator; rotations for the other sets), five gradients out
            if s == 0:
                d["d_out"] = torch.from_numpy(synth.make_grad_input(cfg).view(np.int16)).cuda().view(torch.bfloat16)
            else:
                d["d_out"] = torch.roll(self.sets[0]["d_out"].flatten(), 7919 * s).view_as(d["v"]).contiguous()
            for n, like in (("dq", "q"), ("dk", "k"), ("dv", "v"), ("dla_f", "q"), ("dla_b", "q")):
                d[n] = torch.empty_like(d[like])
            d["la_f"] = torch.empty_like(d["g_fwd"])
            d["la_b"] = torch.empty_like(d["g_bwd"])
            d["out"] = torch.empty_like(d["v"])
            self.sets.append(d)
        sp = stream.cuda_stream
        dims = (cfg.B, cfg.H, cfg.L, cfg.dk)
        self.calls = []
        for d in self.sets:
            gate = (d["g_fwd"].data_ptr(), d["g_bwd"].data_ptr(), d["la_f"].data_ptr(), d["la_b"].data_ptr(),
                    *dims, float(cfg.tau), sp)
            fwd = (d["q"].data_ptr(), d["k"].data_ptr(), d["v"].data_ptr(), d["la_f"].data_ptr(), d["la_b"].data_ptr(),
                   d["out"].data_ptr(), cfg.B, cfg.H, cfg.L, cfg.dk, cfg.dv, sp)
            fused = (d["q"].data_ptr(), d["k"].data_ptr(), d["v"].data_ptr(), d["g_fwd"].data_ptr(), d["g_bwd"].data_ptr(),
                     d["out"].data_ptr(), cfg.B, cfg.H, cfg.L, cfg.dk, cfg.dv, float(cfg.tau), sp)
            blend = (d["q"].data_ptr(), d["k"].data_ptr(), d["v"].data_ptr(), d["g_fwd"].data_ptr(), d["g_bwd"].data_ptr(),
                     d["o_local"].data_ptr(), d["z2d"].data_ptr(), d["out"].data_ptr(), cfg.B, cfg.H, cfg.L, cfg.dk, cfg.dv,
                     float(cfg.tau), sp)
            bwd = (d["q"].data_ptr(), d["k"].data_ptr(), d["v"].data_ptr(), d["la_f"].data_ptr(), d["la_b"].data_ptr(),
                   d["d_out"].data_ptr(), d["dq"].data_ptr(), d["dk"].data_ptr(), d["dv"].data_ptr(), d["dla_f"].data_ptr(),
                   d["dla_b"].data_ptr(), cfg.B, cfg.H, cfg.L, cfg.dk, cfg.dv, sp)
            self.calls.append((gate, fwd, fused, blend, bwd))

    # one step of each kind on buffer set i
    def fused(self, i):
        if self.lib.vig_bigla_fwd_gates_bf16(*self.calls[i % self.n_sets][2]) != 0:
            raise RuntimeError("vig_bigla_fwd_gates_bf16 failed")

    def unfused(self, i):
        gate, fwd = self.calls[i % self.n_sets][:2]
        if (self.lib.vig_gate_prep_bf16(*gate) | self.lib.vig_bigla_fwd_bf16(*fwd)) != 0:
            raise RuntimeError("vig_gate_prep_bf16 + vig_bigla_fwd_bf16 failed")

    def blend(self, i):
        if self.lib.vig_bigla_fwd_blend_bf16(*self.calls[i % self.n_sets][3]) != 0:
            raise RuntimeError("vig_bigla_fwd_blend_bf16 failed")

    def dwconv(self, i):
        """Depth-wise 3x3 convolution of Eq. 7 over the patch grid of the configuration, [B, sqrt(L), sqrt(L), H dv] channels last:
        the bytes of an O_local tensor serve as the image, those of `out` take the result."""
        cfg, d = self.cfg, self.sets[i % self.n_sets]
        side = int(round(cfg.L ** 0.5))
        if side * side != cfg.L:
            raise RuntimeError("the patch grid of this workload is not square")
        if not hasattr(self, "dw_w"):
            g = self.torch.Generator(device="cuda").manual_seed(cfg.seed)
            self.dw_w = (self.torch.randn(cfg.H * cfg.dv, 3, 3, device="cuda", generator=g) / 3).to(self.torch.bfloat16)
            self.dw_b = self.torch.randn(cfg.H * cfg.dv, device="cuda", generator=g).to(self.torch.bfloat16)
        if self.lib.vig_dwconv3x3_bf16(d["o_local"].data_ptr(), self.dw_w.data_ptr(), self.dw_b.data_ptr(), d["out"].data_ptr(),
                                       cfg.B, side, side, cfg.H * cfg.dv, self.stream.cuda_stream) != 0:
            raise RuntimeError("vig_dwconv3x3_bf16 failed")

    def bwd(self, i):   # (log alpha of every set is in place once the un-fused step has run over the sets)
        if self.lib.vig_bigla_bwd_bf16(*self.calls[i % self.n_sets][4]) != 0:
            raise RuntimeError("vig_bigla_bwd_bf16 failed")

    def scan(self, i):
        if self.lib.vig_bigla_fwd_bf16(*self.calls[i % self.n_sets][1]) != 0:
            raise RuntimeError("vig_bigla_fwd_bf16 failed")

    def time(self, fn, steps, warmup, min_total_ms, dist=None, vdist=None):
        """`steps` calls between one CUDA event pair on the launching stream, repeated at least five times and until
        min_total_ms of device time have been spent; every repeat is bracketed by a barrier + synchronize and counts with
        the slowest rank's time.  Returns the per-step times (ms) of the repeats and the host time stamps around them."""
        torch = self.torch
        for i in range(warmup):
            fn(i)
        torch.cuda.synchronize()
        per_step, total, rep = [], 0.0, 0
        t0 = time.perf_counter()
        while rep < 5 or total < min_total_ms:
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            for i in range(steps):
                fn(rep * steps + i)
            e1.record(self.stream)
            torch.cuda.synchronize()
            if dist is not None:
                dist.barrier()
            ms = e0.elapsed_time(e1)
            if vdist is not None:
                ms = vdist.max_over_ranks(ms, dist, device="cuda")   # slowest rank
            per_step.append(ms / steps)
            total += ms
            rep += 1
            if rep >= 2000:
                break
        return per_step, t0, time.perf_counter()


def _summary(per_step_ms):
    a = np.asarray(per_step_ms)
    return {"median_us": float(np.median(a) * 1e3), "min_us": float(a.min() * 1e3), "max_us": float(a.max() * 1e3),
            "repeats": int(a.size)}


def run_profile(args, cfg):
    """A handful of launches of one call sequence over the rotating sets, for a profiler to capture."""
    import torch

    import paper_2405_18425_b200 as vig

    torch.cuda.set_device(0)
    lib = vig.load()
    w = _Workload(cfg, lib, torch, torch.cuda.current_stream())
    fn = {"fused": w.fused, "unfused": w.unfused, "scan": w.scan, "bwd": w.bwd, "dwconv": w.dwconv, "blend": w.blend}[args.profile]
    if args.profile in ("scan", "bwd"):
        w.unfused(0)   # log alpha of set 0 in place; the other sets' log alpha buffers hold arbitrary finite values
        for d in w.sets[1:]:
            d["la_f"].copy_(w.sets[0]["la_f"])
            d["la_b"].copy_(w.sets[0]["la_b"])
    torch.cuda.synchronize()
    for i in range(args.warmup + args.steps):
        fn(i)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    print(json.dumps({"profile": args.profile, "workload": cfg.name, "launch_sequences": args.warmup + args.steps}))


def run_gpu(args, cfg):
    import torch

    import paper_2405_18425_b200 as vig
    from paper_2405_18425_b200 import dist as vdist
    from paper_2405_18425_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    lib = vig.load()   # raises if the CUDA library is missing: there is no fallback path

    if cfg.dtype != "bf16":
        raise SystemExit("the benchmark workloads are the bf16 configurations")
    stream = torch.cuda.current_stream()
    peak, peak_kind = _peaks()
    traffic = _ncu_traffic()

    def roofline_of(c, us, kernel):
        achieved = c.algorithmic_bytes / (us * 1e-6) / 1e9
        t = traffic.get(c.name)
        return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": t["bytes"] if t else None, "traffic_source": t, "peak_source": f"of {peak_kind}",
                "kernel": kernel, "kernel_us": us, "algorithmic_bytes": c.algorithmic_bytes}

    # ---- the headline workload: fused step (the step of `value`), un-fused step, scan call alone ----
    sampler = ClockSampler(local_rank)
    sampler.start()
    w = _Workload(cfg, lib, torch, stream)
    launches0 = vig.vig_kernel_launch_count()
    step_ms, t_host0, t_host1 = w.time(w.fused, args.steps, args.warmup, 50.0, dist, vdist)
    launches = vig.vig_kernel_launch_count() - launches0
    clocks = sampler.summary(t_host0, t_host1)
    unfused_ms, _, _ = w.time(w.unfused, args.steps, args.warmup, 20.0, dist, vdist)   # also leaves log alpha in place for the scan
    scan_ms, _, _ = w.time(w.scan, min(args.steps, 2000), args.warmup, 20.0, dist, vdist)
    blend_ms, _, _ = w.time(w.blend, min(args.steps, 2000), args.warmup, 20.0, dist, vdist)
    dw_ms, _, _ = w.time(w.dwconv, min(args.steps, 2000), args.warmup, 10.0, dist, vdist)
    bwd_ms, _, _ = w.time(w.bwd, min(args.steps, 200), args.warmup, 20.0, dist, vdist)
    assert vig.vig_last_device_status() == 0, "a device-side bounded wait expired"
    ms_per_step = float(np.median(step_ms))
    scan_us = float(np.median(scan_ms)) * 1e3
    tokens_per_step = cfg.tokens
    value = vdist.job_throughput(tokens_per_step, ms_per_step, world)

    line = {
        "metric": "bigla_fwd_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "L": cfg.L, "dk": cfg.dk, "dv": cfg.dv,
                   "step": "vig_bigla_fwd_gates_bf16 (gate preparation fused into the forward pass)",
                   "parallelism": f"batch-sharded x{world}, no collective",
                   "l2": f"{w.n_sets} rotating buffer sets, {w.n_sets * w.set_bytes / 2**20:.0f} MiB touched per rotation (> 2x L2)",
                   "timing": f"{len(step_ms)} repeats of the {args.steps}-step region, median reported"},
        "us_per_call": ms_per_step * 1e3, "step_spread": _summary(step_ms),
        "unfused_step": dict(_summary(unfused_ms), step="vig_gate_prep_bf16 + vig_bigla_fwd_bf16"),
        "scan_only_us": scan_us, "scan_only": _summary(scan_ms),
        "scan_only_tokens_per_s": tokens_per_step / (scan_us * 1e-6),
        # the forward kernel proper, vig_bigla_fwd_bf16 (log alpha in), timed back to back over the rotating sets
        "roofline": roofline_of(cfg, scan_us, "vig_bigla_fwd_bf16 (all launches of one call)"),
        # the single kernel of the fused step: the same algorithmic bytes (g in place of log alpha) plus the gate arithmetic
        "roofline_step": roofline_of(cfg, ms_per_step * 1e3, "vig_bigla_fwd_gates_bf16"),
        "clocks": clocks, "gpu_launches": int(launches),
    }
    line["roofline_step"]["traffic"] = None   # no capture of the fused kernel yet
    # the layer's call with the 2-D gate blend of the locality injection behind the forward pass: two more [B,H,L,dv] inputs
    blend_bytes = cfg.algorithmic_bytes + 2 * cfg.units * cfg.L * cfg.dv * cfg.elem_bytes
    blend_us = float(np.median(blend_ms)) * 1e3
    line["blend_step"] = dict(_summary(blend_ms), step="vig_bigla_fwd_blend_bf16", algorithmic_bytes=blend_bytes,
                              achieved_gbs=blend_bytes / (blend_us * 1e-6) / 1e9, frac=blend_bytes / (blend_us * 1e-6) / 1e9 / peak)

    # the depth-wise convolution in front of the mixer (Eq. 7 line 1): one read and one write of [B, L, H dv]
    dw_bytes = 2 * cfg.units * cfg.L * cfg.dv * cfg.elem_bytes
    dw_us = float(np.median(dw_ms)) * 1e3
    line["dwconv_step"] = dict(_summary(dw_ms), step="vig_dwconv3x3_bf16", algorithmic_bytes=dw_bytes,
                               achieved_gbs=dw_bytes / (dw_us * 1e-6) / 1e9, frac=dw_bytes / (dw_us * 1e-6) / 1e9 / peak)
    # the gradient call (log alpha and d_out in, five gradients out): 8 dk + 3 dv elements per token-head cross HBM; the two
    # recurrence walks do 20 dk dv fp32 flops per token-head on the CUDA cores (peak: SMs x 128 lanes x 2 x max SM clock)
    bwd_bytes = cfg.units * cfg.L * (8 * cfg.dk + 3 * cfg.dv) * cfg.elem_bytes
    bwd_us = float(np.median(bwd_ms)) * 1e3
    walk_flops = 20.0 * cfg.dk * cfg.dv * cfg.units * cfg.L
    alu_peak = torch.cuda.get_device_properties(0).multi_processor_count * 128 * 2 * 1.965e9
    line["bwd_step"] = dict(_summary(bwd_ms), step="vig_bigla_bwd_bf16", algorithmic_bytes=bwd_bytes,
                            achieved_gbs=bwd_bytes / (bwd_us * 1e-6) / 1e9, frac_hbm=bwd_bytes / (bwd_us * 1e-6) / 1e9 / peak,
                            walk_fp32_tflops=walk_flops / (bwd_us * 1e-6) / 1e12, frac_alu=walk_flops / (bwd_us * 1e-6) / alu_peak,
                            tokens_per_s=tokens_per_step / (bwd_us * 1e-6),
                            roofline={"bound": "alu", "achieved": walk_flops / (bwd_us * 1e-6) / 1e12, "peak": alu_peak / 1e12,
                                      "unit": "TFLOP/s", "frac": walk_flops / (bwd_us * 1e-6) / alu_peak, "traffic": None,
                                      "peak_source": "SMs x 128 fp32 lanes x 2 x 1.965 GHz",
                                      "kernel": "bigla_bwd_kernel (the walks' flops over the time of the whole call)"})

    if rank == 0:
        # ---- end to end through the host-buffer entry point (H2D + kernels + D2H in the timed region) ----
        pinned = {n: torch.from_numpy(a.view(np.int16)).pin_memory() for n, a in w.host.items()}
        out_h = torch.empty(w.host["v"].shape, dtype=torch.int16).pin_memory()
        hp = (pinned["q"].data_ptr(), pinned["k"].data_ptr(), pinned["v"].data_ptr(), pinned["g_fwd"].data_ptr(),
              pinned["g_bwd"].data_ptr(), out_h.data_ptr(), cfg.B, cfg.H, cfg.L, cfg.dk, cfg.dv, float(cfg.tau),
              vig.VIG_DTYPE_BF16, stream.cuda_stream)
        n_e2e = max(5, min(args.steps, 20))
        for _ in range(3):
            assert lib.vig_bigla_fwd_host(*hp) == 0
        torch.cuda.synchronize()
        e2e_ms = []
        for _ in range(n_e2e):
            t0 = time.perf_counter()
            assert lib.vig_bigla_fwd_host(*hp) == 0      # synchronises the stream before returning
            e2e_ms.append((time.perf_counter() - t0) * 1e3)
        h2d = sum(int(pinned[n].numel()) * 2 for n in ("q", "k", "v", "g_fwd", "g_bwd"))
        d2h = int(out_h.numel()) * 2
        e2e_med = float(np.median(e2e_ms))
        line["e2e"] = {"value": tokens_per_step / (e2e_med * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": e2e_med,
                       "ms_min": float(min(e2e_ms)), "ms_max": float(max(e2e_ms)),
                       "api": "vig_bigla_fwd_host (pinned host buffers, sliced copy / compute / copy-back pipeline)"}
        # the result of the last e2e step must be the device path's result for set 0
        w.fused(0)
        torch.cuda.synchronize()
        line["e2e"]["matches_device_path"] = bool(torch.equal(w.sets[0]["out"].view(torch.int16).cpu(), out_h))
        del pinned, out_h

    # ---- every bf16 workload, so that one record carries all shapes (shorter regions for the others) ----
    per = {cfg.name: {"us_per_call": ms_per_step * 1e3, "unfused_us_per_call": float(np.median(unfused_ms)) * 1e3,
                      "scan_only_us": scan_us, "bwd_us_per_call": bwd_us,
                      "roofline": {"frac": line["roofline"]["frac"], "traffic": line["roofline"]["traffic"]},
                      "B": cfg.B, "H": cfg.H, "L": cfg.L, "dk": cfg.dk, "dv": cfg.dv}}
    del w
    torch.cuda.empty_cache()
    if world == 1 and not args.only_headline:
        k_small = min(args.steps, 1000)
        pool = synth.CONFIGS + (synth.SWEEP_CONFIGS if args.sweep else ())
        for other in [c for c in pool if c.dtype == "bf16" and c.name != cfg.name]:
            wo = _Workload(other, lib, torch, stream)
            f_ms, _, _ = wo.time(wo.fused, k_small, args.warmup, 10.0)
            u_ms, _, _ = wo.time(wo.unfused, k_small, args.warmup, 10.0)
            s_ms, _, _ = wo.time(wo.scan, k_small, args.warmup, 10.0)
            s_us = float(np.median(s_ms)) * 1e3
            b_ms, _, _ = wo.time(wo.bwd, min(k_small, 20), args.warmup, 5.0)   # the gradient call (log alpha is in place)
            r = roofline_of(other, s_us, "vig_bigla_fwd_bf16")
            per[other.name] = {"us_per_call": float(np.median(f_ms)) * 1e3, "unfused_us_per_call": float(np.median(u_ms)) * 1e3,
                               "scan_only_us": s_us, "bwd_us_per_call": float(np.median(b_ms)) * 1e3, "roofline": {"frac": r["frac"], "traffic": r["traffic"]},
                               "B": other.B, "H": other.H, "L": other.L, "dk": other.dk, "dv": other.dv}
            del wo
            torch.cuda.empty_cache()
        assert vig.vig_last_device_status() == 0, "a device-side bounded wait expired"
    line["workloads"] = per

    if rank == 0 and world == 1:
        line["cpu_baseline"] = _cpu_baseline(cfg, max(1, min(os.cpu_count() or 1, 64)))
    sampler.stop()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


def main():
    from paper_2405_18425_b200 import synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=[c.name for c in synth.CONFIGS + synth.SWEEP_CONFIGS if c.dtype == "bf16"])
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--only-headline", action="store_true", help="skip the shorter runs of the other bf16 workloads")
    ap.add_argument("--sweep", action="store_true",
                    help="also time the second workload (resolution sweep, hierarchical stage shapes) in the `workloads` object")
    ap.add_argument("--profile", choices=["fused", "unfused", "scan", "bwd", "dwconv", "blend"],
                    help="for profilers: W warm-up and K steps of one call sequence only, nothing else is launched or timed")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    cfg = synth.CONFIG_BY_NAME[args.workload]
    if args.profile:
        run_profile(args, cfg)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_gpu(args, cfg)


if __name__ == "__main__":
    main()
