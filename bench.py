#!/usr/bin/env python
"""Benchmark of the BiGLA forward hot path (gate preparation + bidirectional GLA scan) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole path over one batch of the workload: vig_gate_prep_bf16
(log alpha = logsigmoid(g)/tau for both directions) followed by vig_bigla_fwd_bf16, called through
the C ABI with device buffers.  Inputs are seeded synthetic tensors of the workload's shape that
are resident in HBM before the timed region; several buffer sets are rotated so that the bytes
touched between two uses of a set exceed twice the L2 capacity.  Prints ONE JSON line.

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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (None where no capture exists yet).
NCU_TRAFFIC_BYTES = {
    "vig_b_224": 59_593_216,    # bigla_umma_kernel<32,64>: 57.87 MB read + 1.72 MB written (profiles/bigla_umma_kernel_vig_b_224.md)
    # vig_t_1024 runs three launches per call; their captures (profiles/bigla_long_kernels_vig_t_1024.md) were taken with
    # flushed caches, which does not describe the L2-resident hand-over between them: no per-call figure is given.
}


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

    def __init__(self, index: int, period_s: float = 0.01):
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
    tdtype = torch.bfloat16

    # ---- resident inputs: several rotating sets, different seeds per set (same distribution) ----
    set_bytes = cfg.algorithmic_bytes + 2 * cfg.units * cfg.L * cfg.dk * cfg.elem_bytes   # + the two g tensors
    n_sets = max(3, int(np.ceil(2.0 * L2_BYTES / set_bytes)) + 1)
    host = synth.make_inputs(cfg)
    base = {n: torch.from_numpy(a.view(np.int16)).cuda().view(tdtype) for n, a in host.items()}
    sets = []
    for s in range(n_sets):
        d = {}
        for n, t in base.items():
            # a cheap re-draw for the extra sets: a rotation of the flattened tensor keeps the value
            # distribution and the [B,H,L,d] structure-free i.i.d. statistics of the generator
            d[n] = t if s == 0 else torch.roll(t.flatten(), 7919 * s).view_as(t).contiguous()
        d["la_f"] = torch.empty_like(d["g_fwd"])
        d["la_b"] = torch.empty_like(d["g_bwd"])
        d["out"] = torch.empty_like(d["v"])
        sets.append(d)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    dims = (cfg.B, cfg.H, cfg.L, cfg.dk)
    calls = []
    for d in sets:
        gate = (d["g_fwd"].data_ptr(), d["g_bwd"].data_ptr(), d["la_f"].data_ptr(), d["la_b"].data_ptr(),
                *dims, float(cfg.tau), sp)
        fwd = (d["q"].data_ptr(), d["k"].data_ptr(), d["v"].data_ptr(), d["la_f"].data_ptr(), d["la_b"].data_ptr(),
               d["out"].data_ptr(), cfg.B, cfg.H, cfg.L, cfg.dk, cfg.dv, sp)
        calls.append((gate, fwd))

    def step(i):
        gate, fwd = calls[i % n_sets]
        st = lib.vig_gate_prep_bf16(*gate)
        st |= lib.vig_bigla_fwd_bf16(*fwd)
        if st != 0:
            raise RuntimeError(f"C-ABI call failed with status {st}")

    sampler = ClockSampler(local_rank)
    sampler.start()
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()

    # ---- timed region 1: K steps back to back, one event pair around the region ----
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = vig.vig_kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_host0 = time.perf_counter()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    t_host1 = time.perf_counter()
    if dist is not None:
        dist.barrier()
    launches = vig.vig_kernel_launch_count() - launches0
    total_ms = vdist.max_over_ranks(e0.elapsed_time(e1), dist, device="cuda")   # slowest rank
    ms_per_step = total_ms / args.steps
    clocks = sampler.summary(t_host0, t_host1)

    # ---- timed region 2: the scan call alone, back to back over the same rotating sets (log alpha is in place from
    # the steps above), one event pair around the region -> average duration of one vig_bigla_fwd_bf16 call ----
    n_k = min(args.steps, 2000)
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(3):
        assert lib.vig_bigla_fwd_bf16(*calls[i % n_sets][1]) == 0
    torch.cuda.synchronize()
    k0.record(stream)
    for i in range(n_k):
        if lib.vig_bigla_fwd_bf16(*calls[i % n_sets][1]) != 0:
            raise RuntimeError("vig_bigla_fwd_bf16 failed")
    k1.record(stream)
    torch.cuda.synchronize()
    scan_us = k0.elapsed_time(k1) * 1e3 / n_k
    assert vig.vig_last_device_status() == 0, "a device-side bounded wait expired"

    tokens_per_step = cfg.tokens
    value = vdist.job_throughput(tokens_per_step, ms_per_step, world)
    peak, peak_kind = _peaks()
    achieved = cfg.algorithmic_bytes / (scan_us * 1e-6) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES.get(cfg.name), "peak_source": f"of {peak_kind}",
                "kernel": "vig_bigla_fwd_bf16 (all launches of one call)", "kernel_us": scan_us,
                "algorithmic_bytes": cfg.algorithmic_bytes}

    line = {
        "metric": "bigla_fwd_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "L": cfg.L, "dk": cfg.dk, "dv": cfg.dv,
                   "step": "vig_gate_prep_bf16 + vig_bigla_fwd_bf16", "parallelism": f"batch-sharded x{world}, no collective",
                   "l2": f"{n_sets} rotating buffer sets, {n_sets * set_bytes / 2**20:.0f} MiB touched per rotation (> 2x L2)"},
        "us_per_call": ms_per_step * 1e3, "scan_only_us": scan_us,
        "scan_only_tokens_per_s": tokens_per_step / (scan_us * 1e-6),
        "roofline": roofline, "clocks": clocks, "gpu_launches": int(launches),
    }

    if rank == 0:
        # ---- end to end through the host-buffer entry point (H2D + both kernels + D2H in the timed region) ----
        pinned = {n: torch.from_numpy(a.view(np.int16)).pin_memory() for n, a in host.items()}
        out_h = torch.empty(host["v"].shape, dtype=torch.int16).pin_memory()
        hp = (pinned["q"].data_ptr(), pinned["k"].data_ptr(), pinned["v"].data_ptr(), pinned["g_fwd"].data_ptr(),
              pinned["g_bwd"].data_ptr(), out_h.data_ptr(), cfg.B, cfg.H, cfg.L, cfg.dk, cfg.dv, float(cfg.tau),
              vig.VIG_DTYPE_BF16, sp)
        n_e2e = max(3, min(args.steps, 20))
        for _ in range(3):
            assert lib.vig_bigla_fwd_host(*hp) == 0
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            assert lib.vig_bigla_fwd_host(*hp) == 0      # synchronises the stream before returning
        t1 = time.perf_counter()
        h2d = sum(int(pinned[n].numel()) * 2 for n in ("q", "k", "v", "g_fwd", "g_bwd"))
        d2h = int(out_h.numel()) * 2
        line["e2e"] = {"value": tokens_per_step / ((t1 - t0) / n_e2e), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": 1e3 * (t1 - t0) / n_e2e,
                       "api": "vig_bigla_fwd_host (pinned host buffers)"}
        # the result of the last e2e step must be the device path's result for set 0
        ref = sets[0]["out"].view(torch.int16).cpu()
        step(0)
        torch.cuda.synchronize()
        line["e2e"]["matches_device_path"] = bool(torch.equal(sets[0]["out"].view(torch.int16).cpu(), out_h)) and \
            bool(torch.equal(ref, out_h))

        if world == 1:
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
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=[c.name for c in synth.CONFIGS if c.dtype == "bf16"])
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    cfg = synth.CONFIG_BY_NAME[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_gpu(args, cfg)


if __name__ == "__main__":
    main()
