"""Shared helpers of the GPU parity tests: move stored inputs to the device, run the oracle."""
import os

import numpy as np
import torch

from paper_2405_18425_b200 import synth

NTHREADS = max(1, min(32, os.cpu_count() or 1))
TOL = {"f32": 1e-4, "bf16": 2e-2}     # max|gpu - oracle| <= TOL * max|oracle| over the whole output tensor


def to_device(stored: np.ndarray, dtype: str) -> torch.Tensor:
    """Stored array (float32, or uint16 bf16 bit patterns) -> CUDA tensor with the same bytes."""
    if dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(stored)).cuda()
    return torch.from_numpy(np.ascontiguousarray(stored).view(np.int16)).cuda().view(torch.bfloat16)


def to_stored(t: torch.Tensor, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return t.detach().cpu().numpy()
    return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)


def device_to_f64(t: torch.Tensor, dtype: str) -> np.ndarray:
    return synth.stored_to_f64(to_stored(t, dtype), dtype)


def oracle_log_alpha(oracle, g_stored, dtype, tau):
    """Oracle gate preparation on the stored logits, rounded to the storage dtype the way the
    un-fused path stores log alpha (round to nearest even).  Returns the stored array."""
    la = oracle.gate_prep(synth.stored_to_f64(g_stored, dtype), tau)
    return synth.store(la, dtype)


def oracle_out(oracle, q, k, v, la_f, la_b, dtype):
    f = lambda a: synth.stored_to_f64(a, dtype)
    return oracle.bigla_fwd(f(q), f(k), f(v), f(la_f), f(la_b), nthreads=NTHREADS)


def rel_err(gpu_f64: np.ndarray, ref: np.ndarray) -> float:
    scale = np.abs(ref).max()
    return float(np.abs(gpu_f64 - ref).max() / scale) if scale > 0 else float(np.abs(gpu_f64).max())


def random_problem(seed, B, H, L, dk, dv, dtype, gate_mean=0.0, tau=16.0):
    cfg = synth.BiglaConfig(f"rand{seed}", B=B, H=H, L=L, dk=dk, dv=dv, dtype=dtype, gate_mean=gate_mean,
                            seed=seed, tau=tau)
    return cfg, synth.make_inputs(cfg)
