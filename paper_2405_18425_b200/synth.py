"""Seeded synthetic inputs for the BiGLA forward pass, and the benchmark configurations.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only draws numbers, scales q by dk^-0.5
(the paper's equations carry no scale, so the generator applies it) and rounds
to the storage dtype.  Gate logits g are returned raw; turning them into
log alpha is the job of the gate-preparation step on either side.

The generator is counter based and self contained, so the same seed yields the
same bytes on every machine and library version:
    word(seed, stream, n) = splitmix64 finaliser of (seed, stream, n)
    element x of a tensor uses words 2x and 2x+1 as two uniforms in (0, 1]
    and [0, 1), and the Box-Muller transform makes one standard normal of them.
Streams 0..4 are q, k, v, g_fwd, g_bwd, drawn in that order.

The inputs stand in for ImageNet-shaped ViG activations (patch size 16, so
L = 196 at 224x224 and L = 4096 at 1024x1024); the dataset, the trained weights
and the real gate statistics are not available, so the value distributions are
the ones the benchmark configurations state.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


@dataclass(frozen=True)
class BiglaConfig:
    name: str
    B: int
    H: int
    L: int
    dk: int
    dv: int
    dtype: str          # "f32" or "bf16": storage dtype of every tensor
    gate_mean: float    # gate logits ~ N(gate_mean, 1)
    seed: int
    tau: float = 16.0

    @property
    def units(self) -> int:
        return self.B * self.H

    @property
    def tokens(self) -> int:
        return self.B * self.L

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def algorithmic_bytes(self) -> int:
        """Read q, k, log alpha (2 directions), v once and write out once."""
        return (4 * self.dk + 2 * self.dv) * self.elem_bytes * self.B * self.H * self.L


# The five benchmark configurations (index = position in the configuration list).
CONFIGS = (
    BiglaConfig("tiny_8x8_f32", B=1, H=2, L=64, dk=16, dv=32, dtype="f32", gate_mean=0.0, seed=0),
    BiglaConfig("vig_t_224", B=128, H=4, L=196, dk=24, dv=48, dtype="bf16", gate_mean=0.0, seed=1),
    BiglaConfig("vig_s_224", B=128, H=6, L=196, dk=32, dv=64, dtype="bf16", gate_mean=0.0, seed=2),
    BiglaConfig("vig_b_224", B=64, H=12, L=196, dk=32, dv=64, dtype="bf16", gate_mean=2.0, seed=3),
    BiglaConfig("vig_t_1024", B=8, H=4, L=4096, dk=24, dv=48, dtype="bf16", gate_mean=0.0, seed=4),
)

# Second workload: the resolution sweep of the paper's efficiency figure (224^2 .. 2048^2 at patch size 16:
# L = 196 .. 16384, ViG-T-like heads, batch shrunk as the image grows so that the token count stays near 32 K)
# and the four stages of the hierarchical ViG-H-T at 224^2 (patch size 4: L = 3136, 784, 196, 49; channels
# 96 .. 768 over 3 .. 24 heads, i.e. dk = 16, dv = 32 per head).  Same value distributions as the benchmark
# configurations; they stand in for activations of those model variants, which are not available.
SWEEP_CONFIGS = (
    BiglaConfig("res_224", B=168, H=4, L=196, dk=24, dv=48, dtype="bf16", gate_mean=0.0, seed=11),
    BiglaConfig("res_448", B=42, H=4, L=784, dk=24, dv=48, dtype="bf16", gate_mean=0.0, seed=12),
    BiglaConfig("res_896", B=10, H=4, L=3136, dk=24, dv=48, dtype="bf16", gate_mean=0.0, seed=13),
    BiglaConfig("res_1024", B=8, H=4, L=4096, dk=24, dv=48, dtype="bf16", gate_mean=0.0, seed=14),
    BiglaConfig("res_2048", B=2, H=4, L=16384, dk=24, dv=48, dtype="bf16", gate_mean=0.0, seed=15),
    BiglaConfig("vig_h_t_stage1", B=16, H=3, L=3136, dk=16, dv=32, dtype="bf16", gate_mean=0.0, seed=21),
    BiglaConfig("vig_h_t_stage2", B=16, H=6, L=784, dk=16, dv=32, dtype="bf16", gate_mean=0.0, seed=22),
    BiglaConfig("vig_h_t_stage3", B=16, H=12, L=196, dk=16, dv=32, dtype="bf16", gate_mean=0.0, seed=23),
    BiglaConfig("vig_h_t_stage4", B=16, H=24, L=49, dk=16, dv=32, dtype="bf16", gate_mean=0.0, seed=24),
)
CONFIG_BY_NAME = {c.name: c for c in CONFIGS + SWEEP_CONFIGS}


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 output function on uint64 arrays (arithmetic wraps mod 2^64)."""
    with np.errstate(over="ignore"):
        x = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = x
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _words(seed: int, stream: int, first: int, count: int) -> np.ndarray:
    """count 64-bit words of (seed, stream), counters first .. first+count-1."""
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([(int(seed) * 0x51ED27 + 0x1234567) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
        key = _splitmix64(key ^ np.uint64((int(stream) + 1) * 0xD1B54A32D192ED03 & 0xFFFFFFFFFFFFFFFF))
        ctr = np.arange(first, first + count, dtype=np.uint64)
        return _splitmix64(ctr * np.uint64(0x2545F4914F6CDD1D) + key)


def standard_normal(seed: int, stream: int, count: int, first: int = 0) -> np.ndarray:
    """count i.i.d. N(0, 1) draws as fp64; element x depends only on (seed, stream, first + x)."""
    out = np.empty(count, dtype=np.float64)
    step = 1 << 20
    for lo in range(0, count, step):
        n = min(step, count - lo)
        w = _words(seed, stream, 2 * (first + lo), 2 * n)
        u1 = ((w[0::2] >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)  # (0, 1]
        u2 = (w[1::2] >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)          # [0, 1)
        out[lo:lo + n] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp64 -> bf16 (round to nearest even, via fp32) and return the uint16 bit patterns."""
    f = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    u = f.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    with np.errstate(over="ignore"):
        r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns as fp64."""
    u = np.ascontiguousarray(np.asarray(b, dtype=np.uint16)).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def store(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round an fp64 array to the storage dtype: float32 array for "f32", uint16 bf16 bits for "bf16"."""
    if dtype == "f32":
        return np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    if dtype == "bf16":
        return f64_to_bf16_bits(x)
    raise ValueError(f"unknown dtype {dtype!r}")


def stored_to_f64(a: np.ndarray, dtype: str) -> np.ndarray:
    """Exact fp64 copy of a stored array (inverse view of `store`)."""
    if dtype == "f32":
        return np.asarray(a, dtype=np.float32).astype(np.float64)
    if dtype == "bf16":
        return bf16_bits_to_f64(a)
    raise ValueError(f"unknown dtype {dtype!r}")


def make_inputs(cfg: BiglaConfig, units: slice | None = None) -> dict:
    """Stored q, k, v, g_fwd, g_bwd of a configuration.

    Returns arrays shaped [B, H, L, d] in the storage dtype (float32, or uint16
    bf16 bit patterns).  `units` selects a range of the flattened (b, h) units;
    the result is then [n_units, 1, L, d] and bit-identical to the same units of
    the full tensors, which lets a test draw a sample of a large configuration.
    """
    n_units = cfg.units
    lo, hi, _ = (units or slice(None)).indices(n_units)
    count_k = (hi - lo) * cfg.L * cfg.dk
    count_v = (hi - lo) * cfg.L * cfg.dv
    first_k = lo * cfg.L * cfg.dk
    first_v = lo * cfg.L * cfg.dv
    shape_k = (cfg.B, cfg.H, cfg.L, cfg.dk) if units is None else (hi - lo, 1, cfg.L, cfg.dk)
    shape_v = shape_k[:3] + (cfg.dv,)
    q = standard_normal(cfg.seed, 0, count_k, first_k) * (float(cfg.dk) ** -0.5)
    k = standard_normal(cfg.seed, 1, count_k, first_k)
    v = standard_normal(cfg.seed, 2, count_v, first_v)
    g_f = standard_normal(cfg.seed, 3, count_k, first_k) + cfg.gate_mean
    g_b = standard_normal(cfg.seed, 4, count_k, first_k) + cfg.gate_mean
    return {
        "q": store(q, cfg.dtype).reshape(shape_k),
        "k": store(k, cfg.dtype).reshape(shape_k),
        "v": store(v, cfg.dtype).reshape(shape_v),
        "g_fwd": store(g_f, cfg.dtype).reshape(shape_k),
        "g_bwd": store(g_b, cfg.dtype).reshape(shape_k),
    }


def make_locality_inputs(cfg: BiglaConfig, units: slice | None = None) -> dict:
    """Stored O_local and 2-D gate logits z of the locality injection (Eq. 7), [B, H, L, dv] like v and out: streams 5
    and 6 of the configuration's seed, both N(0, 1) (stand-ins for the depth-wise convolution's output laid out per
    head and for its projection O_local W + b).  `units` as in make_inputs."""
    lo, hi, _ = (units or slice(None)).indices(cfg.units)
    count, first = (hi - lo) * cfg.L * cfg.dv, lo * cfg.L * cfg.dv
    shape = (cfg.B, cfg.H, cfg.L, cfg.dv) if units is None else (hi - lo, 1, cfg.L, cfg.dv)
    return {
        "o_local": store(standard_normal(cfg.seed, 5, count, first), cfg.dtype).reshape(shape),
        "z2d": store(standard_normal(cfg.seed, 6, count, first), cfg.dtype).reshape(shape),
    }


def make_grad_input(cfg: BiglaConfig, units: slice | None = None) -> np.ndarray:
    """Stored d_out = dLoss/d_out of the gradient call, [B, H, L, dv] like out: stream 7 of the configuration's seed,
    N(0, 1) (a stand-in for what the layers after the mixer send back).  `units` as in make_inputs."""
    lo, hi, _ = (units or slice(None)).indices(cfg.units)
    count, first = (hi - lo) * cfg.L * cfg.dv, lo * cfg.L * cfg.dv
    shape = (cfg.B, cfg.H, cfg.L, cfg.dv) if units is None else (hi - lo, 1, cfg.L, cfg.dv)
    return store(standard_normal(cfg.seed, 7, count, first), cfg.dtype).reshape(shape)
