"""GPU parity of the 2-D gating locality injection around the mixer (paper Eq. 7): the depth-wise 3x3 convolution, the
gate blend on its own, and the blend in the same call as the forward pass, each against the fp64 oracle (oracle/locality.py and
the Eq. 6 recurrence) on the same seeded inputs.  Bars as for the mixer: 1e-4 (fp32) / 2e-2 (bf16) of max|oracle|."""
import numpy as np
import pytest
import torch

import paper_2405_18425_b200 as vig
from paper_2405_18425_b200 import synth

from helpers import NTHREADS, TOL, device_to_f64, random_problem, rel_err, to_device, to_stored

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("B,Hh,Ww,C", [(2, 14, 14, 192), (1, 1, 1, 8), (3, 1, 9, 16), (2, 7, 1, 24), (1, 56, 56, 96),
                                       (2, 5, 6, 1024), (1, 64, 64, 200), (1, 3, 300, 8), (1, 19, 257, 8)])
def test_dwconv3x3_matches_oracle(oracle, dtype, B, Hh, Ww, C):
    """Grids with a single row, a single column or a single pixel (only some taps exist), the patch grids of the
    configurations, channel counts that are not powers of two; bias given and absent."""
    r = np.random.default_rng(B * 1000 + Hh * 10 + C)
    x = synth.store(r.standard_normal((B, Hh, Ww, C)), dtype)
    w = synth.store(r.standard_normal((C, 3, 3)) * 0.3, dtype)
    b = synth.store(r.standard_normal(C), dtype)
    f = lambda a: synth.stored_to_f64(a, dtype)
    for bias in (b, None):
        out = torch.full_like(to_device(x, dtype), float("nan"))
        vig.vig_dwconv3x3(to_device(x, dtype), to_device(w, dtype), to_device(bias, dtype) if bias is not None else None, out)
        torch.cuda.synchronize()
        ref = oracle.dwconv3x3(f(x), f(w), f(bias) if bias is not None else None)
        got = device_to_f64(out, dtype)
        assert np.isfinite(got).all()
        assert rel_err(got, ref) <= (1e-5 if dtype == "f32" else 2.0 ** -8)   # fp32 accumulation, one rounding to storage


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("n", [1, 7, 8, 4099, 196 * 64 * 5])
def test_gate_blend_matches_oracle(oracle, dtype, n):
    r = np.random.default_rng(n)
    a, z, c = (synth.store(r.standard_normal(n) * s, dtype) for s in (1.0, 4.0, 1.0))
    zz = synth.stored_to_f64(z, dtype).copy()
    zz[: min(n, 4)] = [90.0, -90.0, 0.0, -0.0][: min(n, 4)]            # both asymptotes and the midpoint
    z = synth.store(zz, dtype)
    f = lambda t: synth.stored_to_f64(t, dtype)
    out = torch.full_like(to_device(a, dtype), float("nan"))
    vig.vig_gate_blend(to_device(a, dtype), to_device(z, dtype), to_device(c, dtype), out)
    ref = oracle.gate_blend(f(a), f(z), f(c))
    got = device_to_f64(out, dtype)
    assert np.abs(got - ref).max() <= (2e-6 if dtype == "f32" else 2.0 ** -8) * max(1.0, np.abs(ref).max())
    # in place over the global branch
    cg = to_device(c, dtype)
    vig.vig_gate_blend(to_device(a, dtype), to_device(z, dtype), cg, cg)
    assert torch.equal(cg, out)


def _run_blend(oracle, cfg, x, loc):
    d = {n: to_device(a, cfg.dtype) for n, a in {**x, **loc}.items()}
    out = torch.full_like(d["v"], float("nan"))
    vig.vig_bigla_fwd_blend_bf16(d["q"], d["k"], d["v"], d["g_fwd"], d["g_bwd"], d["o_local"], d["z2d"], out, cfg.tau)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    for n, a in {**x, **loc}.items():   # inputs are never written
        np.testing.assert_array_equal(to_stored(d[n], cfg.dtype), a)
    f = lambda a: synth.stored_to_f64(a, cfg.dtype)
    glob = oracle.bigla_fwd(f(x["q"]), f(x["k"]), f(x["v"]), oracle.gate_prep(f(x["g_fwd"]), cfg.tau),
                            oracle.gate_prep(f(x["g_bwd"]), cfg.tau), nthreads=NTHREADS)
    return device_to_f64(out, cfg.dtype), oracle.gate_blend(f(loc["o_local"]), f(loc["z2d"]), glob)


@pytest.mark.parametrize("idx", [1, 2, 3, 4], ids=[c.name for c in synth.CONFIGS[1:]])
def test_fused_blend_full_size(oracle, idx):
    """Eq. 5 line 1 + Eq. 6 + Eq. 7 lines 3-4 in one call on the four bf16 configurations at full size (the 1024^2 one
    through the forward launches followed by the blend launch), every element compared."""
    cfg = synth.CONFIGS[idx]
    got, ref = _run_blend(oracle, cfg, synth.make_inputs(cfg), synth.make_locality_inputs(cfg))
    assert np.isfinite(got).all()
    err = rel_err(got, ref)
    print(f"fused blend {cfg.name}: max|gpu-oracle|/max|oracle| = {err:.3e}")
    assert err <= TOL["bf16"]


@pytest.mark.parametrize("dk,dv", [(16, 32), (24, 48), (32, 64), (40, 72)])
@pytest.mark.parametrize("L", [1, 17, 128, 129, 196, 256, 300])
def test_fused_blend_small_and_ragged(oracle, dk, dv, L):
    cfg, x = random_problem(3100 + L, 3, 2, L, dk, dv, "bf16", gate_mean=1.0)
    got, ref = _run_blend(oracle, cfg, x, synth.make_locality_inputs(cfg))
    assert np.isfinite(got).all()
    assert rel_err(got, ref) <= TOL["bf16"]


def test_fused_blend_gate_limits(oracle):
    """Gate logits far out: the call returns O_local where the 2-D gate is open and the mixer's output where it is shut."""
    cfg, x = random_problem(3300, 2, 2, 196, 32, 64, "bf16")
    loc = synth.make_locality_inputs(cfg)
    z = np.where(np.arange(64) < 32, 60.0, -60.0) * np.ones((2, 2, 196, 64))
    loc["z2d"] = synth.store(z, "bf16")
    got, ref = _run_blend(oracle, cfg, x, loc)
    assert rel_err(got, ref) <= TOL["bf16"]
    np.testing.assert_array_equal(got[..., :32], synth.stored_to_f64(loc["o_local"], "bf16")[..., :32])
    d = {n: to_device(a, "bf16") for n, a in x.items()}
    plain = torch.empty_like(d["v"])
    vig.vig_bigla_fwd_gates_bf16(d["q"], d["k"], d["v"], d["g_fwd"], d["g_bwd"], plain, cfg.tau)
    np.testing.assert_array_equal(got[..., 32:], device_to_f64(plain, "bf16")[..., 32:])


def test_fused_blend_on_a_unit_handed_to_the_recurrence(oracle):
    """A unit whose gates leave the range of the factorised tiles is evaluated by the recurrence inside the same launch;
    its output must be blended like every other unit's."""
    cfg, x = random_problem(3400, 2, 3, 196, 32, 64, "bf16")
    g = synth.stored_to_f64(x["g_fwd"], "bf16").copy()
    g[1, 1, 10:140] = -10.0            # log alpha = -10 / 16 per token: -80 over a chunk
    x["g_fwd"] = synth.store(g, "bf16")
    vig.vig_test_take_fallback_count()
    got, ref = _run_blend(oracle, cfg, x, synth.make_locality_inputs(cfg))
    assert vig.vig_test_take_fallback_count() == 1
    assert rel_err(got[1, 1], ref[1, 1]) <= TOL["bf16"]
    assert rel_err(got, ref) <= TOL["bf16"]


def test_dwconv3x3_many_channels_in_slabs(oracle):
    """More than 256 sixteen-byte channel groups: the groups are split over the grid's second dimension, raggedly."""
    rng = np.random.default_rng(77)
    B, Hh, Ww, C = 1, 5, 6, 2056
    x = synth.store(rng.standard_normal((B, Hh, Ww, C)), "bf16")
    w = synth.store(rng.standard_normal((C, 3, 3)) / 3, "bf16")
    b = synth.store(rng.standard_normal(C), "bf16")
    out = torch.full((B, Hh, Ww, C), float("nan"), device="cuda", dtype=torch.bfloat16)
    vig.vig_dwconv3x3(to_device(x, "bf16"), to_device(w, "bf16"), to_device(b, "bf16"), out)
    f = lambda a: synth.stored_to_f64(a, "bf16")
    ref = oracle.dwconv3x3(f(x), f(w), f(b))
    assert rel_err(device_to_f64(out, "bf16"), ref) <= TOL["bf16"]


def test_locality_entry_points_validate_arguments():
    lib = vig.load()
    buf = torch.empty(4096, device="cuda", dtype=torch.bfloat16)
    p = buf.data_ptr()
    before = vig.vig_kernel_launch_count()
    assert lib.vig_dwconv3x3_bf16(None, p, p, p, 1, 4, 4, 8, None) == -1
    assert lib.vig_dwconv3x3_bf16(p, p, None, p, 1, 4, 4, 12, None) == -3        # channels not a multiple of 8
    assert lib.vig_dwconv3x3_bf16(p, p, None, p, 1, -4, 4, 8, None) == -2
    assert lib.vig_dwconv3x3_bf16(p + 2, p, None, p, 1, 4, 4, 8, None) == -4
    assert lib.vig_dwconv3x3_bf16(p, p, None, p, 0, 4, 4, 8, None) == 0          # empty
    assert lib.vig_gate_blend_bf16(p, None, p, p, 16, None) == -1
    assert lib.vig_gate_blend_bf16(p, p, p, p, -1, None) == -2
    assert lib.vig_gate_blend_bf16(p, p, p, p, 0, None) == 0
    assert lib.vig_bigla_fwd_blend_bf16(p, p, p, p, p, None, p, p, 1, 1, 8, 16, 32, 16.0, None) == -1
    assert lib.vig_bigla_fwd_blend_bf16(p, p, p, p, p, p, p + 2, p, 1, 1, 8, 16, 32, 16.0, None) == -4
    assert vig.vig_kernel_launch_count() == before
