"""Seeded input generator and the golden fixture (CPU only)."""
import os

import numpy as np
import torch

from paper_2405_18425_b200 import synth


def test_generator_is_deterministic_and_counter_based():
    a = synth.standard_normal(7, 2, 1000)
    b = synth.standard_normal(7, 2, 1000)
    np.testing.assert_array_equal(a, b)
    # element x depends only on (seed, stream, x): a sub-range is the same numbers
    np.testing.assert_array_equal(synth.standard_normal(7, 2, 100, first=250), a[250:350])
    assert np.abs(synth.standard_normal(8, 2, 1000) - a).max() > 0.1
    assert np.abs(synth.standard_normal(7, 3, 1000) - a).max() > 0.1


def test_generator_moments():
    z = synth.standard_normal(11, 0, 400_000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01
    assert abs((z ** 3).mean()) < 0.03 and abs((z ** 4).mean() - 3.0) < 0.1
    assert np.isfinite(z).all() and np.abs(z).max() < 9.0
    # neighbouring draws and different streams are uncorrelated
    assert abs(np.corrcoef(z[:-1], z[1:])[0, 1]) < 0.01
    assert abs(np.corrcoef(z, synth.standard_normal(11, 1, 400_000))[0, 1]) < 0.01


def test_bf16_rounding_matches_torch_rne():
    r = np.random.default_rng(0)
    x = np.concatenate([r.standard_normal(50_000) * 10.0 ** r.integers(-6, 6, 50_000),
                        np.array([0.0, -0.0, 1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -9, -2.5, 65504.0])])
    bits = synth.f64_to_bf16_bits(x)
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16)
    np.testing.assert_array_equal(bits, ref.view(torch.int16).numpy().view(np.uint16))
    np.testing.assert_array_equal(synth.bf16_bits_to_f64(bits), ref.to(torch.float64).numpy())


def test_configs_mirror_the_benchmark_list():
    shapes = [(c.B, c.H, c.L, c.dk, c.dv, c.dtype, c.gate_mean, c.seed) for c in synth.CONFIGS]
    assert shapes == [
        (1, 2, 64, 16, 32, "f32", 0.0, 0),
        (128, 4, 196, 24, 48, "bf16", 0.0, 1),
        (128, 6, 196, 32, 64, "bf16", 0.0, 2),
        (64, 12, 196, 32, 64, "bf16", 2.0, 3),
        (8, 4, 4096, 24, 48, "bf16", 0.0, 4),
    ]
    assert [c.algorithmic_bytes for c in synth.CONFIGS] == [65536, 38535168, 77070336, 77070336, 50331648]


def test_make_inputs_shapes_scale_and_unit_slices():
    cfg = synth.CONFIGS[0]
    x = synth.make_inputs(cfg)
    assert x["q"].shape == (1, 2, 64, 16) and x["v"].shape == (1, 2, 64, 32) and x["q"].dtype == np.float32
    cfg = synth.BiglaConfig("t", B=3, H=4, L=50, dk=24, dv=48, dtype="bf16", gate_mean=2.0, seed=5)
    x = synth.make_inputs(cfg)
    assert x["k"].dtype == np.uint16
    q = synth.stored_to_f64(x["q"], "bf16")
    assert abs(q.std() - 24 ** -0.5) < 0.01 and abs(synth.stored_to_f64(x["k"], "bf16").std() - 1.0) < 0.02
    assert abs(synth.stored_to_f64(x["g_bwd"], "bf16").mean() - 2.0) < 0.03
    part = synth.make_inputs(cfg, units=slice(5, 8))
    for name in x:
        full = x[name].reshape(12, 1, 50, -1)
        np.testing.assert_array_equal(part[name], full[5:8])


def test_golden_fixture_matches_oracle(oracle):
    """tests/golden/bigla_samples.txt was written by tests/golden/make_golden.py from the oracle alone."""
    path = os.path.join(os.path.dirname(__file__), "golden", "bigla_samples.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 60
    cache = {}
    for name, u, t, j, val in rows:
        cfg = synth.CONFIG_BY_NAME[name]
        key = (name, int(u))
        if key not in cache:
            x = synth.make_inputs(cfg, units=slice(int(u), int(u) + 1))
            f = {n: synth.stored_to_f64(a, cfg.dtype) for n, a in x.items()}
            cache[key] = oracle.bigla_fwd(f["q"], f["k"], f["v"], oracle.gate_prep(f["g_fwd"], cfg.tau),
                                          oracle.gate_prep(f["g_bwd"], cfg.tau))[0, 0]
        assert cache[key][int(t), int(j)] == float(val)
