"""GPU parity of the gradient of the forward pass (vig_bigla_bwd_*) against the fp64 gradient oracle
(oracle/backward.py) on the same seeded inputs.  Bars as for the forward pass, per gradient tensor:
max|gpu - oracle| <= 1e-4 (fp32) / 2e-2 (bf16) of max|oracle|."""
import numpy as np
import pytest
import torch

import paper_2405_18425_b200 as vig
from paper_2405_18425_b200 import synth

from helpers import TOL, device_to_f64, oracle_log_alpha, random_problem, rel_err, to_device, to_stored

pytestmark = pytest.mark.gpu

NAMES = ("dq", "dk", "dv", "dlog_alpha_fwd", "dlog_alpha_bwd")


def _run(oracle, cfg, x, d_out, units=None):
    """GPU gradient of the whole problem; the oracle on `units` (a slice of the flattened (b, h) units) or on all."""
    la_f = oracle_log_alpha(oracle, x["g_fwd"], cfg.dtype, cfg.tau)
    la_b = oracle_log_alpha(oracle, x["g_bwd"], cfg.dtype, cfg.tau)
    host = dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b, g=d_out)
    d = {n: to_device(a, cfg.dtype) for n, a in host.items()}
    outs = [torch.full_like(d[n], float("nan")) for n in ("q", "k", "v", "f", "b")]
    vig.vig_bigla_bwd(d["q"], d["k"], d["v"], d["f"], d["b"], d["g"], *outs)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    for n, a in host.items():   # inputs are never written
        np.testing.assert_array_equal(to_stored(d[n], cfg.dtype), a)
    sel = (lambda a: a) if units is None else (lambda a: a.reshape((-1, 1) + a.shape[2:])[units])
    f = lambda a: synth.stored_to_f64(sel(a), cfg.dtype)
    ref = oracle.bigla_bwd(f(x["q"]), f(x["k"]), f(x["v"]), f(la_f), f(la_b), f(d_out))
    got = [sel(device_to_f64(o, cfg.dtype)) for o in outs]
    return got, ref


def _check(got, ref, dtype, label=""):
    for name, g, r in zip(NAMES, got, ref):
        assert np.isfinite(g).all(), name
        err = rel_err(g, r)
        if label:
            print(f"observed {label} {name}: max|gpu-oracle|/max|oracle| = {err:.3e} (bar {TOL[dtype]:g})")
        assert err <= TOL[dtype], (name, err)


@pytest.mark.parametrize("dk,dv", [(16, 32), (24, 48), (32, 64), (8, 16), (40, 72), (64, 128)])
@pytest.mark.parametrize("L", [1, 2, 15, 16, 17, 100, 196, 300])
def test_bf16_gradient_small_and_ragged(oracle, dk, dv, L):
    """Lengths below, at and across the sixteen-token staging, one and two tokens, head sizes on and off the
    tensor-core path of the forward pass that supplies dv."""
    cfg, x = random_problem(4000 + L, 2, 2, L, dk, dv, "bf16", gate_mean=1.0)
    got, ref = _run(oracle, cfg, x, synth.make_grad_input(cfg))
    _check(got, ref, "bf16")


@pytest.mark.parametrize("dk,dv,L", [(16, 32, 7), (5, 3, 33), (32, 64, 130), (24, 48, 50), (3, 2, 6), (128, 128, 20)])
def test_f32_gradient_shapes(oracle, dk, dv, L):
    cfg, x = random_problem(4100 + L, 2, 2, L, dk, dv, "f32", gate_mean=0.5)
    got, ref = _run(oracle, cfg, x, synth.make_grad_input(cfg))
    _check(got, ref, "f32")


def test_gradient_strong_gates(oracle):
    """Gates far below one (log alpha down to about -1 per token): states die within a few tokens, the gate
    gradients are sums of strongly cancelling terms."""
    cfg, x = random_problem(4200, 2, 2, 150, 32, 64, "f32", gate_mean=-3.0, tau=4.0)
    got, ref = _run(oracle, cfg, x, synth.make_grad_input(cfg))
    _check(got, ref, "f32")


def test_bf16_gradient_with_a_unit_beyond_the_tensor_core_range(oracle):
    """One unit whose gates sum to about -80 over a chunk: the forward kernel that supplies dv hands that unit to its
    in-kernel recurrence (the counter says so); all five gradients must still meet the bar."""
    cfg, x = random_problem(4300, 2, 3, 196, 32, 64, "bf16", gate_mean=1.0)
    g = synth.stored_to_f64(x["g_bwd"], "bf16").copy()
    g[1, 1, 10:140] = -10.0            # log alpha< = -10 / 16 per token; moved by one token it gates dv's forward pass
    x["g_bwd"] = synth.store(g, "bf16")
    vig.vig_test_take_fallback_count()
    got, ref = _run(oracle, cfg, x, synth.make_grad_input(cfg))
    assert vig.vig_test_take_fallback_count() == 1
    _check(got, ref, "bf16")


@pytest.mark.parametrize("idx", [0, 1, 3, 4], ids=[synth.CONFIGS[i].name for i in (0, 1, 3, 4)])
def test_gradient_benchmark_config_full_size(oracle, idx):
    """Configurations at full size through the entry point the benchmark times; the oracle (which keeps every state of
    the sequence) on a sample of units spread over the batch: units are independent."""
    cfg = synth.CONFIGS[idx]
    x, g = synth.make_inputs(cfg), synth.make_grad_input(cfg)
    step = max(1, cfg.units // 6)
    units = slice(0, cfg.units, step) if cfg.L <= 256 else slice(0, cfg.units, max(1, cfg.units // 2))
    got, ref = _run(oracle, cfg, x, g, units)
    _check(got, ref, cfg.dtype, cfg.name)


def test_gradient_entry_point_validates_arguments():
    lib = vig.load()
    buf = torch.zeros(1 << 16, device="cuda", dtype=torch.bfloat16)
    p = buf.data_ptr()
    before = vig.vig_kernel_launch_count()
    args = [p + 8192 * n for n in range(11)]   # eleven separate 4096-element regions
    assert lib.vig_bigla_bwd_bf16(*args, 1, 1, 8, 16, 32, None) == 0
    torch.cuda.synchronize()
    launched = vig.vig_kernel_launch_count() - before
    assert launched >= 3                                                        # gates moved, forward pass for dv, the walks
    for missing in range(11):
        a = list(args)
        a[missing] = None
        assert lib.vig_bigla_bwd_bf16(*a, 1, 1, 8, 16, 32, None) == -1
    a = list(args)
    a[7] = p + 2
    assert lib.vig_bigla_bwd_bf16(*a, 1, 1, 8, 16, 32, None) == -4
    assert lib.vig_bigla_bwd_bf16(*args, 1, -1, 8, 16, 32, None) == -2
    assert lib.vig_bigla_bwd_bf16(*args, 1, 1, 8, 200, 32, None) == -3          # head size beyond the kernel's
    assert lib.vig_bigla_bwd_bf16(*args, 0, 1, 8, 16, 32, None) == 0            # empty
    assert vig.vig_kernel_launch_count() - before == launched


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("shape", [(2, 3, 196, 32), (1, 1, 1, 8), (1, 2, 5, 3), (3, 1, 33, 20)])
def test_gate_prep_gradient_matches_oracle(oracle, dtype, shape):
    """dg = dlog_alpha * sigmoid(-g) / tau against the oracle, vector body and scalar tail, separately and in place."""
    r = np.random.default_rng(sum(shape))
    g = [synth.store(r.standard_normal(shape) * 3, dtype) for _ in range(2)]
    d = [synth.store(r.standard_normal(shape), dtype) for _ in range(2)]
    f = lambda a: synth.stored_to_f64(a, dtype)
    tg = [to_device(a, dtype) for a in g]
    td = [to_device(a, dtype) for a in d]
    out = [torch.full_like(t, float("nan")) for t in td]
    vig.vig_gate_prep_bwd(tg[0], tg[1], td[0], td[1], out[0], out[1], 16.0)
    vig.vig_gate_prep_bwd(tg[0], tg[1], td[0], td[1], td[0], td[1], 16.0)   # in place over the incoming gradients
    torch.cuda.synchronize()
    for x in range(2):
        ref = oracle.gate_prep_bwd(f(g[x]), f(d[x]), 16.0)
        assert rel_err(device_to_f64(out[x], dtype), ref) <= (2.0 ** -8 if dtype == "bf16" else 1e-6)
        np.testing.assert_array_equal(to_stored(out[x], dtype), to_stored(td[x], dtype))


@pytest.mark.parametrize("B,H,L,dk,dv", [(16, 4, 196, 32, 64), (2, 2, 1100, 24, 48), (3, 2, 300, 40, 72)])
def test_gradient_is_bitwise_reproducible(B, H, L, dk, dv):
    """Whole units, segmented walks and the element-wise staging: four calls on the same inputs give the same bytes (the
    asynchronous staging and the in-place results leave no room for a race that this would not show sooner or later)."""
    cfg, x = random_problem(4400 + L, B, H, L, dk, dv, "bf16", gate_mean=1.0)
    d = {n: to_device(a, "bf16") for n, a in x.items()}
    d["d_out"] = to_device(synth.make_grad_input(cfg), "bf16")
    la_f, la_b = torch.empty_like(d["g_fwd"]), torch.empty_like(d["g_bwd"])
    vig.vig_gate_prep_bf16(d["g_fwd"], d["g_bwd"], la_f, la_b, cfg.tau)
    first = None
    for _ in range(4):
        outs = [torch.full_like(d[n], float("nan")) for n in ("q", "k", "v", "q", "q")]
        vig.vig_bigla_bwd(d["q"], d["k"], d["v"], la_f, la_b, d["d_out"], *outs)
        torch.cuda.synchronize()
        got = [to_stored(o, "bf16") for o in outs]
        if first is None:
            first = got
        for a, b in zip(first, got):
            np.testing.assert_array_equal(a, b)
