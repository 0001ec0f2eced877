"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded
inputs.  Bar: max|gpu - oracle| <= 1e-4 * max|oracle| for fp32 storage and <= 2e-2 * max|oracle|
for bf16 storage, the maximum taken over the whole output tensor."""
import os

import numpy as np
import pytest
import torch

import paper_2405_18425_b200 as vig
from paper_2405_18425_b200 import synth

from helpers import (NTHREADS, TOL, device_to_f64, oracle_log_alpha, oracle_out, random_problem, rel_err, to_device,
                     to_stored)

pytestmark = pytest.mark.gpu


def _fwd(dtype):
    return vig.vig_bigla_fwd_f32 if dtype == "f32" else vig.vig_bigla_fwd_bf16


def _run_unfused(oracle, cfg, x):
    """Oracle gate prep -> stored log alpha (same bytes for both sides) -> GPU forward vs oracle forward."""
    la_f = oracle_log_alpha(oracle, x["g_fwd"], cfg.dtype, cfg.tau)
    la_b = oracle_log_alpha(oracle, x["g_bwd"], cfg.dtype, cfg.tau)
    d = {n: to_device(a, cfg.dtype) for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    out = torch.empty_like(d["v"])
    _fwd(cfg.dtype)(d["q"], d["k"], d["v"], d["f"], d["b"], out)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    ref = oracle_out(oracle, x["q"], x["k"], x["v"], la_f, la_b, cfg.dtype)
    return device_to_f64(out, cfg.dtype), ref


@pytest.mark.parametrize("idx", range(len(synth.CONFIGS)), ids=[c.name for c in synth.CONFIGS])
def test_benchmark_config_full_size(oracle, idx):
    """All five configurations at full size, every output element compared."""
    cfg = synth.CONFIGS[idx]
    got, ref = _run_unfused(oracle, cfg, synth.make_inputs(cfg))
    assert np.isfinite(got).all()
    err = rel_err(got, ref)
    print(f"observed {cfg.name}: max|gpu-oracle|/max|oracle| = {err:.3e} (bar {TOL[cfg.dtype]:g})")   # shown with pytest -s
    assert err <= TOL[cfg.dtype]


@pytest.mark.parametrize("dk,dv", [(16, 32), (24, 48), (32, 64), (64, 128), (16, 48), (8, 16), (40, 72)])
@pytest.mark.parametrize("L", [1, 5, 16, 17, 33, 100, 250])
def test_bf16_small_and_ragged(oracle, dk, dv, L):
    """Lengths below, at and across the 16-token tile, several head sizes (the last two are not on
    the tensor-core path and exercise the SIMT recurrence kernel through the same entry point)."""
    cfg, x = random_problem(100 + L, 2, 3, L, dk, dv, "bf16")
    got, ref = _run_unfused(oracle, cfg, x)
    assert rel_err(got, ref) <= TOL["bf16"]


@pytest.mark.parametrize("dk,dv,L", [(16, 32, 7), (16, 32, 130), (24, 48, 50), (5, 3, 33), (128, 256, 20),
                                     (32, 64, 600)])
def test_f32_shapes(oracle, dk, dv, L):
    cfg, x = random_problem(200 + L, 2, 2, L, dk, dv, "f32")
    got, ref = _run_unfused(oracle, cfg, x)
    assert rel_err(got, ref) <= TOL["f32"]


@pytest.mark.parametrize("dk,dv", [(32, 64), (24, 48)])
@pytest.mark.parametrize("L", [127, 128, 129, 130, 144, 145, 208, 255, 256, 257, 258, 384, 385, 513])
def test_bf16_chunk_boundaries(oracle, dk, dv, L):
    """Lengths just below, at and just above a multiple of the 128-token chunk: a second (or last) chunk of one
    or two tokens, the hand-over of the running states across the boundary, the step from the single-block
    kernel (L <= 256) to the chunk-task kernels; several units per persistent block."""
    cfg, x = random_problem(700 + L, 5, 3, L, dk, dv, "bf16", gate_mean=1.0)
    got, ref = _run_unfused(oracle, cfg, x)
    assert np.isfinite(got).all()
    assert rel_err(got, ref) <= TOL["bf16"]


@pytest.mark.parametrize("case", range(24))
def test_bf16_random_shapes_repeatable(oracle, case):
    """Seeded random shapes on the tensor-core path (head sizes, lengths on both sides of the 128- and 256-token
    limits, one to several hundred units, slow and fast gates): parity with the oracle, and the same bits from
    three back-to-back calls (no result may depend on how the blocks and their pipelines happen to interleave)."""
    rng = np.random.default_rng(9000 + case)
    dk, dv = int(rng.choice([16, 24, 32])), int(rng.choice([32, 48, 64]))
    kind = case % 4
    L = int(rng.integers(1, 129)) if kind == 0 else int(rng.integers(129, 257)) if kind == 1 else \
        int(rng.integers(257, 900)) if kind == 2 else int(rng.choice([128, 196, 256, 384, 512]))
    units = int(rng.integers(1, 40)) if L > 256 else int(rng.integers(1, 700))
    B = int(rng.integers(1, min(units, 8) + 1))
    H = max(1, units // B)
    cfg, x = random_problem(9100 + case, B, H, L, dk, dv, "bf16", gate_mean=float(rng.choice([0.0, 2.0, -1.0, 4.0])))
    la_f = oracle_log_alpha(oracle, x["g_fwd"], cfg.dtype, cfg.tau)
    la_b = oracle_log_alpha(oracle, x["g_bwd"], cfg.dtype, cfg.tau)
    d = {n: to_device(a, cfg.dtype) for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    outs = []
    for _ in range(3):
        out = torch.full_like(d["v"], float("nan"))
        vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out)
        outs.append(out)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    assert all(torch.equal(outs[0].view(torch.int16), o.view(torch.int16)) for o in outs[1:])
    got = device_to_f64(outs[0], cfg.dtype)
    assert np.isfinite(got).all()
    assert rel_err(got, oracle_out(oracle, x["q"], x["k"], x["v"], la_f, la_b, cfg.dtype)) <= TOL["bf16"]


@pytest.mark.parametrize("L", [196, 700])
def test_cuda_graph_replay(L):
    """Gate preparation + forward captured into a CUDA graph (the programmatic dependent launches included; the long
    path with caller-owned scratch, so that nothing allocates during capture) and replayed: same bits as the direct calls."""
    B, H, dk, dv = 4, 6, 32, 64
    gen = torch.Generator(device="cuda").manual_seed(77 + L)
    def mk(d):
        return torch.randn(B, H, L, d, device="cuda", dtype=torch.bfloat16, generator=gen)
    q, k, v, gf, gb = mk(dk) * dk ** -0.5, mk(dk), mk(dv), mk(dk) + 1, mk(dk) + 1
    lf, lb, ref = torch.empty_like(gf), torch.empty_like(gb), torch.empty_like(v)
    ws = torch.empty(max(vig.vig_bigla_workspace_bytes(B, H, L, dk, dv), 256), dtype=torch.uint8, device="cuda")
    vig.vig_gate_prep_bf16(gf, gb, lf, lb, 16.0)
    vig.vig_bigla_fwd_ws_bf16(q, k, v, lf, lb, ref, ws)     # also the first call per device: one-time set-up before capture
    torch.cuda.synchronize()
    out = torch.zeros_like(v)
    s, g = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            vig.vig_gate_prep_bf16(gf, gb, lf, lb, 16.0, stream=s)
            vig.vig_bigla_fwd_ws_bf16(q, k, v, lf, lb, out, ws, stream=s)
    for _ in range(3):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert vig.vig_last_device_status() == 0
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_two_streams_interleaved(oracle):
    """Calls of different shapes issued alternately on two streams (the long path allocates its scratch per call
    on the stream it is given): every result equals, bit for bit, the one the same call gives on its own."""
    problems = []
    for i, (B, H, L, dk, dv) in enumerate([(3, 4, 196, 32, 64), (1, 3, 1000, 24, 48), (40, 5, 130, 16, 32), (2, 2, 600, 32, 64)]):
        cfg, x = random_problem(9500 + i, B, H, L, dk, dv, "bf16", gate_mean=1.0)
        la_f = oracle_log_alpha(oracle, x["g_fwd"], cfg.dtype, cfg.tau)
        la_b = oracle_log_alpha(oracle, x["g_bwd"], cfg.dtype, cfg.tau)
        d = {n: to_device(a, cfg.dtype) for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
        alone = torch.empty_like(d["v"])
        vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], alone)
        problems.append((d, alone))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = []
    for rep in range(3):
        for i, (d, _) in enumerate(problems):
            out = torch.full_like(d["v"], float("nan"))
            st = streams[(i + rep) % 2]
            st.wait_stream(torch.cuda.current_stream())
            vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out, stream=st)
            outs.append((i, out))
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    for i, out in outs:
        assert torch.equal(out.view(torch.int16), problems[i][1].view(torch.int16))


@pytest.fixture
def chunk_task_path():
    """Sequences of more than 256 tokens on the three chunk-task launches instead of the segmented launch."""
    vig.vig_test_set_kernel_preference(vig.VIG_TEST_KERNEL_CHUNK_TASKS)
    yield
    vig.vig_test_set_kernel_preference(vig.VIG_TEST_KERNEL_AUTO)


@pytest.fixture
def segment_path():
    """Sequences of 257 .. 8192 tokens on the segmented single launch whatever the segment and unit counts."""
    vig.vig_test_set_kernel_preference(vig.VIG_TEST_KERNEL_SEGMENTS)
    yield
    vig.vig_test_set_kernel_preference(vig.VIG_TEST_KERNEL_AUTO)


def _long_sequences(oracle, L):
    cfg, x = random_problem(300 + L, 1, 3, L, 24, 48, "bf16")
    got, ref = _run_unfused(oracle, cfg, x)
    assert rel_err(got, ref) <= TOL["bf16"]
    cfg, x = random_problem(301 + L, 1, 2, L, 32, 64, "bf16", gate_mean=2.0)
    got, ref = _run_unfused(oracle, cfg, x)
    assert rel_err(got, ref) <= TOL["bf16"]


@pytest.mark.parametrize("L", [600, 2049, 4096 + 37, 8192, 8192 + 5, 16384])
def test_bf16_long_sequences(oracle, L):
    """Sequences split into several segments with a ragged last segment: one block per 256-token segment inside one
    launch up to 8192 tokens, chunk tasks over three launches beyond."""
    _long_sequences(oracle, L)


@pytest.mark.parametrize("L", [300, 600, 2049, 4096 + 37])
def test_bf16_long_sequences_chunk_tasks(oracle, chunk_task_path, L):
    _long_sequences(oracle, L)


@pytest.mark.parametrize("L", [300, 600, 2049, 4096 + 37, 8192])
def test_bf16_long_sequences_segments(oracle, segment_path, L):
    _long_sequences(oracle, L)


@pytest.mark.parametrize("units,L", [(1, 257), (3, 384), (40, 513), (700, 300), (5, 8000), (37, 4096)])
def test_bf16_segmented_groups(oracle, segment_path, units, L):
    """The segmented launch with fewer units than groups, more units than groups (several rounds per block), a
    one-token last segment and the longest sequences; three calls must give the same bits."""
    cfg, x = random_problem(1300 + L, units, 1, L, 24, 48, "bf16", gate_mean=1.0)
    la_f = oracle_log_alpha(oracle, x["g_fwd"], cfg.dtype, cfg.tau)
    la_b = oracle_log_alpha(oracle, x["g_bwd"], cfg.dtype, cfg.tau)
    d = {n: to_device(a, cfg.dtype) for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    outs = []
    for _ in range(3):
        out = torch.full_like(d["v"], float("nan"))
        vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out)
        outs.append(out)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    assert all(torch.equal(outs[0].view(torch.int16), o.view(torch.int16)) for o in outs[1:])
    got = device_to_f64(outs[0], cfg.dtype)
    assert np.isfinite(got).all()
    assert rel_err(got, oracle_out(oracle, x["q"], x["k"], x["v"], la_f, la_b, cfg.dtype)) <= TOL["bf16"]


@pytest.mark.parametrize("dk,dv", [(32, 64), (24, 48)])
@pytest.mark.parametrize("L", [196, 700, 3000])
@pytest.mark.parametrize("gate", [-0.2, -0.35, -0.45, "mix"])
def test_steep_gates_inside_the_factorised_range(oracle, dk, dv, L, gate):
    """Gates whose sum over a 128-token chunk lies between -20 and -59: the growing operand factor reaches e^59, yet
    the unit must stay on the tensor-core tiles (the fallback counter stays at zero) and meet the bar."""
    cfg, x = random_problem(1700 + L, 2, 2, L, dk, dv, "bf16")
    rng = np.random.default_rng(L + dk)
    if gate == "mix":
        la = [-(0.16 + 0.29 * rng.random((2, 2, L, dk))) for _ in range(2)]      # -0.16 .. -0.45 per token
    else:
        la = [np.full((2, 2, L, dk), gate) for _ in range(2)]
    la_f, la_b = synth.store(la[0], "bf16"), synth.store(la[1], "bf16")
    totals = synth.stored_to_f64(la_f, "bf16")[0, 0, :128].sum(axis=0) if L >= 128 else None
    assert totals is None or (totals.min() > -60.0 and totals.max() < -20.0)
    d = {n: to_device(a, "bf16") for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    vig.vig_test_take_fallback_count()
    out = torch.empty_like(d["v"])
    vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out)
    assert vig.vig_last_device_status() == 0
    assert vig.vig_test_take_fallback_count() == 0
    got = device_to_f64(out, "bf16")
    ref = oracle_out(oracle, x["q"], x["k"], x["v"], la_f, la_b, "bf16")
    assert np.isfinite(got).all()
    assert rel_err(got, ref) <= TOL["bf16"]


def test_fallback_counter_counts_out_of_range_units(oracle):
    cfg, x = random_problem(1800, 2, 3, 196, 32, 64, "bf16")
    la = np.full((2, 3, 196, 32), -0.05)
    la[1, 1, 10:140] = -0.6          # 128 x -0.6 = -77 inside chunk 0 of one unit
    la_s = synth.store(la, "bf16")
    d = {n: to_device(a, "bf16") for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_s, b=la_s).items()}
    vig.vig_test_take_fallback_count()
    out = torch.empty_like(d["v"])
    vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out)
    assert vig.vig_test_take_fallback_count() == 1
    assert vig.vig_test_take_fallback_count() == 0
    assert rel_err(device_to_f64(out, "bf16"), oracle_out(oracle, x["q"], x["k"], x["v"], la_s, la_s, "bf16")) <= TOL["bf16"]


def test_expired_device_wait_is_reported_and_leaves_the_library_usable(oracle):
    """A bounded device-side wait that runs out (a test hook makes every block wait, for a few dozen polls, on an
    mbarrier nothing completes): the call returns, nothing is stored, the status reads VIG_ERR_DEVICE_TIMEOUT once,
    and the next ordinary call is correct."""
    cfg, x = random_problem(1900, 2, 2, 196, 32, 64, "bf16")
    la_f = oracle_log_alpha(oracle, x["g_fwd"], "bf16", 16.0)
    la_b = oracle_log_alpha(oracle, x["g_bwd"], "bf16", 16.0)
    d = {n: to_device(a, "bf16") for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    assert vig.vig_last_device_status() == 0
    out = torch.full_like(d["v"], 7.0)
    vig.vig_test_expire_next_wait()
    vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out)     # the call itself succeeds: the wait expires on the device
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == -7                                # VIG_ERR_DEVICE_TIMEOUT
    assert vig.status_string(-7) == "a bounded device-side wait expired"
    assert bool((out == 7.0).all())                                          # nothing was stored
    assert vig.vig_last_device_status() == 0                                 # read and cleared
    vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out)
    assert vig.vig_last_device_status() == 0
    assert rel_err(device_to_f64(out, "bf16"), oracle_out(oracle, x["q"], x["k"], x["v"], la_f, la_b, "bf16")) <= TOL["bf16"]


@pytest.mark.parametrize("name", [c.name for c in synth.SWEEP_CONFIGS])
def test_second_workload_resolution_sweep_and_hierarchical_stages(oracle, name):
    """The resolution sweep (L = 196 .. 16384) and the stage shapes of the hierarchical variant (dk = 16, dv = 32,
    L = 3136 .. 49) at full size through the fused entry point; a sample of units spread over the batch is compared
    with the oracle chain element by element (units are independent, so a unit's result does not depend on the batch)."""
    cfg = synth.CONFIG_BY_NAME[name]
    x = synth.make_inputs(cfg)
    d = {n: to_device(a, cfg.dtype) for n, a in x.items()}
    out = torch.full_like(d["v"], float("nan"))
    vig.vig_bigla_fwd_gates_bf16(d["q"], d["k"], d["v"], d["g_fwd"], d["g_bwd"], out, cfg.tau)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    got = device_to_f64(out, cfg.dtype).reshape(cfg.units, cfg.L, cfg.dv)
    assert np.isfinite(got).all()
    budget = max(2, min(cfg.units, int(2.0e5 // cfg.L)))          # about 2e5 tokens through the oracle
    pick = sorted(set(np.linspace(0, cfg.units - 1, budget).astype(int).tolist()))
    f = lambda n, dd: synth.stored_to_f64(x[n], cfg.dtype).reshape(cfg.units, 1, cfg.L, dd)[pick]
    ref = oracle.bigla_fwd(f("q", cfg.dk), f("k", cfg.dk), f("v", cfg.dv), oracle.gate_prep(f("g_fwd", cfg.dk), cfg.tau),
                           oracle.gate_prep(f("g_bwd", cfg.dk), cfg.tau), nthreads=NTHREADS)[:, 0]
    err = rel_err(got[pick], ref)
    print(f"observed {name}: {len(pick)} of {cfg.units} units, max|gpu-oracle|/max|oracle| = {err:.3e}")
    assert err <= TOL["bf16"]


def _gate_cases(L, dk, rng):
    zero = np.zeros((1, 1, L, dk))
    closed = np.full((1, 1, L, dk), -1.0e3)
    wall = zero.copy()
    wall[0, 0, L // 2] = -1.0e3
    mixed = -rng.random((1, 1, L, dk)) * np.where(rng.random((1, 1, L, dk)) < 0.1, 40.0, 0.05)
    steep = np.full((1, 1, L, dk), -6.0)            # decays by e^-96 inside a 16-token block
    return {"alpha_one": zero, "closed": closed, "wall": wall, "mixed": mixed, "steep": steep}


@pytest.mark.parametrize("case", ["alpha_one", "closed", "wall", "mixed", "steep"])
@pytest.mark.parametrize("dtype,dk,dv,L", [("bf16", 32, 64, 196), ("bf16", 24, 48, 700), ("f32", 16, 32, 64)])
def test_degenerate_gates(oracle, case, dtype, dk, dv, L):
    """alpha == 1 (plain linear attention), fully closed gates (only the s = t term survives), a single
    closed gate, and gates mixing slow decay with hard resets: the result must stay finite and match."""
    rng = np.random.default_rng(7)
    cfg, x = random_problem(400, 1, 2, L, dk, dv, dtype)
    la = [np.broadcast_to(_gate_cases(L, dk, rng)[case], (1, 2, L, dk)) for _ in range(2)]
    la_f, la_b = synth.store(la[0], dtype), synth.store(la[1], dtype)
    d = {n: to_device(a, dtype) for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    out = torch.empty_like(d["v"])
    _fwd(dtype)(d["q"], d["k"], d["v"], d["f"], d["b"], out)
    torch.cuda.synchronize()
    got = device_to_f64(out, dtype)
    ref = oracle_out(oracle, x["q"], x["k"], x["v"], la_f, la_b, dtype)
    assert np.isfinite(got).all()
    assert rel_err(got, ref) <= TOL[dtype]
    if case == "closed":
        f = lambda n: synth.stored_to_f64(x[n], dtype)
        diag = np.einsum("bhti,bhti->bht", f("q"), f("k"))[..., None] * f("v")
        assert rel_err(got, diag) <= TOL[dtype]


def test_mixed_units_fast_and_exact_paths(oracle):
    """One unit with out-of-range gates among ordinary units must not disturb its neighbours."""
    cfg, x = random_problem(500, 2, 3, 196, 32, 64, "bf16")
    la_f = synth.stored_to_f64(oracle_log_alpha(oracle, x["g_fwd"], "bf16", 16.0), "bf16")
    la_b = synth.stored_to_f64(oracle_log_alpha(oracle, x["g_bwd"], "bf16", 16.0), "bf16")
    la_f[1, 0, 40:60] = -7.0
    la_b[0, 2, 100:101] = -90.0
    la_f, la_b = synth.store(la_f, "bf16"), synth.store(la_b, "bf16")
    d = {n: to_device(a, "bf16") for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    out = torch.empty_like(d["v"])
    vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], out)
    got = device_to_f64(out, "bf16")
    ref = oracle_out(oracle, x["q"], x["k"], x["v"], la_f, la_b, "bf16")
    assert rel_err(got, ref) <= TOL["bf16"]
    for b in range(2):
        for h in range(3):
            assert rel_err(got[b, h], ref[b, h]) <= TOL["bf16"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gate_prep_matches_oracle(oracle, dtype):
    r = np.random.default_rng(3)
    g = np.concatenate([r.standard_normal(5000) * 3.0, np.array([0.0, -0.0, 50.0, -50.0, 88.0, -88.0, 200.0, -200.0,
                                                                  1e-3, -1e-3]), r.standard_normal(6) * 30.0])
    g = np.resize(g, (2, 3, 19, 44))                       # n = 5016 elements: vector body and scalar tail
    gs = synth.store(g, dtype)
    for tau in (16.0, 1.0, 3.0):
        gf, gb = to_device(gs, dtype), to_device(synth.store(-g, dtype), dtype)
        of, ob = torch.empty_like(gf), torch.empty_like(gb)
        fn = vig.vig_gate_prep_f32 if dtype == "f32" else vig.vig_gate_prep_bf16
        fn(gf, gb, of, ob, tau)
        torch.cuda.synchronize()
        for got_t, g_in in ((of, gs), (ob, synth.store(-g, dtype))):
            ref = oracle.gate_prep(synth.stored_to_f64(g_in, dtype), tau)
            got = device_to_f64(got_t, dtype)
            assert np.isfinite(got).all() and (got <= 0).all()
            # fp32 evaluation then rounding to storage: a few fp32 ulps, plus one storage ulp for bf16
            ulp = 2.0 ** -22 if dtype == "f32" else 2.0 ** -8
            assert np.all(np.abs(got - ref) <= ulp * np.abs(ref) + 1e-37)
    # in place
    gf = to_device(gs, dtype)
    keep = gf.clone()
    o2 = torch.empty_like(gf)
    fn(keep, keep.clone(), o2, torch.empty_like(gf), 16.0)
    gb = gf.clone()
    fn(gf, gb, gf, gb, 16.0)
    assert torch.equal(gf, o2)


def test_whole_path_gate_prep_then_forward(oracle):
    """GPU gate prep feeding the GPU forward, against the oracle chain from the same logits (the
    oracle keeps log alpha in fp64, the un-fused GPU path rounds it to bf16 in between)."""
    cfg = synth.CONFIGS[3]
    x = synth.make_inputs(cfg, units=slice(0, 24))
    d = {n: to_device(a, cfg.dtype) for n, a in x.items()}
    la_f, la_b = torch.empty_like(d["g_fwd"]), torch.empty_like(d["g_bwd"])
    vig.vig_gate_prep_bf16(d["g_fwd"], d["g_bwd"], la_f, la_b, cfg.tau)
    out = torch.empty_like(d["v"])
    vig.vig_bigla_fwd(d["q"], d["k"], d["v"], la_f, la_b, out)
    f = lambda n: synth.stored_to_f64(x[n], cfg.dtype)
    ref = oracle.bigla_fwd(f("q"), f("k"), f("v"), oracle.gate_prep(f("g_fwd"), cfg.tau),
                           oracle.gate_prep(f("g_bwd"), cfg.tau), nthreads=8)
    assert rel_err(device_to_f64(out, cfg.dtype), ref) <= TOL["bf16"]


def _run_fused(oracle, cfg, x, tau=None):
    """GPU forward from the gate logits against the oracle chain gate_prep -> bigla_fwd with fp64 gates in between."""
    tau = cfg.tau if tau is None else tau
    d = {n: to_device(a, cfg.dtype) for n, a in x.items()}
    out = torch.full_like(d["v"], float("nan"))
    vig.vig_bigla_fwd_gates_bf16(d["q"], d["k"], d["v"], d["g_fwd"], d["g_bwd"], out, tau)
    torch.cuda.synchronize()
    assert vig.vig_last_device_status() == 0
    f = lambda n: synth.stored_to_f64(x[n], cfg.dtype)
    ref = oracle.bigla_fwd(f("q"), f("k"), f("v"), oracle.gate_prep(f("g_fwd"), tau), oracle.gate_prep(f("g_bwd"), tau),
                           nthreads=NTHREADS)
    for n in x:   # inputs are never written
        np.testing.assert_array_equal(to_stored(d[n], cfg.dtype), x[n])
    return device_to_f64(out, cfg.dtype), ref


@pytest.mark.parametrize("idx", [1, 2, 3, 4], ids=[c.name for c in synth.CONFIGS[1:]])
def test_fused_gates_full_size(oracle, idx):
    """Eq. 5 line 1 + Eq. 6 in one call on the four bf16 configurations at full size, every element compared."""
    cfg = synth.CONFIGS[idx]
    got, ref = _run_fused(oracle, cfg, synth.make_inputs(cfg))
    assert np.isfinite(got).all()
    err = rel_err(got, ref)
    print(f"fused gates {cfg.name}: max|gpu-oracle|/max|oracle| = {err:.3e}")
    assert err <= TOL["bf16"]


@pytest.mark.parametrize("dk,dv", [(16, 32), (24, 48), (32, 64), (24, 64), (40, 72)])
@pytest.mark.parametrize("L", [1, 5, 16, 17, 100, 128, 129, 196, 250, 255, 256, 300])
def test_fused_gates_small_and_ragged(oracle, dk, dv, L):
    """Ragged lengths on both sides of the chunk boundary (the padded rows and columns of the gate tiles must stay
    out of the sums), the last shape off the tensor-core set, L = 300 through gate preparation into scratch."""
    cfg, x = random_problem(2100 + L, 3, 2, L, dk, dv, "bf16", gate_mean=1.0)
    got, ref = _run_fused(oracle, cfg, x)
    assert np.isfinite(got).all()
    assert rel_err(got, ref) <= TOL["bf16"]


@pytest.mark.parametrize("tau", [1.0, 3.0, 16.0, 64.0])
def test_fused_gates_temperature_and_extreme_logits(oracle, tau):
    """tau = 1 makes the gates steep (padded columns must not trip the range check), tau = 64 nearly open; logits
    of +-50 and -200 reach both asymptotes of logsigmoid, the last ones through the in-kernel recurrence."""
    cfg, x = random_problem(2300, 2, 3, 196, 24, 48, "bf16", gate_mean=2.0, tau=tau)
    got, ref = _run_fused(oracle, cfg, x)
    assert rel_err(got, ref) <= TOL["bf16"]
    g = synth.stored_to_f64(x["g_fwd"], "bf16").copy()
    g[0, 1, 30:34] = 50.0
    g[1, 0, 100:103] = -50.0
    g[1, 2, 7] = -200.0
    x2 = dict(x, g_fwd=synth.store(g, "bf16"), g_bwd=synth.store(g[:, :, ::-1].copy(), "bf16"))
    got, ref = _run_fused(oracle, cfg, x2, tau)
    assert np.isfinite(got).all()
    assert rel_err(got, ref) <= TOL["bf16"]


def test_fused_gates_match_unfused_chain_closely():
    """The fused kernel rounds log alpha to bf16 at the same point as the un-fused chain, so the two GPU results agree
    far inside the tolerance (not bit for bit: log alpha may round the other way here and there, which moves an
    output by a bf16 unit in the last place: up to 2^-8 of its own size)."""
    cfg = synth.CONFIGS[3]
    x = synth.make_inputs(cfg, units=slice(0, 48))
    d = {n: to_device(a, cfg.dtype) for n, a in x.items()}
    la_f, la_b = torch.empty_like(d["g_fwd"]), torch.empty_like(d["g_bwd"])
    vig.vig_gate_prep_bf16(d["g_fwd"], d["g_bwd"], la_f, la_b, cfg.tau)
    a, b = torch.empty_like(d["v"]), torch.empty_like(d["v"])
    vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], la_f, la_b, a)
    vig.vig_bigla_fwd_gates_bf16(d["q"], d["k"], d["v"], d["g_fwd"], d["g_bwd"], b, cfg.tau)
    torch.cuda.synchronize()
    fa, fb = device_to_f64(a, "bf16"), device_to_f64(b, "bf16")
    assert np.abs(fa - fb).max() <= 1e-2 * np.abs(fa).max()


@pytest.mark.parametrize("idx", [0, 3, 4])
def test_host_entry_point_matches_device_path(oracle, idx):
    """Host buffers in and out (pinned and pageable), the batch cut into slices inside the call: the same bits as the
    device entry points on the whole batch."""
    cfg = synth.CONFIGS[idx]
    n_units = min(cfg.units, 96 if idx == 3 else 16)   # config 4: enough bytes for the sliced pipeline
    x = synth.make_inputs(cfg, units=slice(0, n_units))
    host = {n: torch.from_numpy(a.view(np.int16) if cfg.dtype == "bf16" else a).pin_memory() for n, a in x.items()}
    out_h = torch.empty(x["v"].shape, dtype=host["v"].dtype).pin_memory()
    code = vig.VIG_DTYPE_F32 if cfg.dtype == "f32" else vig.VIG_DTYPE_BF16
    vig.vig_bigla_fwd_host(host["q"], host["k"], host["v"], host["g_fwd"], host["g_bwd"], out_h, cfg.tau, code)
    # the device calls the host path makes: the forward pass from the logits (bf16), gate preparation + forward (fp32)
    d = {n: to_device(a, cfg.dtype) for n, a in x.items()}
    out_d = torch.empty_like(d["v"])
    if cfg.dtype == "f32":
        la_f, la_b = torch.empty_like(d["g_fwd"]), torch.empty_like(d["g_bwd"])
        vig.vig_gate_prep_f32(d["g_fwd"], d["g_bwd"], la_f, la_b, cfg.tau)
        vig.vig_bigla_fwd_f32(d["q"], d["k"], d["v"], la_f, la_b, out_d)
    else:
        vig.vig_bigla_fwd_gates_bf16(d["q"], d["k"], d["v"], d["g_fwd"], d["g_bwd"], out_d, cfg.tau)
    torch.cuda.synchronize()
    ref_bytes = to_stored(out_d, cfg.dtype)
    got_bytes = out_h.numpy().view(np.uint16) if cfg.dtype == "bf16" else out_h.numpy()
    np.testing.assert_array_equal(got_bytes, ref_bytes)
    # and numpy arrays (pageable memory) work as well
    out_n = np.empty_like(x["v"])
    vig.vig_bigla_fwd_host(x["q"], x["k"], x["v"], x["g_fwd"], x["g_bwd"], out_n, cfg.tau, code)
    np.testing.assert_array_equal(out_n, ref_bytes)


def test_workspace_variant_and_determinism(oracle):
    cfg = synth.CONFIGS[4]
    x = synth.make_inputs(cfg, units=slice(0, 6))
    la_f = oracle_log_alpha(oracle, x["g_fwd"], "bf16", 16.0)
    la_b = oracle_log_alpha(oracle, x["g_bwd"], "bf16", 16.0)
    d = {n: to_device(a, "bf16") for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    need = vig.vig_bigla_workspace_bytes(6, 1, cfg.L, cfg.dk, cfg.dv)
    assert need > 0
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(2):
        o = torch.full_like(d["v"], float("nan"))
        vig.vig_bigla_fwd_ws_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], o, ws)
        outs.append(o)
        o = torch.full_like(d["v"], float("nan"))
        vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], o)
        outs.append(o)
    torch.cuda.synchronize()
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16))     # bit-identical run to run
    with pytest.raises(vig.VigError) as e:
        vig.vig_bigla_fwd_ws_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], outs[0], ws[: need - 256])
    assert e.value.status == -6


def test_short_sequence_determinism_and_streams(oracle):
    cfg = synth.CONFIGS[2]
    x = synth.make_inputs(cfg, units=slice(0, 40))
    la_f = oracle_log_alpha(oracle, x["g_fwd"], "bf16", 16.0)
    la_b = oracle_log_alpha(oracle, x["g_bwd"], "bf16", 16.0)
    d = {n: to_device(a, "bf16") for n, a in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items()}
    a = torch.empty_like(d["v"])
    vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], a)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    b = torch.full_like(d["v"], float("nan"))
    before = vig.vig_kernel_launch_count()
    with torch.cuda.stream(s):
        vig.vig_bigla_fwd_bf16(d["q"], d["k"], d["v"], d["f"], d["b"], b)
    s.synchronize()
    assert vig.vig_kernel_launch_count() > before
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    # inputs are never written
    for n, src in dict(q=x["q"], k=x["k"], v=x["v"], f=la_f, b=la_b).items():
        np.testing.assert_array_equal(to_stored(d[n], "bf16"), src)


def test_empty_calls_on_device():
    z = torch.empty(0, 2, 8, 16, device="cuda", dtype=torch.bfloat16)
    zv = torch.empty(0, 2, 8, 32, device="cuda", dtype=torch.bfloat16)
    # data_ptr() of an empty tensor is NULL, so pass a real allocation with a zero batch
    buf = torch.empty(64, device="cuda", dtype=torch.bfloat16)
    lib = vig.load()
    p = buf.data_ptr()
    assert lib.vig_bigla_fwd_bf16(p, p, p, p, p, p, 0, 2, 8, 16, 32, None) == 0
    assert lib.vig_bigla_fwd_f32(p, p, p, p, p, p, 2, 2, 0, 16, 32, None) == 0
    assert lib.vig_gate_prep_bf16(p, p, p, p, 2, 0, 8, 16, 16.0, None) == 0
    assert z.numel() == 0 and zv.numel() == 0


def test_golden_samples(oracle):
    """Sampled outputs of every configuration stored by tests/golden/make_golden.py (oracle only;
    gates kept in fp64 there, rounded to storage here, which the tolerance covers)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "bigla_samples.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    by_unit = {}
    for name, u, t, j, val in rows:
        by_unit.setdefault((name, int(u)), []).append((int(t), int(j), float(val)))
    for (name, u), samples in by_unit.items():
        cfg = synth.CONFIG_BY_NAME[name]
        x = synth.make_inputs(cfg, units=slice(u, u + 1))
        d = {n: to_device(a, cfg.dtype) for n, a in x.items()}
        la_f, la_b = torch.empty_like(d["g_fwd"]), torch.empty_like(d["g_bwd"])
        (vig.vig_gate_prep_f32 if cfg.dtype == "f32" else vig.vig_gate_prep_bf16)(d["g_fwd"], d["g_bwd"], la_f, la_b, cfg.tau)
        out = torch.empty_like(d["v"])
        _fwd(cfg.dtype)(d["q"], d["k"], d["v"], la_f, la_b, out)
        got = device_to_f64(out, cfg.dtype)[0, 0]
        scale = np.abs(got).max()
        for t, j, val in samples:
            assert abs(got[t, j] - val) <= TOL[cfg.dtype] * scale


@pytest.mark.parametrize("pref", [vig.VIG_TEST_KERNEL_AUTO, vig.VIG_TEST_KERNEL_SIMT, vig.VIG_TEST_KERNEL_CHUNK_TASKS,
                                  vig.VIG_TEST_KERNEL_SEGMENTS])
@pytest.mark.parametrize("dk,dv,L", [(32, 64, 196), (24, 48, 196), (32, 48, 128), (24, 64, 129), (32, 64, 256),
                                     (32, 64, 40), (24, 48, 300)])
def test_every_kernel_family_meets_the_bar(oracle, pref, dk, dv, L):
    """The tcgen05 kernels and the SIMT recurrence kernel behind the same entry point."""
    cfg, x = random_problem(600 + L, 3, 2, L, dk, dv, "bf16")
    vig.vig_test_set_kernel_preference(pref)
    try:
        got, ref = _run_unfused(oracle, cfg, x)
    finally:
        vig.vig_test_set_kernel_preference(vig.VIG_TEST_KERNEL_AUTO)
    assert np.isfinite(got).all()
    assert rel_err(got, ref) <= TOL["bf16"]


def test_kernel_preference_rejects_unknown_values():
    lib = vig.load()
    assert lib.vig_test_set_kernel_preference(7) == -3
    assert lib.vig_test_set_kernel_preference(vig.VIG_TEST_KERNEL_AUTO) == 0
