"""Pins for the fp64 oracle: everything here runs on the CPU.

The paper prints no worked numeric example of BiGLA, so the oracle is pinned to
what Eq. 3-6 and the mathematics fix: the unrolled double sum, the alpha == 1
reduction to (anti)causal linear attention built from numpy's cumsum, the flip
symmetry between the two directions, a geometric-series closed form, a "gate
wall" that fixes which position's gate decays which pair, the diagonal limit,
linearity and unit independence.  Each pin is a function of an implementation,
so the same pins are also run against deliberately wrong variants (planted on
the CPU) to show that a dropped term, a shifted index or a swapped gate fails
at least one of them.
"""
import mpmath
import numpy as np
import pytest

from oracle.quadratic import bigla_quadratic


def _rand(seed, B=1, H=2, L=9, dk=3, dv=4, gate_scale=1.0):
    r = np.random.default_rng(seed)
    q = r.standard_normal((B, H, L, dk))
    k = r.standard_normal((B, H, L, dk))
    v = r.standard_normal((B, H, L, dv))
    la_f = -gate_scale * r.random((B, H, L, dk))
    la_b = -gate_scale * r.random((B, H, L, dk))
    return q, k, v, la_f, la_b


# ----------------------------------------------------------------------------------------------
# Pins.  impl(q, k, v, la_f, la_b) -> (o, o_fwd, o_bwd); each pin raises AssertionError on failure.
# ----------------------------------------------------------------------------------------------

def pin_quadratic_form(impl):
    """Unrolled Eq. 6 (explicit sum over pairs with gate-by-gate products)."""
    for seed, shape in ((1, dict(L=9, dk=3, dv=4)), (2, dict(B=2, H=1, L=16, dk=4, dv=2, gate_scale=3.0))):
        args = _rand(seed, **shape)
        got = impl(*args)
        ref = bigla_quadratic(*args)
        for g, r in zip(got, ref):
            np.testing.assert_allclose(g, r, rtol=1e-12, atol=1e-12)


def pin_alpha_one_is_linear_attention(impl):
    """log alpha = 0: Eq. 5 collapses to Eq. 3-4, o>_t = q_t sum_{s<=t} k_s^T v_s (numpy cumsum)."""
    q, k, v, la_f, la_b = _rand(3, L=11, dk=4, dv=5)
    zero = np.zeros_like(la_f)
    o, o_f, o_b = impl(q, k, v, zero, zero)
    kv = np.einsum("bhti,bhtj->bhtij", k, v)
    causal = np.cumsum(kv, axis=2)
    anti = np.flip(np.cumsum(np.flip(kv, axis=2), axis=2), axis=2)
    np.testing.assert_allclose(o_f, np.einsum("bhti,bhtij->bhtj", q, causal), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(o_b, np.einsum("bhti,bhtij->bhtj", q, anti), rtol=1e-12, atol=1e-12)
    # o>_t + o<_t = q_t (sum over all s of k_s^T v_s) + (q_t . k_t) v_t : the self pair is in both directions
    total = kv.sum(axis=2, keepdims=True)
    both = np.einsum("bhti,bhtij->bhtj", q, np.broadcast_to(total, kv.shape)) + \
        np.einsum("bhti,bhti->bht", q, k)[..., None] * v
    np.testing.assert_allclose(2.0 * o, both, rtol=1e-12, atol=1e-12)


def pin_flip_symmetry(impl):
    """The backward scan is the forward scan of the reversed sequence with reversed gates."""
    q, k, v, la_f, la_b = _rand(4, L=13, dk=3, dv=3, gate_scale=2.0)
    _, o_f, o_b = impl(q, k, v, la_f, la_b)
    fl = lambda a: np.ascontiguousarray(np.flip(a, axis=2))
    _, o_f2, o_b2 = impl(fl(q), fl(k), fl(v), fl(la_b), fl(la_f))
    np.testing.assert_allclose(o_b, fl(o_f2), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(o_f, fl(o_b2), rtol=1e-12, atol=1e-13)


def pin_diagonal_limit(impl):
    """log alpha very negative: every state is forgotten at once, only s = t survives, weight 1/2 + 1/2."""
    q, k, v, la_f, la_b = _rand(5, L=7, dk=4, dv=3)
    big = np.full_like(la_f, -1.0e3)  # exp(-1000) is exactly 0 in fp64
    o, o_f, o_b = impl(q, k, v, big, big)
    diag = np.einsum("bhti,bhti->bht", q, k)[..., None] * v
    np.testing.assert_allclose(o, diag, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(o_f, diag, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(o_b, diag, rtol=1e-13, atol=1e-13)


def pin_geometric_closed_form(impl):
    """q = k = v = 1 and a constant scalar alpha: o>_t = dk (1 - alpha^t)/(1 - alpha) with t counted
    from 1, o<_t = dk (1 - alpha^(L-t+1))/(1 - alpha).  Different alpha per direction."""
    L, dk, dv = 10, 3, 2
    one_k = np.ones((1, 1, L, dk))
    one_v = np.ones((1, 1, L, dv))
    af, ab = 0.8, 0.55
    o, o_f, o_b = impl(one_k, one_k, one_v, np.full_like(one_k, np.log(af)), np.full_like(one_k, np.log(ab)))
    t = np.arange(1, L + 1, dtype=np.float64)
    ref_f = dk * (1.0 - af ** t) / (1.0 - af)
    ref_b = dk * (1.0 - ab ** (L - t + 1)) / (1.0 - ab)
    np.testing.assert_allclose(o_f[0, 0, :, 0], ref_f, rtol=1e-12)
    np.testing.assert_allclose(o_b[0, 0, :, 1], ref_b, rtol=1e-12)
    np.testing.assert_allclose(o[0, 0, :, 0], (ref_f + ref_b) / 2.0, rtol=1e-12)


def pin_gate_wall(impl):
    """One fully closed gate at position p (all other gates open) fixes the index convention:
    forward, a query t >= p sees only keys s >= p (the gate at the query position acts, the gate at
    the key position does not), queries t < p see all s <= t; mirrored for the backward direction."""
    L, dk, dv, p = 8, 2, 3, 3
    q, k, v, _, _ = _rand(6, H=1, L=L, dk=dk, dv=dv)
    open_ = np.zeros((1, 1, L, dk))
    wall = open_.copy()
    wall[0, 0, p, :] = -1.0e3
    kv = np.einsum("bhti,bhtj->bhtij", k, v)[0, 0]

    def attend(t, keys):
        S = sum((kv[s] for s in keys), np.zeros((dk, dv)))
        return q[0, 0, t] @ S

    _, o_f, _ = impl(q, k, v, wall, open_)
    for t in range(L):
        keys = range(p, t + 1) if t >= p else range(0, t + 1)
        np.testing.assert_allclose(o_f[0, 0, t], attend(t, keys), rtol=1e-12, atol=1e-13)
    _, _, o_b = impl(q, k, v, open_, wall)
    for t in range(L):
        keys = range(t, p + 1) if t <= p else range(t, L)
        np.testing.assert_allclose(o_b[0, 0, t], attend(t, keys), rtol=1e-12, atol=1e-13)


def pin_per_key_dim_gate(impl):
    """G_t = alpha_t^T 1: the gate indexes the key dimension (rows of S), not the value dimension.
    Closing key dim 0 only, everywhere, leaves key dim 1 as plain linear attention."""
    L, dk, dv = 6, 2, 3
    q, k, v, _, _ = _rand(7, H=1, L=L, dk=dk, dv=dv)
    la = np.zeros((1, 1, L, dk))
    la[..., 0] = -1.0e3
    _, o_f, _ = impl(q, k, v, la, la)
    kv1 = np.cumsum(k[0, 0, :, 1, None] * v[0, 0], axis=0)             # key dim 1: running sum
    ref = q[0, 0, :, 0, None] * k[0, 0, :, 0, None] * v[0, 0] + q[0, 0, :, 1, None] * kv1
    np.testing.assert_allclose(o_f[0, 0], ref, rtol=1e-12, atol=1e-13)


def pin_linearity_and_independence(impl):
    q, k, v, la_f, la_b = _rand(8, B=2, H=2, L=5, dk=3, dv=4)
    o1 = impl(q, k, v, la_f, la_b)[0]
    r = np.random.default_rng(80)
    v2 = r.standard_normal(v.shape)
    o2 = impl(q, k, v2, la_f, la_b)[0]
    o12 = impl(q, k, 2.0 * v - 3.0 * v2, la_f, la_b)[0]
    np.testing.assert_allclose(o12, 2.0 * o1 - 3.0 * o2, rtol=1e-11, atol=1e-12)
    # changing one (b, h) unit leaves every other unit's output unchanged
    q3, k3 = q.copy(), k.copy()
    q3[1, 0] = r.standard_normal(q3[1, 0].shape)
    k3[1, 0] = r.standard_normal(k3[1, 0].shape)
    o3 = impl(q3, k3, v, la_f, la_b)[0]
    keep = np.ones((2, 2), dtype=bool)
    keep[1, 0] = False
    np.testing.assert_array_equal(o3[keep], o1[keep])
    assert np.abs(o3[1, 0] - o1[1, 0]).max() > 1e-3


def pin_single_token(impl):
    q, k, v, la_f, la_b = _rand(9, L=1, dk=5, dv=3)
    o = impl(q, k, v, la_f, la_b)[0]
    np.testing.assert_allclose(o, np.einsum("bhti,bhti->bht", q, k)[..., None] * v, rtol=1e-13, atol=1e-14)


PINS = [
    pin_quadratic_form,
    pin_alpha_one_is_linear_attention,
    pin_flip_symmetry,
    pin_diagonal_limit,
    pin_geometric_closed_form,
    pin_gate_wall,
    pin_per_key_dim_gate,
    pin_linearity_and_independence,
    pin_single_token,
]


@pytest.fixture(scope="module")
def oracle_impl(oracle):
    def impl(q, k, v, la_f, la_b):
        o, o_f, o_b, _ = oracle.bigla_fwd_directions(q, k, v, la_f, la_b, nthreads=2)
        return o, o_f, o_b

    return impl


@pytest.mark.parametrize("pin", PINS, ids=lambda p: p.__name__)
def test_oracle_passes_pin(oracle_impl, pin):
    pin(oracle_impl)


def test_oracle_matches_quadratic_on_tiny_config(oracle):
    """The smallest benchmark configuration itself (fp32 storage, L = 64), one head to keep it quick."""
    from paper_2405_18425_b200 import synth

    cfg = synth.CONFIGS[0]
    x = synth.make_inputs(cfg)
    f = lambda name: synth.stored_to_f64(x[name], cfg.dtype)[:, :1]
    la_f, la_b = oracle.gate_prep(f("g_fwd"), cfg.tau), oracle.gate_prep(f("g_bwd"), cfg.tau)
    o, o_f, o_b, _ = oracle.bigla_fwd_directions(f("q"), f("k"), f("v"), la_f, la_b)
    ro, rf, rb = bigla_quadratic(f("q"), f("k"), f("v"), la_f, la_b)
    scale = np.abs(ro).max()
    assert np.abs(o - ro).max() <= 1e-12 * scale
    assert np.abs(o_f - rf).max() <= 1e-12 * np.abs(rf).max()
    assert np.abs(o_b - rb).max() <= 1e-12 * np.abs(rb).max()


def test_oracle_thread_count_does_not_change_result(oracle):
    args = _rand(10, B=3, H=3, L=17, dk=4, dv=6)
    a = oracle.bigla_fwd_directions(*args, nthreads=1)
    b = oracle.bigla_fwd_directions(*args, nthreads=5)
    assert a[3] == 1 and b[3] == 5
    for x, y in zip(a[:3], b[:3]):
        np.testing.assert_array_equal(x, y)


def test_oracle_empty_inputs(oracle):
    z = np.zeros((0, 2, 5, 3))
    o = oracle.bigla_fwd(z, z, np.zeros((0, 2, 5, 4)), z, z)
    assert o.shape == (0, 2, 5, 4)
    z = np.zeros((1, 2, 0, 3))
    o = oracle.bigla_fwd(z, z, np.zeros((1, 2, 0, 4)), z, z)
    assert o.shape == (1, 2, 0, 4)


# ----------------------------------------------------------------------------------------------
# Planted mistakes (CPU only): a numpy restatement of the recurrence with one switchable error.
# Every mutant must fail at least one pin; the unmutated restatement must pass all of them.
# ----------------------------------------------------------------------------------------------

def _mutant(mistake):
    def impl(q, k, v, la_f, la_b):
        B, H, L, dk = q.shape
        dv = v.shape[3]
        o_f = np.zeros((B, H, L, dv))
        o_b = np.zeros((B, H, L, dv))
        for b in range(B):
            for h in range(H):
                for direction, la, o in ((+1, la_f, o_f), (-1, la_b, o_b)):
                    if mistake == "bwd_uses_fwd_gate":
                        la = la_f
                    S = np.zeros((dk, dv))
                    order = range(L) if direction > 0 else range(L - 1, -1, -1)
                    for t in order:
                        a = np.exp(la[b, h, t])
                        kv = np.outer(k[b, h, t], v[b, h, t])
                        if mistake == "gate_at_key":          # decays the new pair too
                            S = a[:, None] * (S + kv)
                        elif mistake == "gate_over_dv":        # gate indexes the wrong state axis
                            S = S * np.resize(a, dv)[None, :] + kv
                        elif mistake == "transposed_kv":
                            S = a[:, None] * S + np.resize(np.outer(v[b, h, t], k[b, h, t]), (dk, dv))
                        else:
                            S = a[:, None] * S + kv
                        if mistake == "output_before_update" and direction > 0:
                            o[b, h, t] = q[b, h, t] @ (S - kv)  # o_t = q_t S_{t-1}: drops the self pair
                        elif mistake == "bwd_excludes_self" and direction < 0:
                            o[b, h, t] = q[b, h, t] @ (S - kv)
                        else:
                            o[b, h, t] = q[b, h, t] @ S
        if mistake == "no_half":
            return o_f + o_b, o_f, o_b
        return (o_f + o_b) / 2.0, o_f, o_b

    return impl


def _failed_pins(impl):
    failed = []
    for pin in PINS:
        try:
            pin(impl)
        except AssertionError:
            failed.append(pin.__name__)
    return failed


def test_unmutated_restatement_passes_all_pins():
    assert _failed_pins(_mutant(None)) == []


@pytest.mark.parametrize("mistake", [
    "gate_at_key", "gate_over_dv", "transposed_kv", "output_before_update",
    "bwd_excludes_self", "bwd_uses_fwd_gate", "no_half",
])
def test_planted_mistake_is_caught(mistake):
    assert _failed_pins(_mutant(mistake)), f"no pin notices the mistake {mistake!r}"


# ----------------------------------------------------------------------------------------------
# Gate preparation: log alpha = log(sigmoid(g)^(1/tau))
# ----------------------------------------------------------------------------------------------

def test_gate_prep_closed_forms(oracle):
    la = oracle.gate_prep(np.array([0.0]), 16.0)
    assert la[0] == pytest.approx(-np.log(2.0) / 16.0, rel=1e-15)
    assert la[0] == pytest.approx(-0.0433216987849966, rel=1e-13)
    g = np.linspace(-30.0, 30.0, 241)
    plus, minus = oracle.gate_prep(g, 1.0), oracle.gate_prep(-g, 1.0)
    np.testing.assert_allclose(plus - minus, g, rtol=1e-13, atol=1e-13)   # logsigmoid(g) - logsigmoid(-g) = g
    assert np.all(oracle.gate_prep(g, 16.0) < 0.0)
    # asymptotes: g -> -inf gives g / tau, g -> +inf gives -exp(-g) / tau -> 0 from below, no overflow
    far = oracle.gate_prep(np.array([-800.0, 800.0, 40.0]), 16.0)
    assert far[0] == pytest.approx(-50.0, rel=1e-15)
    assert far[1] <= 0.0 and abs(far[1]) < 1e-300
    assert far[2] == pytest.approx(-np.exp(-40.0) / 16.0, rel=1e-12)


def test_gate_prep_matches_literal_definition(oracle):
    """alpha = sigmoid(g)^(1/tau) evaluated literally (safe for moderate g) and in 50-digit arithmetic."""
    g = np.linspace(-20.0, 20.0, 81)
    for tau in (16.0, 1.0, 4.0):
        alpha = (1.0 / (1.0 + np.exp(-g))) ** (1.0 / tau)
        np.testing.assert_allclose(np.exp(oracle.gate_prep(g, tau)), alpha, rtol=1e-14)
    mpmath.mp.dps = 50
    for gx in (-37.5, -3.25, -0.5, 0.0, 0.125, 2.0, 17.0, 36.0):
        exact = mpmath.log(1 / (1 + mpmath.exp(-mpmath.mpf(gx)))) / 16
        got = oracle.gate_prep(np.array([gx]), 16.0)[0]
        assert abs(got - float(exact)) <= 4e-16 * abs(float(exact))


# ----------------------------------------------------------------------------------------------
# Eq. 7: depth-wise 3x3 convolution and the 2-D gate blend (oracle/locality.py)
# ----------------------------------------------------------------------------------------------

def _pins_dwconv(conv):
    from scipy import ndimage

    r = np.random.default_rng(70)
    x = r.standard_normal((2, 5, 7, 3))
    w = r.standard_normal((3, 3, 3))
    b = r.standard_normal(3)
    got = conv(x, w, b)
    # a library routine on the special case of one image and one channel: zero-padded cross-correlation
    for n in range(2):
        for c in range(3):
            ref = ndimage.correlate(x[n, :, :, c], w[c], mode="constant", cval=0.0) + b[c]
            np.testing.assert_allclose(got[n, :, :, c], ref, rtol=1e-13, atol=1e-13)
    # brute force, tap by tap
    for (n, i, j, c) in [(0, 0, 0, 0), (1, 4, 6, 2), (0, 2, 3, 1), (1, 0, 6, 0)]:
        acc = b[c]
        for di in (-1, 0, 1):
            for dj in (-1, 0, 1):
                if 0 <= i + di < 5 and 0 <= j + dj < 7:
                    acc += w[c, di + 1, dj + 1] * x[n, i + di, j + dj, c]
        assert abs(got[n, i, j, c] - acc) < 1e-13
    # the centre tap alone is the identity; the tap above the centre reads the row above (zero at the top border)
    delta = np.zeros((3, 3, 3)); delta[:, 1, 1] = 1.0
    np.testing.assert_array_equal(conv(x, delta, None), x)
    up = np.zeros((3, 3, 3)); up[:, 0, 1] = 1.0
    s = conv(x, up, None)
    np.testing.assert_array_equal(s[:, 1:], x[:, :-1])
    np.testing.assert_array_equal(s[:, 0], 0.0)
    left = np.zeros((3, 3, 3)); left[:, 1, 0] = 1.0
    s = conv(x, left, None)
    np.testing.assert_array_equal(s[:, :, 1:], x[:, :, :-1])
    np.testing.assert_array_equal(s[:, :, 0], 0.0)
    # zero padding: ones * ones counts the neighbours inside the grid (4 in a corner, 6 on an edge, 9 inside)
    cnt = conv(np.ones((1, 4, 5, 1)), np.ones((1, 3, 3)), None)[0, :, :, 0]
    assert cnt[0, 0] == 4 and cnt[0, 2] == 6 and cnt[2, 0] == 6 and cnt[2, 2] == 9 and cnt[3, 4] == 4
    # depth-wise: a channel sees only its own filter and its own input; linear in x
    x2 = x.copy(); x2[..., 1] += 5.0
    d = conv(x2, w, b) - got
    assert np.abs(d[..., 0]).max() == 0 and np.abs(d[..., 2]).max() == 0 and np.abs(d[..., 1]).max() > 0
    np.testing.assert_allclose(conv(2.0 * x, w, None), 2.0 * conv(x, w, None), rtol=1e-13)
    # a 1 x 1 grid keeps only the centre tap
    one = conv(np.full((1, 1, 1, 2), 3.0), np.arange(18.0).reshape(2, 3, 3), np.array([1.0, -1.0]))
    np.testing.assert_allclose(one[0, 0, 0], [3.0 * 4.0 + 1.0, 3.0 * 13.0 - 1.0])


def _pins_blend(blend):
    r = np.random.default_rng(71)
    a, c = r.standard_normal((3, 4)), r.standard_normal((3, 4))
    np.testing.assert_allclose(blend(a, np.zeros((3, 4)), c), 0.5 * (a + c), rtol=1e-15)
    np.testing.assert_allclose(blend(a, np.full((3, 4), 50.0), c), a, rtol=1e-15, atol=1e-15)      # gate open: the local branch
    np.testing.assert_allclose(blend(a, np.full((3, 4), -50.0), c), c, rtol=1e-15, atol=1e-15)     # gate closed: the global branch
    assert np.isfinite(blend(a, np.full((3, 4), 800.0), c)).all() and np.isfinite(blend(a, np.full((3, 4), -800.0), c)).all()
    z = r.standard_normal((3, 4)) * 3
    np.testing.assert_allclose(blend(a, z, a), a, rtol=1e-15)                                   # the weights sum to one
    # sigmoid(z) + sigmoid(-z) = 1: swapping the branches and negating z changes nothing
    np.testing.assert_allclose(blend(a, z, c), blend(c, -z, a), rtol=1e-14)
    mpmath.mp.dps = 50
    for zz in (-7.5, -0.3, 0.0, 1.25, 11.0):
        g = mpmath.mpf(1) / (1 + mpmath.e ** (-mpmath.mpf(zz)))
        ref = g * mpmath.mpf(2) + (1 - g) * mpmath.mpf(-3)
        assert abs(blend(np.array([2.0]), np.array([zz]), np.array([-3.0]))[0] - float(ref)) < 1e-15


def test_dwconv_and_blend_oracle_pins():
    from oracle.locality import dwconv3x3, gate_blend

    _pins_dwconv(dwconv3x3)
    _pins_blend(gate_blend)


def test_planted_mistakes_in_eq7_are_caught():
    from oracle.locality import dwconv3x3, gate_blend

    def flipped(x, w, b):                     # a true convolution (kernel flipped) instead of the cross-correlation
        return dwconv3x3(x, w[:, ::-1, ::-1], b)

    def replicate(x, w, b):                   # edge replication instead of zero padding
        xp = np.pad(np.asarray(x, dtype=np.float64), ((0, 0), (1, 1), (1, 1), (0, 0)), mode="edge")
        out = np.zeros_like(np.asarray(x, dtype=np.float64))
        for di in range(3):
            for dj in range(3):
                out += np.asarray(w)[None, None, None, :, di, dj] * xp[:, di:di + x.shape[1], dj:dj + x.shape[2], :]
        return out + (0 if b is None else np.asarray(b)[None, None, None, :])

    def shared_filter(x, w, b):               # one filter for every channel (not depth-wise)
        return dwconv3x3(x, np.broadcast_to(np.asarray(w)[:1], np.asarray(w).shape), b)

    for wrong in (flipped, replicate, shared_filter):
        with pytest.raises(AssertionError):
            _pins_dwconv(wrong)

    def swapped(a, z, c):                     # the gate on the global branch
        return gate_blend(c, z, a)

    def tanh_gate(a, z, c):                   # a different squashing function
        g = 0.5 * (1 + np.tanh(z))
        return g * a + (1 - g) * c

    for wrong in (swapped, tanh_gate):
        with pytest.raises(AssertionError):
            _pins_blend(wrong)
