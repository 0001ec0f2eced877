"""Pins of the gradient oracle (oracle/backward.py) to things other than itself, CPU only.

The paper prints no gradient formula and no worked example; what fixes the gradient is Eq. 6 and calculus.  So the pins
are: central finite differences of the (already pinned) forward oracle for every input element; the single-token closed
form; log alpha = 0, where the layer is a dense masked matrix product with a textbook gradient; Euler's homogeneity
relations; reverse-mode autodiff (torch.autograd, fp64) of a literal restatement of Eq. 6 at a size finite differences
would take long on.  Planted mistakes (in copies of the oracle's results, on the CPU) must each trip a pin.
"""
import numpy as np
import pytest
import torch

import mpmath

from oracle.backward import bigla_bwd, gate_prep_bwd


def _rand(seed, B=1, H=2, L=6, dk=3, dv=2, gate_scale=1.0):
    r = np.random.default_rng(seed)
    q, k = r.standard_normal((B, H, L, dk)), r.standard_normal((B, H, L, dk))
    v, g = r.standard_normal((B, H, L, dv)), r.standard_normal((B, H, L, dv))
    la_f, la_b = -gate_scale * r.random((B, H, L, dk)), -gate_scale * r.random((B, H, L, dk))
    return q, k, v, la_f, la_b, g


def pin_finite_differences(bwd, fwd):
    """d/dx sum(out * W) by central differences of the forward oracle, every element of every input."""
    for seed, shape in ((11, dict()), (12, dict(B=2, H=1, L=4, dk=2, dv=3, gate_scale=3.0))):
        q, k, v, la_f, la_b, w = _rand(seed, **shape)
        got = bwd(q, k, v, la_f, la_b, w)
        prim = [q, k, v, la_f, la_b]
        h = 1e-6
        for which, (x, gx) in enumerate(zip(prim, got)):
            num = np.zeros_like(x)
            for idx in np.ndindex(*x.shape):
                vals = []
                for s in (+h, -h):
                    args = [a.copy() for a in prim]
                    args[which][idx] += s
                    vals.append(float((fwd(*args) * w).sum()))
                num[idx] = (vals[0] - vals[1]) / (2 * h)
            np.testing.assert_allclose(gx, num, rtol=2e-7, atol=2e-8, err_msg=f"input {which}")


def pin_single_token(bwd, fwd):
    """L = 1: out = (q . k) v (both states hold just k^T v; the gates act on empty states)."""
    q, k, v, la_f, la_b, g = _rand(13, L=1, dk=4, dv=3)
    dq, dk, dv, dlf, dlb = bwd(q, k, v, la_f, la_b, g)
    gv = (g * v).sum(-1, keepdims=True)
    np.testing.assert_allclose(dq, gv * k, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(dk, gv * q, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(dv, (q * k).sum(-1, keepdims=True) * g, rtol=1e-13, atol=1e-13)
    assert not dlf.any() and not dlb.any()


def pin_alpha_one_dense(bwd, fwd):
    """log alpha = 0: out = (M * (Q K^T)) V with M = (lower + upper triangle) / 2 (diagonal weight 1); the gradient of
    a masked matrix product: dV = (M * QK^T)^T dO, dQ = (M * dO V^T) K, dK = (M * dO V^T)^T Q."""
    q, k, v, _, _, g = _rand(14, L=7, dk=3, dv=4)
    zero = np.zeros_like(q)
    dq, dk, dv, _, _ = bwd(q, k, v, zero, zero, g)
    L = q.shape[2]
    M = 0.5 * (np.tril(np.ones((L, L))) + np.triu(np.ones((L, L))))
    A = M * np.einsum("bhti,bhsi->bhts", q, k)
    dA = M * np.einsum("bhtj,bhsj->bhts", g, v)
    np.testing.assert_allclose(dv, np.einsum("bhts,bhtj->bhsj", A, g), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dq, np.einsum("bhts,bhsi->bhti", dA, k), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dk, np.einsum("bhts,bhti->bhsi", dA, q), rtol=1e-12, atol=1e-12)


def pin_homogeneity(bwd, fwd):
    """out is linear in q and in v, and unchanged by k -> c k, q -> q / c per key dimension (and unit):
    sum(q dq) = sum(v dv) = sum(out d_out), and sum_t (q_t dq_t - k_t dk_t) = 0 for every key dimension."""
    q, k, v, la_f, la_b, g = _rand(15, B=2, H=2, L=8, dk=3, dv=3, gate_scale=2.0)
    dq, dk, dv, _, _ = bwd(q, k, v, la_f, la_b, g)
    total = (fwd(q, k, v, la_f, la_b) * g).sum(axis=(2, 3))
    np.testing.assert_allclose((q * dq).sum(axis=(2, 3)), total, rtol=1e-12)
    np.testing.assert_allclose((v * dv).sum(axis=(2, 3)), total, rtol=1e-12)
    np.testing.assert_allclose((q * dq - k * dk).sum(axis=2), 0.0, atol=1e-12)


def _torch_eq6(q, k, v, la_f, la_b):
    """Eq. 6 as written, in torch fp64 (for autograd)."""
    B, H, L, dk = q.shape
    outs = []
    for la, order in ((la_f, range(L)), (la_b, range(L - 1, -1, -1))):
        S = torch.zeros(B, H, dk, v.shape[3], dtype=torch.float64)
        o = [None] * L
        for t in order:
            S = torch.exp(la[:, :, t, :, None]) * S + k[:, :, t, :, None] * v[:, :, t, None, :]
            o[t] = torch.einsum("bhi,bhij->bhj", q[:, :, t], S)
        outs.append(torch.stack(o, dim=2))
    return 0.5 * (outs[0] + outs[1])


def pin_autograd(bwd, fwd):
    args = _rand(16, B=1, H=3, L=37, dk=5, dv=6, gate_scale=1.5)
    t = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in args[:5]]
    out = _torch_eq6(*t)
    np.testing.assert_allclose(out.detach().numpy(), fwd(*args[:5]), rtol=1e-12, atol=1e-12)   # the restatement is Eq. 6
    out.backward(torch.tensor(args[5]))
    for got, ref in zip(bwd(*args), t):
        np.testing.assert_allclose(got, ref.grad.numpy(), rtol=1e-11, atol=1e-12)


PINS = [pin_finite_differences, pin_single_token, pin_alpha_one_dense, pin_homogeneity, pin_autograd]


@pytest.fixture(scope="module")
def fwd(oracle):
    return lambda q, k, v, la_f, la_b: oracle.bigla_fwd(q, k, v, la_f, la_b)


@pytest.mark.parametrize("pin", PINS, ids=lambda p: p.__name__)
def test_backward_oracle_passes_pin(fwd, pin):
    pin(bigla_bwd, fwd)


def test_backward_oracle_empty_and_shapes():
    z = lambda d: np.zeros((2, 3, 0, d))
    for g, d in zip(bigla_bwd(z(4), z(4), z(5), z(4), z(4), z(5)), (4, 4, 5, 4, 4)):
        assert g.shape == (2, 3, 0, d)
    args = _rand(17, B=2, H=1, L=5, dk=4, dv=3)
    for g, a in zip(bigla_bwd(*args), args):
        assert g.shape == a.shape and g.dtype == np.float64


def _mutant(mistake):
    def wrong(q, k, v, la_f, la_b, g):
        dq, dk, dv, dlf, dlb = bigla_bwd(q, k, v, la_f, la_b, g)
        if mistake == "no_half":                 # the 1/2 of Eq. 6 dropped
            return 2 * dq, 2 * dk, 2 * dv, 2 * dlf, 2 * dlb
        if mistake == "grad_wrt_alpha":          # d/d alpha instead of d/d log alpha
            return dq, dk, dv, dlf / np.exp(la_f), dlb / np.exp(la_b)
        if mistake == "gate_directions_swapped":
            return dq, dk, dv, dlb, dlf
        if mistake == "gate_one_token_late":     # the gate of token t credited to token t + 1
            return dq, dk, dv, np.roll(dlf, 1, axis=2), dlb
        if mistake == "gate_uses_new_state":     # rowsum(Z * S_t) instead of rowsum(Z * S_{t-1}): adds k_t dk>_t
            kd = bigla_bwd(q, k, v, la_f, np.full_like(la_b, -1e3), g)[1]   # dk with the <- direction shut: the -> part plus the self pair
            return dq, dk, dv, dlf + np.exp(la_f) * k * kd, dlb
        if mistake == "one_direction_only":
            return tuple(bigla_bwd(q, k, v, la_f, np.full_like(la_b, -1e3), g))
        if mistake == "dq_dk_swapped":
            return dk, dq, dv, dlf, dlb
        raise ValueError(mistake)
    return wrong


@pytest.mark.parametrize("mistake", ["no_half", "grad_wrt_alpha", "gate_directions_swapped", "gate_one_token_late",
                                     "gate_uses_new_state", "one_direction_only", "dq_dk_swapped"])
def test_planted_mistake_in_gradient_is_caught(fwd, mistake):
    failed = []
    for pin in PINS:
        try:
            pin(_mutant(mistake), fwd)
        except AssertionError:
            failed.append(pin.__name__)
    assert failed, f"no pin catches {mistake}"


# ----------------------------------------------------------------------------------------------
# Gradient through the gate preparation (Eq. 5 line 1)
# ----------------------------------------------------------------------------------------------

def _pins_gate_prep_bwd(fn, oracle):
    r = np.random.default_rng(31)
    g = np.concatenate([r.standard_normal(40) * 3, [-30.0, -1.0, 0.0, 1.0, 30.0]])
    d = r.standard_normal(g.size)
    for tau in (16.0, 3.0):
        got = fn(g, d, tau)
        h = 1e-6
        num = (oracle.gate_prep(g + h, tau) - oracle.gate_prep(g - h, tau)) / (2 * h)   # the pinned forward oracle
        np.testing.assert_allclose(got, d * num, rtol=1e-8, atol=1e-10)
        np.testing.assert_allclose(fn(np.zeros(3), np.ones(3), tau), 0.5 / tau, rtol=1e-15)         # sigmoid(0) = 1/2
        np.testing.assert_allclose(fn(g, np.ones_like(g), tau) + fn(-g, np.ones_like(g), tau), 1.0 / tau, rtol=1e-14)   # sigmoid(g) + sigmoid(-g) = 1
    assert fn(np.array([800.0]), np.array([1.0]), 1.0)[0] == 0.0 and fn(np.array([-800.0]), np.array([1.0]), 1.0)[0] == 1.0
    mpmath.mp.dps = 50
    for gg in (-7.5, -0.3, 2.25, 11.0):
        ref = mpmath.mpf(3) / (1 + mpmath.e ** mpmath.mpf(gg)) / 16
        assert abs(fn(np.array([gg]), np.array([3.0]), 16.0)[0] - float(ref)) < 1e-16


def test_gate_prep_gradient_oracle_pins(oracle):
    _pins_gate_prep_bwd(gate_prep_bwd, oracle)


@pytest.mark.parametrize("wrong", [
    lambda g, d, tau: gate_prep_bwd(g, d, tau) * tau,                 # the temperature forgotten
    lambda g, d, tau: gate_prep_bwd(-g, d, tau),                      # sigmoid(g) instead of 1 - sigmoid(g)
    lambda g, d, tau: gate_prep_bwd(g, d, tau) * (1 - gate_prep_bwd(g, np.ones_like(g), 1.0)),   # the derivative of sigmoid, not of its logarithm
], ids=["no_tau", "wrong_sign", "sigmoid_derivative"])
def test_planted_mistake_in_gate_prep_gradient_is_caught(oracle, wrong):
    with pytest.raises(AssertionError):
        _pins_gate_prep_bwd(wrong, oracle)
