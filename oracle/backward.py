"""fp64 CPU oracle for the gradient of the BiGLA forward pass.  TEST INFRASTRUCTURE ONLY.

The paper trains with the layer of Eq. 6 but does not describe its gradient; what the gradient IS follows from Eq. 6 by
the chain rule alone, so the oracle is the reverse-mode adjoint of the two recurrences, step by step, in fp64:

    forward (Eq. 6):  S>_t = diag(alpha>_t) S>_{t-1} + k_t^T v_t,   S<_t = diag(alpha<_t) S<_{t+1} + k_t^T v_t,
                      out_t = (q_t S>_t + q_t S<_t) / 2,            alpha = exp(log alpha), zero states outside 1..L.

Given d_out = dLoss/d_out it returns dLoss/d{q, k, v, log alpha>, log alpha<}.  For the -> direction, walking t = L..1 with
Z = dLoss/dS>_t:
    Z      += q_t^T d_out_t / 2
    dq_t   += S>_t d_out_t^T / 2
    dk_t   += Z v_t^T,   dv_t += k_t Z
    dlog alpha>_t = alpha>_t * rowsum(Z * S>_{t-1})        (d/d alpha of diag(alpha) S_{t-1}, times d alpha / d log alpha)
    Z       = diag(alpha>_t) Z                             (what reaches S>_{t-1})
The <- direction is the same walk on the time-reversed sequence.  All S>_t are kept from a forward walk (the oracle is
for test sizes; units are independent, so a full-size check samples units).

Pinned in tests/test_oracle_pins.py against central finite differences of the forward oracle, closed forms (L = 1,
alpha = 1 through the dense masked-attention matrices) and planted mistakes.  Shares no code with the CUDA path.
"""
from __future__ import annotations

import numpy as np


def _one_direction(q, k, v, la, d_out):
    """Gradient of o_t = q_t S_t / 2 with S_t = diag(exp(la_t)) S_{t-1} + k_t^T v_t, t ascending; arrays [U, L, d]."""
    U, L, dk = q.shape
    dv_ = v.shape[2]
    a = np.exp(la)
    S = np.zeros((L + 1, U, dk, dv_))                       # S[t] = state after token t (1-based), S[0] = 0
    for t in range(1, L + 1):
        S[t] = a[:, t - 1, :, None] * S[t - 1] + k[:, t - 1, :, None] * v[:, t - 1, None, :]
    dq, dk_, dvv, dla = (np.zeros_like(x) for x in (q, k, v, la))
    Z = np.zeros((U, dk, dv_))
    for t in range(L, 0, -1):
        g = d_out[:, t - 1]                                  # [U, dv]
        Z = Z + 0.5 * q[:, t - 1, :, None] * g[:, None, :]
        dq[:, t - 1] = 0.5 * np.einsum("uij,uj->ui", S[t], g)
        dk_[:, t - 1] = np.einsum("uij,uj->ui", Z, v[:, t - 1])
        dvv[:, t - 1] = np.einsum("ui,uij->uj", k[:, t - 1], Z)
        dla[:, t - 1] = a[:, t - 1] * np.einsum("uij,uij->ui", Z, S[t - 1])
        Z = a[:, t - 1, :, None] * Z
    return dq, dk_, dvv, dla


def bigla_bwd(q, k, v, log_alpha_fwd, log_alpha_bwd, d_out):
    """All arrays [B, H, L, d] (q, k, log alpha: dk; v, d_out: dv), any float dtype; fp64 arithmetic.
    Returns (dq, dk, dv, dlog_alpha_fwd, dlog_alpha_bwd), fp64, shaped like their primal."""
    q, k, v, laf, lab, g = (np.asarray(x, dtype=np.float64) for x in (q, k, v, log_alpha_fwd, log_alpha_bwd, d_out))
    B, H, L, dk = q.shape
    dv_ = v.shape[3]
    if B * H * L == 0:
        return tuple(np.zeros_like(x) for x in (q, k, v, laf, lab))
    r3 = lambda x: x.reshape(B * H, L, x.shape[3])
    fq, fk, fv, fl = _one_direction(r3(q), r3(k), r3(v), r3(laf), r3(g))
    flip = lambda x: r3(x)[:, ::-1]
    bq, bk, bv, bl = _one_direction(flip(q), flip(k), flip(v), flip(lab), flip(g))
    unflip = lambda x: x[:, ::-1]
    out = (fq + unflip(bq), fk + unflip(bk), fv + unflip(bv), fl, unflip(bl))
    shapes = (q.shape, k.shape, v.shape, laf.shape, lab.shape)
    return tuple(np.ascontiguousarray(x).reshape(s) for x, s in zip(out, shapes))


def gate_prep_bwd(g, dlog_alpha, tau: float = 16.0):
    """Gradient through the gate preparation log alpha = logsigmoid(g) / tau (Eq. 5 line 1):
    dg = dlog_alpha * sigmoid(-g) / tau, since d/dg log(sigmoid(g)) = 1 - sigmoid(g).  fp64, shaped like g.
    (exp is only taken of non-positive numbers.)"""
    g = np.asarray(g, dtype=np.float64)
    d = np.asarray(dlog_alpha, dtype=np.float64)
    e = np.exp(-np.abs(g))
    sig_neg = np.where(g >= 0, e / (1.0 + e), 1.0 / (1.0 + e))   # sigmoid(-g)
    return d * sig_neg / float(tau)
