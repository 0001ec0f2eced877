"""Explicit (unrolled) form of BiGLA, for tiny inputs.  TEST INFRASTRUCTURE ONLY.

Unrolling the two recurrences of Eq. 6 from zero initial states gives, for every
(batch, head) unit,

    o>_t = sum_{s <= t} ( q_t * prod_{r = s+1 .. t} alpha>_r ) . k_s  v_s
    o<_t = sum_{s >= t} ( q_t * prod_{r = t .. s-1} alpha<_r ) . k_s  v_s
    o_t  = (o>_t + o<_t) / 2

(* is the element-wise product over the key dimension, . the dot product over
it).  The gate at the query position t is inside the product, the gate at the
key position s is not, and the pair s = t appears once in each direction with
an empty product.  The code below is that double sum written out with the
products taken gate by gate; it keeps no running state and is O(L^2 dk dv).
It exists to pin oracle/bigla_oracle.c to something other than itself.
"""
from __future__ import annotations

import numpy as np


def bigla_quadratic(q, k, v, log_alpha_fwd, log_alpha_bwd):
    """Returns (o, o_fwd, o_bwd), fp64, for [B, H, L, d] inputs."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    alpha_f = np.exp(np.asarray(log_alpha_fwd, dtype=np.float64))
    alpha_b = np.exp(np.asarray(log_alpha_bwd, dtype=np.float64))
    B, H, L, dk = q.shape
    dv = v.shape[3]
    o_f = np.zeros((B, H, L, dv))
    o_b = np.zeros((B, H, L, dv))
    for b in range(B):
        for h in range(H):
            for t in range(L):
                for s in range(0, t + 1):
                    decay = np.ones(dk)
                    for r in range(s + 1, t + 1):
                        decay = decay * alpha_f[b, h, r]
                    w = float(np.sum(q[b, h, t] * decay * k[b, h, s]))
                    o_f[b, h, t] += w * v[b, h, s]
                for s in range(t, L):
                    decay = np.ones(dk)
                    for r in range(t, s):
                        decay = decay * alpha_b[b, h, r]
                    w = float(np.sum(q[b, h, t] * decay * k[b, h, s]))
                    o_b[b, h, t] += w * v[b, h, s]
    return (o_f + o_b) / 2.0, o_f, o_b
