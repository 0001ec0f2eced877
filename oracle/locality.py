"""fp64 CPU oracle of the 2-D gating locality injection around BiGLA (paper Eq. 7).  TEST INFRASTRUCTURE ONLY.

    O_local  = DWConv3x3(X)                       (line 1)
    O_global = BiGLA(O_local)                     (line 2: the mixer itself, oracle.bigla_fwd after the projections)
    G_2D     = sigmoid(O_local W + b)             (line 3)
    O        = G_2D * O_local + (1 - G_2D) * O_global          (line 4)

Plain loops over the nine taps and element-wise numpy arithmetic: the definitions written out, nothing blocked or
fused.  The dense projections (q, k, v, the gate logits of Eq. 5 and `O_local W + b`) are ordinary matrix products
outside the hot path; the blend takes the logits z = O_local W + b as an input.
"""
from __future__ import annotations

import numpy as np


def dwconv3x3(x, w, b=None):
    """Depth-wise 3x3 convolution of Eq. 7 line 1 over the patch grid, one filter per channel, stride 1, zero padding 1.

    x: [B, Hh, Ww, C] (channels last: the flattened sequence of the mixer is the row-major Hh x Ww grid);
    w: [C, 3, 3]; b: [C] or None.  Cross-correlation, the convention of deep-learning convolutions:
        out[n, i, j, c] = b[c] + sum_{di, dj in {-1, 0, 1}} w[c, di + 1, dj + 1] * x[n, i + di, j + dj, c]
    with x taken as zero outside the grid.
    """
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    B, Hh, Ww, C = x.shape
    if w.shape != (C, 3, 3):
        raise ValueError("w must be [C, 3, 3]")
    out = np.zeros_like(x)
    for di in (-1, 0, 1):
        for dj in (-1, 0, 1):
            i0, i1 = max(0, -di), min(Hh, Hh - di)      # output rows whose tap (i + di) lies inside the grid
            j0, j1 = max(0, -dj), min(Ww, Ww - dj)
            if i0 >= i1 or j0 >= j1:
                continue
            out[:, i0:i1, j0:j1, :] += w[None, None, None, :, di + 1, dj + 1] * x[:, i0 + di:i1 + di, j0 + dj:j1 + dj, :]
    if b is not None:
        out += np.asarray(b, dtype=np.float64)[None, None, None, :]
    return out


def gate_blend(o_local, z, o_global):
    """Eq. 7 lines 3-4 with z = O_local W + b given: G = sigmoid(z), O = G * O_local + (1 - G) * O_global (same shapes)."""
    o_local = np.asarray(o_local, dtype=np.float64)
    z = np.asarray(z, dtype=np.float64)
    o_global = np.asarray(o_global, dtype=np.float64)
    # sigmoid without overflow: e^{-|z|} is at most 1
    e = np.exp(-np.abs(z))
    g = np.where(z >= 0, 1.0 / (1.0 + e), e / (1.0 + e))
    return g * o_local + (1.0 - g) * o_global
