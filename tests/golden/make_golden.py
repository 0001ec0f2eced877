"""Writes tests/golden/bigla_samples.txt: fp64 oracle outputs at a few sampled positions of each
benchmark configuration.  Calls only the CPU oracle and the seeded input generator, never the CUDA
path.  The paper prints no numeric example of BiGLA, so these are regression values of the pinned
oracle (Eq. 6), not values from the paper.  Run from the repository root:

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2405_18425_b200 import synth  # noqa: E402

UNITS_PER_CONFIG = 2     # the first and the last (b, h) unit of every configuration
POSITIONS = 6


def sample_lines():
    yield "# config unit t j o(fp64)   -- gates: log alpha = logsigmoid(g)/tau in fp64 from the stored g"
    for cfg in synth.CONFIGS:
        for u in sorted({0, cfg.units - 1})[:UNITS_PER_CONFIG]:
            x = synth.make_inputs(cfg, units=slice(u, u + 1))
            f = {n: synth.stored_to_f64(a, cfg.dtype) for n, a in x.items()}
            la_f = oracle.gate_prep(f["g_fwd"], cfg.tau)
            la_b = oracle.gate_prep(f["g_bwd"], cfg.tau)
            o = oracle.bigla_fwd(f["q"], f["k"], f["v"], la_f, la_b)[0, 0]
            ts = np.linspace(0, cfg.L - 1, POSITIONS).astype(int)
            for n, t in enumerate(ts):
                j = (7 * n + 3) % cfg.dv
                yield f"{cfg.name} {u} {t} {j} {o[t, j]!r}".replace("np.float64(", "").replace(")", "")


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "bigla_samples.txt")
    with open(path, "w") as fh:
        fh.write("\n".join(sample_lines()) + "\n")
    print("wrote", path)
