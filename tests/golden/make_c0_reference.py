"""Writes tests/golden/c0_oracle_samples.txt from the CPU oracle alone.

Inputs are built here with numpy (seeded, same recipe as the tiny fp32
configuration: iid N(0,1), Q and K rows L2-normalised and scaled by sqrt(h)),
so the file depends on nothing but numpy and oracle/.
Run:  python tests/golden/make_c0_reference.py
"""
import math
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
from oracle import polysketch as orc  # noqa: E402


def build():
    n, h, r = 1024, 64, 16
    g = np.random.default_rng(0)
    Q, K, V = (g.standard_normal((n, h)) for _ in range(3))
    Q *= math.sqrt(h) / np.linalg.norm(Q, axis=1, keepdims=True)
    K *= math.sqrt(h) / np.linalg.norm(K, axis=1, keepdims=True)
    gg = np.random.default_rng(1)
    G1, G2 = gg.standard_normal((h, r)), gg.standard_normal((h, r))
    return Q, K, V, G1, G2


ROWS = (0, 1, 127, 128, 500, 1023)

if __name__ == "__main__":
    Q, K, V, G1, G2 = build()
    O, d = orc.causal_polysketch_attention(Q, K, V, G1, G2)
    with open(os.path.join(HERE, "c0_oracle_samples.txt"), "w") as f:
        f.write("# row d O[0] O[31] O[63]  (oracle, Section 3 definition, numpy seeds 0/1)\n")
        for i in ROWS:
            f.write("%d %.17g %.17g %.17g %.17g\n" % (i, d[i], O[i, 0], O[i, 31], O[i, 63]))
