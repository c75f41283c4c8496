"""The oracle still reproduces the rows it wrote to tests/golden/ (regression anchor)."""
import importlib.util
import os

import numpy as np

from oracle import polysketch as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def test_c0_samples_unchanged():
    spec = importlib.util.spec_from_file_location("make_c0_reference",
                                                  os.path.join(HERE, "golden", "make_c0_reference.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    Q, K, V, G1, G2 = mod.build()
    O, d = orc.causal_polysketch_attention_blocked(Q, K, V, G1, G2, 128)
    rows = np.loadtxt(os.path.join(HERE, "golden", "c0_oracle_samples.txt"))
    for i, di, o0, o31, o63 in rows:
        i = int(i)
        np.testing.assert_allclose([d[i], O[i, 0], O[i, 31], O[i, 63]], [di, o0, o31, o63], rtol=1e-10)
