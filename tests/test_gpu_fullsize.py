"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py
times: sampled (batch, head) slices against the block-form oracle (outputs and gradients),
sampled rows against Section 3's definition, and a finiteness sweep of the full tensors."""
import numpy as np
import pytest
import torch

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200 import inputs as wl
from parity_util import TOL, check, check_tiles, oracle_backward, oracle_forward, oracle_rows

pytestmark = pytest.mark.gpu


def _sample_heads(w, k=3):
    g = np.random.default_rng(w.data_seed)
    heads = [(0, 0), (w.B - 1, w.H - 1)]
    while len(heads) < k:
        h = (int(g.integers(w.B)), int(g.integers(w.H)))
        if h not in heads:
            heads.append(h)
    return heads


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_full_size_configuration(name):
    w = wl.WORKLOADS[name]
    inp = wl.make_inputs(w, "cuda")
    Q, K, V, G1, G2 = (inp[k] for k in ("Q", "K", "V", "G1", "G2"))
    # as bench.py runs it: forward and backward share the workspace and the forward's states
    flags = psk.FLAG_KEEP_STATES if w.backward else 0
    shp = psk.binding.make_shape(Q, G1, w.r, w.b, flags=flags)
    ws = torch.empty(max(psk.workspace_bytes(shp, False), psk.workspace_bytes(shp, w.backward)),
                     dtype=torch.uint8, device="cuda")
    O, den = psk.causal_attn_fwd(Q, K, V, G1, G2, w.b, workspace=ws, flags=flags)
    assert psk.check(ws) == 0
    grads = None
    if w.backward:
        grads = psk.causal_attn_bwd(Q, K, V, G1, G2, O, den, inp["dO"], w.b, workspace=ws, flags=flags)
        assert psk.check(ws) == 0
    tol = TOL[w.dtype]
    for t in (O, den) + tuple(grads or ()):
        assert torch.isfinite(t).all()
    assert (den >= 1).all()
    heads = _sample_heads(w, 3 if name != "c4" else 2)
    for idx, (bi, hi) in enumerate(heads):
        O_ref, d_ref = oracle_forward(inp, bi, hi, w.b)
        check("%s O[%d,%d]" % (name, bi, hi), O[bi, hi], O_ref, tol)
        check("%s denom[%d,%d]" % (name, bi, hi), den[bi, hi], d_ref, tol)
        # the slice norm cannot see a bad tile among thousands: every 128-row tile beyond the first
        # block holds the same tolerance on its own; the first block's figure is printed (run with -s)
        first, later = check_tiles("%s O[%d,%d]" % (name, bi, hi), O[bi, hi], O_ref, tol, w.b)
        print("%s O[%d,%d]: worst 128-row tile, first block %.2e, later blocks %.2e" % (name, bi, hi, first, later))
        if idx == 0:
            # single rows straight from the definition (quadratic form, no blocks)
            rows = [0, 1, w.b - 1, w.b, w.n // 2 + 3, w.n - 1]
            ref = oracle_rows(inp, bi, hi, rows)
            got = np.stack([O[bi, hi, i].double().cpu().numpy() for i in rows])
            exp = np.stack([ref[i][0] for i in rows])
            assert np.linalg.norm(got - exp) / np.linalg.norm(exp) <= tol
            # the target tolerance is a relative L2 over a tensor, not a per-element bound: a row
            # with one or two keys can be off by several percent in bf16 (its single score is a
            # cancelling dot product of bf16-rounded half sketches)
            dg = np.array([float(den[bi, hi, i]) for i in rows])
            de = np.array([ref[i][1] for i in rows])
            assert np.linalg.norm(dg - de) / np.linalg.norm(de) <= tol
            late = [i for i in rows if i >= w.b]
            for i in late:
                assert abs(float(den[bi, hi, i]) / ref[i][1] - 1) <= tol
        if w.backward and idx < 2:
            for nm, got, ref in zip(("dQ", "dK", "dV"), grads, oracle_backward(inp, bi, hi, w.b)):
                check("%s %s[%d,%d]" % (name, nm, bi, hi), got[bi, hi], ref, tol)
                first, later = check_tiles("%s %s[%d,%d]" % (name, nm, bi, hi), got[bi, hi], ref, 2 * tol, w.b)
                print("%s %s[%d,%d]: worst 128-row tile, first block %.2e, later blocks %.2e" % (name, nm, bi, hi, first, later))
