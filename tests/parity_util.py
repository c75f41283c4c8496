"""Helpers for the GPU parity tests: run the oracle on (batch, head) slices of the
stored tensors and compare element by element."""
import numpy as np
import torch

from oracle import polysketch as orc
from paper_2310_01655_b200.inputs import head_slice_f64

# Tolerances of the build target: relative L2 over a whole tensor.
TOL = {"f32": 1e-4, "bf16": 2e-2}


def g_slice(G, hi):
    return G[hi if G.shape[0] > 1 else 0].detach().cpu().to(torch.float64).numpy()


def oracle_forward(inp, bi, hi, b):
    Q, K, V = (head_slice_f64(inp[k], bi, hi) for k in "QKV")
    return orc.causal_polysketch_attention_blocked(Q, K, V, g_slice(inp["G1"], hi), g_slice(inp["G2"], hi), b)


def oracle_backward(inp, bi, hi, b):
    Q, K, V, dO = (head_slice_f64(inp[k], bi, hi) for k in ("Q", "K", "V", "dO"))
    return orc.causal_polysketch_attention_backward_blocked(
        Q, K, V, g_slice(inp["G1"], hi), g_slice(inp["G2"], hi), dO, b)


def oracle_rows(inp, bi, hi, rows):
    """Section 3's definition for single rows i: weights (m(q_i).m(k_j))^2, j <= i."""
    Q, K, V = (head_slice_f64(inp[k], bi, hi) for k in "QKV")
    G1, G2 = g_slice(inp["G1"], hi), g_slice(inp["G2"], hi)
    Mk = orc.half_sketch(K, G1, G2)
    out = {}
    for i in rows:
        mq = orc.half_sketch(Q[i:i + 1], G1, G2)[0]
        w = (Mk[:i + 1] @ mq) ** 2
        d = 1.0 + w.sum()
        out[i] = ((w @ V[:i + 1]) / d, d)
    return out


def check(name, got, ref, tol):
    err = orc.rel_l2(got.detach().cpu().to(torch.float64).numpy(), ref)
    assert np.isfinite(err) and err <= tol, "%s: rel L2 %.3e > %.1e" % (name, err, tol)
    return err


def tile_errors(got, ref, rows=128):
    """Relative L2 of every tile of `rows` consecutive rows of a [n, ...] tensor: the slice-level norm
    is dominated by late rows (large normalisers), so the worst tile is reported beside it."""
    g = got.detach().cpu().to(torch.float64).numpy()
    g = g.reshape(g.shape[0], -1)
    r = np.asarray(ref, dtype=np.float64).reshape(g.shape[0], -1)
    n = g.shape[0] // rows * rows
    num = np.linalg.norm((g[:n] - r[:n]).reshape(n // rows, -1), axis=1)
    den = np.linalg.norm(r[:n].reshape(n // rows, -1), axis=1)
    return num / np.maximum(den, 1e-300)


def check_tiles(name, got, ref, tol, first_block_rows, rows=128):
    """Per-tile bound for tiles beyond the first block (every row there has at least a block of keys
    behind it); the first block's worst tile is returned for the record, not asserted: a row with one
    or two keys has a single cancelling score and is outside what a tensor-level tolerance covers."""
    e = tile_errors(got, ref, rows)
    k = first_block_rows // rows
    later = float(e[k:].max()) if len(e) > k else 0.0
    assert np.isfinite(e).all() and later <= tol, "%s: worst 128-row tile beyond the first block %.3e > %.1e" % (name, later, tol)
    return float(e[:k].max()) if k else 0.0, later
