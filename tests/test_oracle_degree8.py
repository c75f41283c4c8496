"""Pins for the oracle's degree-8 case (one more level of Algorithm 1's recursion)."""
import math

import numpy as np
import pytest

from oracle import polysketch as orc


def _gaussians(g, h, r):
    return [g.standard_normal((h, r)) for _ in range(4)] + [g.standard_normal((r, r)) for _ in range(2)]


def test_half_sketch_is_the_recursion_written_out():
    g = np.random.default_rng(50)
    h, r = 6, 4
    X = g.standard_normal((7, h))
    Gs = _gaussians(g, h, r)
    M1 = (X @ Gs[0]) * (X @ Gs[1]) / math.sqrt(r)
    M2 = (X @ Gs[2]) * (X @ Gs[3]) / math.sqrt(r)
    np.testing.assert_allclose(orc.half_sketch_degree4(X, Gs), (M1 @ Gs[4]) * (M2 @ Gs[5]) / math.sqrt(r), rtol=1e-13)


def test_half_sketch_inner_product_is_unbiased_for_the_fourth_power():
    # E[M(q) . M(k)] = (q . k)^4 over the Gaussians (each level is unbiased and they are independent)
    g = np.random.default_rng(51)
    h, r, trials = 5, 8, 60000
    q, k = g.standard_normal(h) * 0.8, g.standard_normal(h) * 0.8
    X = np.stack([q, k])
    vals = np.empty(trials)
    for t in range(trials):
        M = orc.half_sketch_degree4(X, _gaussians(g, h, r))
        vals[t] = M[0] @ M[1]
    target = float(q @ k) ** 4
    assert abs(vals.mean() - target) < 5 * vals.std() / math.sqrt(trials)


def test_weights_are_nonnegative_and_block_algorithm_matches_definition():
    g = np.random.default_rng(52)
    n, h, r = 32, 8, 6
    Q, K, V = g.standard_normal((n, h)) * 0.6, g.standard_normal((n, h)) * 0.6, g.standard_normal((n, h))
    Gs = _gaussians(g, h, r)
    O_ref, d_ref = orc.causal_polysketch8_attention(Q, K, V, Gs)
    assert (d_ref >= 1).all()
    Mq, Mk = orc.half_sketch_degree4(Q, Gs), orc.half_sketch_degree4(K, Gs)
    for b in (1, 8, 32):
        O, d = orc.causal_attention_blocked_from_half_sketches(Mq, Mk, V, b)
        assert orc.rel_l2(O, O_ref) < 1e-10 and orc.rel_l2(d, d_ref) < 1e-10
    # the same function on p = 4 half sketches is the p = 4 block algorithm
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    O4, d4 = orc.causal_polysketch_attention_blocked(Q, K, V, G1, G2, 8)
    O4b, d4b = orc.causal_attention_blocked_from_half_sketches(orc.half_sketch(Q, G1, G2), orc.half_sketch(K, G1, G2), V, 8)
    assert orc.rel_l2(O4b, O4) < 1e-12 and orc.rel_l2(d4b, d4) < 1e-12


def test_backward_against_central_differences():
    g = np.random.default_rng(53)
    n, h, r = 8, 4, 3
    Q, K, V = g.standard_normal((n, h)) * 0.7, g.standard_normal((n, h)) * 0.7, g.standard_normal((n, h))
    Gs = _gaussians(g, h, r)
    dO = g.standard_normal((n, h))
    grads = orc.causal_polysketch8_attention_backward(Q, K, V, Gs, dO)

    def loss(q, k, v):
        return float((orc.causal_polysketch8_attention(q, k, v, Gs)[0] * dO).sum())

    eps = 1e-6
    for which, grad in zip("QKV", grads):
        num = np.zeros((n, h))
        for i in range(n):
            for c in range(h):
                a = {"Q": Q.copy(), "K": K.copy(), "V": V.copy()}
                a[which][i, c] += eps
                up = loss(a["Q"], a["K"], a["V"])
                a[which][i, c] -= 2 * eps
                dn = loss(a["Q"], a["K"], a["V"])
                num[i, c] = (up - dn) / (2 * eps)
        assert orc.rel_l2(grad, num) < 1e-5, which
