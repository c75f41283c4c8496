"""Pins for the oracle's degree-2 case (Algorithm 1 with p = 2: no sketch, phi'(x) = x (x) x)."""
import numpy as np
import pytest

from oracle import polysketch as orc


def _looped(Q, K, V):
    n = Q.shape[0]
    O, d = np.zeros_like(V), np.zeros(n)
    for i in range(n):
        den, num = 1.0, np.zeros(V.shape[1])
        for j in range(i + 1):
            w = float(np.dot(Q[i], K[j])) ** 2
            den += w
            num += w * V[j]
        O[i], d[i] = num / den, den
    return O, d


def _case(seed, n, h):
    g = np.random.default_rng(seed)
    return g, g.standard_normal((n, h)), g.standard_normal((n, h)), g.standard_normal((n, h))


@pytest.mark.parametrize("b", [1, 4, 8, 24])
def test_block_algorithm_is_exact_degree2_attention(b):
    _, Q, K, V = _case(40, 24, 5)
    O_ref, d_ref = _looped(Q, K, V)
    O, d = orc.causal_degree2_attention_blocked(Q, K, V, b)
    assert orc.rel_l2(O, O_ref) < 1e-12 and orc.rel_l2(d, d_ref) < 1e-12
    # Algorithm 1's recursion bottoms out at p = 1 with the matrix itself
    M, rest = orc.polysketch_with_negativity(Q, [], 1)
    assert np.array_equal(M, Q) and rest == []
    # and the features' inner products are the squared inner products
    np.testing.assert_allclose(orc.self_tensor(Q) @ orc.self_tensor(K).T, (Q @ K.T) ** 2, rtol=1e-12, atol=1e-12)
    O2, d2 = orc.causal_exact_polynomial_attention(Q, K, V, 2)
    assert orc.rel_l2(O2, O_ref) < 1e-12 and orc.rel_l2(d2, d_ref) < 1e-12


def test_backward_against_central_differences():
    g, Q, K, V = _case(41, 10, 4)
    Q, K = 0.7 * Q, 0.7 * K
    dO = g.standard_normal(V.shape)
    grads = orc.causal_degree2_attention_backward(Q, K, V, dO)

    def loss(q, k, v):
        return float((orc.causal_exact_polynomial_attention(q, k, v, 2)[0] * dO).sum())

    eps = 1e-6
    for which, grad in zip("QKV", grads):
        num = np.zeros_like(V)
        for i in range(V.shape[0]):
            for c in range(V.shape[1]):
                a = {"Q": Q.copy(), "K": K.copy(), "V": V.copy()}
                a[which][i, c] += eps
                up = loss(a["Q"], a["K"], a["V"])
                a[which][i, c] -= 2 * eps
                dn = loss(a["Q"], a["K"], a["V"])
                num[i, c] = (up - dn) / (2 * eps)
        assert orc.rel_l2(grad, num) < 1e-6, which
