"""Pins for the oracle's local-exact variant (Section 3.2): inside a block of b rows the
weights are the exact polynomial weights (q_i . k_j)^4, across blocks the Polysketch weights.
Each test ties it to something the paper or the mathematics fixes, not to the oracle itself."""
import math

import numpy as np
import pytest

from oracle import polysketch as orc


def rng(seed):
    return np.random.default_rng(seed)


def normalised(g, n, h, scale=1.0):
    x = g.standard_normal((n, h))
    return x * (scale * math.sqrt(h) / np.linalg.norm(x, axis=1, keepdims=True))


def _looped_local_exact(Q, K, V, G1, G2, b):
    """Section 3.2 with plain loops: token pairs of one block use (q.k)^4, all other causal
    pairs use (m(q).m(k))^2 with m written out entry by entry (Algorithm 1, degree-2 level)."""
    n, h = Q.shape
    r = G1.shape[1]

    def m(x):
        out = np.zeros(r)
        for c in range(r):
            a1 = sum(x[t] * G1[t, c] for t in range(h))
            a2 = sum(x[t] * G2[t, c] for t in range(h))
            out[c] = a1 * a2 / math.sqrt(r)
        return out

    O = np.zeros_like(V)
    d = np.zeros(n)
    for i in range(n):
        mq = m(Q[i])
        den, num = 1.0, np.zeros(V.shape[1])
        for j in range(i + 1):
            if i // b == j // b:
                w = float(np.dot(Q[i], K[j])) ** 4
            else:
                w = float(np.dot(mq, m(K[j]))) ** 2
            den += w
            num += w * V[j]
        O[i], d[i] = num / den, den
    return O, d


def _case(seed, n, h, r, scale=1.0):
    g = rng(seed)
    Q, K, V = normalised(g, n, h, scale), normalised(g, n, h, scale), g.standard_normal((n, h))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    return g, Q, K, V, G1, G2


def test_looped_definition():
    _, Q, K, V, G1, G2 = _case(20, 24, 5, 3)
    for b in (1, 4, 8, 24):
        O_ref, d_ref = _looped_local_exact(Q, K, V, G1, G2, b)
        O, d = orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, b)
        assert orc.rel_l2(O, O_ref) < 1e-12 and orc.rel_l2(d, d_ref) < 1e-12


def test_one_block_is_exact_polynomial_attention():
    # b = n: every causal pair shares the block, so the sketch drops out altogether (Section 2.1)
    _, Q, K, V, G1, G2 = _case(21, 32, 8, 4)
    O_ref, d_ref = orc.causal_exact_polynomial_attention(Q, K, V, 4)
    for fn in (orc.causal_polysketch_local_exact_attention,
               lambda *a: orc.causal_polysketch_attention_blocked(*a, diagonal="exact")):
        O, d = fn(Q, K, V, G1, G2, 32)
        assert orc.rel_l2(O, O_ref) < 1e-12 and orc.rel_l2(d, d_ref) < 1e-12
    # and different sketch matrices give the same result
    O2, _ = orc.causal_polysketch_local_exact_attention(Q, K, V, 2 * G1, G2[:, ::-1], 32)
    assert np.array_equal(O2, orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, 32)[0])


@pytest.mark.parametrize("b", [1, 4, 8, 16])
def test_block_algorithm_matches_masked_definition(b):
    # Section 3.1's algorithm with P_l = lt((Q_l K_l^T)^4) [V_l | 1] against the n x n definition
    _, Q, K, V, G1, G2 = _case(22, 32, 8, 5)
    O_ref, d_ref = orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, b)
    O, d = orc.causal_polysketch_attention_blocked(Q, K, V, G1, G2, b, diagonal="exact")
    assert orc.rel_l2(O, O_ref) < 1e-12 and orc.rel_l2(d, d_ref) < 1e-12


def test_block_size_matters_only_through_the_sketch_error():
    # with a real sketch the result depends on b ...
    _, Q, K, V, G1, G2 = _case(23, 32, 8, 4)
    O4, _ = orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, 4)
    O16, _ = orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, 16)
    assert orc.rel_l2(O4, O16) > 1e-3
    # ... and is closer to exact polynomial attention with larger blocks (more exact pairs)
    O_ex, _ = orc.causal_exact_polynomial_attention(Q, K, V, 4)
    errs = [orc.rel_l2(orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, b)[0], O_ex) for b in (1, 8, 32)]
    assert errs[2] < 1e-12 and errs[1] < errs[0]
    # when the degree-2 map is exact, (m(q).m(k))^2 = (q.k)^4 and b drops out: h = 3, m(x) = x (x) x
    # written as a "sketch" with G1 = I (x) 1^T, G2 = 1^T (x) I and r = h^2 (so 1/sqrt(r) is undone below)
    h = 3
    g = rng(24)
    Q, K, V = g.standard_normal((16, h)), g.standard_normal((16, h)), g.standard_normal((16, h))
    G1 = np.kron(np.eye(h), np.ones((1, h))) * math.sqrt(h)       # (x G1)[a*h+c] = sqrt(h) x_a
    G2 = np.kron(np.ones((1, h)), np.eye(h)) * math.sqrt(h)       # (x G2)[a*h+c] = sqrt(h) x_c
    M = orc.half_sketch(Q, G1, G2)
    np.testing.assert_allclose(M, orc.self_tensor(Q), rtol=1e-13, atol=1e-14)
    O_ex, d_ex = orc.causal_exact_polynomial_attention(Q, K, V, 4)
    for b in (1, 2, 4, 16):
        O, d = orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, b)
        assert orc.rel_l2(O, O_ex) < 1e-10 and orc.rel_l2(d, d_ex) < 1e-10


def test_weights_nonnegative_and_causal():
    g, Q, K, V, G1, G2 = _case(25, 32, 8, 4)
    W = orc.causal_weights_local_exact(Q, K, G1, G2, 8)
    assert (W >= 0).all() and np.abs(np.triu(W, 1)).max() == 0
    cut = 13
    K2, V2 = K.copy(), V.copy()
    K2[cut:] = g.standard_normal((32 - cut, 8))
    V2[cut:] = g.standard_normal((32 - cut, 8))
    Oa, da = orc.causal_polysketch_attention_blocked(Q, K, V, G1, G2, 8, diagonal="exact")
    Ob, db = orc.causal_polysketch_attention_blocked(Q, K2, V2, G1, G2, 8, diagonal="exact")
    assert np.array_equal(Oa[:cut], Ob[:cut]) and np.array_equal(da[:cut], db[:cut])
    assert not np.allclose(Oa[cut:], Ob[cut:])


def _loss(Q, K, V, G1, G2, dO, b):
    O, _ = orc.causal_polysketch_local_exact_attention(Q, K, V, G1, G2, b)
    return float((O * dO).sum())


@pytest.mark.parametrize("b", [2, 5, 10])
def test_backward_against_central_differences(b):
    g, Q, K, V, G1, G2 = _case(26, 10, 5, 3, scale=0.6)
    n, h = V.shape
    dO = g.standard_normal((n, h))
    grads = orc.causal_polysketch_local_exact_attention_backward(Q, K, V, G1, G2, dO, b)
    eps = 1e-6
    for which, grad in zip("QKV", grads):
        num = np.zeros((n, h))
        for i in range(n):
            for c in range(h):
                args = {"Q": Q.copy(), "K": K.copy(), "V": V.copy()}
                args[which][i, c] += eps
                up = _loss(args["Q"], args["K"], args["V"], G1, G2, dO, b)
                args[which][i, c] -= 2 * eps
                dn = _loss(args["Q"], args["K"], args["V"], G1, G2, dO, b)
                num[i, c] = (up - dn) / (2 * eps)
        assert orc.rel_l2(grad, num) < 1e-6, which


@pytest.mark.parametrize("b", [1, 8, 32])
def test_block_backward_matches_quadratic_backward(b):
    g, Q, K, V, G1, G2 = _case(27, 32, 12, 6)
    dO = g.standard_normal(V.shape)
    ref = orc.causal_polysketch_local_exact_attention_backward(Q, K, V, G1, G2, dO, b)
    got = orc.causal_polysketch_attention_backward_blocked(Q, K, V, G1, G2, dO, b, diagonal="exact")
    for a, e in zip(got, ref):
        assert orc.rel_l2(a, e) < 1e-10


def test_dV_is_transposed_weight_matrix():
    g, Q, K, V, G1, G2 = _case(28, 20, 6, 4)
    dO = g.standard_normal(V.shape)
    W = orc.causal_weights_local_exact(Q, K, G1, G2, 5)
    A = W / (1 + W.sum(1))[:, None]
    _, _, dV = orc.causal_polysketch_local_exact_attention_backward(Q, K, V, G1, G2, dO, 5)
    np.testing.assert_allclose(dV, A.T @ dO, rtol=1e-12, atol=1e-14)
