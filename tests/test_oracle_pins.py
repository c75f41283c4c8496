"""Pins for the CPU oracle: each test ties a part of oracle/polysketch.py to
something fixed by the paper or by mathematics, not to the oracle itself."""
from fractions import Fraction
import math

import numpy as np
import pytest

from oracle import polysketch as orc


def rng(seed):
    return np.random.default_rng(seed)


def normalised(g, n, h):
    x = g.standard_normal((n, h))
    return x * (math.sqrt(h) / np.linalg.norm(x, axis=1, keepdims=True))


# ---------------------------------------------------------------------------
# Hand-worked rational example (looped, exact arithmetic; Sections 2.2 and 3).
# ---------------------------------------------------------------------------
def _looped_polysketch_attention_fraction(Q, K, V, G1, G2, rsq):
    """Definition of Section 3 with plain loops over exact rationals.
    m(x)_c = (x.G1[:,c]) (x.G2[:,c]) / sqrt(r); the weights only use products
    m(q)_c m(k)_c, so 1/sqrt(r)^2 = 1/r stays rational (rsq = r)."""
    n, h, r = len(Q), len(Q[0]), len(G1[0])

    def raw(x):
        out = []
        for c in range(r):
            a1 = sum(x[t] * G1[t][c] for t in range(h))
            a2 = sum(x[t] * G2[t][c] for t in range(h))
            out.append(a1 * a2)
        return out

    O, D = [], []
    for i in range(n):
        mq = raw(Q[i])
        num = [Fraction(0)] * len(V[0])
        den = Fraction(1)
        for j in range(i + 1):
            mk = raw(K[j])
            s = sum(a * b for a, b in zip(mq, mk)) / rsq
            w = s * s
            den += w
            num = [x + w * v for x, v in zip(num, V[j])]
        O.append([x / den for x in num])
        D.append(den)
    return O, D


def test_hand_worked_rational_example():
    F = Fraction
    Q = [[F(1), F(2)], [F(0), F(-1)], [F(3), F(1)]]
    K = [[F(2), F(1)], [F(1), F(1)], [F(-1), F(2)]]
    V = [[F(1), F(0)], [F(0), F(2)], [F(3), F(-1)]]
    G1 = [[F(1), F(0), F(2), F(-1)], [F(0), F(1), F(1), F(1)]]
    G2 = [[F(1), F(1), F(0), F(2)], [F(-1), F(0), F(1), F(1)]]
    O_ref, d_ref = _looped_polysketch_attention_fraction(Q, K, V, G1, G2, 4)
    # first row by hand: m(q1)*2 = [(1)(-1), (2)(1), (4)(2), (1)(4)] = [-1,2,8,4];
    # m(k1)*2 = [(2)(1), (1)(2), (5)(1), (-1)(5)] = [2,2,5,-5]; s = (-2+4+40-20)/4 = 11/2
    assert d_ref[0] == 1 + Fraction(121, 4)
    assert O_ref[0] == [Fraction(121, 4) / (1 + Fraction(121, 4)), 0]
    f = lambda M: np.array([[float(x) for x in row] for row in M])
    O, d = orc.causal_polysketch_attention(f(Q), f(K), f(V), f(G1), f(G2))
    np.testing.assert_allclose(O, f(O_ref), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(d, [float(x) for x in d_ref], rtol=1e-13)
    O2, d2 = orc.causal_polysketch_attention_blocked(f(Q), f(K), f(V), f(G1), f(G2), 1)
    np.testing.assert_allclose(O2, f(O_ref), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(d2, [float(x) for x in d_ref], rtol=1e-13)


# ---------------------------------------------------------------------------
# Check 1: exact tensor features x (x) x reproduce brute-force (q.k)^4 attention.
# ---------------------------------------------------------------------------
def _looped_exact_poly_attention(Q, K, V, p):
    n = Q.shape[0]
    O = np.zeros_like(V)
    d = np.zeros(n)
    for i in range(n):
        den = 1.0
        num = np.zeros(V.shape[1])
        for j in range(i + 1):
            w = float(np.dot(Q[i], K[j])) ** p
            den += w
            num += w * V[j]
        O[i] = num / den
        d[i] = den
    return O, d


@pytest.mark.parametrize("h", [3, 4])
def test_exact_features_reproduce_degree4_attention(h):
    g = rng(h)
    n = 24
    Q, K = g.standard_normal((n, h)), g.standard_normal((n, h))
    V = g.standard_normal((n, h))
    O_ref, d_ref = _looped_exact_poly_attention(Q, K, V, 4)
    # the sketch replaced by the exact degree-2 map m(x) = x (x) x, then self-tensored
    PhiQ = orc.self_tensor(orc.self_tensor(Q))
    PhiK = orc.self_tensor(orc.self_tensor(K))
    O, d = orc.causal_attention_from_features(PhiQ, PhiK, V)
    assert orc.rel_l2(O, O_ref) < 1e-10
    assert orc.rel_l2(d, d_ref) < 1e-10
    O3, d3 = orc.causal_exact_polynomial_attention(Q, K, V, 4)
    assert orc.rel_l2(O3, O_ref) < 1e-12 and orc.rel_l2(d3, d_ref) < 1e-12
    # same through the block algorithm with C = [V | 1]
    C = np.concatenate([V, np.ones((n, 1))], axis=1)
    for b in (1, 4, 8, n):
        N = orc.lt_multiply_blocked(PhiQ, PhiK, C, b)
        assert orc.rel_l2(N[:, :h] / (1 + N[:, h:]), O_ref) < 1e-10


def test_kronecker_order_and_inner_product_identity():
    # a (x) b ordering of Section 1.2 and <a^(x)2, b^(x)2> = <a,b>^2 (Section 2.2)
    a = np.array([[1.0, 2.0, 3.0]])
    np.testing.assert_array_equal(orc.self_tensor(a)[0], [1, 2, 3, 2, 4, 6, 3, 6, 9])
    g = rng(0)
    A, B = g.standard_normal((5, 7)), g.standard_normal((6, 7))
    np.testing.assert_allclose(orc.self_tensor(A) @ orc.self_tensor(B).T, (A @ B.T) ** 2, rtol=1e-12)


# ---------------------------------------------------------------------------
# Check 2: block algorithm is independent of b; lt multiply vs dense triangle.
# ---------------------------------------------------------------------------
def test_lt_multiply_matches_dense_triangle():
    g = rng(1)
    n, m, k = 48, 10, 5
    A, B, C = g.standard_normal((n, m)), g.standard_normal((n, m)), g.standard_normal((n, k))
    dense = np.zeros((n, k))
    for i in range(n):
        for j in range(i + 1):           # j <= i: the diagonal is kept
            dense[i] += float(A[i] @ B[j]) * C[j]
    for b in (1, 2, 6, 16, n):
        np.testing.assert_allclose(orc.lt_multiply_blocked(A, B, C, b), dense, rtol=1e-11, atol=1e-11)
    with pytest.raises(ValueError):
        orc.lt_multiply_blocked(A, B, C, 5)


@pytest.mark.parametrize("diag", ["phi", "LR"])
def test_block_size_invariance(diag):
    g = rng(2)
    n, h, r = 64, 16, 8
    Q, K, V = normalised(g, n, h), normalised(g, n, h), g.standard_normal((n, h))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    O_ref, d_ref = orc.causal_polysketch_attention(Q, K, V, G1, G2)
    for b in (1, 16, n):
        O, d = orc.causal_polysketch_attention_blocked(Q, K, V, G1, G2, b, diagonal=diag)
        assert orc.rel_l2(O, O_ref) < 1e-11
        assert orc.rel_l2(d, d_ref) < 1e-11


# ---------------------------------------------------------------------------
# Check 3: non-negativity (Theorem 1.1 item 1).
# ---------------------------------------------------------------------------
def test_feature_inner_products_are_nonnegative():
    g = rng(3)
    n, h, r = 40, 64, 16
    Q, K = normalised(g, n, h), normalised(g, n, h)
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    PQ, PK = orc.polysketch_non_negative(Q, G1, G2), orc.polysketch_non_negative(K, G1, G2)
    assert PQ.shape == (n, r * r)
    gram = PQ @ PK.T
    assert (gram >= -1e-9 * np.abs(gram).max()).all()
    # and the un-tensored sketch does go negative, so the property is not vacuous
    assert (orc.half_sketch(Q, G1, G2) @ orc.half_sketch(K, G1, G2).T < 0).any()
    W = orc.causal_weights(Q, K, G1, G2)
    assert (W >= 0).all() and np.allclose(np.triu(W, 1), 0)
    np.testing.assert_allclose(W, np.tril(gram), rtol=1e-9, atol=1e-9 * gram.max())
    _, d = orc.causal_polysketch_attention(Q, K, g.standard_normal((n, h)), G1, G2)
    assert (d >= 1.0).all()


# ---------------------------------------------------------------------------
# Check 4: Monte-Carlo mean of the degree-2 sketch, with its closed-form variance.
# For Gaussian G: E[m(q).m(k)] = (q.k)^2 and
# Var = [ (|q|^2 |k|^2 + 2 (q.k)^2)^2 - (q.k)^4 ] / r   (fourth moments of a Gaussian).
# ---------------------------------------------------------------------------
def test_sketch_is_unbiased_with_known_variance():
    g = rng(4)
    h, r, trials = 12, 8, 20000
    q, k = g.standard_normal(h), g.standard_normal(h)
    qk, qq, kk = q @ k, q @ q, k @ k
    vals = np.empty(trials)
    for t in range(trials):
        G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
        vals[t] = (orc.half_sketch(q[None], G1, G2) @ orc.half_sketch(k[None], G1, G2).T)[0, 0]
    var = ((qq * kk + 2 * qk ** 2) ** 2 - qk ** 4) / r
    z = (vals.mean() - qk ** 2) / math.sqrt(var / trials)
    assert abs(z) < 4.5, z
    assert abs(vals.var() / var - 1.0) < 0.15


def test_sketch_error_falls_with_r():
    # Theorem 1.1 item 2 (trend only): Frobenius error of the weights ~ 1/sqrt(r)
    g = rng(5)
    n, h = 48, 16
    Q, K = normalised(g, n, h), normalised(g, n, h)
    exact = (Q @ K.T) ** 4
    errs = []
    for r in (8, 128):
        e = []
        for _ in range(8):
            G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
            s = orc.half_sketch(Q, G1, G2) @ orc.half_sketch(K, G1, G2).T
            e.append(np.linalg.norm(s * s - exact))
        errs.append(np.mean(e))
    assert errs[1] < 0.5 * errs[0]


def test_identity_sketch_closed_form():
    # G1 = G2 = I (r = h): m(x) = x*x/sqrt(h), so m(q).m(k) = sum_a q_a^2 k_a^2 / h
    g = rng(6)
    h = 6
    q, k = g.standard_normal((3, h)), g.standard_normal((4, h))
    I = np.eye(h)
    np.testing.assert_allclose(orc.half_sketch(q, I, I), q * q / math.sqrt(h), rtol=1e-14)
    s = orc.half_sketch(q, I, I) @ orc.half_sketch(k, I, I).T
    np.testing.assert_allclose(s, (q ** 2) @ (k ** 2).T / h, rtol=1e-13)


def test_recursion_levels_of_algorithm_1():
    g = rng(7)
    A = g.standard_normal((5, 6))
    M, rest = orc.polysketch_with_negativity(A, [], 1)
    assert M is not None and np.array_equal(M, A) and rest == []
    # p = 4: two independent degree-2 sketches, then r x r Gaussians
    r = 4
    Gs = [g.standard_normal((6, r)) for _ in range(4)] + [g.standard_normal((r, r)) for _ in range(2)]
    M4, rest = orc.polysketch_with_negativity(A, Gs, 4)
    M1 = (A @ Gs[0]) * (A @ Gs[1]) / 2.0
    M2 = (A @ Gs[2]) * (A @ Gs[3]) / 2.0
    np.testing.assert_allclose(M4, (M1 @ Gs[4]) * (M2 @ Gs[5]) / 2.0, rtol=1e-13)
    assert rest == []


# ---------------------------------------------------------------------------
# Normaliser, degenerate sizes, causality.
# ---------------------------------------------------------------------------
def test_all_ones_values_and_single_token():
    g = rng(8)
    n, h, r = 32, 8, 4
    Q, K = normalised(g, n, h), normalised(g, n, h)
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    O, d = orc.causal_polysketch_attention(Q, K, np.ones((n, h)), G1, G2)
    np.testing.assert_allclose(O, np.repeat(((d - 1) / d)[:, None], h, 1), rtol=1e-13)
    assert (O < 1).all()
    v = g.standard_normal((1, h))
    O1, d1 = orc.causal_polysketch_attention(Q[:1], K[:1], v, G1, G2)
    w11 = float((orc.half_sketch(Q[:1], G1, G2) @ orc.half_sketch(K[:1], G1, G2).T)[0, 0]) ** 2
    np.testing.assert_allclose(O1, w11 * v / (1 + w11), rtol=1e-13)
    np.testing.assert_allclose(d1, [1 + w11], rtol=1e-14)


def test_causality_forward_and_backward():
    g = rng(9)
    n, h, r, b = 32, 8, 4, 8
    Q, K, V = normalised(g, n, h), normalised(g, n, h), g.standard_normal((n, h))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    cut = 13
    K2, V2 = K.copy(), V.copy()
    K2[cut:] = g.standard_normal((n - cut, h))
    V2[cut:] = g.standard_normal((n - cut, h))
    for fn in (lambda k, v: orc.causal_polysketch_attention(Q, k, v, G1, G2),
               lambda k, v: orc.causal_polysketch_attention_blocked(Q, k, v, G1, G2, b)):
        Oa, da = fn(K, V)
        Ob, db = fn(K2, V2)
        assert np.array_equal(Oa[:cut], Ob[:cut]) and np.array_equal(da[:cut], db[:cut])
        assert not np.allclose(Oa[cut:], Ob[cut:])
    dO = np.zeros((n, h))
    dO[:cut] = g.standard_normal((cut, h))
    for grads in (orc.causal_polysketch_attention_backward(Q, K, V, G1, G2, dO),
                  orc.causal_polysketch_attention_backward_blocked(Q, K, V, G1, G2, dO, b)):
        dQ, dK, dV = grads
        assert np.abs(dK[cut:]).max() == 0 and np.abs(dV[cut:]).max() == 0
        assert np.abs(dQ[cut:]).max() == 0
        assert np.abs(dK[:cut]).max() > 0


# ---------------------------------------------------------------------------
# Backward: finite differences, explicit weight matrix, block form vs quadratic form.
# ---------------------------------------------------------------------------
def _loss(Q, K, V, G1, G2, dO):
    O, _ = orc.causal_polysketch_attention(Q, K, V, G1, G2)
    return float((O * dO).sum())


def test_backward_against_central_differences():
    g = rng(10)
    n, h, r = 10, 5, 3
    Q, K, V = normalised(g, n, h) * 0.6, normalised(g, n, h) * 0.6, g.standard_normal((n, h))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    dO = g.standard_normal((n, h))
    grads = orc.causal_polysketch_attention_backward(Q, K, V, G1, G2, dO)
    eps = 1e-6
    for which, grad in zip("QKV", grads):
        num = np.zeros((n, h))
        for i in range(n):
            for c in range(h):
                args = {"Q": Q.copy(), "K": K.copy(), "V": V.copy()}
                args[which][i, c] += eps
                up = _loss(args["Q"], args["K"], args["V"], G1, G2, dO)
                args[which][i, c] -= 2 * eps
                dn = _loss(args["Q"], args["K"], args["V"], G1, G2, dO)
                num[i, c] = (up - dn) / (2 * eps)
        assert orc.rel_l2(grad, num) < 1e-6, which


def test_dV_is_transposed_weight_matrix():
    # O is linear in V: O = A V with A_ij = W_ij / d_i, hence dV = A^T dO
    g = rng(11)
    n, h, r = 20, 6, 4
    Q, K, V = normalised(g, n, h), normalised(g, n, h), g.standard_normal((n, h))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    dO = g.standard_normal((n, h))
    W = orc.causal_weights(Q, K, G1, G2)
    A = W / (1 + W.sum(1))[:, None]
    _, _, dV = orc.causal_polysketch_attention_backward(Q, K, V, G1, G2, dO)
    np.testing.assert_allclose(dV, A.T @ dO, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("b", [1, 8, 32])
def test_block_backward_matches_quadratic_backward(b):
    g = rng(12)
    n, h, r = 32, 12, 6
    Q, K, V = normalised(g, n, h), normalised(g, n, h), g.standard_normal((n, h))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    dO = g.standard_normal((n, h))
    ref = orc.causal_polysketch_attention_backward(Q, K, V, G1, G2, dO)
    got = orc.causal_polysketch_attention_backward_blocked(Q, K, V, G1, G2, dO, b)
    for a, e in zip(got, ref):
        assert orc.rel_l2(a, e) < 1e-10


def test_rel_l2_metric():
    assert orc.rel_l2([3.0, 4.0], [3.0, 4.0]) == 0
    assert abs(orc.rel_l2([3.0, 5.0], [3.0, 4.0]) - 0.2) < 1e-15
