"""Pins for the oracle's non-causal Polysketch attention (Section 3, first formula: no mask,
one state phi'(K)^T [V | 1] per head)."""
import numpy as np

from oracle import polysketch as orc


def _data(n=24, h=6, r=5, seed=0):
    g = np.random.default_rng(seed)
    Q, K, V, dO = (g.standard_normal((n, h)) for _ in range(4))
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    return Q, K, V, dO, G1, G2


def test_exact_features_give_looped_degree4_attention_over_all_keys():
    # with exact degree-2 features m(x) = x (x) x the weights are (q.k)^4: Section 2.1 without a mask
    g = np.random.default_rng(1)
    n, h = 9, 3
    Q, K, V = (g.standard_normal((n, h)) for _ in range(3))
    Mq, Mk = orc.self_tensor(Q), orc.self_tensor(K)
    O, d = orc.attention_from_features(orc.self_tensor(Mq), orc.self_tensor(Mk), V)
    for i in range(n):
        num, den = np.zeros(h), 1.0
        for j in range(n):                                   # every key, also j > i
            w = float(Q[i] @ K[j]) ** 4
            num += w * V[j]
            den += w
        np.testing.assert_allclose(O[i], num / den, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(d[i], den, rtol=1e-10)


def test_looped_definition_with_the_sketch_written_out():
    Q, K, V, _, G1, G2 = _data(n=7, h=4, r=3, seed=2)
    O, d = orc.polysketch_attention(Q, K, V, G1, G2)
    r = G1.shape[1]
    m = lambda x: np.array([(x @ G1[:, c]) * (x @ G2[:, c]) / np.sqrt(r) for c in range(r)])
    for i in range(7):
        w = np.array([float(m(Q[i]) @ m(K[j])) ** 2 for j in range(7)])
        np.testing.assert_allclose(d[i], 1.0 + w.sum(), rtol=1e-12)
        np.testing.assert_allclose(O[i], (w[:, None] * V).sum(0) / (1.0 + w.sum()), rtol=1e-11, atol=1e-13)


def test_last_row_equals_the_causal_form_and_earlier_rows_do_not():
    Q, K, V, _, G1, G2 = _data(seed=3)
    O, d = orc.polysketch_attention(Q, K, V, G1, G2)
    Oc, dc = orc.causal_polysketch_attention(Q, K, V, G1, G2)
    np.testing.assert_allclose(O[-1], Oc[-1], rtol=1e-12)
    np.testing.assert_allclose(d[-1], dc[-1], rtol=1e-12)
    assert np.all(d[:-1] > dc[:-1])                          # every earlier row sees more keys
    assert np.abs(O[0] - Oc[0]).max() > 1e-3


def test_joint_permutation_of_keys_and_values_changes_nothing():
    Q, K, V, _, G1, G2 = _data(seed=4)
    perm = np.random.default_rng(5).permutation(K.shape[0])
    O, d = orc.polysketch_attention(Q, K, V, G1, G2)
    Op, dp = orc.polysketch_attention(Q, K[perm], V[perm], G1, G2)
    np.testing.assert_allclose(Op, O, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dp, d, rtol=1e-12)


def test_linear_time_form_equals_the_definition():
    Q, K, V, dO, G1, G2 = _data(n=40, h=8, r=6, seed=6)
    O, d = orc.polysketch_attention(Q, K, V, G1, G2)
    Ol, dl = orc.polysketch_attention_linear(Q, K, V, G1, G2)
    np.testing.assert_allclose(Ol, O, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(dl, d, rtol=1e-12)
    for a, b in zip(orc.polysketch_attention_backward(Q, K, V, G1, G2, dO),
                    orc.polysketch_attention_backward_linear(Q, K, V, G1, G2, dO)):
        np.testing.assert_allclose(b, a, rtol=1e-9, atol=1e-11)


def test_weights_non_negative_and_values_of_ones():
    Q, K, V, _, G1, G2 = _data(seed=7)
    O, d = orc.polysketch_attention(Q, K, np.ones_like(V), G1, G2)
    assert np.all(d >= 1.0)
    np.testing.assert_allclose(O, ((d - 1.0) / d)[:, None] * np.ones_like(V), rtol=1e-12)


def test_backward_matches_central_differences():
    Q, K, V, dO, G1, G2 = _data(n=6, h=4, r=3, seed=8)
    Q, K = 0.5 * Q, 0.5 * K
    grads = orc.polysketch_attention_backward(Q, K, V, G1, G2, dO)
    loss = lambda q, k, v: float((orc.polysketch_attention(q, k, v, G1, G2)[0] * dO).sum())
    eps = 1e-6
    for which, (X, G) in enumerate(zip((Q, K, V), grads)):
        num = np.zeros_like(X)
        for idx in np.ndindex(*X.shape):
            Xp, Xm = X.copy(), X.copy()
            Xp[idx] += eps
            Xm[idx] -= eps
            args_p = [Q, K, V]; args_m = [Q, K, V]
            args_p[which], args_m[which] = Xp, Xm
            num[idx] = (loss(*args_p) - loss(*args_m)) / (2 * eps)
        np.testing.assert_allclose(G, num, rtol=2e-6, atol=1e-8)


def test_dV_is_the_transposed_weight_matrix_times_dO():
    Q, K, V, dO, G1, G2 = _data(seed=9)
    s = orc.half_sketch(Q, G1, G2) @ orc.half_sketch(K, G1, G2).T
    W = s * s
    A = W / (1.0 + W.sum(axis=1))[:, None]
    np.testing.assert_allclose(orc.polysketch_attention_backward(Q, K, V, G1, G2, dO)[2], A.T @ dO, rtol=1e-11, atol=1e-13)
