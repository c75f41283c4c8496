"""Pins for the oracle's learnable sketch (Algorithm 2 of the appendix) and the attention built on it."""
import math

import numpy as np

from oracle import polysketch as orc


def make_net(g, h, r, scale=0.3):
    return {"g0": 1.0 + 0.1 * g.standard_normal(h), "c0": 0.1 * g.standard_normal(h),
            "W1": scale * g.standard_normal((h, 8 * r)) / np.sqrt(h), "b1": 0.1 * g.standard_normal(8 * r),
            "g1": 1.0 + 0.1 * g.standard_normal(8 * r), "c1": 0.1 * g.standard_normal(8 * r),
            "W2": g.standard_normal((8 * r, r)) / np.sqrt(8 * r), "b2": 0.1 * g.standard_normal(r),
            "W3": g.standard_normal((r, 8 * r)) / np.sqrt(r), "b3": 0.1 * g.standard_normal(8 * r),
            "W4": g.standard_normal((8 * r, r)) / np.sqrt(8 * r), "b4": 0.1 * g.standard_normal(r)}


def test_one_row_entry_by_entry():
    g = np.random.default_rng(0)
    h, r = 6, 2
    P = make_net(g, h, r)
    x = g.standard_normal(h)

    def ln(v, gain, bias):
        mu = sum(v) / len(v)
        var = sum((a - mu) ** 2 for a in v) / len(v)
        return [(a - mu) / math.sqrt(var + 1e-6) * gain[i] + bias[i] for i, a in enumerate(v)]

    gl = lambda u: 0.5 * u * (1.0 + math.erf(u / math.sqrt(2.0)))
    z0 = ln(list(x), P["g0"], P["c0"])
    a1 = [gl(sum(z0[k] * P["W1"][k, j] for k in range(h)) + P["b1"][j]) for j in range(8 * r)]
    z1 = ln(a1, P["g1"], P["c1"])
    a2 = [sum(z1[k] * P["W2"][k, j] for k in range(8 * r)) + P["b2"][j] for j in range(r)]
    a3 = [gl(sum(a2[k] * P["W3"][k, j] for k in range(r)) + P["b3"][j]) for j in range(8 * r)]
    f = [sum(a3[k] * P["W4"][k, j] for k in range(8 * r)) + P["b4"][j] for j in range(r)]
    np.testing.assert_allclose(orc.learned_net(x[None, :], P)[0], f, rtol=1e-12, atol=1e-14)
    P2 = make_net(g, h, r)
    f2 = orc.learned_net(x[None, :], P2)[0]
    want = [math.sqrt(r) * math.tanh(f[j] * f2[j] / math.sqrt(r)) for j in range(r)]
    np.testing.assert_allclose(orc.learned_half_sketch(x[None, :], P, P2)[0], want, rtol=1e-12, atol=1e-14)


def test_output_is_bounded_by_sqrt_r():
    g = np.random.default_rng(1)
    h, r = 8, 4
    P1, P2 = make_net(g, h, r), make_net(g, h, r)
    P1["W4"] *= 40.0                                           # large products: deep into the tanh
    P2["W4"] *= 40.0
    M = orc.learned_half_sketch(10.0 * g.standard_normal((50, h)), P1, P2)
    assert np.all(np.abs(M) <= np.sqrt(r)) and np.abs(M).max() > 0.9 * np.sqrt(r)


def reducing_net(g, h, r, G, shift=12.0):
    """Parameters under which f(x) = LN(x) G up to the gelu tail at `shift`: W1 has orthonormal rows
    that each sum to zero, so the first hidden layer keeps the norm and adds a constant mean; the
    second normalisation then only rescales by sqrt(8r / h); the last two layers pass a2 through."""
    m = 8 * r
    A = g.standard_normal((h, m))
    A -= A.mean(axis=1, keepdims=True)                        # rows sum to zero
    Qm, _ = np.linalg.qr(A.T)                                 # m x h, orthonormal columns in the zero-sum subspace
    W1 = Qm.T
    W3 = np.zeros((r, m)); W3[:, :r] = np.eye(r)
    W4 = np.zeros((m, r)); W4[:r, :] = np.eye(r)
    b4 = -shift * np.ones(r)
    return {"g0": np.ones(h), "c0": np.zeros(h), "W1": W1, "b1": shift * np.ones(m),
            "g1": np.ones(m), "c1": np.zeros(m), "W2": np.sqrt(h / m) * W1.T @ G, "b2": np.zeros(r),
            "W3": W3, "b3": shift * np.ones(m), "W4": W4, "b4": b4}


def test_reduces_to_the_random_sketch_for_linear_networks_and_small_products():
    g = np.random.default_rng(2)
    h, r, n = 16, 4, 30
    X = g.standard_normal((n, h))
    Xn = (X - X.mean(axis=1, keepdims=True)) / np.sqrt(X.var(axis=1, keepdims=True) + orc.LN_EPS)
    G1, G2 = g.standard_normal((h, r)), g.standard_normal((h, r))
    eps = 0.02
    P1, P2 = reducing_net(g, h, r, eps * G1), reducing_net(g, h, r, eps * G2)
    # (exact up to the eps of the second normalisation, 1e-6 against a variance of h / 8r, and the gelu tail)
    np.testing.assert_allclose(orc.learned_net(X, P1), Xn @ (eps * G1), rtol=5e-6, atol=1e-9)
    M = orc.learned_half_sketch(X, P1, P2)
    # sqrt(r) tanh(u / sqrt(r)) -> u for small u = f1 * f2, and Algorithm 1 gives (x G1')(x G2') / sqrt(r):
    # the two agree for G' = r^(1/4) eps G
    c = eps * r ** 0.25
    want = orc.half_sketch(Xn, c * G1, c * G2)
    np.testing.assert_allclose(M, want, rtol=1e-4, atol=1e-9)
    assert np.abs(want).max() > 1e-4


def test_block_algorithm_equals_the_definition_also_with_exact_same_block_weights():
    g = np.random.default_rng(3)
    h, r, n = 6, 3, 24
    P1, P2 = make_net(g, h, r), make_net(g, h, r)
    Q, K, V = (g.standard_normal((n, h)) for _ in range(3))
    O, d = orc.causal_learned_polysketch_attention(Q, K, V, P1, P2)
    for b in (1, 4, 24):
        Ob, db = orc.causal_learned_polysketch_attention_blocked(Q, K, V, P1, P2, b)
        np.testing.assert_allclose(Ob, O, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(db, d, rtol=1e-11)
    Oe, de = orc.causal_learned_polysketch_attention_blocked(Q, K, V, P1, P2, n, diagonal="exact")
    Ox, dx = orc.causal_exact_polynomial_attention(Q, K, V, 4)      # one block: all pairs exact
    np.testing.assert_allclose(Oe, Ox, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(de, dx, rtol=1e-11)
    assert np.all(d >= 1.0)


def _numgrad(fun, x, eps=1e-6):
    gnum = np.zeros_like(x)
    for idx in np.ndindex(*x.shape):
        old = x[idx]
        x[idx] = old + eps; fp = fun()
        x[idx] = old - eps; fm = fun()
        x[idx] = old
        gnum[idx] = (fp - fm) / (2 * eps)
    return gnum


def test_backward_matches_central_differences_for_inputs_and_every_parameter_group():
    g = np.random.default_rng(4)
    h, r, n, b = 4, 2, 6, 3
    P1, P2 = make_net(g, h, r), make_net(g, h, r)
    Q, K, V, dO = (g.standard_normal((n, h)) for _ in range(4))
    for diag in ("LR", "exact"):
        if diag == "exact":
            fwd = lambda: orc.causal_learned_polysketch_attention_blocked(Q, K, V, P1, P2, b, diagonal="exact")[0]
        else:
            fwd = lambda: orc.causal_learned_polysketch_attention(Q, K, V, P1, P2)[0]
        loss = lambda: float((fwd() * dO).sum())
        dQ, dK, dV, g1, g2 = orc.causal_learned_polysketch_attention_backward(Q, K, V, P1, P2, dO, b, diag)
        for X, G in ((Q, dQ), (K, dK), (V, dV)):
            np.testing.assert_allclose(G, _numgrad(loss, X), rtol=2e-5, atol=2e-8)
        for P, gP in ((P1, g1), (P2, g2)):
            for key in orc.NET_KEYS:
                np.testing.assert_allclose(gP[key], _numgrad(loss, P[key]), rtol=5e-5, atol=5e-8, err_msg=key)


def test_gelu_and_its_derivative():
    x = np.linspace(-4, 4, 41)
    phi = np.array([0.5 * (1 + math.erf(v / math.sqrt(2))) for v in x])
    np.testing.assert_allclose(orc.gelu(x), x * phi, rtol=1e-14, atol=1e-16)
    e = 1e-6
    np.testing.assert_allclose(orc._gelu_grad(x), (orc.gelu(x + e) - orc.gelu(x - e)) / (2 * e), rtol=1e-7, atol=1e-9)
