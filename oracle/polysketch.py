"""CPU oracle for causal polynomial-sketch (Polysketch) attention, fp64.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference that the
CUDA library is checked against.  It shares no code with the CUDA path and the
product never imports it: only the tests, the smoke check and the benchmark's
CPU-baseline leg may call it.

Everything here works on ONE (batch, head) slice: Q, K, V are (n, h) arrays,
G1, G2 are (h, r).  Arithmetic is float64 throughout.  Matrix products use
numpy's matmul as a library primitive; nothing is blocked, fused or reordered
beyond what the cited definition or algorithm states.

Notation (paper -> here)
  M = A^{(x)2} S               half sketch, Section 2.2 / Algorithm 1 (p = 2 level)
  phi'(A) = M^{(x)2}           self-tensored features, Algorithm 1 (PolySketchNonNegative)
  lt(.)                        keep the lower triangle INCLUDING the diagonal (Section 1.2)
  D~ = diag(1 + lt(..) 1)      row normaliser of Section 3 (the "1 +" is part of it)
  H_l, Z_l, P_l                per-block state, exclusive prefix, diagonal block (Section 3.1)
  P_l = lt((Q_l K_l^T)^p) X_l  exact polynomial weights inside a block (Section 3.2)

Pins (tests/test_oracle_*.py): exact-feature case against looped (q.k)^4
attention, hand-worked rational example, G = I closed form, Monte-Carlo mean and
closed-form variance of the sketch, V = 1 closed form, n = 1 closed form,
causality, block-size invariance, lt-multiply against a dense triangle, central
finite differences for every gradient, dV against the explicit weight matrix;
for the local-exact variant (Section 3.2): one block = exact polynomial
attention, exact features = no dependence on the block size, looped definition,
block algorithm against the masked definition, finite differences; for
degree 2 (no sketch): looped (q.k)^2 attention, finite differences; for degree 8:
the recursion written out, Monte-Carlo mean (q.k)^4 of the half sketch, exact
features, block algorithm against the definition, finite differences.
the non-causal form of Section 3: looped (q.k)^4 attention over all keys, invariance
under a joint permutation of keys and values, last row of the causal form, linear-time
evaluation against the definition, finite differences.
for the learnable sketch (Algorithm 2): one row evaluated entry by entry, the bound |M| <= sqrt(r),
weights under which each network reduces to x -> LN(x) G so that the result approaches the random
sketch's, finite differences for inputs and every parameter group.
Every function in this file has at least one such pin.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _f64(x):
    return np.asarray(x, dtype=F64)


# ---------------------------------------------------------------------------
# Algorithm 1
# ---------------------------------------------------------------------------
def polysketch_with_negativity(A, gaussians, p):
    """Algorithm 1, PolySketchWithNegativity(A, r, p): A^{(x)p} S.

    `gaussians` supplies the matrices the algorithm would sample, in the order
    the recursion consumes them (left sub-call first, then right sub-call, then
    this level's own G1, G2), so that the same S can be applied to Q and to K
    (Definition 2.1 uses one S on both sides).  p = 1 returns A; p = 2 uses two
    (m x r) matrices; p = 4 uses 2 + 2 (m x r) and then two (r x r).
    """
    A = _f64(A)
    if p == 1:
        return A, gaussians
    if p < 1 or p % 2:
        raise ValueError("p must be a power of two")
    M1, rest = polysketch_with_negativity(A, gaussians, p // 2)
    M2, rest = polysketch_with_negativity(A, rest, p // 2)
    G1, G2 = _f64(rest[0]), _f64(rest[1])
    r = G1.shape[1]
    return np.sqrt(1.0 / r) * ((M1 @ G1) * (M2 @ G2)), rest[2:]


def half_sketch(X, G1, G2):
    """Degree-2 level of Algorithm 1 (Section 2.2): sqrt(1/r) [(X G1) * (X G2)]."""
    M, rest = polysketch_with_negativity(X, [G1, G2], 2)
    assert len(rest) == 0
    return M


def self_tensor(M):
    """Row-wise M^{(x)2}: entry (a, b) of the Kronecker square sits at a*r + b
    (the ordering of the Kronecker product in Section 1.2)."""
    M = _f64(M)
    n, r = M.shape
    return (M[:, :, None] * M[:, None, :]).reshape(n, r * r)


def polysketch_non_negative(A, G1, G2):
    """Algorithm 1, PolySketchNonNegative(A, r, 4): phi'(A) = (A^{(x)2} S)^{(x)2}."""
    return self_tensor(half_sketch(A, G1, G2))


# ---------------------------------------------------------------------------
# Definitions: Section 2.1 (exact polynomial attention), Section 3 (causal
# Polysketch attention).  Quadratic in n; these are the plain definitions.
# ---------------------------------------------------------------------------
def lt(M):
    """Lower-triangular part including the diagonal (j <= i), Section 1.2."""
    return np.tril(_f64(M))


def causal_attention_from_features(PhiQ, PhiK, V):
    """Section 3: D~^{-1} lt(phi'(Q) phi'(K)^T) V with D~ = diag(1 + lt(..) 1).

    Returns (O, d) with d the diagonal of D~.
    """
    W = lt(_f64(PhiQ) @ _f64(PhiK).T)
    d = 1.0 + W.sum(axis=1)
    return (W @ _f64(V)) / d[:, None], d


def causal_polysketch_attention(Q, K, V, G1, G2):
    """Section 3 with phi' from Algorithm 1 (p = 4), features materialised."""
    return causal_attention_from_features(
        polysketch_non_negative(Q, G1, G2), polysketch_non_negative(K, G1, G2), V)


def causal_weights(Q, K, G1, G2):
    """lt(phi'(Q) phi'(K)^T) through the identity <a^{(x)2}, b^{(x)2}> = <a,b>^2
    (Section 2.2): entries (m(q_i) . m(k_j))^2 for j <= i, zero above."""
    s = half_sketch(Q, G1, G2) @ half_sketch(K, G1, G2).T
    return lt(s * s)


def causal_exact_polynomial_attention(Q, K, V, p):
    """Section 2.1 with a causal mask: weights <q_i,k_j>^p / (1 + sum_{j'<=i} <q_i,k_j'>^p)."""
    W = lt((_f64(Q) @ _f64(K).T) ** p)
    d = 1.0 + W.sum(axis=1)
    return (W @ _f64(V)) / d[:, None], d


# ---------------------------------------------------------------------------
# Section 3.1: block lower-triangular multiplication
# ---------------------------------------------------------------------------
def lt_multiply_blocked(A, B, C, b, diag_block=None):
    """lt(A B^T) C by the block algorithm of Section 3.1.

    Blocks of b consecutive rows (n = t*b).  H_l = sum_{i in block l} b_i c_i^T,
    Z_l = sum_{j<l} H_j (sequential prefix, as the authors use),
    P_l = lt(A_l B_l^T) C_l, and rows of block l are P_l + A_l Z_l.
    `diag_block(l)` may return lt(A_l B_l^T) computed some other way (the
    (L R^T)^2 shortcut of Section 3.1); default is the direct product.
    """
    A, B, C = _f64(A), _f64(B), _f64(C)
    n, m = A.shape
    k = C.shape[1]
    if n % b:
        raise ValueError("n must be a multiple of the block size")
    t = n // b
    out = np.empty((n, k), dtype=F64)
    Z = np.zeros((m, k), dtype=F64)
    for l in range(t):
        rows = slice(l * b, (l + 1) * b)
        Al, Bl, Cl = A[rows], B[rows], C[rows]
        T = lt(Al @ Bl.T) if diag_block is None else diag_block(l)
        P = T @ Cl
        out[rows] = P + Al @ Z
        H = Bl.T @ Cl
        Z = Z + H
    return out


def same_block(n, b):
    """Boolean n x n matrix: tokens i and j lie in the same block of b rows (Section 3.1's B_l)."""
    blk = np.arange(n) // b
    return blk[:, None] == blk[None, :]


def causal_weights_local_exact(Q, K, G1, G2, b, p=4):
    """Section 3.2 as a definition: the weight of (i, j), j <= i, is the exact polynomial
    weight <q_i, k_j>^p when i and j share a block of b rows, and the Polysketch weight
    (m(q_i) . m(k_j))^2 otherwise."""
    Q, K = _f64(Q), _f64(K)
    s = half_sketch(Q, G1, G2) @ half_sketch(K, G1, G2).T
    return lt(np.where(same_block(Q.shape[0], b), (Q @ K.T) ** p, s * s))


def causal_polysketch_local_exact_attention(Q, K, V, G1, G2, b):
    """Section 3 with the weights of Section 3.2; returns (O, d), d including its "1 +"."""
    W = causal_weights_local_exact(Q, K, G1, G2, b)
    d = 1.0 + W.sum(axis=1)
    return (W @ _f64(V)) / d[:, None], d


def causal_polysketch_attention_blocked(Q, K, V, G1, G2, b, diagonal="LR"):
    """Causal Polysketch attention in time linear in n (Section 3.1).

    A = phi'(Q), B = phi'(K), C = [V | 1_n]; the last output column is the
    normaliser without its "1 +".  diagonal="phi" forms the diagonal blocks from
    the r^2-dimensional features, diagonal="LR" from (L R^T)^2 with L, R the
    b x r half sketches of the block, diagonal="exact" from the block's own
    queries and keys, lt((Q_l K_l^T)^4) (Section 3.2, p = 4).
    """
    V = _f64(V)
    n, h = V.shape
    Mq, Mk = half_sketch(Q, G1, G2), half_sketch(K, G1, G2)
    C = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    if diagonal == "phi":
        diag_block = None
    elif diagonal == "LR":
        def diag_block(l):
            L, R = Mq[l * b:(l + 1) * b], Mk[l * b:(l + 1) * b]
            return lt((L @ R.T) ** 2)
    elif diagonal == "exact":
        Qf, Kf = _f64(Q), _f64(K)

        def diag_block(l):
            return lt((Qf[l * b:(l + 1) * b] @ Kf[l * b:(l + 1) * b].T) ** 4)
    else:
        raise ValueError(diagonal)
    N = lt_multiply_blocked(self_tensor(Mq), self_tensor(Mk), C, b, diag_block)
    d = 1.0 + N[:, h]
    return N[:, :h] / d[:, None], d


# ---------------------------------------------------------------------------
# Backward.  The paper differentiates automatically and prints no formulas;
# these are the derivatives of the definitions above, taken by hand:
#   O_i = N_i / d_i,  N_i = sum_{j<=i} W_ij v_j,  d_i = 1 + sum_{j<=i} W_ij,
#   W_ij = s_ij^2,  s_ij = m(q_i) . m(k_j),  m(x) = (x G1)*(x G2)/sqrt(r).
# With g = dL/dO:  dL/dN_i = g_i/d_i,  dL/dd_i = -(g_i . O_i)/d_i, so with
#   E_i = [ g_i/d_i | -(g_i . O_i)/d_i ]  and  V~_j = [ v_j | 1 ]
# dL/dW_ij = E_i . V~_j for j <= i.
# ---------------------------------------------------------------------------
def _backward_rows(O, d, dO):
    O, d, dO = _f64(O), _f64(d), _f64(dO)
    return np.concatenate([dO / d[:, None],
                           -((dO * O).sum(axis=1) / d)[:, None]], axis=1)


def _sketch_backward(X, G1, G2, dM):
    """Chain rule through m(x): dX = ((dM*A2) G1^T + (dM*A1) G2^T)/sqrt(r)."""
    X, G1, G2 = _f64(X), _f64(G1), _f64(G2)
    r = G1.shape[1]
    A1, A2 = X @ G1, X @ G2
    return ((dM * A2) @ G1.T + (dM * A1) @ G2.T) / np.sqrt(r)


def causal_polysketch_attention_backward(Q, K, V, G1, G2, dO):
    """Gradients (dQ, dK, dV) of sum(dO * O) through the quadratic definition."""
    V = _f64(V)
    n, h = V.shape
    Mq, Mk = half_sketch(Q, G1, G2), half_sketch(K, G1, G2)
    s = Mq @ Mk.T
    W = lt(s * s)
    d = 1.0 + W.sum(axis=1)
    O = (W @ V) / d[:, None]
    E = _backward_rows(O, d, dO)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    dW = lt(E @ Vt.T)
    dV = W.T @ E[:, :h]
    ds = 2.0 * s * dW
    dMq = ds @ Mk
    dMk = ds.T @ Mq
    return (_sketch_backward(Q, G1, G2, dMq), _sketch_backward(K, G1, G2, dMk), dV)


def causal_polysketch_local_exact_attention_backward(Q, K, V, G1, G2, dO, b):
    """Gradients (dQ, dK, dV) of sum(dO * O) for the weights of Section 3.2, through the
    quadratic definition.  Same-block pairs: W_ij = x_ij^4 with x_ij = q_i . k_j, so
    dL/dx_ij = 4 x_ij^3 dL/dW_ij reaches Q and K directly; other pairs go through the half
    sketches as in causal_polysketch_attention_backward."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    n, h = V.shape
    Mq, Mk = half_sketch(Q, G1, G2), half_sketch(K, G1, G2)
    same = same_block(n, b)
    s = Mq @ Mk.T
    x = Q @ K.T
    W = lt(np.where(same, x ** 4, s * s))
    d = 1.0 + W.sum(axis=1)
    O = (W @ V) / d[:, None]
    E = _backward_rows(O, d, dO)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    dW = lt(E @ Vt.T)
    dV = W.T @ E[:, :h]
    ds = np.where(same, 0.0, 2.0 * s * dW)
    dx = np.where(same, 4.0 * x ** 3 * dW, 0.0)
    dQ = _sketch_backward(Q, G1, G2, ds @ Mk) + dx @ K
    dK = _sketch_backward(K, G1, G2, ds.T @ Mq) + dx.T @ Q
    return dQ, dK, dV


def causal_polysketch_attention_backward_blocked(Q, K, V, G1, G2, dO, b, diagonal="LR"):
    """Same gradients in time linear in n, in the style of Section 3.1.

    diagonal="exact": the same-block pairs carry the weights of Section 3.2,
    (q_i . k_j)^4, whose gradient 4 (q_i . k_j)^3 dW_ij reaches Q and K directly.

    Forward sweep carries Z_l = sum_{blocks < l} phi'(K)^T V~ (the forward's
    own prefix); reverse sweep carries R_l = sum_{blocks > l} phi'(Q)^T E.
    For a row in block l:  d phi'(q_i) = Z_l E_i,  d phi'(k_j) = R_l V~_j,
    dV~_j = R_l^T phi'(k_j); the same-block pairs go through the b x b tile
    exactly as in the forward.  d m = (mat(d phi') + mat(d phi')^T) m because
    phi'(m)[a*r+b] = m_a m_b.
    """
    V = _f64(V)
    n, h = V.shape
    if n % b:
        raise ValueError("n must be a multiple of the block size")
    t = n // b
    G1 = _f64(G1)
    r = G1.shape[1]
    Mq, Mk = half_sketch(Q, G1, G2), half_sketch(K, G1, G2)
    if diagonal not in ("LR", "exact"):
        raise ValueError(diagonal)
    exact = diagonal == "exact"
    Qf, Kf = _f64(Q), _f64(K)
    dQl = np.zeros_like(Qf)
    dKl = np.zeros_like(Kf)
    O, d = causal_polysketch_attention_blocked(Q, K, V, G1, G2, b, diagonal=diagonal)
    E = _backward_rows(O, d, dO)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    PhiQ, PhiK = self_tensor(Mq), self_tensor(Mk)
    dMq = np.zeros_like(Mq)
    dMk = np.zeros_like(Mk)
    dVt = np.zeros_like(Vt)

    def untensor(dPhi, M):
        T = dPhi.reshape(-1, r, r)
        return np.einsum("nab,nb->na", T + T.transpose(0, 2, 1), M)

    # same-block pairs and the forward sweep (earlier blocks -> queries)
    Z = np.zeros((r * r, h + 1), dtype=F64)
    for l in range(t):
        rows = slice(l * b, (l + 1) * b)
        dW = lt(E[rows] @ Vt[rows].T)
        if exact:
            x = Qf[rows] @ Kf[rows].T
            W = lt(x ** 4)
            dx = 4.0 * x ** 3 * dW
            dQl[rows] += dx @ Kf[rows]
            dKl[rows] += dx.T @ Qf[rows]
        else:
            s = Mq[rows] @ Mk[rows].T
            W = lt(s * s)
            ds = 2.0 * s * dW
            dMq[rows] += ds @ Mk[rows]
            dMk[rows] += ds.T @ Mq[rows]
        dVt[rows] += W.T @ E[rows]
        dMq[rows] += untensor(E[rows] @ Z.T, Mq[rows])
        Z = Z + PhiK[rows].T @ Vt[rows]
    # reverse sweep (later blocks -> keys and values)
    R = np.zeros((r * r, h + 1), dtype=F64)
    for l in range(t - 1, -1, -1):
        rows = slice(l * b, (l + 1) * b)
        dMk[rows] += untensor(Vt[rows] @ R.T, Mk[rows])
        dVt[rows] += PhiK[rows] @ R
        R = R + PhiQ[rows].T @ E[rows]
    return (_sketch_backward(Q, G1, G2, dMq) + dQl, _sketch_backward(K, G1, G2, dMk) + dKl, dVt[:, :h])


# ---------------------------------------------------------------------------
# Degree p = 2: Algorithm 1 with p/2 = 1 has no sketch at all (PolySketchWithNegativity(A, r, 1)
# is A), so phi'(A) = A^{(x)2} with h^2 entries and the attention is exact degree-2 polynomial
# attention (Section 2.1 with p = 2).
# ---------------------------------------------------------------------------
def causal_degree2_attention_blocked(Q, K, V, b):
    """Section 3.1's block algorithm on phi'(A) = A^{(x)2} (Algorithm 1, p = 2), diagonal
    blocks through (Q_l K_l^T)^2.  Returns (O, d)."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    n, h = V.shape
    C = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)

    def diag_block(l):
        return lt((Q[l * b:(l + 1) * b] @ K[l * b:(l + 1) * b].T) ** 2)

    N = lt_multiply_blocked(self_tensor(Q), self_tensor(K), C, b, diag_block)
    d = 1.0 + N[:, h]
    return N[:, :h] / d[:, None], d


def causal_degree2_attention_backward(Q, K, V, dO):
    """Gradients (dQ, dK, dV) of sum(dO * O) for the weights (q_i . k_j)^2, j <= i, through the
    quadratic definition: ds = 2 s dW reaches Q and K directly (there is no sketch)."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    n, h = V.shape
    s = Q @ K.T
    W = lt(s * s)
    d = 1.0 + W.sum(axis=1)
    O = (W @ V) / d[:, None]
    E = _backward_rows(O, d, dO)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    dW = lt(E @ Vt.T)
    ds = 2.0 * s * dW
    return ds @ K, ds.T @ Q, W.T @ E[:, :h]


# ---------------------------------------------------------------------------
# Degree p = 8: one more level of Algorithm 1's recursion.  PolySketchWithNegativity(A, r, 4)
# combines two independent degree-2 sketches M1, M2 of A through two r x r Gaussians,
#   M = sqrt(1/r) [(M1 Gc1) * (M2 Gc2)],   M1 = sqrt(1/r) [(A Ga1) * (A Ga2)],  M2 likewise with Gb,
# and phi'(A) = M^{(x)2}: <phi'(q), phi'(k)> = (M_q . M_k)^2 approximates (q . k)^8.
# Everything after the half sketch M is the p = 4 algorithm unchanged.
# ---------------------------------------------------------------------------
def half_sketch_degree4(X, gaussians):
    """PolySketchWithNegativity(X, r, 4) with gaussians = [Ga1, Ga2, Gb1, Gb2, Gc1, Gc2]."""
    M, rest = polysketch_with_negativity(X, list(gaussians), 4)
    assert len(rest) == 0
    return M


def causal_attention_blocked_from_half_sketches(Mq, Mk, V, b):
    """Section 3.1 on phi' = M^{(x)2} for given half sketches (diagonal blocks through (L R^T)^2)."""
    Mq, Mk, V = _f64(Mq), _f64(Mk), _f64(V)
    n, h = V.shape
    C = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)

    def diag_block(l):
        return lt((Mq[l * b:(l + 1) * b] @ Mk[l * b:(l + 1) * b].T) ** 2)

    N = lt_multiply_blocked(self_tensor(Mq), self_tensor(Mk), C, b, diag_block)
    d = 1.0 + N[:, h]
    return N[:, :h] / d[:, None], d


def causal_polysketch8_attention(Q, K, V, gaussians):
    """Section 3 with phi' = PolySketchNonNegative(., r, 8): the n x n definition.  Returns (O, d)."""
    s = half_sketch_degree4(Q, gaussians) @ half_sketch_degree4(K, gaussians).T
    W = lt(s * s)
    d = 1.0 + W.sum(axis=1)
    return (W @ _f64(V)) / d[:, None], d


def _sketch_degree4_backward(X, gaussians, dM):
    """Chain rule through M = sqrt(1/r) [(M1 Gc1) * (M2 Gc2)] and the two degree-2 sketches."""
    X = _f64(X)
    Ga1, Ga2, Gb1, Gb2, Gc1, Gc2 = (_f64(g) for g in gaussians)
    r = Gc1.shape[1]
    rs = 1.0 / np.sqrt(r)
    M1 = rs * (X @ Ga1) * (X @ Ga2)
    M2 = rs * (X @ Gb1) * (X @ Gb2)
    C1, C2 = M1 @ Gc1, M2 @ Gc2
    dM1 = (rs * dM * C2) @ Gc1.T
    dM2 = (rs * dM * C1) @ Gc2.T
    return _sketch_backward(X, Ga1, Ga2, dM1) + _sketch_backward(X, Gb1, Gb2, dM2)


def causal_polysketch8_attention_backward(Q, K, V, gaussians, dO):
    """Gradients (dQ, dK, dV) of sum(dO * O) for degree 8, through the quadratic definition."""
    V = _f64(V)
    n, h = V.shape
    Mq, Mk = half_sketch_degree4(Q, gaussians), half_sketch_degree4(K, gaussians)
    s = Mq @ Mk.T
    W = lt(s * s)
    d = 1.0 + W.sum(axis=1)
    O = (W @ V) / d[:, None]
    E = _backward_rows(O, d, dO)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    dW = lt(E @ Vt.T)
    ds = 2.0 * s * dW
    return (_sketch_degree4_backward(Q, gaussians, ds @ Mk), _sketch_degree4_backward(K, gaussians, ds.T @ Mq),
            W.T @ E[:, :h])


# ---------------------------------------------------------------------------
# Section 3, first formula: Polysketch attention WITHOUT the causal mask,
#   D~^{-1} phi'(Q) phi'(K)^T V,   D~ = diag(1 + phi'(Q) phi'(K)^T 1),
# which the paper evaluates in time linear in n by forming phi'(K)^T V first.
# ---------------------------------------------------------------------------
def attention_from_features(PhiQ, PhiK, V):
    """The definition: all n x n weights <phi'(q_i), phi'(k_j)>, no mask.  Returns (O, d)."""
    W = _f64(PhiQ) @ _f64(PhiK).T
    d = 1.0 + W.sum(axis=1)
    return (W @ _f64(V)) / d[:, None], d


def polysketch_attention(Q, K, V, G1, G2):
    """Non-causal Polysketch attention from the definition (features materialised)."""
    return attention_from_features(polysketch_non_negative(Q, G1, G2), polysketch_non_negative(K, G1, G2), V)


def polysketch_attention_linear(Q, K, V, G1, G2):
    """The same in time linear in n (Section 3): one state S = phi'(K)^T [V | 1] per head, then
    every row is phi'(q_i)^T S; its last entry is the normaliser's sum."""
    V = _f64(V)
    n, h = V.shape
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    S = polysketch_non_negative(K, G1, G2).T @ Vt
    N = polysketch_non_negative(Q, G1, G2) @ S
    d = 1.0 + N[:, h]
    return N[:, :h] / d[:, None], d


def polysketch_attention_backward(Q, K, V, G1, G2, dO):
    """Gradients (dQ, dK, dV) of sum(dO * O) for the non-causal form, through the n x n
    definition: W_ij = s_ij^2 for every pair, dL/dW_ij = E_i . V~_j (derivation above)."""
    V = _f64(V)
    n, h = V.shape
    Mq, Mk = half_sketch(Q, G1, G2), half_sketch(K, G1, G2)
    s = Mq @ Mk.T
    W = s * s
    d = 1.0 + W.sum(axis=1)
    O = (W @ V) / d[:, None]
    E = _backward_rows(O, d, dO)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    dW = E @ Vt.T
    dV = W.T @ E[:, :h]
    ds = 2.0 * s * dW
    return (_sketch_backward(Q, G1, G2, ds @ Mk), _sketch_backward(K, G1, G2, ds.T @ Mq), dV)


def polysketch_attention_backward_linear(Q, K, V, G1, G2, dO):
    """The same gradients in time linear in n: with S = phi'(K)^T V~ and R = phi'(Q)^T E,
    d phi'(q_i) = S E_i,  d phi'(k_j) = R V~_j,  dV~_j = R^T phi'(k_j), and
    dm = (mat(d phi') + mat(d phi')^T) m  because phi'(m)[a*r+b] = m_a m_b."""
    V = _f64(V)
    n, h = V.shape
    r = _f64(G1).shape[1]
    Mq, Mk = half_sketch(Q, G1, G2), half_sketch(K, G1, G2)
    Pq, Pk = self_tensor(Mq), self_tensor(Mk)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    S = Pk.T @ Vt
    N = Pq @ S
    d = 1.0 + N[:, h]
    O = N[:, :h] / d[:, None]
    E = _backward_rows(O, d, dO)
    R = Pq.T @ E
    dPq = E @ S.T
    dPk = Vt @ R.T
    dV = (Pk @ R)[:, :h]

    def untensor(dP, M):
        D = dP.reshape(n, r, r)
        return np.einsum("nab,nb->na", D + D.transpose(0, 2, 1), M)

    return (_sketch_backward(Q, G1, G2, untensor(dPq, Mq)), _sketch_backward(K, G1, G2, untensor(dPk, Mk)), dV)


# ---------------------------------------------------------------------------
# Algorithm 2 (appendix "Replacing Random Projections with Learnable Transformations"):
# the products M_1 G_1 and M_2 G_2 of Algorithm 1 become f_1(M_1), f_2(M_2) for two dense networks
# of equal structure and separate parameters, and the result goes through
# sqrt(r) tanh(sqrt(1/r) [f_1 * f_2]).  Each network: output dimension r, three hidden layers of
# sizes [8r, r, 8r], gelu after the first and the third hidden layer, layer normalisation before the
# input and before the second hidden layer.
# Readings where the appendix is silent: dense layers carry biases; each layer normalisation has a
# learnable gain and bias and eps = 1e-6 inside the square root; gelu is x Phi(x) (the erf form);
# one pair of networks serves every head.  For p = 4 the recursion bottoms out at M_1 = M_2 = A.
# A network's parameters are a dict with keys
#   g0, c0 (h)  W1 (h x 8r), b1 (8r)  g1, c1 (8r)  W2 (8r x r), b2 (r)  W3 (r x 8r), b3 (8r)  W4 (8r x r), b4 (r).
# ---------------------------------------------------------------------------
LN_EPS = 1e-6
NET_KEYS = ("g0", "c0", "W1", "b1", "g1", "c1", "W2", "b2", "W3", "b3", "W4", "b4")


def _erf(x):
    import math
    return np.vectorize(math.erf, otypes=[F64])(x)


def gelu(x):
    x = _f64(x)
    return 0.5 * x * (1.0 + _erf(x / np.sqrt(2.0)))


def _gelu_grad(x):
    x = _f64(x)
    return 0.5 * (1.0 + _erf(x / np.sqrt(2.0))) + x * np.exp(-0.5 * x * x) / np.sqrt(2.0 * np.pi)


def layer_norm(x, gain, bias):
    x = _f64(x)
    mu = x.mean(axis=1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=1, keepdims=True)
    return (x - mu) / np.sqrt(var + LN_EPS) * _f64(gain) + _f64(bias)


def learned_net(X, P):
    """One network f of Algorithm 2 applied to the rows of X."""
    z0 = layer_norm(X, P["g0"], P["c0"])
    a1 = gelu(z0 @ _f64(P["W1"]) + _f64(P["b1"]))
    z1 = layer_norm(a1, P["g1"], P["c1"])
    a2 = z1 @ _f64(P["W2"]) + _f64(P["b2"])
    a3 = gelu(a2 @ _f64(P["W3"]) + _f64(P["b3"]))
    return a3 @ _f64(P["W4"]) + _f64(P["b4"])


def learned_half_sketch(X, P1, P2):
    """LearnablePolysketchWithNegativity(X, r, 2): sqrt(r) tanh(sqrt(1/r) [f_1(X) * f_2(X)])."""
    f1, f2 = learned_net(X, P1), learned_net(X, P2)
    r = f1.shape[1]
    return np.sqrt(r) * np.tanh(f1 * f2 / np.sqrt(r))


def causal_learned_polysketch_attention(Q, K, V, P1, P2):
    """Section 3 with phi' = LearnablePolysketchNonNegative(., r, 4) = M^{(x)2}: the n x n definition."""
    s = learned_half_sketch(Q, P1, P2) @ learned_half_sketch(K, P1, P2).T
    W = lt(s * s)
    d = 1.0 + W.sum(axis=1)
    return (W @ _f64(V)) / d[:, None], d


def causal_learned_polysketch_attention_blocked(Q, K, V, P1, P2, b, diagonal="LR"):
    """The same by Section 3.1's block algorithm; diagonal="exact" gives the same-block pairs the
    weights (q_i . k_j)^4 of Section 3.2 (the paper's "learned + local" variant)."""
    Mq, Mk = learned_half_sketch(Q, P1, P2), learned_half_sketch(K, P1, P2)
    if diagonal == "LR":
        return causal_attention_blocked_from_half_sketches(Mq, Mk, V, b)
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    n, h = V.shape
    C = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)

    def diag_block(l):
        return lt((Q[l * b:(l + 1) * b] @ K[l * b:(l + 1) * b].T) ** 4)

    N = lt_multiply_blocked(self_tensor(Mq), self_tensor(Mk), C, b, diag_block)
    d = 1.0 + N[:, h]
    return N[:, :h] / d[:, None], d


def _layer_norm_backward(x, gain, dz):
    """z = n * gain + bias with n = (x - mean) / sqrt(var + eps): returns (dx, dgain, dbias)."""
    x, dz = _f64(x), _f64(dz)
    mu = x.mean(axis=1, keepdims=True)
    sig = np.sqrt(((x - mu) ** 2).mean(axis=1, keepdims=True) + LN_EPS)
    nrm = (x - mu) / sig
    dn = dz * _f64(gain)
    dx = (dn - dn.mean(axis=1, keepdims=True) - nrm * (dn * nrm).mean(axis=1, keepdims=True)) / sig
    return dx, (dz * nrm).sum(axis=0), dz.sum(axis=0)


def learned_net_backward(X, P, df):
    """Gradients of sum(df * f(X)): (dX, dict of parameter gradients)."""
    X = _f64(X)
    W1, W2, W3, W4 = (_f64(P[k]) for k in ("W1", "W2", "W3", "W4"))
    z0 = layer_norm(X, P["g0"], P["c0"])
    p1 = z0 @ W1 + _f64(P["b1"])
    a1 = gelu(p1)
    z1 = layer_norm(a1, P["g1"], P["c1"])
    a2 = z1 @ W2 + _f64(P["b2"])
    p3 = a2 @ W3 + _f64(P["b3"])
    a3 = gelu(p3)
    df = _f64(df)
    g = {"W4": a3.T @ df, "b4": df.sum(axis=0)}
    dp3 = (df @ W4.T) * _gelu_grad(p3)
    g["W3"], g["b3"] = a2.T @ dp3, dp3.sum(axis=0)
    da2 = dp3 @ W3.T
    g["W2"], g["b2"] = z1.T @ da2, da2.sum(axis=0)
    da1, g["g1"], g["c1"] = _layer_norm_backward(a1, P["g1"], da2 @ W2.T)
    dp1 = da1 * _gelu_grad(p1)
    g["W1"], g["b1"] = z0.T @ dp1, dp1.sum(axis=0)
    dX, g["g0"], g["c0"] = _layer_norm_backward(X, P["g0"], dp1 @ W1.T)
    return dX, g


def learned_half_sketch_backward(X, P1, P2, dM):
    """Gradients of sum(dM * M) for M = learned_half_sketch(X, P1, P2): (dX, grads of P1, grads of P2)."""
    f1, f2 = learned_net(X, P1), learned_net(X, P2)
    r = f1.shape[1]
    t = np.tanh(f1 * f2 / np.sqrt(r))
    du = _f64(dM) * (1.0 - t * t)                 # d/du of sqrt(r) tanh(u / sqrt(r)) at u = f1 * f2
    dX1, g1 = learned_net_backward(X, P1, du * f2)
    dX2, g2 = learned_net_backward(X, P2, du * f1)
    return dX1 + dX2, g1, g2


def causal_learned_polysketch_attention_backward(Q, K, V, P1, P2, dO, b=None, diagonal="LR"):
    """Gradients (dQ, dK, dV, grads of P1, grads of P2) of sum(dO * O), through the n x n definition.
    The networks see the queries and the keys, so their gradients are the sum of both uses.
    diagonal="exact" (with the block size b): same-block pairs carry (q_i . k_j)^4, whose gradient
    reaches Q and K directly."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    n, h = V.shape
    Mq, Mk = learned_half_sketch(Q, P1, P2), learned_half_sketch(K, P1, P2)
    s = Mq @ Mk.T
    if diagonal == "exact":
        same = same_block(n, b)
        x = Q @ K.T
        W = lt(np.where(same, x ** 4, s * s))
    else:
        same = np.zeros((n, n), dtype=bool)
        x = np.zeros((n, n))
        W = lt(s * s)
    d = 1.0 + W.sum(axis=1)
    O = (W @ V) / d[:, None]
    E = _backward_rows(O, d, dO)
    Vt = np.concatenate([V, np.ones((n, 1), dtype=F64)], axis=1)
    dW = lt(E @ Vt.T)
    ds = np.where(same, 0.0, 2.0 * s * dW)
    dx = np.where(same, 4.0 * x ** 3 * dW, 0.0)
    dQ, gq1, gq2 = learned_half_sketch_backward(Q, P1, P2, ds @ Mk)
    dK, gk1, gk2 = learned_half_sketch_backward(K, P1, P2, ds.T @ Mq)
    g1 = {k: gq1[k] + gk1[k] for k in NET_KEYS}
    g2 = {k: gq2[k] + gk2[k] for k in NET_KEYS}
    return dQ + dx @ K, dK + dx.T @ Q, W.T @ E[:, :h], g1, g2


# ---------------------------------------------------------------------------
# Error metric used by the parity tests and the benchmark
# ---------------------------------------------------------------------------
def rel_l2(x, ref):
    """|| x - ref ||_2 / || ref ||_2 over the whole tensor (fp64)."""
    x, ref = _f64(x), _f64(ref)
    den = np.linalg.norm(ref.ravel())
    num = np.linalg.norm((x - ref).ravel())
    return num / den if den > 0 else num
