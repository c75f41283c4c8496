"""Host-only checks of the tensor-core path's feature order (no GPU).

Section 2.2: phi'(x) = m (x) m, so <phi'(q), phi'(k)> = sum over ORDERED pairs (a, b) of
(q_a q_b)(k_a k_b).  The kernels keep one feature per unordered pair and put the multiplicity into
the weights of their state rows.  Whatever the order, it is correct iff every unordered pair
{a, b} carries total weight 2 (a != b) or 1 (a == b); then the weighted feature product equals
the r^2-dimensional one, which the last test checks against the oracle's self-tensoring."""
import numpy as np
import pytest

import paper_2310_01655_b200 as psk
from oracle import polysketch as orc


@pytest.mark.parametrize("r", [16, 32, 64])
def test_every_pair_carries_its_multiplicity(r):
    a, b, w = psk.binding.feature_table(r)
    assert len(a) == len(b) == len(w)
    assert ((0 <= a) & (a < r) & (0 <= b) & (b < r)).all()
    total = np.zeros((r, r))
    for ai, bi, wi in zip(a, b, w):
        lo, hi = min(ai, bi), max(ai, bi)
        total[lo, hi] += wi
    expect = np.triu(np.full((r, r), 2.0), 1) + np.eye(r)
    assert np.array_equal(total, expect)
    # weights are 0, 1 or 2: exact in bf16, so folding them into stored rows costs no accuracy
    assert set(np.unique(w)) <= {0.0, 1.0, 2.0}


@pytest.mark.parametrize("r", [16, 32, 64])
def test_stored_extent_matches_the_chunking(r):
    a, b, w = psk.binding.feature_table(r)
    F = len(a)
    assert F % 16 == 0                       # whole MMA K steps
    assert F >= r * (r + 1) // 2             # at least one feature per unordered pair
    assert (F + 127) // 128 * 128 <= {16: 256, 32: 640, 64: 2176}[r]


@pytest.mark.parametrize("r", [16, 32, 64])
def test_weighted_features_reproduce_the_self_tensored_product(r):
    rng = np.random.default_rng(r)
    mq, mk = rng.standard_normal(r), rng.standard_normal(r)
    a, b, w = psk.binding.feature_table(r)
    got = float(np.sum(w * (mq[a] * mq[b]) * (mk[a] * mk[b])))
    ref = float(orc.self_tensor(mq[None, :])[0] @ orc.self_tensor(mk[None, :])[0])
    assert abs(got - ref) <= 1e-12 * max(1.0, abs(ref))
    assert abs(ref - float(mq @ mk) ** 2) <= 1e-12 * max(1.0, abs(ref))


def test_bad_arguments():
    import ctypes
    L = psk.lib()
    buf = (ctypes.c_int * 8)()
    fb = (ctypes.c_float * 8)()
    assert L.psk_feature_table(48, buf, buf, fb, 8) == -2
    assert L.psk_feature_table(32, None, buf, fb, 8) == -1
    assert L.psk_feature_table(32, buf, buf, fb, 8) == -5
