"""Pins for the relatedness-head checker (oracle/relatedness.py)."""
import math

import numpy as np

from oracle import relatedness as orl


def _rand(seed, n=6, H=7, Hs=4, K=5):
    rng = np.random.default_rng(seed)
    return (rng.uniform(-1, 1, (n, H)), rng.uniform(-1, 1, (Hs, H)), rng.uniform(-1, 1, (Hs, H)), rng.uniform(-1, 1, Hs),
            rng.uniform(-1, 1, (K, Hs)), rng.uniform(-1, 1, K))


def test_scalar_pair_by_hand():
    """H = Hs = 1, K = 2, every number written with math.exp."""
    h = np.array([[0.6], [-0.3]])
    y, p = orl.head(h, [0], [1], [[0.8]], [[-0.5]], [0.1], [[1.5], [-2.0]], [0.2, 0.4])
    hx, hp = 0.6 * -0.3, abs(0.6 + 0.3)
    hs = 1.0 / (1.0 + math.exp(-(0.8 * hx - 0.5 * hp + 0.1)))
    z1, z2 = 1.5 * hs + 0.2, -2.0 * hs + 0.4
    p1 = math.exp(z1) / (math.exp(z1) + math.exp(z2))
    assert abs(p[0, 0] - p1) < 1e-15 and abs(p[0, 1] - (1 - p1)) < 1e-15
    assert abs(y[0] - (1 * p1 + 2 * (1 - p1))) < 1e-15


def test_probabilities_range_symmetry_and_uniform_case():
    h, Wx, Wp, bh, Wq, bq = _rand(3)
    left, right = [0, 2, 4, 1], [1, 3, 5, 1]
    y, p = orl.head(h, left, right, Wx, Wp, bh, Wq, bq)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-15) and np.all(p > 0)
    assert np.all(y > 1.0) and np.all(y < 5.0)
    y2, p2 = orl.head(h, right, left, Wx, Wp, bh, Wq, bq)          # both features are symmetric in the pair
    assert np.array_equal(y, y2) and np.array_equal(p, p2)
    # a tree paired with itself: h_+ = 0 and h_x = h^2
    hs = 1.0 / (1.0 + np.exp(-(Wx @ (h[1] * h[1]) + bh)))
    z = Wq @ hs + bq
    assert np.allclose(p[3], np.exp(z) / np.exp(z).sum(), atol=1e-15)
    # no output weights: every class equally likely, the expectation is the middle of 1..K
    y0, p0 = orl.head(h, left, right, Wx, Wp, bh, np.zeros_like(Wq), np.zeros_like(bq))
    assert np.allclose(p0, 0.2, atol=1e-16) and np.allclose(y0, 3.0, atol=1e-15)
    # a constant added to every logit changes nothing
    y3, _ = orl.head(h, left, right, Wx, Wp, bh, Wq, bq + 100.0)
    assert np.allclose(y3, y, atol=1e-12)
