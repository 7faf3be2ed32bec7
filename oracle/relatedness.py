"""Relatedness head over pairs of root states, one pair at a time in fp64.  TEST INFRASTRUCTURE ONLY.

The paper's workload is the semantic-relatedness task on sentence pairs (Section 5): each sample is two trees, and
what is scored is a function of their two root states.  The paper does not write that function out; it is the head
of the Tree-LSTM model it cites, for a pair (h_L, h_R), K classes and r = (1, ..., K):

    h_x = h_L * h_R                    h_+ = |h_L - h_R|
    h_s = sigmoid(W_x h_x + W_+ h_+ + b_h)
    p   = softmax(W_p h_s + b_p)
    y   = r . p                        (the predicted relatedness, between 1 and K)

Readings where the paper is silent: the whole definition above (taken from the cited model), K = 5 for its dataset,
softmax evaluated after subtracting the largest logit.

Nothing here is shared with the CUDA path.  Pins: tests/test_oracle_relatedness.py.
"""
from __future__ import annotations

import numpy as np


def head(h, left, right, Wx, Wp, bh, Wq, bq):
    """h [n, H]; left/right [P] root node ids; Wx, Wp [Hs, H]; bh [Hs]; Wq [K, Hs]; bq [K].  Returns (y [P], p [P, K])."""
    h = np.asarray(h, dtype=np.float64)
    Wx, Wp, bh, Wq, bq = (np.asarray(a, dtype=np.float64) for a in (Wx, Wp, bh, Wq, bq))
    K = Wq.shape[0]
    r = np.arange(1, K + 1, dtype=np.float64)
    ys, ps = [], []
    for a, b in zip(left, right):
        hl, hr = h[int(a)], h[int(b)]
        hs = 1.0 / (1.0 + np.exp(-(Wx @ (hl * hr) + Wp @ np.abs(hl - hr) + bh)))
        z = Wq @ hs + bq
        e = np.exp(z - np.max(z))
        p = e / np.sum(e)
        ps.append(p)
        ys.append(float(r @ p))
    return np.asarray(ys), np.asarray(ps).reshape(len(ys), K)
