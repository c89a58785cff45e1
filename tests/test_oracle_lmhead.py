"""Pins of the oracle for the fused output projection + Eq. 4 (``oracle.lmhead_confidence``).

The function is the composition z = W h followed by c = max softmax(z), x^ = argmax z, so it is pinned
against the mathematics of each part and against the already pinned Eq. 4 oracle on the special case
where the projection is the identity."""
import numpy as np
import pytest
import torch

import oracle


def test_identity_projection_reduces_to_eq4_oracle():
    rng = np.random.default_rng(0)
    h = (2 * rng.standard_normal((7, 50))).astype(np.float32)
    conf, tok = oracle.lmhead_confidence(h, np.eye(50, dtype=np.float32))
    c4, t4 = oracle.confidence(h)
    assert np.array_equal(tok, t4) and np.abs(conf - c4).max() < 1e-15


def test_logits_are_the_matrix_product_and_confidence_matches_logsumexp():
    rng = np.random.default_rng(1)
    h = rng.standard_normal((5, 33)).astype(np.float32)
    w = rng.standard_normal((101, 33)).astype(np.float32)
    conf, tok, z = oracle.lmhead_confidence(h, w, want_logits=True)
    ref = h.astype(np.float64) @ w.astype(np.float64).T               # library routine on the same definition
    assert np.abs(z - ref).max() < 1e-12
    zt = torch.from_numpy(ref)
    assert np.abs(conf - torch.exp(zt.max(1).values - torch.logsumexp(zt, 1)).numpy()).max() < 1e-14
    assert np.array_equal(tok, ref.argmax(1))
    # a transposed weight (a plausible mistake) gives different logits
    w2 = rng.standard_normal((33, 33)).astype(np.float32)
    _, _, z2 = oracle.lmhead_confidence(h, w2, want_logits=True)
    assert np.abs(z2 - h.astype(np.float64) @ w2.astype(np.float64)).max() > 1e-3


def test_closed_forms():
    # zero weights: every logit is 0 -> confidence 1/V, lowest index
    conf, tok = oracle.lmhead_confidence(np.ones((3, 8), np.float32), np.zeros((40, 8), np.float32))
    assert np.allclose(conf, 1 / 40, rtol=0, atol=1e-16) and (tok == 0).all()
    # h = e_k picks column k of W: logits (a, 0, ..., 0) -> e^a / (e^a + V - 1)
    V, a = 25, 3.0
    w = np.zeros((V, 4), np.float32)
    w[7, 2] = a
    h = np.zeros((1, 4), np.float32)
    h[0, 2] = 1.0
    conf, tok = oracle.lmhead_confidence(h, w)
    assert tok[0] == 7 and abs(conf[0] - np.exp(a) / (np.exp(a) + V - 1)) < 1e-14
    # scaling h by s scales the logits: (s a, 0, ...) 
    conf2, _ = oracle.lmhead_confidence(2 * h, w)
    assert abs(conf2[0] - np.exp(2 * a) / (np.exp(2 * a) + V - 1)) < 1e-14


def test_ties_and_shift_invariance():
    rng = np.random.default_rng(2)
    h = rng.standard_normal((4, 16)).astype(np.float32)
    w = rng.standard_normal((30, 16)).astype(np.float32)
    w[21] = w[9]                                   # duplicate output embedding: equal logits
    w[9] *= 1.0
    big = 5.0 * h[0] / np.dot(h[0], h[0])
    w[9] += big.astype(np.float32)                 # make 9 / 21 compete for row 0 ... and restore equality
    w[21] = w[9]
    conf, tok, z = oracle.lmhead_confidence(h, w, want_logits=True)
    for r in range(4):
        if z[r].argmax() in (9, 21):
            assert tok[r] == 9                     # lowest index among equal maxima
    # adding one vector c to every output embedding shifts all logits of a row by <h, c>: softmax unchanged
    c = rng.standard_normal(16).astype(np.float32)
    conf_s, tok_s = oracle.lmhead_confidence(h.astype(np.float64), w.astype(np.float64) + c.astype(np.float64))
    # (float32 rounding of w + c perturbs the logits slightly: compare loosely, the identity is exact in reals)
    assert np.abs(conf_s - conf).max() < 1e-5
