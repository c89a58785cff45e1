"""Pins for the Eq. 4 oracle (c = max softmax(z), x^ = argmax): closed forms,
shift invariance, tie rule, and a library log-sum-exp."""
import math

import numpy as np
import torch

import oracle


def test_all_equal_logits():
    conf, tok = oracle.confidence(np.full((3, 1000), 2.5, np.float32))
    np.testing.assert_allclose(conf, 1.0 / 1000, rtol=1e-14)
    assert tok.tolist() == [0, 0, 0]


def test_single_spike_closed_form():
    V, a = 4096, 7.0
    z = np.zeros((2, V), np.float32)
    z[0, 17] = a
    z[1, V - 1] = a
    conf, tok = oracle.confidence(z)
    expect = math.exp(a) / (math.exp(a) + V - 1)
    np.testing.assert_allclose(conf, expect, rtol=1e-13)
    assert tok.tolist() == [17, V - 1]


def test_shift_invariance_and_lse():
    rng = np.random.default_rng(1)
    z = (2.0 * rng.standard_normal((5, 777))).astype(np.float32)
    conf, tok = oracle.confidence(z)
    conf2, tok2 = oracle.confidence(z + np.float32(4.0))
    # softmax is shift invariant; z + 4 rounds in float32, so the shifted result is
    # compared with the float64 definition on the shifted values, and with the
    # unshifted result at float32 resolution
    np.testing.assert_allclose(conf2, conf, rtol=1e-5)
    zs = (z + np.float32(4.0)).astype(np.float64)
    ref2 = np.exp(zs.max(1) - torch.logsumexp(torch.from_numpy(zs), 1).numpy())
    np.testing.assert_allclose(conf2, ref2, rtol=1e-12)
    assert (tok2 == zs.argmax(1)).all()
    zd = torch.from_numpy(z.astype(np.float64))
    ref = torch.exp(zd.max(1).values - torch.logsumexp(zd, 1)).numpy()
    np.testing.assert_allclose(conf, ref, rtol=1e-12)
    assert (tok == z.argmax(1)).all()
    # conf equals the largest softmax probability of the library softmax
    np.testing.assert_allclose(conf, torch.softmax(zd, 1).max(1).values.numpy(), rtol=1e-12)


def test_two_equal_maxima_lowest_index():
    z = np.full((1, 50), -1e4, np.float32)
    z[0, 31] = 3.0
    z[0, 12] = 3.0
    conf, tok = oracle.confidence(z)
    assert tok[0] == 12
    assert abs(conf[0] - 0.5) < 1e-15


def test_v_equal_one_and_odd_sizes():
    conf, tok = oracle.confidence(np.array([[3.0], [-2.0]], np.float32))
    assert conf.tolist() == [1.0, 1.0] and tok.tolist() == [0, 0]
    rng = np.random.default_rng(2)
    for V in (2, 7, 9, 1025):
        z = rng.standard_normal((3, V)).astype(np.float32)
        conf, tok = oracle.confidence(z)
        e = np.exp(z.astype(np.float64) - z.max(1, keepdims=True))
        np.testing.assert_allclose(conf, 1.0 / e.sum(1), rtol=1e-13)
        assert (tok == z.argmax(1)).all()


def test_confidence_bounds():
    rng = np.random.default_rng(3)
    z = (2 * rng.standard_normal((20, 300))).astype(np.float32)
    conf, _ = oracle.confidence(z)
    assert ((conf >= 1.0 / 300) & (conf <= 1.0)).all()
