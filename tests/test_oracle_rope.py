"""Pins of ``oracle.rope_gather``: rotary encoding of the retained rows with their original position ids
(the suffix pruning of Eq. 7 keeps token order "via RoPE position IDs") plus the gather of Eq. 8's rows."""
import numpy as np

import oracle


def _raw(B=2, Hq=4, Hkv=2, T=40, D=16, seed=0):
    rng = np.random.default_rng(seed)
    f = lambda h: rng.standard_normal((B, h, T, D)).astype(np.float32)
    return f(Hq), f(Hkv), f(Hkv)


def test_matches_complex_rotation_and_fancy_indexing():
    q, k, v = _raw()
    idx = np.array([0, 1, 2, 5, 6, 39])
    off, theta = 100, 10000.0
    qo, ko, vo = oracle.rope_gather(q, k, v, idx, off, theta)
    D = q.shape[-1]
    pos = (off + idx).astype(np.float64)
    inv = theta ** (-2.0 * np.arange(D // 2) / D)
    rot = np.exp(1j * pos[:, None] * inv[None, :])                       # independent formulation: complex multiply
    for src, out in ((q, qo), (k, ko)):
        x = src[:, :, idx].astype(np.float64)
        z = (x[..., : D // 2] + 1j * x[..., D // 2:]) * rot
        assert np.abs(out[..., : D // 2] - z.real).max() < 1e-12 and np.abs(out[..., D // 2:] - z.imag).max() < 1e-12
    assert np.array_equal(vo, v[:, :, idx].astype(np.float64))            # values: gathered, not rotated


def test_position_zero_is_identity_and_norms_are_preserved():
    q, k, v = _raw(seed=1)
    qo, ko, _ = oracle.rope_gather(q, k, v, np.array([0]), 0)
    assert np.abs(qo[:, :, 0] - q[:, :, 0]).max() < 1e-15 and np.abs(ko[:, :, 0] - k[:, :, 0]).max() < 1e-15
    idx = np.arange(0, 40, 3)
    qo, ko, _ = oracle.rope_gather(q, k, v, idx, 777)
    assert np.abs(np.linalg.norm(qo, axis=-1) - np.linalg.norm(q[:, :, idx].astype(np.float64), axis=-1)).max() < 1e-12


def test_scores_depend_on_position_difference_only():
    """<R_m q, R_n k> is a function of m - n: shifting every position id by the same amount (a longer prefix)
    leaves all query-key scores unchanged, which is why pruned rows must keep their ORIGINAL ids: renumbering
    the retained rows 0..Lq-1 changes the distances and therefore the scores."""
    q, k, v = _raw(B=1, Hq=2, Hkv=2, seed=2)
    idx = np.array([0, 1, 2, 3, 30, 39])
    qa, ka, _ = oracle.rope_gather(q, k, v, idx, 64)
    qb, kb, _ = oracle.rope_gather(q, k, v, idx, 64 + 1000)
    sa = np.einsum("bhid,bhjd->bhij", qa, ka)
    sb = np.einsum("bhid,bhjd->bhij", qb, kb)
    assert np.abs(sa - sb).max() < 1e-9
    # compact renumbering (what dropping the ids would do): gather first, then positions 0..Lq-1
    qc, kc, _ = oracle.rope_gather(q[:, :, idx], k[:, :, idx], v[:, :, idx], np.arange(len(idx)), 64)
    sc = np.einsum("bhid,bhjd->bhij", qc, kc)
    assert np.abs(sa - sc).max() > 1e-2


def test_per_batch_index_lists_and_frequency_ladder():
    q, k, v = _raw(B=2, seed=3)
    idx = np.array([[0, 4, 9], [1, 2, 39]])
    qo, _, vo = oracle.rope_gather(q, k, v, idx, 5)
    for b in range(2):
        qs, _, vs = oracle.rope_gather(q[b:b + 1], k[b:b + 1], v[b:b + 1], idx[b], 5)
        assert np.array_equal(qo[b], qs[0]) and np.array_equal(vo[b], vs[0])
    # the slowest pair (d = D/2 - 1) turns by p * theta^(-(D-2)/D); the fastest (d = 0) by p radians
    x = np.zeros((1, 1, 1, 8), np.float32)
    x[..., 0] = 1.0
    x[..., 3] = 1.0
    o, _, _ = oracle.rope_gather(x, x, x, np.array([0]), 2, theta=100.0)
    assert abs(o[0, 0, 0, 0] - np.cos(2.0)) < 1e-15 and abs(o[0, 0, 0, 4] - np.sin(2.0)) < 1e-15
    a = 2.0 * 100.0 ** (-6.0 / 8.0)
    assert abs(o[0, 0, 0, 3] - np.cos(a)) < 1e-15 and abs(o[0, 0, 0, 7] - np.sin(a)) < 1e-15
