"""Pins for the selection oracle: Eq. 10 hand-worked thresholds (golden file),
Eq. 9 hand-worked accept sets, boundary values, invariants, and exhaustive
enumeration on tiny blocks against a second, separately written predicate."""
import itertools

import numpy as np
import pytest

import oracle


def _cases(golden_dir):
    out = []
    for line in (golden_dir / "threshold_cases.txt").read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        K, n, extra, tau0, alpha, tau = line.split()
        out.append((int(K), int(n), int(extra), float(tau0), float(alpha), float(tau)))
    return out


def test_threshold_hand_worked(golden_dir):
    cases = _cases(golden_dir)
    assert len(cases) >= 8
    for K, n, extra, tau0, alpha, tau in cases:
        got = oracle.threshold(n, K, tau0, alpha, extra)
        assert abs(got - tau) < 2e-7, (K, n, extra, tau0, alpha, got, tau)


def test_threshold_boundaries():
    # r_mask = 1 -> tau0 exactly; r_mask -> 0 approaches tau0 * (1 - alpha)
    assert oracle.threshold(32, 32, 0.9, 0.6) == np.float32(0.9)
    lim = 0.9 * (1 - 0.6)
    taus = [oracle.threshold(n, 1024, 0.9, 0.6) for n in (1024, 512, 64, 1)]
    assert all(a > b for a, b in zip(taus, taus[1:]))          # monotone in the masked ratio
    assert abs(taus[-1] - lim) < 1e-3 and taus[-1] > lim
    # alpha = 0: fixed threshold for every ratio
    assert {oracle.threshold(n, 32, 0.9, 0.0) for n in range(1, 33)} == {float(np.float32(0.9))}


def _run(conf, tok, masked, x=None, **kw):
    conf = np.asarray(conf, np.float32).reshape(1, -1)
    K = conf.shape[1]
    tok = np.asarray(tok, np.int32).reshape(1, K)
    masked = np.asarray(masked, np.uint8).reshape(1, K)
    x = np.full((1, K), -7, np.int32) if x is None else np.asarray(x, np.int32).reshape(1, K)
    return oracle.select(conf, tok, masked, x, **kw)


def test_accept_above_threshold_ignores_unmasked():
    # all four positions' confidences; position 3 is already decoded
    r = _run([0.95, 0.7, 0.91, 0.99], [10, 11, 12, 13], [1, 1, 1, 0], x=[-7, -7, -7, 55], tau0=0.9, alpha=0.0)
    assert r["sel_cnt"][0] == 2 and r["sel_idx"][0].tolist() == [0, 2, -1, -1]
    assert r["x_block"][0].tolist() == [10, -7, 12, 55]
    assert r["masked"][0].tolist() == [0, 1, 0, 0]
    assert r["block_done"][0] == 0 and r["active_seq"].tolist() == [0]


def test_fallback_picks_exactly_one_lowest_index_on_ties():
    r = _run([0.3, 0.5, 0.5, 0.99], [1, 2, 3, 4], [1, 1, 1, 0], tau0=0.9, alpha=0.0)
    assert r["sel_cnt"][0] == 1 and r["sel_idx"][0, 0] == 1
    assert r["x_block"][0].tolist() == [-7, 2, -7, -7]
    assert r["masked"][0].tolist() == [1, 0, 1, 0]


def test_threshold_is_inclusive():
    tau = oracle.threshold(4, 4, 0.9, 0.0)
    r = _run([tau, np.nextafter(np.float32(tau), np.float32(0)), 0.1, 0.2], [1, 2, 3, 4], [1, 1, 1, 1],
             tau0=0.9, alpha=0.0)
    assert r["sel_idx"][0].tolist() == [0, -1, -1, -1]


def test_adaptive_threshold_admits_more_late():
    conf = [0.8, 0.75, 0.2, 0.65]
    # 2 of 4 masked, alpha = 0.5: tau = 0.9 * (1 - 0.5 * 0.5) = 0.675
    r = _run(conf, [1, 2, 3, 4], [1, 0, 0, 1], tau0=0.9, alpha=0.5)
    assert abs(r["tau"][0] - 0.675) < 1e-6
    assert r["sel_idx"][0].tolist() == [0, -1, -1, -1]
    # same confidences with alpha = 0.6: tau = 0.63 -> position 3 (0.65) joins
    r = _run(conf, [1, 2, 3, 4], [1, 0, 0, 1], tau0=0.9, alpha=0.6)
    assert r["sel_idx"][0].tolist() == [0, 3, -1, -1] and r["block_done"][0] == 1
    assert r["active_seq"].tolist() == []


def test_ratio_extra_reading():
    # block only: n = 1 of K = 4 -> tau = 0.9 * (1 - 0.5 * 0.75) = 0.5625 -> 0.6 accepted by rule
    r = _run([0.6, 0, 0, 0], [9, 0, 0, 0], [1, 0, 0, 0], tau0=0.9, alpha=0.5)
    assert abs(r["tau"][0] - 0.5625) < 1e-6
    # counting 12 retained suffix rows as masked: r = 13/16 -> tau = 0.9 * (1 - 0.5 * 3/16) = 0.815625
    r = _run([0.6, 0, 0, 0], [9, 0, 0, 0], [1, 0, 0, 0], tau0=0.9, alpha=0.5, ratio_extra=12)
    assert abs(r["tau"][0] - 0.815625) < 1e-6
    assert r["sel_cnt"][0] == 1     # still taken, by the fallback


def test_no_masks_left():
    r = _run([0.99, 0.99], [1, 2], [0, 0], x=[5, 6], tau0=0.9, alpha=0.3)
    assert r["sel_cnt"][0] == 0 and r["block_done"][0] == 1 and r["x_block"][0].tolist() == [5, 6]
    assert r["active_seq"].tolist() == []


def test_early_exit_flag():
    EOS = 2
    # EOS accepted with high confidence -> flag
    r = _run([0.95, 0.2], [EOS, 7], [1, 1], tau0=0.9, alpha=0.0, eos_id=EOS, eos_tau=0.9)
    assert r["eos_exit"][0] == 1
    # EOS taken only by the fallback at low confidence -> no flag
    r = _run([0.3, 0.2], [EOS, 7], [1, 1], tau0=0.9, alpha=0.0, eos_id=EOS, eos_tau=0.9)
    assert r["sel_idx"][0, 0] == 0 and r["eos_exit"][0] == 0
    # EOS predicted but position not masked -> no flag
    r = _run([0.95, 0.95], [EOS, 7], [0, 1], tau0=0.9, alpha=0.0, eos_id=EOS, eos_tau=0.9)
    assert r["eos_exit"][0] == 0
    # disabled; sticky
    r = _run([0.95, 0.2], [EOS, 7], [1, 1], tau0=0.9, alpha=0.0, eos_id=-1)
    assert r["eos_exit"][0] == 0
    r = _run([0.1, 0.2], [5, 7], [1, 1], tau0=0.9, alpha=0.0, eos_id=EOS, eos_exit=[1])
    assert r["eos_exit"][0] == 1


def test_seq_list_and_active_compaction():
    rng = np.random.default_rng(0)
    B, K = 6, 8
    conf = rng.random((B, K)).astype(np.float32)
    tok = rng.integers(0, 100, (B, K)).astype(np.int32)
    masked = np.ones((B, K), np.uint8)
    masked[1] = 0
    masked[4, 1:] = 0           # single mask left -> finishes this step
    x = np.full((B, K), -1, np.int32)
    r = oracle.select(conf, tok, masked, x, 0.9, 0.3, seq_list=[0, 2, 4, 5])
    assert r["active_seq"].tolist() == [0, 2, 5]
    assert np.isnan(r["tau"][[1, 3]]).all()
    assert (r["masked"][3] == 1).all() and (r["x_block"][3] == -1).all() and r["sel_cnt"][3] == 0
    with pytest.raises(ValueError):
        oracle.select(conf, tok, masked, x, 0.9, 0.3, seq_list=[2, 0])


def _second_opinion(conf, tok, masked, tau):
    """Eq. 9 written again from its three cases, as set logic."""
    cand = {i for i in range(len(conf)) if masked[i]}
    above = {i for i in cand if not (conf[i] < tau)}
    if above:
        return sorted(above)
    if not cand:
        return []
    top = max(conf[i] for i in cand)
    return [min(i for i in cand if conf[i] == top)]


def test_exhaustive_small_blocks():
    grid = [np.float32(v) for v in (0.0, 0.45, 0.675, 0.9, 1.0)]
    for K in (1, 2, 3):
        for alpha in (0.0, 0.5):
            for conf in itertools.product(grid, repeat=K):
                for masked in itertools.product((0, 1), repeat=K):
                    tau = oracle.threshold(sum(masked), K, 0.9, alpha)
                    r = _run(conf, list(range(100, 100 + K)), masked, tau0=0.9, alpha=alpha)
                    want = _second_opinion(conf, None, masked, np.float32(tau))
                    got = [i for i in r["sel_idx"][0].tolist() if i >= 0]
                    assert got == want, (K, alpha, conf, masked, tau, got, want)
                    assert r["sel_cnt"][0] == len(want)


def test_block_converges_within_K_steps():
    rng = np.random.default_rng(5)
    B, K = 4, 16
    masked = np.ones((B, K), np.uint8)
    x = np.full((B, K), -1, np.int32)
    active = None
    for step in range(K):
        conf = rng.random((B, K)).astype(np.float32) * 0.8       # never reaches tau0: fallback every step
        tok = rng.integers(0, 50, (B, K)).astype(np.int32)
        before = masked.sum(1)
        r = oracle.select(conf, tok, masked, x, 0.9, 0.3, seq_list=active)
        masked, x = r["masked"], r["x_block"]
        after = masked.sum(1)
        assert ((after < before) | (before == 0)).all()
        assert ((r["sel_cnt"] >= 1) | (before == 0)).all() and (r["sel_cnt"] <= before).all()
        active = r["active_seq"]
        if len(active) == 0:
            break
    assert masked.sum() == 0 and (x >= 0).all()
