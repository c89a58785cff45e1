"""Pins of the oracle's block-wise decoding loop (Eq. 1-5, Eq. 9-10, early exit) against what the paper
and the arithmetic fix: closed-form step counts in the two limiting thresholds, library argmax, a
hand-worked two-block example, the early-exit rule, and invariants of the procedure."""
import numpy as np
import pytest

import oracle

MASK = 100000   # outside every vocabulary used here


def _table_fn(tables):
    return lambda n, t: tables[(n, t)]


def _rand_fn(B, K, V, seed, spike=None):
    def fn(n, t):
        rng = np.random.default_rng([seed, n, t])
        z = rng.normal(size=(B, K, V))
        if spike is not None:
            hot = rng.integers(0, V, (B, K))
            on = rng.random((B, K)) < spike
            bb, kk = np.nonzero(on)
            z[bb, kk, hot[bb, kk]] += 12.0
        return z
    return fn


def test_unreachable_threshold_takes_one_token_per_iteration():
    # tau0 > 1 with alpha = 0: no confidence reaches the threshold, so Eq. 9's second case finalises exactly
    # one token per iteration -> every block takes K iterations, N * K in total (K = 1 steps of Eq. 2's remark)
    B, L, K, V = 3, 24, 8, 50
    r = oracle.decode(_rand_fn(B, K, V, 1), B, L, K, tau0=1.5, alpha=0.0, mask_id=MASK)
    assert r["steps"].tolist() == [K] * (L // K)
    assert (r["seq_steps"] == K).all()
    assert (r["x"] != MASK).all()


def test_zero_threshold_finalises_a_block_in_one_iteration_with_the_argmax():
    B, L, K, V = 4, 32, 8, 64
    fn = _rand_fn(B, K, V, 2)
    r = oracle.decode(fn, B, L, K, tau0=0.0, alpha=0.3, mask_id=MASK)
    assert r["steps"].tolist() == [1] * (L // K)
    want = np.concatenate([np.argmax(fn(n, 0), axis=-1) for n in range(L // K)], axis=1)   # library argmax
    assert np.array_equal(r["x"], want)


def test_hand_worked_two_blocks():
    # B = 1, K = 2, V = 3.  Confidences follow from softmax by hand:
    #   logits (a, 0, 0): c = e^a / (e^a + 2);  a = ln 18 -> 0.9,  a = ln 2 -> 0.5,  a = ln 8 -> 0.8
    # tau0 = 0.85, alpha = 0.4: two masked of two -> tau = 0.85; one masked of two -> tau = 0.85 (1 - 0.4 * 0.5) = 0.68
    ln = np.log
    z = {
        (0, 0): np.array([[[ln(18.0), 0, 0], [0, ln(2.0), 0]]]),   # conf 0.9 (token 0) accepted, 0.5 (token 1) waits
        (0, 1): np.array([[[0, 0, 5.0], [0, 0, ln(8.0)]]]),        # position 1: conf 0.8 >= 0.68, token 2
        (1, 0): np.array([[[0, ln(2.0), 0], [ln(2.0), 0, 0]]]),    # both 0.5 < 0.85: fallback takes the lower index
        (1, 1): np.array([[[9.0, 0, 0], [0, 0, ln(2.0)]]]),        # one masked: tau 0.68 > 0.5: fallback, token 2
    }
    tr = []
    r = oracle.decode(_table_fn(z), 1, 4, 2, tau0=0.85, alpha=0.4, mask_id=MASK, trace=tr)
    assert r["x"].tolist() == [[0, 2, 1, 2]]
    assert r["steps"].tolist() == [2, 2]
    assert [round(float(e["tau"][0]), 6) for e in tr] == [0.85, 0.68, 0.85, 0.68]
    assert np.allclose(tr[0]["conf"][0], [0.9, 0.5], atol=1e-6)


def test_early_exit_skips_later_blocks_of_that_sequence_only():
    B, L, K, V, EOS = 2, 12, 4, 16, 5
    base = _rand_fn(B, K, V, 3)

    def fn(n, t):
        z = base(n, t)
        if n == 1:
            z[0, 2, EOS] += 30.0          # sequence 0 predicts EOS with confidence ~1 inside block 1
        return z
    r = oracle.decode(fn, B, L, K, tau0=0.5, alpha=0.2, mask_id=MASK, eos_id=EOS, eos_tau=0.9)
    assert r["eos_exit"].tolist() == [1, 0]
    assert r["x"][0, 4 + 2] == EOS
    assert (r["x"][0, 8:] == EOS).all() and r["seq_steps"][0, 2] == 0       # block 2 skipped and filled
    assert (r["x"][0, 4:8] != MASK).all() and r["seq_steps"][0, 1] >= 1     # block 1 still completed
    assert r["seq_steps"][1, 2] >= 1 and (r["x"][1] != MASK).all()
    # without an EOS id nothing is skipped
    r2 = oracle.decode(fn, B, L, K, tau0=0.5, alpha=0.2, mask_id=MASK)
    assert (r2["seq_steps"] >= 1).all()
    # a low-confidence EOS does not trigger the exit
    r3 = oracle.decode(base, B, L, K, tau0=0.0, alpha=0.0, mask_id=MASK, eos_id=int(np.argmax(base(0, 0)[1, 0])),
                       eos_tau=0.999)
    assert r3["eos_exit"].tolist() == [0, 0]


@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.6])
def test_invariants_of_the_procedure(alpha):
    B, L, K, V = 5, 64, 16, 200
    fn = _rand_fn(B, K, V, 4, spike=0.4)
    tr = []
    r = oracle.decode(fn, B, L, K, tau0=0.9, alpha=alpha, mask_id=MASK, trace=tr)
    N = L // K
    assert (r["x"] != MASK).all()
    assert ((1 <= r["seq_steps"]) & (r["seq_steps"] <= K)).all()          # at least one token per iteration
    assert (r["steps"] == r["seq_steps"].max(0)).all()
    # every token equals the arg max of the logits of the iteration in which its position was finalised,
    # recomputed here from the trace with numpy
    for e in tr:
        n, t = e["n"], e["t"]
        nxt = [f for f in tr if f["n"] == n and f["t"] == t + 1]
        after = nxt[0]["masked"] if nxt else np.zeros((B, K), np.uint8)
        newly = (e["masked"] == 1) & (after == 0)
        for b in e["active"]:
            assert newly[b].any()
            am = np.argmax(fn(n, t)[b], axis=-1)
            assert np.array_equal(r["x"][b, n * K:(n + 1) * K][newly[b]], am[newly[b]])
            # Eq. 9: everything at or above the threshold went, nothing below it unless it was the fallback
            c, tau = e["conf"][b], e["tau"][b]
            m = e["masked"][b] == 1
            above = m & (c >= tau)
            assert np.array_equal(newly[b], above) if above.any() else newly[b].sum() == 1


def test_ratio_over_the_query_counts_the_retained_suffix_rows():
    # Eq. 10 with r_mask taken over the whole query: K = 2 block positions plus e = 2 retained suffix rows that are
    # always masked.  Two masked: r = 4/4, tau = tau0; one masked: r = 3/4, tau = tau0 (1 - alpha / 4).
    ln = np.log
    z = {
        (0, 0): np.array([[[ln(18.0), 0, 0], [0, ln(2.0), 0]]]),   # confidences 0.9 and 0.5 against tau = 0.85
        (0, 1): np.array([[[0, 0, 5.0], [0, 0, ln(8.0)]]]),        # 0.8 against tau = 0.85 * 0.9 = 0.765: accepted
    }
    tr = []
    r = oracle.decode(_table_fn(z), 1, 2, 2, tau0=0.85, alpha=0.4, mask_id=MASK, extra_fn=lambda n: 2, trace=tr)
    assert [round(float(e["tau"][0]), 6) for e in tr] == [0.85, 0.765]
    assert r["x"].tolist() == [[0, 2]] and r["steps"].tolist() == [2]
    # with the block-only ratio the second threshold is 0.85 (1 - 0.4 / 2) = 0.68
    tr2 = []
    oracle.decode(_table_fn(z), 1, 2, 2, tau0=0.85, alpha=0.4, mask_id=MASK, trace=tr2)
    assert [round(float(e["tau"][0]), 6) for e in tr2] == [0.85, 0.68]
