"""Pins for the attention oracle: closed forms, invariants, a library routine on
the special case it reduces to, and the paper's structural identity that a
window covering the whole suffix is the unpruned method (window-size ablation:
"no suffix windows" = the full size)."""
import numpy as np
import pytest
import torch

import oracle


def _rand(B=2, Hq=4, Hkv=2, D=16, P=5, T=11, seed=0):
    rng = np.random.default_rng(seed)
    f = lambda *s: rng.standard_normal(s).astype(np.float32)
    return dict(q_tail=f(B, Hq, T, D), k_tail=f(B, Hkv, T, D), v_tail=f(B, Hkv, T, D),
                k_pre=f(B, Hkv, P, D), v_pre=f(B, Hkv, P, D))


def test_retained_indices_eq7():
    # K = 32 block, 16 nearest suffix tokens, plus the last position of a 256-token tail
    idx = oracle.retained_indices(256, 32, 0, 16)
    assert idx == list(range(48)) + [255]
    # later block: the tail shrinks by c*K rows
    idx = oracle.retained_indices(256, 32, 3, 32)
    assert idx == list(range(64)) + [256 - 96 - 1]
    # window reaching the end does not duplicate the trailing position
    assert oracle.retained_indices(128, 32, 0, 96) == list(range(128))
    assert oracle.retained_indices(128, 32, 0, 4096) == list(range(128))
    # no window, no trailing position: the block alone
    assert oracle.retained_indices(128, 32, 0, 0, keep_last=False) == list(range(32))
    # last block: nothing after it
    assert oracle.retained_indices(128, 32, 3, 64) == list(range(32))
    # Eq. 2 block positions
    assert oracle.block_indices(10, 4, 2) == [18, 19, 20, 21]


def test_all_retained_equals_unpruned():
    x = _rand()
    T = x["q_tail"].shape[2]
    scale = 0.3
    got = oracle.attn(**x, idx=np.arange(T), scale=scale)
    ref = oracle.attn_full(**x, scale=scale)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_pruned_rows_equal_unpruned_on_pruned_sequence():
    """Pruning = running the unpruned definition on the shortened sequence x~ (Eq. 8)."""
    x = _rand(seed=3)
    idx = np.array([0, 1, 2, 5, 10])
    got = oracle.attn(**x, idx=idx, scale=0.25)
    y = dict(x)
    for k in ("q_tail", "k_tail", "v_tail"):
        y[k] = x[k][:, :, idx, :]
    ref = oracle.attn_full(**y, scale=0.25)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_against_library_sdpa_float64():
    x = _rand(B=1, Hq=3, Hkv=3, D=8, P=7, T=9, seed=5)
    idx = np.array([0, 1, 2, 3, 8])
    scale = 1.0 / np.sqrt(8)
    got = oracle.attn(**x, idx=idx, scale=scale)
    q = torch.from_numpy(x["q_tail"][:, :, idx]).double()
    k = torch.cat([torch.from_numpy(x["k_pre"]), torch.from_numpy(x["k_tail"][:, :, idx])], 2).double()
    v = torch.cat([torch.from_numpy(x["v_pre"]), torch.from_numpy(x["v_tail"][:, :, idx])], 2).double()
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, scale=scale).numpy()
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)


def test_values_all_one_give_one():
    x = _rand(seed=7)
    x["v_tail"][:] = 1.0
    x["v_pre"][:] = 1.0
    got = oracle.attn(**x, idx=np.array([0, 3, 4, 10]), scale=0.5)
    np.testing.assert_allclose(got, 1.0, rtol=0, atol=1e-13)


def test_zero_queries_give_mean_of_values():
    x = _rand(seed=9)
    x["q_tail"][:] = 0.0
    idx = np.array([1, 2, 6])
    got = oracle.attn(**x, idx=idx, scale=0.5)
    B, Hq = got.shape[:2]
    G = Hq // x["k_tail"].shape[1]
    for b in range(B):
        for h in range(Hq):
            vals = np.concatenate([x["v_pre"][b, h // G], x["v_tail"][b, h // G][idx]], 0).astype(np.float64)
            np.testing.assert_allclose(got[b, h], np.broadcast_to(vals.mean(0), got[b, h].shape), atol=1e-13)


def test_single_key_returns_that_value_row():
    x = _rand(B=1, Hq=2, Hkv=2, D=4, P=0, T=6, seed=11)
    got = oracle.attn(**x, idx=np.array([4]), scale=0.7)
    np.testing.assert_allclose(got[0, :, 0, :], x["v_tail"][0, :, 4, :].astype(np.float64), atol=1e-15)


def test_no_suffix_is_prefix_plus_block():
    x = _rand(seed=13)
    K = 4
    got = oracle.attn(**x, idx=np.arange(K), scale=0.2)
    y = {k: (v[:, :, :K] if k.endswith("tail") else v) for k, v in x.items()}
    ref = oracle.attn_full(**y, scale=0.2)
    np.testing.assert_allclose(got, ref, atol=1e-12)


def test_prefix_tail_swap_and_key_order_invariance():
    """Softmax attention is invariant to the order of keys and to which keys are
    counted as cached prefix: move two prefix rows to the front of the tail as
    key-only rows (their outputs are dropped)."""
    x = _rand(B=1, Hq=2, Hkv=1, D=8, P=6, T=5, seed=17)
    idx = np.arange(5)
    base = oracle.attn(**x, idx=idx, scale=0.4)
    perm = np.array([3, 1, 5, 0, 4, 2])
    y = dict(x)
    y["k_pre"] = x["k_pre"][:, :, perm]
    y["v_pre"] = x["v_pre"][:, :, perm]
    np.testing.assert_allclose(oracle.attn(**y, idx=idx, scale=0.4), base, atol=1e-13)
    # move prefix rows 4,5 into the tail (rows 0,1 of a longer tail), query rows unchanged
    z = dict(x)
    z["k_pre"], z["v_pre"] = x["k_pre"][:, :, :4], x["v_pre"][:, :, :4]
    z["k_tail"] = np.concatenate([x["k_pre"][:, :, 4:], x["k_tail"]], 2)
    z["v_tail"] = np.concatenate([x["v_pre"][:, :, 4:], x["v_tail"]], 2)
    z["q_tail"] = np.concatenate([np.zeros((1, 2, 2, 8), np.float32), x["q_tail"]], 2)
    moved = oracle.attn(**z, idx=np.arange(7), scale=0.4)
    np.testing.assert_allclose(moved[:, :, 2:], base, atol=1e-13)


def test_gqa_equals_expanded_mha():
    x = _rand(B=1, Hq=6, Hkv=2, D=8, P=4, T=7, seed=19)
    idx = np.array([0, 1, 2, 6])
    got = oracle.attn(**x, idx=idx, scale=0.35)
    y = dict(x)
    for k in ("k_tail", "v_tail", "k_pre", "v_pre"):
        y[k] = np.repeat(x[k], 3, axis=1)   # consecutive query heads share a KV head
    np.testing.assert_allclose(oracle.attn(**y, idx=idx, scale=0.35), got, atol=1e-14)


def test_lse_and_per_batch_index_lists():
    x = _rand(B=2, Hq=2, Hkv=2, D=8, P=3, T=9, seed=23)
    idx = np.array([[0, 1, 8], [0, 4, 5]])
    out, lse = oracle.attn(**x, idx=idx, scale=0.5, want_lse=True)
    for b in range(2):
        xb = {k: v[b:b + 1] for k, v in x.items()}
        ob, lb = oracle.attn(**xb, idx=idx[b], scale=0.5, want_lse=True)
        np.testing.assert_allclose(out[b], ob[0], atol=1e-14)
        np.testing.assert_allclose(lse[b], lb[0], atol=1e-14)
    # lse against the definition log(sum(exp(scale * q.k)))
    q = x["q_tail"][0, 1, idx[0][2]].astype(np.float64)
    keys = np.concatenate([x["k_pre"][0, 1], x["k_tail"][0, 1][idx[0]]], 0).astype(np.float64)
    assert abs(lse[0, 1, 2] - np.log(np.exp(0.5 * keys @ q).sum())) < 1e-12


def test_planted_mistakes_are_caught():
    """A transposed operand or a dropped prefix would change the result: the pins
    above are not vacuous (checks the brute-force reference disagrees with a
    deliberately wrong variant)."""
    x = _rand(seed=29)
    T = x["q_tail"].shape[2]
    good = oracle.attn(**x, idx=np.arange(T), scale=0.3)
    y = dict(x)
    y["k_pre"], y["v_pre"] = x["k_pre"][:, :, :0], x["v_pre"][:, :, :0]
    assert np.abs(oracle.attn_full(**y, scale=0.3) - good).max() > 1e-3
    y = dict(x)
    y["k_tail"], y["v_tail"] = x["v_tail"], x["k_tail"]
    assert np.abs(oracle.attn_full(**y, scale=0.3) - good).max() > 1e-3


def test_bad_index_rejected():
    x = _rand()
    with pytest.raises(ValueError):
        oracle.attn(**x, idx=np.array([0, 99]), scale=1.0)
