"""One small point of each variant sweep, run through the sweep harness's own functions and checked against the
oracle (the knobs are the ones the paper ablates: the adaptation strength of Eq. 10, the window of Eq. 7 and
its trailing position).  The identities used:

* alpha = 0 is the fixed-threshold rule: the loop needs exactly the iterations ``oracle.decode`` needs with
  alpha = 0 on the same seeded logits, and decodes the same tokens;
* a window that covers the whole suffix is the unpruned method: the output equals ``oracle.attn_full``;
* without the trailing position the output equals the oracle on Eq. 7's list without that row.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_17917_b200 import sweeps
from paper_2601_17917_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


def _np(t):
    return t.float().cpu().numpy()


def _close(out, ref):
    rms_row = np.sqrt((ref ** 2).mean(axis=-1, keepdims=True))       # the bound of tests/test_gpu_attn.py
    assert (np.abs(_np(out) - ref) <= 2.0 ** -8 * np.abs(ref) + 2.5e-2 * rms_row + 1e-6).all()


@pytest.mark.parametrize("alpha", [0.0, 0.3])
def test_alpha_sweep_point_matches_the_oracle_loop(alpha):
    B, K, n_blocks, V = 2, 8, 3, 2048
    rows = sweeps.sweep_alpha(DEV, alphas=(alpha,), B=B, K=K, n_blocks=n_blocks, V=V, w=4, readings=(False,),
                              emit=None)
    assert len(rows) == 1 and rows[0]["alpha"] == alpha and not rows[0]["ratio_counts_suffix"]
    cfg, table = sweeps.alpha_sweep_config(B, K, n_blocks, V)
    trace = []
    ref = oracle.decode(lambda n, t: table(n, t, DEV).float().cpu().numpy().reshape(B, K, V), B, cfg.gen, K, cfg.tau0, alpha,
                        V - 1, trace=trace)
    # parity of integer decisions needs the oracle's trajectory to be clear of near-ties (1e-4 band)
    for e in trace:
        for b in e["active"]:
            c = e["conf"][b][e["masked"][b] == 1].astype(np.float64)
            assert np.abs(c - float(e["tau"][b])).min() >= 1e-4, "near-tie: pick another sweep seed for the test"
    assert rows[0]["iterations"] == ref["steps"].tolist()
    assert np.array_equal(rows[0]["x"].cpu().numpy(), ref["x"])
    if alpha == 0.0:        # the fixed-threshold rule: tau = tau0 at every iteration
        assert all(abs(float(t) - cfg.tau0) < 1e-7 for e in trace for t in np.atleast_1d(e["tau"])[e["active"]])


def test_window_sweep_points_match_the_oracle():
    cfg = wl.shrink(wl.CONFIGS["long32-w64"], B=2, Hq=4, Hkv=4, P=300, gen=448, name="long32-small")
    rows = sweeps.sweep_window(DEV, cfg=cfg, windows=(64, -1), reps=2, keep_outputs=True, emit=None)
    got = {(r["w_tokens"], r["keep_last"]): r for r in rows}
    assert set(got) == {(64, True), (64, False), (-1, True)}
    x = {k: _np(v) for k, v in rows[0]["inputs"].items()}
    scale = rows[0]["scale"]
    # whole suffix = unpruned
    r = got[(-1, True)]
    assert r["Lq"] == cfg.gen
    _close(r["out"], oracle.attn_full(x["q_tail"], x["k_tail"], x["v_tail"], x["k_pre"], x["v_pre"], scale))
    # window 64 with and without the trailing position
    for keep_last in (True, False):
        r = got[(64, keep_last)]
        idx = oracle.retained_indices(cfg.gen, cfg.K, 0, 64, keep_last)
        assert r["idx"] == idx and r["Lq"] == cfg.K + 64 + (1 if keep_last else 0)
        _close(r["out"], oracle.attn(x["q_tail"], x["k_tail"], x["v_tail"], x["k_pre"], x["v_pre"],
                                     np.asarray(idx), scale))
    assert all(r["attn_us"] > 0 and r["GBps"] > 0 for r in rows)
