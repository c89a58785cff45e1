"""GPU parity of the block scheduler (decode.BlockDecoder over ds_block_begin, ds_confidence_listed and
ds_unmask_select) against the oracle's decoding loop, on the same seeded logits.  Tokens, iteration counts
and early-exit flags are integer results: bit-exact.  Eq. 9's comparisons are taken in float32 on both
sides from confidences that differ in the last bits, so the test first checks, on the oracle's trajectory,
that no decision is closer than 1e-4 to flipping (threshold margin, gap of the two best fallback
candidates); a seed that fails that check is not a parity case."""
import numpy as np
import pytest
import torch

import oracle
import paper_2601_17917_b200 as ds
from paper_2601_17917_b200 import workloads as wl
from paper_2601_17917_b200.decode import BlockDecoder

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MASK = 1 << 20


def _cfg(B, K, L, V, seed):
    return wl.shrink(wl.CONFIGS["tiny"], B=B, K=K, gen=L, V=V, dtype="bf16", spike_p=0.7, seed=seed, name="decode")


def _table(cfg, eos=None):
    cache = {}

    def z(n, t):
        if (n, t) not in cache:
            x = wl.logits(cfg, step=n * 4096 + t, spike_range=(8.0, 18.0))
            if eos is not None and n == eos["block"]:
                x[eos["seq"] * cfg.K + eos["pos"], eos["id"]] = 40.0
            cache[(n, t)] = x
        return cache[(n, t)]
    return z


def _margins_ok(trace, eos_tau=None):
    for e in trace:
        for b in e["active"]:
            m = e["masked"][b] == 1
            c = e["conf"][b][m].astype(np.float64)
            if np.abs(c - float(e["tau"][b])).min() < 1e-4:
                return False
            if eos_tau is not None and np.abs(c - eos_tau).min() < 1e-4:
                return False
            if (c < e["tau"][b]).all() and len(c) > 1:
                top = np.sort(c)[-2:]
                if top[1] - top[0] < 1e-4:
                    return False
    return True


def _run(cfg, alpha, lookahead, eos=None, count_suffix=False, w=16):
    B, K, L, V = cfg.B, cfg.K, cfg.gen, cfg.V
    z = _table(cfg, eos)
    eos_id = -1 if eos is None else eos["id"]
    extra = (lambda n: len(oracle.retained_indices(L, K, n, w, True)) - K) if count_suffix else None
    tr = []
    ref = oracle.decode(lambda n, t: z(n, t).float().numpy().reshape(B, K, V), B, L, K, cfg.tau0, alpha, MASK,
                        eos_id=eos_id, eos_tau=0.9, extra_fn=extra, trace=tr)
    assert _margins_ok(tr, 0.9 if eos else None), "near-tie on the oracle's trajectory: pick another seed"
    dec = BlockDecoder(B, L, K, V, tau0=cfg.tau0, alpha=alpha, mask_id=MASK, eos_id=eos_id, eos_tau=0.9,
                       w_tokens=w, keep_last=True, count_suffix=count_suffix, device=DEV, lookahead=lookahead)
    seen = []

    def forward(step):
        seen.append((step.n, step.t, step.refresh, step.idx.numel()))
        step.logits.copy_(z(step.n, step.t).to(DEV))
    got = dec.decode(forward)
    torch.cuda.synchronize()
    assert np.array_equal(got["x"].cpu().numpy(), ref["x"])
    assert got["steps"] == ref["steps"].tolist()
    assert got["eos_exit"].cpu().numpy().tolist() == ref["eos_exit"].tolist()
    for need, ran in zip(got["steps"], got["launched"]):
        assert need <= ran <= min(K, need + lookahead)
    # first iteration of a block is the refresh (all rows of the tail), the others use Eq. 7's retained rows
    for n, t, refresh, n_idx in seen:
        assert refresh == (t == 0)
        assert n_idx == (L - n * K if t == 0 else len(oracle.retained_indices(L, K, n, w, True)))
    return got, ref


@pytest.mark.parametrize("lookahead", [0, 2, 5])
@pytest.mark.parametrize("alpha", [0.0, 0.3])
def test_decode_matches_the_oracle_loop(alpha, lookahead):
    got, ref = _run(_cfg(4, 16, 64, 512, seed=11), alpha, lookahead)
    assert 1 < max(got["steps"]) <= 16


def test_ratio_counts_the_retained_suffix_rows():
    _run(_cfg(3, 16, 96, 512, seed=12), 0.5, 2, count_suffix=True)


def test_early_exit_skips_the_remaining_blocks():
    cfg = _cfg(4, 16, 64, 512, seed=13)
    got, ref = _run(cfg, 0.3, 2, eos=dict(block=1, seq=2, pos=5, id=77))
    assert ref["eos_exit"].tolist() == [0, 0, 1, 0]
    x = got["x"].cpu().numpy()
    assert (x[2, 32:] == 77).all() and (x[[0, 1, 3]] != MASK).all()


def test_every_sequence_exits_and_the_last_blocks_take_no_iteration():
    cfg = _cfg(2, 8, 32, 256, seed=14)
    z = _table(cfg)

    def rig(n, t):
        x = z(n, t).clone()
        if n == 0:
            x[0 * 8 + 1, 9] = 40.0
            x[1 * 8 + 6, 9] = 40.0
        return x
    ref = oracle.decode(lambda n, t: rig(n, t).float().numpy().reshape(2, 8, 256), 2, 32, 8, 0.9, 0.3, MASK,
                        eos_id=9, eos_tau=0.9)
    assert ref["steps"].tolist()[1:] == [0, 0, 0]
    for lookahead in (0, 3):
        dec = BlockDecoder(2, 32, 8, 256, tau0=0.9, alpha=0.3, mask_id=MASK, eos_id=9, eos_tau=0.9, device=DEV,
                           lookahead=lookahead)
        got = dec.decode(lambda s: s.logits.copy_(rig(s.n, s.t).to(DEV)))
        assert got["steps"] == ref["steps"].tolist()
        assert np.array_equal(got["x"].cpu().numpy(), ref["x"])


def test_iterations_as_cuda_graphs():
    # one graph launch per iteration; the logits are staged by the eager hook, the captured callback is fixed
    cfg = _cfg(4, 16, 64, 512, seed=11)
    B, K, L, V = cfg.B, cfg.K, cfg.gen, cfg.V
    z = _table(cfg)
    ref = oracle.decode(lambda n, t: z(n, t).float().numpy().reshape(B, K, V), B, L, K, cfg.tau0, 0.3, MASK)
    dec = BlockDecoder(B, L, K, V, tau0=cfg.tau0, alpha=0.3, mask_id=MASK, w_tokens=16, device=DEV, lookahead=2)
    stage = lambda n, t: dec.logits.copy_(z(n, t).to(DEV))
    n0 = ds.ds_launch_count()
    for _ in range(2):                                  # the second run replays the graphs captured by the first
        got = dec.decode(lambda st: None, before_iteration=stage, graphs=True)
        torch.cuda.synchronize()
        assert np.array_equal(got["x"].cpu().numpy(), ref["x"])
        assert got["steps"] == ref["steps"].tolist()
    assert len(dec._graphs) == 2 * (L // K)


def test_block_begin_lists():
    B, K = 70, 24
    rng = np.random.default_rng(3)
    ex = (rng.random(B) < 0.4).astype(np.uint8)
    t = lambda *s, dt=torch.int32: torch.full(s, -9, dtype=dt, device=DEV)
    masked, xb = torch.full((B, K), 7, dtype=torch.uint8, device=DEV), t(B, K)
    act, cnt, rows, rcnt = t(B), t(1), t(B * K), t(1)
    ds.ds_block_begin(torch.tensor(ex, device=DEV), masked, xb, MASK, 5, act, cnt, rows, rcnt)
    torch.cuda.synchronize()
    live = np.nonzero(ex == 0)[0]
    assert cnt.item() == len(live) and act[:len(live)].cpu().tolist() == live.tolist()
    assert rcnt.item() == len(live) * K
    assert rows[:len(live) * K].cpu().tolist() == [b * K + i for b in live for i in range(K)]
    assert (rows[len(live) * K:] == -9).all()
    assert np.array_equal(masked.cpu().numpy(), np.repeat((ex == 0).astype(np.uint8)[:, None], K, 1))
    assert np.array_equal(xb.cpu().numpy(), np.where(ex[:, None] == 0, MASK, 5) * np.ones((1, K), np.int64))
