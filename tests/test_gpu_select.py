"""GPU parity of ds_unmask_select (Eq. 9, Eq. 10, Eq. 5, flags) against the CPU
oracle, through the C ABI.  Everything here is integer/flag output: bit-exact.

(A) isolated: both sides consume the same fp32 confidences.
(B) chained: GPU confidence -> GPU select against oracle confidence -> oracle
    select over several steps; a sequence is dropped from the comparison from
    the step where an oracle confidence lies within 1e-4 of the threshold (or
    the two best fallback candidates lie within 1e-4 of each other)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2601_17917_b200 as ds
from paper_2601_17917_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _gpu_select(conf, tok, masked, x, **kw):
    c = torch.as_tensor(conf, dtype=torch.float32).to(DEV).contiguous()
    t = torch.as_tensor(tok, dtype=torch.int32).to(DEV).contiguous()
    m = torch.as_tensor(masked, dtype=torch.uint8).to(DEV).contiguous().clone()
    xb = torch.as_tensor(x, dtype=torch.int32).to(DEV).contiguous().clone()
    for k in ("seq_list", "n_seq_dev"):
        if kw.get(k) is not None:
            kw[k] = torch.as_tensor(kw[k], dtype=torch.int32).to(DEV)
    eos_init = kw.pop("eos_exit", None)
    B, K = c.shape
    out = dict(sel_idx=torch.full((B, K), -5, dtype=torch.int32, device=DEV),
               sel_cnt=torch.zeros(B, dtype=torch.int32, device=DEV),
               block_done=torch.zeros(B, dtype=torch.uint8, device=DEV),
               eos_exit=(torch.zeros(B, dtype=torch.uint8, device=DEV) if eos_init is None
                         else torch.as_tensor(eos_init, dtype=torch.uint8).to(DEV)),
               active_seq=torch.full((max(B, 1),), -5, dtype=torch.int32, device=DEV),
               active_cnt=torch.full((1,), -5, dtype=torch.int32, device=DEV),
               masked_rows=torch.full((max(B * K, 1),), -5, dtype=torch.int32, device=DEV),
               masked_cnt=torch.full((1,), -5, dtype=torch.int32, device=DEV))
    ds.ds_unmask_select(c, t, m, xb, out=out, **kw)
    torch.cuda.synchronize()
    n = int(out["active_cnt"].item())
    nr = int(out["masked_cnt"].item())
    assert (out["masked_rows"][nr:] == -5).all()
    return dict(masked_rows=out["masked_rows"].cpu().numpy()[:nr], masked=m.cpu().numpy(), x_block=xb.cpu().numpy(), sel_idx=out["sel_idx"].cpu().numpy(),
                sel_cnt=out["sel_cnt"].cpu().numpy(), block_done=out["block_done"].cpu().numpy(),
                eos_exit=out["eos_exit"].cpu().numpy(), active_seq=out["active_seq"].cpu().numpy()[:n])


def _same(g, o, seqs=None):
    B = g["masked"].shape[0]
    seqs = list(range(B)) if seqs is None else list(seqs)
    for b in seqs:
        for k in ("masked", "x_block", "sel_idx", "sel_cnt", "block_done", "eos_exit"):
            assert np.array_equal(g[k][b], o[k][b]), (k, b, g[k][b], o[k][b])
    assert g["active_seq"].tolist() == o["active_seq"].tolist()
    # the rows still masked after the step, over the processed sequences (all of them when none are listed)
    if seqs is not None:
        K = o["masked"].shape[1]
        want = [b * K + i for b in sorted(seqs) for i in np.nonzero(o["masked"][b])[0]]
        assert g["masked_rows"].tolist() == want


@pytest.mark.parametrize("name", ["tiny", "llada1", "llada8x32", "dream16", "long32-w64"])
@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.6])
def test_isolated_uniform_confidences(name, alpha):
    cfg = wl.CONFIGS[name]
    EOS = 7
    conf, tok = wl.uniform_confidences(cfg, eos_id=EOS, eos_p=0.05)
    for mode in ("all", "half", "few"):
        x, masked = wl.block_state(cfg, mode)
        kw = dict(tau0=cfg.tau0, alpha=alpha, eos_id=EOS, eos_tau=0.9)
        g = _gpu_select(conf, tok, masked, x, **kw)
        o = oracle.select(conf.numpy(), tok.numpy(), masked.numpy(), x.numpy(), **kw)
        _same(g, o)
        # the other reading of r_mask: count the retained suffix rows as masked too
        kw["ratio_extra"] = 65
        _same(_gpu_select(conf, tok, masked, x, **kw),
              oracle.select(conf.numpy(), tok.numpy(), masked.numpy(), x.numpy(), **kw))


@pytest.mark.parametrize("K", [1, 5, 31, 32, 33, 100, 1024, 4096])
def test_block_sizes_and_fallback(K):
    rng = np.random.default_rng(K)
    B = 7
    conf = rng.random((B, K)).astype(np.float32)
    conf[1] *= 0.5                       # nothing reaches the threshold: fallback
    conf[2] = 0.25                       # all equal: fallback takes the lowest masked index
    tok = rng.integers(0, 1000, (B, K)).astype(np.int32)
    masked = (rng.random((B, K)) < 0.7).astype(np.uint8)
    masked[3] = 0                        # finished block
    masked[4] = 0
    masked[4, K - 1] = 1                 # single mask in the last position
    x = np.full((B, K), -1, np.int32)
    kw = dict(tau0=0.9, alpha=0.3, eos_id=3, eos_tau=0.5)
    _same(_gpu_select(conf, tok, masked, x, **kw), oracle.select(conf, tok, masked, x, **kw))


def test_hand_worked_cases_on_gpu():
    conf = np.array([[0.95, 0.7, 0.91, 0.99]], np.float32)
    g = _gpu_select(conf, [[10, 11, 12, 13]], [[1, 1, 1, 0]], [[-7, -7, -7, 55]], tau0=0.9, alpha=0.0)
    assert g["sel_idx"][0].tolist() == [0, 2, -1, -1] and g["x_block"][0].tolist() == [10, -7, 12, 55]
    assert g["masked"][0].tolist() == [0, 1, 0, 0] and g["block_done"][0] == 0
    g = _gpu_select([[0.3, 0.5, 0.5, 0.99]], [[1, 2, 3, 4]], [[1, 1, 1, 0]], [[-7] * 4], tau0=0.9, alpha=0.0)
    assert g["sel_cnt"][0] == 1 and g["sel_idx"][0, 0] == 1
    # threshold is inclusive; tau = 0.9 * (1 - 0.5 * 0.5) = 0.675 with 2 of 4 masked
    tau = np.float32(oracle.threshold(2, 4, 0.9, 0.5))
    g = _gpu_select([[tau, 0.1, 0.2, np.nextafter(tau, np.float32(0))]], [[1, 2, 3, 4]], [[1, 0, 0, 1]],
                    [[-7] * 4], tau0=0.9, alpha=0.5)
    assert g["sel_idx"][0].tolist() == [0, -1, -1, -1]
    # early exit: accepted EOS at high confidence sets the flag, a fallback pick at 0.3 does not
    g = _gpu_select([[0.95, 0.2], [0.3, 0.2]], [[2, 7], [2, 7]], [[1, 1], [1, 1]], [[-1, -1], [-1, -1]],
                    tau0=0.9, alpha=0.0, eos_id=2, eos_tau=0.9)
    assert g["eos_exit"].tolist() == [1, 0]


def test_thresholds_match_for_every_mask_count():
    """Bit-exact tau on both sides: put confidences exactly at and just below the oracle's
    float32 threshold for every n."""
    K = 32
    for alpha in (0.1, 0.3, 0.4, 0.6, 0.7):
        for extra in (0, 65):
            rows_c, rows_m = [], []
            for n in range(1, K + 1):
                tau = np.float32(oracle.threshold(n, K, 0.9, alpha, extra))
                c = np.full(K, np.nextafter(tau, np.float32(0)), np.float32)
                c[n - 1] = tau
                m = np.zeros(K, np.uint8)
                m[:n] = 1
                rows_c.append(c)
                rows_m.append(m)
            conf, masked = np.stack(rows_c), np.stack(rows_m)
            tok = np.ones((K, K), np.int32)
            x = np.zeros((K, K), np.int32)
            kw = dict(tau0=0.9, alpha=alpha, ratio_extra=extra)
            g = _gpu_select(conf, tok, masked, x, **kw)
            o = oracle.select(conf, tok, masked, x, **kw)
            _same(g, o)
            assert (g["sel_cnt"] == 1).all() and [int(g["sel_idx"][i, 0]) for i in range(K)] == list(range(K))


def test_seq_list_device_count_and_large_batch():
    rng = np.random.default_rng(11)
    B, K = 3000, 32                      # spreads over the grid + separate compaction kernel
    conf = rng.random((B, K)).astype(np.float32)
    tok = rng.integers(0, 50, (B, K)).astype(np.int32)
    masked = (rng.random((B, K)) < 0.3).astype(np.uint8)
    x = np.full((B, K), -1, np.int32)
    kw = dict(tau0=0.9, alpha=0.3, eos_id=5, eos_tau=0.8)
    _same(_gpu_select(conf, tok, masked, x, **kw), oracle.select(conf, tok, masked, x, **kw))
    seqs = sorted(rng.choice(B, 1200, replace=False).tolist())
    g = _gpu_select(conf, tok, masked, x, seq_list=seqs, **kw)
    o = oracle.select(conf, tok, masked, x, seq_list=seqs, **kw)
    _same(g, o, seqs)
    rest = sorted(set(range(B)) - set(seqs))
    assert np.array_equal(g["masked"][rest], masked[rest]) and (g["sel_idx"][rest] == -5).all()
    # count taken from a device scalar smaller than the list
    g = _gpu_select(conf[:64], tok[:64], masked[:64], x[:64], seq_list=list(range(0, 64, 2)), n_seq_dev=[10], **kw)
    o = oracle.select(conf[:64], tok[:64], masked[:64], x[:64], seq_list=list(range(0, 20, 2)), **kw)
    _same(g, o, list(range(0, 20, 2)))
    # empty list
    g = _gpu_select(conf[:8], tok[:8], masked[:8], x[:8], seq_list=torch.zeros(0, dtype=torch.int32), **kw)
    assert g["active_seq"].tolist() == []


@pytest.mark.parametrize("B", [40, 3000])
def test_active_list_updated_in_place(B):
    # active_seq aliases seq_list and active_cnt aliases n_seq_dev: the list shrinks in place over the steps
    rng = np.random.default_rng(21)
    K = 32
    masked = np.ones((B, K), np.uint8)
    x = np.full((B, K), -1, np.int32)
    lst = torch.arange(B, dtype=torch.int32, device=DEV)
    cnt = torch.tensor([B], dtype=torch.int32, device=DEV)
    gm, gx = torch.tensor(masked, device=DEV), torch.tensor(x, device=DEV)
    out = dict(sel_idx=torch.empty((B, K), dtype=torch.int32, device=DEV),
               sel_cnt=torch.zeros(B, dtype=torch.int32, device=DEV),
               block_done=torch.zeros(B, dtype=torch.uint8, device=DEV),
               eos_exit=torch.zeros(B, dtype=torch.uint8, device=DEV), active_seq=lst, active_cnt=cnt,
               masked_rows=torch.empty(B * K, dtype=torch.int32, device=DEV),
               masked_cnt=torch.zeros(1, dtype=torch.int32, device=DEV))
    active = list(range(B))
    for step in range(6):
        conf = rng.random((B, K)).astype(np.float32) ** 0.25
        tok = rng.integers(0, 50, (B, K)).astype(np.int32)
        o = oracle.select(conf, tok, masked, x, 0.9, 0.3, seq_list=active)
        ds.ds_unmask_select(torch.tensor(conf, device=DEV), torch.tensor(tok, device=DEV), gm, gx, 0.9, 0.3,
                            seq_list=lst, n_seq=B, n_seq_dev=cnt, out=out)
        torch.cuda.synchronize()
        masked, x, active = o["masked"], o["x_block"], o["active_seq"].tolist()
        assert cnt.item() == len(active) and lst[:len(active)].cpu().tolist() == active
        assert np.array_equal(gm.cpu().numpy(), masked) and np.array_equal(gx.cpu().numpy(), x)
        want_rows = [b * K + i for b in range(B) for i in np.nonzero(masked[b])[0]]
        assert out["masked_rows"][:out["masked_cnt"].item()].cpu().tolist() == want_rows
    assert len(active) < B


def _chain(cfg, steps, alpha, eos_id):
    """Config-4 style simulation: few masks per sequence, fresh logits each step."""
    x0, m0 = wl.block_state(cfg, "few")
    gx, gm = x0.to(DEV), m0.to(DEV)
    ox, om = x0.numpy().copy(), m0.numpy().copy()
    B, K = cfg.B, cfg.K
    g_eos = torch.zeros(B, dtype=torch.uint8, device=DEV)
    o_eos = np.zeros(B, np.uint8)
    g_active = None
    o_active = None
    valid = np.ones(B, bool)
    fired = dict(done=0, eos=0, rule=0, fallback=0)
    for step in range(steps):
        z = wl.logits(cfg, device=DEV, step=step, spike_range=(12.0, 20.0))
        if eos_id >= 0:
            z[::5, eos_id] = 22.0        # some rows predict EOS confidently
        gc, gt = ds.ds_confidence(z)
        oc, ot = oracle.confidence(z.float().cpu().numpy())
        assert np.abs(gc.cpu().numpy() - oc).max() < 2e-5 and (gt.cpu().numpy() == ot).all()
        kw = dict(tau0=cfg.tau0, alpha=alpha, eos_id=eos_id, eos_tau=cfg.tau0)
        out = ds.ds_unmask_select(gc.view(B, K), gt.view(B, K), gm, gx, seq_list=g_active, **kw,
                                  out=dict(sel_idx=torch.full((B, K), -1, dtype=torch.int32, device=DEV),
                                           sel_cnt=torch.zeros(B, dtype=torch.int32, device=DEV),
                                           block_done=torch.zeros(B, dtype=torch.uint8, device=DEV),
                                           eos_exit=g_eos,
                                           active_seq=torch.empty(B, dtype=torch.int32, device=DEV),
                                           active_cnt=torch.zeros(1, dtype=torch.int32, device=DEV)))
        ocf = oc.reshape(B, K).astype(np.float32)
        o = oracle.select(ocf, ot.reshape(B, K), om, ox, seq_list=o_active, eos_exit=o_eos, **kw)
        listed = range(B) if o_active is None else o_active
        for b in listed:                 # exclusion band around the decision
            mk = om[b].astype(bool)
            if not mk.any():
                continue
            c = ocf[b][mk]
            near_tau = np.abs(c - o["tau"][b]).min() < 1e-4
            top2 = np.sort(c)[-2:]
            near_tie = (o["sel_cnt"][b] == 1 and c.max() < o["tau"][b] and len(top2) == 2
                        and top2[1] - top2[0] < 1e-4)
            if near_tau or near_tie:
                valid[b] = False
        n = int(out["active_cnt"].item())
        ga = out["active_seq"][:n].clone()
        for b in listed:
            if not valid[b]:
                continue
            assert np.array_equal(out["sel_idx"][b].cpu().numpy(), o["sel_idx"][b]), (step, b)
            assert int(out["sel_cnt"][b]) == o["sel_cnt"][b] and int(out["block_done"][b]) == o["block_done"][b]
            assert int(g_eos[b]) == o["eos_exit"][b]
            fired["rule" if (ocf[b][om[b].astype(bool)] >= o["tau"][b]).any() else "fallback"] += 1
        if valid.all():
            assert ga.cpu().tolist() == o["active_seq"].tolist()
        om, ox, o_eos, o_active = o["masked"], o["x_block"], o["eos_exit"], o["active_seq"]
        g_active = ga
        fired["done"] += int(o["block_done"][list(listed)].sum())
        fired["eos"] = int(o_eos.sum())
        if len(o_active) == 0 or n == 0:
            break
    for b in range(B):
        if valid[b]:
            assert np.array_equal(gm[b].cpu().numpy(), om[b]) and np.array_equal(gx[b].cpu().numpy(), ox[b])
    return fired, valid


def test_chained_eight_steps_dream_shape():
    cfg = wl.CONFIGS["dream16"]
    fired, valid = _chain(cfg, steps=8, alpha=0.3, eos_id=11)
    assert valid.sum() >= cfg.B - 2
    assert fired["done"] > 0 and fired["eos"] > 0 and fired["rule"] > 0 and fired["fallback"] > 0


def test_chained_literal_distribution_tiny():
    # literal inputs (+8 spike): nearly every step is a fallback pick
    cfg = wl.CONFIGS["tiny"]
    x, masked = wl.block_state(cfg, "half")
    z = wl.logits(cfg, device=DEV)
    gc, gt = ds.ds_confidence(z)
    oc, ot = oracle.confidence(z.float().cpu().numpy())
    kw = dict(tau0=cfg.tau0, alpha=cfg.alpha)
    g = _gpu_select(gc.view(1, -1).cpu(), gt.view(1, -1).cpu(), masked, x, **kw)
    o = oracle.select(oc.reshape(1, -1).astype(np.float32), ot.reshape(1, -1), masked.numpy(), x.numpy(), **kw)
    mk = masked.numpy()[0].astype(bool)
    if np.abs(oc[mk] - o["tau"][0]).min() >= 1e-4:
        _same(g, o)
