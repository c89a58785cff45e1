"""The prefix-cache life cycle, end to end, on two consecutive blocks (Method, "Dynamic Confidence Aware
Parallel Decoding": the prefix KV is computed at the first step of a block, reused by the block's later steps,
and the finished block joins the prefix).

A toy model stands in for the network: per layer and position, seeded un-rotated Q/K/V projections (they do
not depend on the tokens), and the block's logits from a seeded table.  The GPU run drives the block scheduler
with a forward callback that does what a layer's attention does at every iteration:

  first iteration of block n (refresh)   the finished block n-1 is appended to the cache
                                         (ds_rope_gather with n_append = K); dense attention over prefix + block
                                         + retained suffix with nothing cached (ds_rope_gather over all rows, then
                                         ds_attn_pruned with P = 0)
  later iterations (pruned)              ds_rope_gather of the retained tail rows, ds_attn_pruned over
                                         [cache rows 0 .. P0 + n K) ; retained rows]

so block 1's attention reads rows that block 0 appended.  The same chain of oracle calls (rope_gather for the
cache and the retained rows, attn, decode) gives the reference.  Attention outputs are compared within the
tolerance of the rope -> attention pipeline test (the GPU cache is bf16, the oracle's is not rounded); tokens,
iteration counts and the cache's untouched rows exactly."""
import math

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
THETA = 10000.0


def _np(t):
    return t.float().cpu().numpy()


def _raw(B, Hq, Hkv, S, D, seed):
    g = torch.Generator().manual_seed(seed)
    mk = lambda h: torch.randn(B, h, S, D, generator=g).to(torch.bfloat16).to(DEV)
    return mk(Hq), mk(Hkv), mk(Hkv)


@pytest.mark.parametrize("w_tokens", [16, 0])
def test_two_blocks_second_block_attends_over_what_the_first_appended(w_tokens):
    B, Hq, Hkv, D, P0, K, N, V, n_layers = 2, 4, 2, 128, 160, 32, 2, 512, 2
    L = N * K
    S = P0 + L
    scale = 1.0 / math.sqrt(D)
    raw = [_raw(B, Hq, Hkv, S, D, seed=100 + l) for l in range(n_layers)]
    cfg = wl.shrink(wl.CONFIGS["tiny"], B=B, K=K, gen=L, V=V, dtype="bf16", spike_p=0.7, seed=4242, name="lifecycle")
    table = {}

    def z(n, t):
        if (n, t) not in table:
            table[(n, t)] = wl.logits(cfg, step=n * 4096 + t, spike_range=(8.0, 18.0))
        return table[(n, t)]

    # ---------------- GPU run ----------------
    kc = [torch.zeros(B, Hkv, S, D, dtype=torch.bfloat16, device=DEV) for _ in range(n_layers)]
    vc = [torch.zeros_like(kc[0]) for _ in range(n_layers)]
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for l, (q, k, v) in enumerate(raw):       # prompt prefill: rotated K and plain V of positions 0 .. P0-1
        ds.ds_rope_gather(q, k, v, torch.arange(P0, dtype=torch.int32, device=DEV), 0, THETA, k_cache=kc[l], v_cache=vc[l],
                          cache_row0=0, n_append=P0, status=status)
    seen = {}

    def forward(st):
        base = P0 + st.n * K                  # absolute position of tail row 0 = rows of the cache in use
        for l, (q, k, v) in enumerate(raw):
            if st.refresh:
                if st.n > 0:                  # the finished block joins the prefix
                    ds.ds_rope_gather(q[:, :, base - K:], k[:, :, base - K:], v[:, :, base - K:],
                                      torch.arange(K, dtype=torch.int32, device=DEV), base - K, THETA, k_cache=kc[l],
                                      v_cache=vc[l], cache_row0=base - K, n_append=K, status=status)
                keep = torch.tensor(ds.retained_indices(L, K, st.n, w_tokens, True), dtype=torch.int32, device=DEV) + base
                rows = torch.cat([torch.arange(base, dtype=torch.int32, device=DEV), keep])
                qo, ko, vo = ds.ds_rope_gather(q, k, v, rows, 0, THETA, status=status)
                out = ds.ds_attn_pruned(qo, ko, vo, None, None, torch.arange(rows.numel(), dtype=torch.int32, device=DEV),
                                        scale, status=status)
            else:
                qo, ko, vo = ds.ds_rope_gather(q[:, :, base:], k[:, :, base:], v[:, :, base:], st.idx, base, THETA,
                                               status=status)
                out = ds.ds_attn_pruned(qo, ko, vo, kc[l][:, :, :base], vc[l][:, :, :base],
                                        torch.arange(st.idx.numel(), dtype=torch.int32, device=DEV), scale, status=status)
            if (st.n, st.t) in ((0, 1), (1, 0), (1, 1), (1, 2)):
                seen[(st.n, st.t, l)] = out.clone()
        st.logits.copy_(z(st.n, st.t).to(DEV))

    dec = BlockDecoder(B, L, K, V, tau0=cfg.tau0, alpha=0.3, mask_id=MASK, w_tokens=w_tokens, keep_last=True, device=DEV,
                       lookahead=0)
    got = dec.decode(forward)
    torch.cuda.synchronize()
    assert ds.ds_read_status(status) == 0

    # ---------------- the same chain of oracle calls ----------------
    ref = oracle.decode(lambda n, t: z(n, t).float().numpy().reshape(B, K, V), B, L, K, cfg.tau0, 0.3, MASK)
    assert np.array_equal(got["x"].cpu().numpy(), ref["x"]) and got["steps"] == ref["steps"].tolist()
    assert min(got["steps"]) >= 3, "the seeded logits are meant to give every block several pruned iterations"
    for l, (q, k, v) in enumerate(raw):
        fq, fk, fv = _np(q), _np(k), _np(v)
        # the oracle's cache after block 0: prompt rows, then block 0's rows, each rotated with its own position
        _, ck0, cv0 = oracle.rope_gather(fq, fk, fv, np.arange(P0), 0, THETA)
        _, ck1, cv1 = oracle.rope_gather(fq[:, :, P0:], fk[:, :, P0:], fv[:, :, P0:], np.arange(K), P0, THETA)
        ock, ocv = np.concatenate([ck0, ck1], 2), np.concatenate([cv0, cv1], 2)
        # cache contents: rows written are the rotated keys / plain values (bf16 rounding), the rest untouched
        assert (np.abs(_np(kc[l][:, :, :P0 + K]) - ock) <= 2.0 ** -8 * np.abs(ock) + 1e-6).all()
        assert np.array_equal(_np(vc[l][:, :, :P0 + K]), ocv)
        assert (kc[l][:, :, P0 + K:] == 0).all() and (vc[l][:, :, P0 + K:] == 0).all()
        for n, t in ((0, 1), (1, 1), (1, 2)):               # pruned iterations: cache prefix + retained rows
            base = P0 + n * K
            idx = np.asarray(oracle.retained_indices(L, K, n, w_tokens, True))
            rq, rk, rv = oracle.rope_gather(fq[:, :, base:], fk[:, :, base:], fv[:, :, base:], idx, base, THETA)
            want = oracle.attn(rq, rk, rv, ock[:, :, :base], ocv[:, :, :base], np.arange(len(idx)), scale)
            err = np.abs(_np(seen[(n, t, l)]) - want).max()
            assert err <= 1e-2 and err <= 6e-3, (l, n, t, err)
            if n == 1:
                # block 1 really depends on the appended rows: without them the result is far off
                hole_k, hole_v = ock[:, :, :base].copy(), ocv[:, :, :base].copy()
                hole_k[:, :, P0:] = 0.0
                hole_v[:, :, P0:] = 0.0
                other = oracle.attn(rq, rk, rv, hole_k, hole_v, np.arange(len(idx)), scale)
                assert np.abs(other - want).max() > 10 * 6e-3
        # the refresh iteration of block 1: every row a query and a key, nothing cached
        base = P0 + K
        rows = np.concatenate([np.arange(base), base + np.asarray(oracle.retained_indices(L, K, 1, w_tokens, True))])
        rq, rk, rv = oracle.rope_gather(fq, fk, fv, rows, 0, THETA)
        want = oracle.attn(rq, rk, rv, np.zeros((B, Hkv, 0, D)), np.zeros((B, Hkv, 0, D)), np.arange(len(rows)), scale)
        err = np.abs(_np(seen[(1, 0, l)]) - want).max()
        assert err <= 1e-2 and err <= 6e-3, (l, "refresh", err)
