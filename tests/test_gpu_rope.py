"""GPU parity of ds_rope_gather against the CPU oracle, through the C ABI, and the two-kernel pipeline
ds_rope_gather -> ds_attn_pruned against oracle.rope_gather -> oracle.attn.

Tolerance of the rotated rows: the kernel's angle is exact to fp32 rounding of the final sine / cosine, so
what remains is the bf16 rounding of the output: |err| <= 2^-8 |value| + 1e-6.  Gathered V rows and the
appended cache rows are compared bit for bit (with the kernel's own outputs for the rotated K rows)."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2601_17917_b200 as ds
from paper_2601_17917_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
f = lambda t: t.float().cpu().numpy()


def _raw(B, Hq, Hkv, T, D, seed):
    cfg = wl.StepConfig("t", B=B, Hq=Hq, Hkv=Hkv, D=D, P=8, gen=T, K=1, w=0, keep_last=False, dtype="bf16", V=8,
                        spike_p=0, seed=seed)
    x = wl.attention_inputs(cfg, device=DEV)
    return x["q_tail"], x["k_tail"], x["v_tail"], x


def _close(got, ref):
    got = f(got).astype(np.float64)
    assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-6).all(), np.abs(got - ref).max()


@pytest.mark.parametrize("B,Hq,Hkv,T,D,Lq,off,theta", [
    (1, 4, 4, 256, 64, 49, 64, 10000.0), (2, 8, 2, 300, 128, 129, 4096, 500000.0), (3, 4, 4, 200, 32, 1, 0, 10000.0),
    (2, 28, 4, 500, 128, 97, 8000, 1000000.0), (1, 2, 2, 64, 256, 64, 100000, 10000.0)])
def test_rotation_and_gather_match_oracle(B, Hq, Hkv, T, D, Lq, off, theta):
    q, k, v, _ = _raw(B, Hq, Hkv, T, D, seed=Lq + D)
    idx = list(range(Lq - 1)) + [T - 1]
    idx_t = torch.tensor(idx, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    qo, ko, vo = ds.ds_rope_gather(q, k, v, idx_t, off, theta, status=status)
    torch.cuda.synchronize()
    assert ds.ds_read_status(status) == 0
    rq, rk, rv = oracle.rope_gather(f(q), f(k), f(v), np.asarray(idx), off, theta)
    _close(qo, rq)
    _close(ko, rk)
    assert torch.equal(vo, v[:, :, idx_t.long()])


def test_per_batch_lists_strided_views_and_cache_append():
    B, Hq, Hkv, T, D, K = 3, 4, 2, 400, 128, 32
    q, k, v, _ = _raw(B, Hq, Hkv, T, D, seed=5)
    rng = np.random.default_rng(1)
    idx = np.stack([np.concatenate([np.arange(K), K + np.sort(rng.choice(T - K, 20, replace=False))]) for _ in range(B)])
    idx_t = torch.tensor(idx, dtype=torch.int32, device=DEV)
    # head-major parents with padded rows: strided views
    def strided(t):
        big = torch.zeros(t.shape[0], t.shape[2], t.shape[1], t.shape[3] + 16, dtype=t.dtype, device=DEV)
        big[..., : t.shape[3]] = t.transpose(1, 2)
        return big.transpose(1, 2)[..., : t.shape[3]]
    qs, ks, vs = strided(q), strided(k), strided(v)
    P = 100
    kc = torch.zeros(B, Hkv, P + K + 5, D, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    qo, ko, vo = ds.ds_rope_gather(qs, ks, vs, idx_t, P, 10000.0, k_cache=kc, v_cache=vc, cache_row0=P, n_append=K)
    torch.cuda.synchronize()
    rq, rk, rv = oracle.rope_gather(f(q), f(k), f(v), idx, P, 10000.0)
    _close(qo, rq)
    _close(ko, rk)
    assert torch.equal(kc[:, :, P:P + K], ko[:, :, :K]) and torch.equal(vc[:, :, P:P + K], vo[:, :, :K])
    assert (kc[:, :, :P] == 0).all() and (kc[:, :, P + K:] == 0).all() and (vc[:, :, P + K:] == 0).all()


def test_pipeline_rope_then_pruned_attention_matches_oracle_pipeline():
    """Un-rotated projections -> ds_rope_gather -> ds_attn_pruned on the compact buffers, against the same
    two steps of the oracle.  The prefix cache holds K rotated with positions 0..P-1 (appended block by block
    in a real run; here rotated by the oracle's routine applied to the prefix as a 'tail' at offset 0)."""
    B, Hq, Hkv, D, P, T, K, w = 2, 8, 2, 128, 384, 512, 32, 64
    q, k, v, x = _raw(B, Hq, Hkv, T, D, seed=9)
    cfg = wl.StepConfig("t", B=B, Hq=Hq, Hkv=Hkv, D=D, P=P, gen=T, K=K, w=w, keep_last=True, dtype="bf16", V=8,
                        spike_p=0, seed=10)
    pre = wl.attention_inputs(cfg, device=DEV)
    idx = ds.retained_indices(T, K, 0, w)
    idx_t = torch.tensor(idx, dtype=torch.int32, device=DEV)
    # prefix cache: rotate the raw prefix keys with positions 0..P-1 on the GPU as well
    allp = torch.arange(P, dtype=torch.int32, device=DEV)
    _, kpre_rot, vpre = ds.ds_rope_gather(pre["k_pre"][:, :1].expand(-1, Hq, -1, -1).contiguous(), pre["k_pre"], pre["v_pre"],
                                          allp, 0, 10000.0)
    qo, ko, vo = ds.ds_rope_gather(q, k, v, idx_t, P, 10000.0)
    scale = 1 / math.sqrt(D)
    out = ds.ds_attn_pruned(qo, ko, vo, kpre_rot, vpre, torch.arange(len(idx), dtype=torch.int32, device=DEV), scale)
    torch.cuda.synchronize()
    # oracle pipeline in float64 on the same raw inputs (its rotated tensors are not rounded to bf16)
    _, rkpre, rvpre = oracle.rope_gather(f(pre["k_pre"][:, :1].expand(-1, Hq, -1, -1)), f(pre["k_pre"]), f(pre["v_pre"]),
                                         np.arange(P), 0, 10000.0)
    rq, rk, rv = oracle.rope_gather(f(q), f(k), f(v), np.asarray(idx), P, 10000.0)
    ref = oracle.attn(rq, rk, rv, rkpre, rvpre, np.arange(len(idx)), scale)
    err = np.abs(f(out) - ref).max()
    assert err <= 1e-2 and err <= 6e-3, err


def test_argument_errors_and_bad_index_flag():
    q, k, v, _ = _raw(1, 2, 2, 64, 64, seed=2)
    idx = torch.tensor([0, 1, 99], dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ds.ds_rope_gather(q, k, v, idx, 0, status=status)
    assert ds.ds_read_status(status) & ds.DS_DEV_INDEX
    with pytest.raises(ds.DsError):
        ds.ds_rope_gather(q, k, v, idx[:2], 0, rope_theta=0.5)
    with pytest.raises(ds.DsError):
        ds.ds_rope_gather(q[..., :40], k[..., :40], v[..., :40], idx[:2], 0)     # D not a multiple of 16
