"""GPU parity of ds_confidence (Eq. 4) against the CPU oracle, through the C ABI.

Tolerances: token index bit-exact (lowest index among equal maxima);
confidence within 1e-3 absolute (the stated bar), and within 2e-5 as this
kernel's own bound (fp32 accumulation of ex2.approx terms, relative error
about 2e-6 on the sum)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2601_17917_b200 as ds
from paper_2601_17917_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CONF_BAR = 1e-3
CONF_OWN = 2e-5


def _check(z_dev, conf, tok, rows=None):
    z = z_dev.float().cpu().numpy()
    rc, rt = oracle.confidence(z)
    conf, tok = conf.cpu().numpy(), tok.cpu().numpy()
    sel = np.arange(z.shape[0]) if rows is None else np.asarray(rows, dtype=np.int64)
    assert (tok[sel] == rt[sel]).all(), "argmax mismatch"
    err = np.abs(conf[sel].astype(np.float64) - rc[sel]).max() if len(sel) else 0.0
    assert err <= CONF_BAR and err <= CONF_OWN, err
    return err


@pytest.mark.parametrize("name", ["tiny", "llada1", "llada8x32", "dream16", "long32-w64"])
def test_config_logits_match_oracle(name):
    cfg = wl.CONFIGS[name]
    z = wl.logits(cfg, device=DEV)
    conf, tok = ds.ds_confidence(z)
    torch.cuda.synchronize()
    _check(z, conf, tok)
    # same distribution with spikes that spread the confidences over (0, 1)
    if cfg.rows <= 512:
        z2 = wl.logits(cfg, device=DEV, step=1, spike_range=(12.0, 20.0))
        conf2, tok2 = ds.ds_confidence(z2)
        _check(z2, conf2, tok2)
        assert conf2.max().item() > 0.5


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1, 2, 7, 8, 9, 63, 1000, 4097, 40000])
def test_ragged_vocab_and_misaligned_rows(dtype, V):
    g = torch.Generator(device="cpu").manual_seed(V)
    rows, ld = 5, V + 3
    buf = (2 * torch.randn(rows * ld + 8, generator=g)).to(dtype).to(DEV)
    for off in (0, 1, 3):   # base pointer not 16-byte aligned, row stride not a multiple of a vector
        z = buf[off: off + rows * ld].view(rows, ld)[:, :V]
        conf, tok = ds.ds_confidence(z)
        _check(z, conf, tok)


def test_ties_resolve_to_lowest_index():
    V = 126464
    z = torch.full((4, V), -3.0, dtype=torch.bfloat16, device=DEV)
    z[0, [70000, 5, 126463]] = 9.0          # same vector-aligned max in three places
    z[1, [126463, 126462]] = 2.5
    z[2, 8] = 1.0
    z[2, 7] = 1.0
    conf, tok = ds.ds_confidence(z)
    assert tok.tolist() == [5, 126462, 7, 0]
    _check(z, conf, tok)
    # literal workload rows: bf16 N(0, 2^2) rows repeat their top value often
    cfg = wl.CONFIGS["llada1"]
    z = wl.logits(cfg, device=DEV)
    zf = z.float()
    n_tied = int(((zf == zf.max(1, keepdim=True).values).sum(1) > 1).sum())
    conf, tok = ds.ds_confidence(z)
    _check(z, conf, tok)
    assert n_tied >= 0


def test_extreme_values():
    z = torch.zeros((4, 5000), dtype=torch.float32, device=DEV)
    z[0, 123] = 1.0e4                        # exp underflows everywhere else: conf = 1
    z[1] = -1.0e4
    z[1, 4000] = -9990.0
    z[2, :] = float("-inf")
    z[2, 77] = 0.5                           # -inf entries contribute nothing
    z[3, 10] = 88.0
    z[3, 11] = 87.0
    conf, tok = ds.ds_confidence(z)
    assert tok.tolist() == [123, 4000, 77, 10]
    _check(z, conf, tok)
    assert abs(conf[0].item() - 1.0) < 1e-6 and abs(conf[2].item() - 1.0) < 1e-6


def test_row_list_and_split_rows():
    cfg = wl.CONFIGS["llada1"]
    z = wl.logits(cfg, device=DEV)
    rows = [0, 3, 4, 31]
    conf = torch.full((cfg.rows,), -1.0, device=DEV)
    tok = torch.full((cfg.rows,), -1, dtype=torch.int32, device=DEV)
    ds.ds_confidence(z, row_list=torch.tensor(rows, dtype=torch.int32, device=DEV), conf=conf, tok=tok)
    _check(z, conf, tok, rows)
    untouched = [r for r in range(cfg.rows) if r not in rows]
    assert (conf[untouched] == -1).all() and (tok[untouched] == -1).all()
    # a list with no entry touches nothing (no list at all would mean every row)
    conf.fill_(-2.0)
    tok.fill_(-2)
    n0 = ds.ds_launch_count()
    ds.ds_confidence(z, row_list=torch.empty(0, dtype=torch.int32, device=DEV), conf=conf, tok=tok)
    torch.cuda.synchronize()
    assert ds.ds_launch_count() == n0 and (conf == -2).all() and (tok == -2).all()
    # one row, widest split over CTAs
    conf1, tok1 = ds.ds_confidence(z[5:6])
    _check(z[5:6], conf1, tok1)
    # padded row stride
    zp = torch.zeros((8, cfg.V + 64), dtype=torch.bfloat16, device=DEV)
    zp[:, :cfg.V] = z[:8]
    c2, t2 = ds.ds_confidence(zp[:, :cfg.V])
    _check(z[:8], c2, t2)


def test_workspace_errors_and_determinism():
    cfg = wl.CONFIGS["llada1"]
    z = wl.logits(cfg, device=DEV)
    with pytest.raises(ds.DsError) as e:
        ds.ds_confidence(z, workspace=torch.empty(16, dtype=torch.uint8, device=DEV))
    assert e.value.code == ds.DS_ERR_WORKSPACE
    ws = torch.empty(ds.ds_confidence_workspace(cfg.rows, cfg.V, z.dtype), dtype=torch.uint8, device=DEV)
    first = None
    for _ in range(10):
        conf, tok = ds.ds_confidence(z, workspace=ws)
        cur = (conf.clone(), tok.clone())
        if first is None:
            first = cur
        assert torch.equal(cur[0], first[0]) and torch.equal(cur[1], first[1])   # bitwise repeatable


@pytest.mark.parametrize("V", [1000, 126464])
def test_listed_rows_with_the_count_on_the_device(V):
    # the rows still masked and their number live on the device (ds_unmask_select's masked_rows / masked_cnt)
    torch.manual_seed(5)
    rows = 96
    z = (torch.randn(rows, V, device=DEV) * 3).to(torch.bfloat16)
    lst = torch.tensor([3, 4, 17, 40, 41, 42, 90, 95, 1, 2], dtype=torch.int32, device=DEV)  # the last two: beyond the count
    for n in (8, 0, 3):
        conf = torch.full((rows,), -7.0, device=DEV)
        tok = torch.full((rows,), -7, dtype=torch.int32, device=DEV)
        cnt = torch.tensor([n], dtype=torch.int32, device=DEV)
        ds.ds_confidence_listed(z, lst, cnt, conf, tok)
        torch.cuda.synchronize()
        used = lst[:n].cpu().tolist()
        _check(z, conf, tok, rows=used)
        rest = sorted(set(range(rows)) - set(used))
        assert (conf[rest] == -7.0).all() and (tok[rest] == -7).all()
    # a count larger than the list is clamped to the list; a row number outside the matrix is skipped
    lst2 = torch.tensor([5, 6, 1000, -1], dtype=torch.int32, device=DEV)
    conf = torch.full((rows,), -7.0, device=DEV)
    tok = torch.full((rows,), -7, dtype=torch.int32, device=DEV)
    ds.ds_confidence_listed(z, lst2, torch.tensor([99], dtype=torch.int32, device=DEV), conf, tok)
    torch.cuda.synchronize()
    _check(z, conf, tok, rows=[5, 6])
    assert (conf[7:] == -7.0).all()
