"""ds_confidence_static: the entry point that allocates nothing.

Some users of this library cannot allocate device memory at the point where they call it (code that
runs inside another framework's memory plan, a plugin whose host forbids allocation after start-up),
so they cannot provide the workspace ds_confidence asks for.  ds_confidence_static keeps that scratch
in a fixed array inside the library instead.  It runs the same kernel, so its results must equal those
of ds_confidence on the same logits, and the CPU oracle's: token ids bit for bit, confidences within the
tolerance the other confidence tests use.  The array is shared by all calls and keeps the last call's
contents, so the check is made on two calls in a row, the second on different logits.  The claim that sets
this entry point apart -- the call allocates nothing -- is checked too: the device's free memory and torch's
allocator counters are the same before and after it.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test.  It passes on its own in a fresh process as well as after the others.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2601_17917_b200 as ds

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CONF_TOL = 2e-5      # the confidence kernel's own bound in tests/test_gpu_confidence.py


def _logits(rows, V, seed, dtype):
    g = torch.Generator(device="cpu").manual_seed(seed)
    z = 2.0 * torch.randn(rows, V, generator=g)
    z[torch.arange(rows), torch.randint(0, V, (rows,), generator=g)] += 8.0
    return z.to(dtype).to(DEV)


@pytest.mark.parametrize("rows,V,dtype", [(32, 126464, torch.bfloat16), (5, 40001, torch.float32),
                                          (700, 8192, torch.bfloat16)])
def test_static_scratch_matches_workspace_entry_point_twice(rows, V, dtype):
    conf = torch.empty(rows, dtype=torch.float32, device=DEV)
    tok = torch.empty(rows, dtype=torch.int32, device=DEV)
    for call in range(2):                       # the second call meets the scratch the first one left
        z = _logits(rows, V, seed=17 * rows + call, dtype=dtype)
        want_conf, want_tok = ds.ds_confidence(z)
        conf.fill_(-1.0)
        tok.fill_(-1)
        torch.cuda.synchronize()
        if call == 1:       # the first call on a device looks up the scratch address; from then on nothing moves
            free0 = torch.cuda.mem_get_info()[0]
            alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
            n_alloc0 = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
        ds.ds_confidence_static(z, conf, tok)
        torch.cuda.synchronize()
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free0, "device memory in use changed across the call"
            assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
            assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == n_alloc0
        assert torch.equal(tok, want_tok), f"call {call}: token ids differ"
        assert (conf - want_conf).abs().max().item() <= CONF_TOL, f"call {call}"
        oc, ot = oracle.confidence(z.float().cpu().numpy())
        assert (tok.cpu().numpy() == ot).all(), f"call {call}: token ids differ from the oracle's"
        assert np.abs(conf.cpu().numpy().astype(np.float64) - oc).max() <= CONF_TOL, f"call {call}"


def test_static_scratch_with_a_row_list_leaves_other_rows_alone():
    rows, V = 48, 50000
    z = _logits(rows, V, seed=5, dtype=torch.bfloat16)
    listed = torch.tensor([1, 7, 8, 40], dtype=torch.int32, device=DEV)
    want_conf, want_tok = ds.ds_confidence(z)
    conf = torch.full((rows,), -1.0, dtype=torch.float32, device=DEV)
    tok = torch.full((rows,), -1, dtype=torch.int32, device=DEV)
    ds.ds_confidence_static(z, conf, tok, row_list=listed)
    torch.cuda.synchronize()
    li = listed.long()
    assert torch.equal(tok[li], want_tok[li])
    assert (conf[li] - want_conf[li]).abs().max().item() <= CONF_TOL
    rest = torch.ones(rows, dtype=torch.bool, device=DEV)
    rest[li] = False
    assert (tok[rest] == -1).all() and (conf[rest] == -1.0).all()
    # a list with no entry touches nothing (it is not the same as "no list", which means every row)
    conf.fill_(-2.0)
    tok.fill_(-2)
    n0 = ds.ds_launch_count()
    ds.ds_confidence_static(z, conf, tok, row_list=listed[:0])
    torch.cuda.synchronize()
    assert ds.ds_launch_count() == n0 and (tok == -2).all() and (conf == -2.0).all()


def test_more_rows_than_the_fixed_scratch_serves_is_refused():
    rows = ds.DS_CONFIDENCE_STATIC_MAX_ROWS + 1
    z = torch.zeros(rows, 64, dtype=torch.bfloat16, device=DEV)
    conf = torch.empty(rows, dtype=torch.float32, device=DEV)
    tok = torch.empty(rows, dtype=torch.int32, device=DEV)
    with pytest.raises(ds.DsError) as e:
        ds.ds_confidence_static(z, conf, tok)
    assert e.value.code == ds.DS_ERR_STATIC_LIMIT
    assert "fixed scratch" in ds.ds_strerror(e.value.code)
    # the limit itself is served
    ds.ds_confidence_static(z[:-1], conf, tok)
    torch.cuda.synchronize()
    assert (tok[:-1] == 0).all() and (conf[:-1] - 1.0 / 64).abs().max().item() <= CONF_TOL
