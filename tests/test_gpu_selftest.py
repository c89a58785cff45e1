"""The bounded on-chip wait runs out cleanly.

Every mbarrier wait inside the tensor-core kernels polls a limited number of times; on expiry the kernel
raises DS_DEV_TIMEOUT in the status word and the CTA leaves in order.  ds_selftest_bounded_wait runs that
same wait function in a one-warp kernel on a barrier nobody arrives on, with a small poll limit, so the
expiry path is exercised without starving a barrier inside a real kernel.  The test checks the status bit,
that the barrier still works afterwards, and that the GPU serves ordinary calls right after."""
import numpy as np
import pytest
import torch

import oracle
import paper_2601_17917_b200 as ds

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("limit", [1, 64, 1024, 4096])
def test_wait_on_a_barrier_nobody_arrives_on_gives_up_and_reports(limit):
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    report = torch.full((3,), -1, dtype=torch.int32, device=DEV)
    ds.ds_selftest_bounded_wait(limit, status, report)
    torch.cuda.synchronize()
    assert ds.ds_read_status(status) == ds.DS_DEV_TIMEOUT
    assert report.tolist() == [1, 1, 1]          # gave up, flagged, and the barrier completed a phase afterwards
    # the bit is sticky and OR-ed: a second run leaves other bits alone
    status.fill_(ds.DS_DEV_INDEX)
    ds.ds_selftest_bounded_wait(limit, status, None)
    assert ds.ds_read_status(status) == ds.DS_DEV_INDEX | ds.DS_DEV_TIMEOUT
    # the context is healthy: an ordinary call right behind it gives the oracle's answer
    z = torch.randn(4, 1000, generator=torch.Generator().manual_seed(limit)).to(DEV)
    conf, tok = ds.ds_confidence(z)
    rc, rt = oracle.confidence(z.cpu().numpy())
    assert (tok.cpu().numpy() == rt).all() and np.abs(conf.cpu().numpy() - rc).max() < 2e-5


def test_selftest_refuses_limits_outside_its_range():
    for limit in (0, 1 << 17):
        with pytest.raises(ds.DsError) as e:
            ds.ds_selftest_bounded_wait(limit)
        assert e.value.code == ds.DS_ERR_INVALID_ARG
