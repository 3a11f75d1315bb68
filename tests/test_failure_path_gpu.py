"""The device-side failure path without faulting anything: a bounded wait
runs out, the status word reports it once, and the context keeps working."""

import pytest
import torch

from paper_2608_20818_b200 import binding as B

pytestmark = pytest.mark.gpu


def test_bounded_wait_times_out_and_context_survives():
    shapes = [(256, 512)]
    opt = B.PeriodicRowwiseMuon(shapes, 2)
    w = torch.zeros(shapes[0], dtype=torch.bfloat16, device="cuda")
    g = torch.full(shapes[0], 1e-3, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(shapes[0], device="cuda")
    assert opt.status() == B.PRM_OK
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.prm_selftest_timeout(opt.h, 20.0, torch.cuda.current_stream().cuda_stream)
    t1.record()
    torch.cuda.synchronize()
    assert 15.0 <= t0.elapsed_time(t1) <= 500.0        # it waited its 20 ms and then returned
    assert opt.status() == B.PRM_ERR_DEVICE_TIMEOUT
    assert "wait" in B.prm_last_error(opt.h)
    assert opt.status() == B.PRM_OK                    # reported once, then cleared
    # the context is intact: a refresh and a row step still run and report no error
    opt.step([w], [g], [m], 0)
    opt.step([w], [g], [m], 1)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    assert torch.isfinite(w.float()).all() and float(w.float().abs().max()) > 0
    with pytest.raises(B.PrmError):
        B.prm_selftest_timeout(opt.h, 5000.0)
    opt.close()
