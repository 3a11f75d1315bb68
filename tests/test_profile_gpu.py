"""prm_profile / prm_profile_read: per-class device times and launch counts
add up to what the handle launched."""

import pytest
import torch

from paper_2608_20818_b200 import binding as B

pytestmark = pytest.mark.gpu


def test_profile_classes_account_for_every_launch():
    shapes = [(256, 512), (512, 256), (256, 512), (256, 256)]
    opt = B.PeriodicRowwiseMuon(shapes, 2, nesterov=True)
    w = [torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    g = [torch.full(s, 1e-3, dtype=torch.bfloat16, device="cuda") + 1e-4 * torch.randn(s, device="cuda").bfloat16()
         for s in shapes]
    m = [torch.zeros(s, device="cuda") for s in shapes]
    opt.step(w, g, m, 0)                      # not profiled
    before = opt.launch_count()
    opt.profile(True)
    opt.step(w, g, m, 1)                      # row step
    opt.step(w, g, m, 2)                      # refresh
    prof = opt.profile_read()
    opt.profile(False)
    assert sum(n for (_, n) in prof.values()) == opt.launch_count() - before
    assert prof["row_wide"][1] == 2 and prof["row_tall"][1] == 3          # 2 wide groups, 3 kernels for the tall one
    assert prof["prepass"][1] == 2 * 3                                      # 3 groups, 2 kernels each
    assert prof["gram"][1] == prof["poly"][1] == 5 * 3
    assert prof["update"][1] == 4 * 3 and prof["update_final"][1] == 3
    assert all(ms > 0 for (ms, n) in prof.values() if n > 0)
    again = opt.profile_read()
    assert all(n == 0 and ms == 0 for (ms, n) in again.values())
    assert opt.status() == B.PRM_OK
    opt.close()
