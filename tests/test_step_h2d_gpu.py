"""prm_step_h2d: gradients copied from pinned host memory on the handle's copy
stream give bit-identical results to prm_step on resident gradients, for both
branches and over several consecutive steps."""

import pytest
import torch

from paper_2608_20818_b200 import binding as B
from tests import util as U

pytestmark = pytest.mark.gpu


def test_step_h2d_matches_step():
    shapes = [(256, 512), (512, 256), (256, 512), (64, 4104), (300, 264)]
    K = 2
    W, G0, M = U.make_inputs(shapes, 51, "bf16", grad_std=1e-3, mom_std=1e-3)
    gens = [[(torch.randn(s, generator=torch.Generator().manual_seed(100 * t + i)) * 1e-3).to(torch.bfloat16)
             for i, s in enumerate(shapes)] for t in range(4)]

    def run(h2d):
        opt = B.PeriodicRowwiseMuon(shapes, K, 0.95, True, 5e-3, 0.01)
        w = [x.cuda() for x in W]
        m = [x.cuda() for x in M]
        g = [torch.zeros_like(x, device="cuda") for x in G0]
        host = [torch.empty_like(x).pin_memory() for x in G0]
        for t in range(4):
            if h2d:
                torch.cuda.synchronize()          # the host buffers are free to be rewritten
                for hb, src in zip(host, gens[t]):
                    hb.copy_(src)
                opt.step_h2d(w, g, host, m, t)
            else:
                for gb, src in zip(g, gens[t]):
                    gb.copy_(src)
                opt.step(w, g, m, t)
        torch.cuda.synchronize()
        assert opt.status() == B.PRM_OK
        opt.close()
        return [x.cpu() for x in w], [x.cpu() for x in m], [x.cpu() for x in g]

    a, b = run(False), run(True)
    for k in range(3):
        for x, y in zip(a[k], b[k]):
            assert torch.equal(x, y)
