"""prm_step inside a CUDA graph.  With unchanged pointers a step only launches kernels (and, for
the streaming tall kernel, one memset), so a K-step period can be captured once and replayed:
the replay must give the bits of the eager steps.  The first step on a handle uploads the
pointer tables and encodes tensor maps and therefore stays outside the capture."""

import numpy as np
import pytest
import torch

from paper_2608_20818_b200 import binding as B
from tests import util as U

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("tall_kernel", [0, 2])
def test_a_period_of_steps_replays_from_a_graph(tall_kernel):
    shapes = [(256, 1024), (1024, 256), (256, 1024), (1024, 2560), (40, 24), (2048, 512)]
    K = 3
    kw = dict(beta=0.95, nesterov=True, lr=5e-3, wd=0.01, tall_kernel=tall_kernel)
    W, G, M = U.make_inputs(shapes, 61, "bf16", grad_std=1e-3, mom_std=1e-3)

    def fresh():
        return [w.cuda() for w in W], [g.cuda() for g in G], [m.cuda() for m in M]

    # eager: warm-up step 0 (refresh), then steps 1, 2, 3 (row, row, refresh)
    opt = B.PeriodicRowwiseMuon(shapes, K, **kw)
    w, g, m = fresh()
    for t in range(0, 4):
        opt.step(w, g, m, t)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    want_w, want_m = [x.clone() for x in w], [x.clone() for x in m]
    opt.close()

    # the same with steps 1..3 captured and replayed
    opt = B.PeriodicRowwiseMuon(shapes, K, **kw)
    w, g, m = fresh()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        opt.step(w, g, m, 0)                  # uploads tables and maps: outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for t in range(1, 4):
            opt.step(w, g, m, t)
    # capture runs nothing: the tensors still hold the state after step 0
    graph.replay()
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    for i, s in enumerate(shapes):
        assert torch.equal(w[i], want_w[i]), s
        assert torch.equal(m[i], want_m[i]), s
    opt.close()
