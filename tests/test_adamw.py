"""AdamW for the parameters outside the Muon set (Algorithm 1 line 11):
oracle pinned to torch.optim.AdamW on CPU, CUDA kernel against the oracle."""

import numpy as np
import pytest
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B

HP = dict(lr=1e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.01)   # the paper's auxiliary AdamW group


def test_oracle_adamw_matches_torch():
    g = torch.Generator().manual_seed(3)
    p0 = torch.randn(37, 5, generator=g, dtype=torch.float64)
    p = torch.nn.Parameter(p0.clone())
    opt = torch.optim.AdamW([p], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]), eps=HP["eps"], weight_decay=HP["wd"])
    po, m, v = p0.numpy().copy(), np.zeros((37, 5)), np.zeros((37, 5))
    for t in range(1, 6):
        grad = torch.randn(37, 5, generator=g, dtype=torch.float64)
        p.grad = grad.clone()
        opt.step()
        po, m, v = O.adamw_step(po, grad.numpy(), m, v, t, **HP)
        np.testing.assert_allclose(po, p.detach().numpy(), rtol=1e-12, atol=1e-15)
    # first step from zero moments moves every entry by lr*sign(g) (bias correction), up to eps
    p1, _, _ = O.adamw_step(np.zeros(4), np.array([3.0, -2.0, 0.5, -1e-3]), np.zeros(4), np.zeros(4), 1, lr=0.1,
                            beta1=0.9, beta2=0.95, eps=0.0, wd=0.0)
    np.testing.assert_allclose(p1, [-0.1, 0.1, -0.1, 0.1], rtol=1e-12)


@pytest.mark.gpu
@pytest.mark.parametrize("io", ["fp32", "bf16"])
def test_adamw_kernel_against_oracle(io):
    dt = torch.float32 if io == "fp32" else torch.bfloat16
    g = torch.Generator().manual_seed(7)
    shapes = [(1,), (7,), (1216,), (4096,), (3, 5, 7), (100003,), (0,)] + [(64 + k,) for k in range(60)]
    P = [(torch.randn(s, generator=g) * 0.1).to(dt) for s in shapes]
    M = [torch.zeros(s) for s in shapes]
    V = [torch.zeros(s) for s in shapes]
    Pd = [x.cuda() for x in P]
    Md = [x.cuda() for x in M]
    Vd = [x.cuda() for x in V]
    Pr = [x.double().numpy() for x in P]
    Mr = [x.double().numpy() for x in M]
    Vr = [x.double().numpy() for x in V]
    for t in range(1, 4):
        G = [(torch.randn(s, generator=g) * 1e-2).to(dt) for s in shapes]
        B.prm_adamw_step(Pd, [x.cuda() for x in G], Md, Vd, t, **HP)
        torch.cuda.synchronize()
        for i in range(len(shapes)):
            # the oracle restarts from the GPU's stored parameters: one rounding per step is compared
            p_in = Pr[i] if io == "fp32" else P[i].double().numpy()
            Pr[i], Mr[i], Vr[i] = O.adamw_step(p_in, G[i].double().numpy(), Mr[i], Vr[i], t, **HP)
            got = Pd[i].double().cpu().numpy()
            tol = 1e-5 * np.abs(Pr[i]) + 1e-9 + (np.abs(Pr[i]) * 2.0 ** -8 if io == "bf16" else 0.0)
            assert np.all(np.abs(got - Pr[i]) <= tol), (shapes[i], t)
            # moments: 1e-5 relative, plus 1e-6 of the tensor's rms where beta*m and (1-beta)*g cancel
            for got_s, ref_s in ((Md[i], Mr[i]), (Vd[i], Vr[i])):
                if ref_s.size:
                    rms = float(np.sqrt(np.mean(ref_s * ref_s)))
                    np.testing.assert_allclose(got_s.double().cpu().numpy(), ref_s, rtol=1e-5, atol=1e-6 * rms + 1e-30)
            P[i] = Pd[i].cpu()
            if io == "fp32":
                Pr[i] = got.copy()
