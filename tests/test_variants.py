"""The ablation variants of the paper's Table 3(a) (vanilla Muon = K 1,
RowNorm at every step, gamma = 1, scalar-controlled = gamma on both branches):
oracle pins on CPU, GPU parity against the oracle."""

import numpy as np
import pytest

from oracle import prm_oracle as O
from tests import util as U


def _case(rng, m, n):
    return rng.standard_normal((m, n)) * 0.02, rng.standard_normal((m, n)), rng.standard_normal((m, n)) * 0.1


def test_oracle_variants_reduce_to_the_base_rules():
    rng = np.random.default_rng(31)
    W, G, M = _case(rng, 6, 10)
    base = dict(K=3, nesterov=True, lr=1e-2, wd=0.0)
    # RowNorm at every step: a refresh index behaves like any other step
    a, _ = O.step_matrix(W, G, M, 3, O.OracleConfig(no_refresh=True, **base))
    b, _ = O.step_matrix(W, G, M, 1, O.OracleConfig(**base))
    np.testing.assert_array_equal(a, b)
    # scalar-controlled: gamma multiplies the NS5 direction as well
    c, _ = O.step_matrix(W, G, M, 3, O.OracleConfig(gamma=0.15, gamma_ns=0.15, **base))
    d, _ = O.step_matrix(W, G, M, 3, O.OracleConfig(gamma=0.15, **base))
    np.testing.assert_allclose(W - c, 0.15 * (W - d), rtol=1e-12)
    # and leaves the row branch alone
    e, _ = O.step_matrix(W, G, M, 1, O.OracleConfig(gamma=0.15, gamma_ns=0.15, **base))
    np.testing.assert_array_equal(e, O.step_matrix(W, G, M, 1, O.OracleConfig(gamma=0.15, **base))[0])
    # vanilla Muon: K = 1 refreshes at every step
    assert all(O.is_refresh(t, 1) for t in range(4))


@pytest.mark.gpu
@pytest.mark.parametrize("variant", ["vanilla", "rownorm_only", "gamma_one", "scalar_controlled"])
def test_variants_on_gpu(variant):
    kw = dict(K=3, nesterov=True, lr=5e-3, wd=0.01, gamma=0.15)
    if variant == "vanilla":
        kw["K"] = 1
    elif variant == "rownorm_only":
        kw["no_refresh"] = True
    elif variant == "gamma_one":
        kw["gamma"] = 1.0
    else:
        kw["gamma_ns"] = 0.15
    cfg = U.oracle_cfg(**kw)
    shapes = [(256, 512), (512, 256)]
    W, G, M = U.make_inputs(shapes, 41, "fp32", grad_std=1e-3, mom_std=1e-3)
    for t in (3, 4):                       # a refresh index of K = 3 and a row-step index
        Wg, Mg = U.gpu_step(shapes, W, G, M, t, cfg, "fp32", True)
        for i in range(2):
            Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), t, cfg)
            U.assert_elementwise(Mg[i], Mr, False, f"momentum {variant} t={t}")
            U.assert_elementwise(Wg[i], Wr, False, f"param {variant} t={t}", rtol=2e-5)
