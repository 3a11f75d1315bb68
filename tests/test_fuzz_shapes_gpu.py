"""Seeded random shapes (ragged, tiny, tall, wide, unaligned column counts)
through both branches and both NS5 modes against the oracle."""

import numpy as np
import pytest

from oracle import prm_oracle as O
from tests import util as U

pytestmark = pytest.mark.gpu


def _shapes(seed, n):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        kind = rng.integers(0, 4)
        if kind == 0:
            out.append((int(rng.integers(1, 40)), int(rng.integers(1, 700))))
        elif kind == 1:
            out.append((int(rng.integers(1, 700)), int(rng.integers(1, 40))))
        elif kind == 2:
            out.append((int(rng.integers(200, 600)), int(rng.integers(200, 600))))
        else:
            out.append((8 * int(rng.integers(1, 60)), 8 * int(rng.integers(1, 90))))
    return out


@pytest.mark.parametrize("seed", [1, 2, 3])
@pytest.mark.parametrize("io", ["fp32", "bf16"])
def test_row_step_random_shapes(seed, io):
    shapes = _shapes(seed, 12)
    cfg = U.oracle_cfg(K=4, nesterov=bool(seed & 1), lr=5e-3, wd=0.01)
    W, G, M = U.make_inputs(shapes, 70 + seed, io)
    Wg, Mg = U.gpu_step(shapes, W, G, M, 1, cfg, io, True)
    for i, sh in enumerate(shapes):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 1, cfg)
        U.assert_elementwise(Mg[i], Mr, False, f"momentum {sh}")
        U.assert_elementwise(Wg[i], Wr, io == "bf16", f"param {sh}")


@pytest.mark.parametrize("seed", [4, 5])
@pytest.mark.parametrize("check_mode", [True, False])
def test_refresh_random_shapes(seed, check_mode):
    shapes = [s for s in _shapes(seed, 10) if min(s) >= 16]
    cfg = U.oracle_cfg(K=1, nesterov=True, lr=1.0, wd=0.0)          # default shape scale
    W, G, M = U.make_inputs(shapes, 80 + seed, "bf16", grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()
    Wg, Mg = U.gpu_step(shapes, W, G, M, 0, cfg, "bf16", check_mode)
    for i, sh in enumerate(shapes):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
        U.assert_elementwise(Mg[i], Mr, False, f"momentum {sh}")
        err = U.rel_fro(Wg[i], Wr)
        assert err <= (4e-3 if check_mode else 2e-2), (sh, err)     # bf16 store: 2^-9


@pytest.mark.parametrize("seed", [6, 7])
def test_refresh_split_input_random_large_shapes(seed):
    """Seeded ragged shapes on both sides of 1024 padded rows, wide and tall, column counts that
    are and are not multiples of 8, with the two-plane NS5 input: every one within 2e-2."""
    rng = np.random.default_rng(seed)
    shapes = []
    for _ in range(5):
        r = int(rng.integers(700, 1500))
        c = int(rng.integers(r, 2600))
        if rng.integers(0, 2):
            c = 8 * (c // 8)
        shapes.append((r, c) if rng.integers(0, 2) else (c, r))
    cfg = U.oracle_cfg(K=1, nesterov=bool(seed & 1), lr=1.0, wd=0.0)
    W, G, M = U.make_inputs(shapes, 90 + seed, "bf16", grad_std=1e-3, mom_std=1e-3)
    for w in W:
        w.zero_()
    Wg, Mg = U.gpu_step(shapes, W, G, M, 0, cfg, "bf16", False, split_input=True)
    for i, sh in enumerate(shapes):
        Wr, Mr = O.step_matrix(U.to_np64(W[i]), U.to_np64(G[i]), U.to_np64(M[i]), 0, cfg)
        U.assert_elementwise(Mg[i], Mr, False, f"momentum {sh}")
        err = U.rel_fro(Wg[i], Wr)
        assert err <= 2e-2, (sh, err)
