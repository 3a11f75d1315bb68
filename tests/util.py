"""Shared helpers of the GPU parity tests (no optimizer arithmetic here)."""

import numpy as np
import torch

from oracle import prm_oracle as O
from paper_2608_20818_b200 import binding as B

GUARD = 64  # elements of canary on both sides of every caller buffer


def to_np64(t):
    return t.detach().float().cpu().double().numpy()


class Guarded:
    """A device tensor embedded in a larger buffer with canary margins."""

    def __init__(self, src: torch.Tensor, device="cuda"):
        n = src.numel()
        self.canary = 1.0 if src.dtype != torch.bfloat16 else 1.0
        self.buf = torch.full((n + 2 * GUARD,), 12345.0, dtype=src.dtype, device=device)
        self.t = self.buf[GUARD:GUARD + n].view(src.shape)
        self.t.copy_(src)
        assert self.t.data_ptr() % 16 == 0

    def intact(self):
        n = self.t.numel()
        return bool((self.buf[:GUARD] == 12345.0).all() and (self.buf[GUARD + n:] == 12345.0).all())


def io_torch_dtype(io):
    return torch.float32 if io == "fp32" else torch.bfloat16


def make_inputs(shapes, seed, io, grad_std=1.0, mom_std=0.1, heavy=False):
    """Seeded CPU tensors in storage dtypes: params, grads, momentum."""
    g = torch.Generator().manual_seed(seed)
    dt = io_torch_dtype(io)
    W, G, M = [], [], []
    for (m, n) in shapes:
        W.append((torch.randn(m, n, generator=g) * 0.02).to(torch.bfloat16).to(dt))
        x = torch.randn(m, n, generator=g)
        if heavy:
            x = x * torch.exp(torch.randn(m, 1, generator=g))
        G.append((x * grad_std).to(dt))
        M.append(torch.randn(m, n, generator=g) * mom_std)
    return W, G, M


def structured_grads(kind, shapes, seed=5, scale=1e-3):
    """Seeded bf16 gradient matrices with a chosen spectrum: "heavy_rows"
    (log-normal row scales, as in the 15B-class configuration),
    "low_rank_mild" (rank-8 signal at the level of the noise), "spiked" (rank-8
    signal two orders of magnitude above the noise floor), "gauss"."""
    g = torch.Generator().manual_seed(seed)
    out = []
    for (m, n) in shapes:
        if kind == "heavy_rows":
            x = torch.randn(m, n, generator=g) * torch.exp(torch.randn(m, 1, generator=g))
        elif kind == "low_rank_mild":
            x = torch.randn(m, 8, generator=g) @ torch.randn(8, n, generator=g) / 8 ** 0.5 + torch.randn(m, n, generator=g)
        elif kind == "spiked":
            x = torch.randn(m, 8, generator=g) @ torch.randn(8, n, generator=g) + 0.1 * torch.randn(m, n, generator=g)
        elif kind == "gauss":
            x = torch.randn(m, n, generator=g)
        else:
            raise ValueError(kind)
        out.append((x * scale).to(torch.bfloat16))
    return out


def oracle_cfg(**kw):
    return O.OracleConfig(**kw)


def gpu_step(shapes, W, G, M, t, cfg, io, check_mode, ns_workspace_bytes=None, steps=1, grads_fn=None,
             gram_span=2, tall_kernel=0, launches=None, split_input=False, wide_kernel=0):
    """Run `steps` steps from step index t on the GPU through the C ABI.
    Returns (W_new list, M_new list) as fp64 numpy, after checking canaries."""
    opt = B.PeriodicRowwiseMuon(shapes, cfg.K, cfg.beta, cfg.nesterov, cfg.lr, cfg.wd, gamma=cfg.gamma,
                                eps_row=cfg.eps_row, eps_ns=cfg.eps_ns, scale_mode=cfg.scale_mode,
                                io_dtype=io, check_mode=check_mode, ns_workspace_bytes=ns_workspace_bytes,
                                gamma_ns=cfg.gamma_ns, no_refresh=cfg.no_refresh, gram_span=gram_span,
                                tall_kernel=tall_kernel, split_input=split_input, wide_kernel=wide_kernel)
    gw = [Guarded(w) for w in W]
    gg = [Guarded(g) for g in G]
    gm = [Guarded(m) for m in M]
    for k in range(steps):
        if grads_fn is not None and k > 0:
            for dst, src in zip(gg, grads_fn(t + k)):
                dst.t.copy_(src)
        opt.step([x.t for x in gw], [x.t for x in gg], [x.t for x in gm], t + k)
    torch.cuda.synchronize()
    assert opt.status() == B.PRM_OK
    for x in gw + gg + gm:
        assert x.intact(), "write outside a caller buffer"
    for g_dev, g_host in zip(gg, G):
        if grads_fn is None:
            assert torch.equal(g_dev.t.cpu(), g_host), "gradients were modified"
    out = [to_np64(x.t) for x in gw], [to_np64(x.t) for x in gm]
    if launches is not None:
        launches.append(opt.launch_count())
    opt.close()
    return out


def bf16_half_ulp(ref):
    a = np.abs(ref)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    return np.where(a > 0, 2.0 ** (e - 8), 0.0)


def assert_elementwise(got, ref, io_is_bf16, what, rtol=1e-5):
    """|got-ref| <= rtol*|ref| + 1e-6*rms(ref row) (+ half a bf16 ulp when the
    value was stored as bf16)."""
    rms = np.sqrt(np.mean(ref * ref, axis=1, keepdims=True))
    tol = rtol * np.abs(ref) + 1e-6 * rms + 1e-30
    if io_is_bf16:
        tol = tol + bf16_half_ulp(ref) * (1 + 1e-3)
    bad = np.abs(got - ref) > tol
    assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} elements off, worst {np.abs(got - ref).max():.3e}"


def rel_fro(got, ref):
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
