"""Seeded synthetic workloads: shape sets and input tensors.

This module holds no arithmetic of the optimizer.  It only names the shape
sets of the five benchmark configurations and draws seeded random inputs with
their stated distributions, so that the CUDA path and the CPU oracle can be
fed identical bits.  The shape sets stand in for the paper's GPIC-trained
MMDiT gradients, which are not available: matrix kinds (attention qkv and
output, MLP up and down, adaLN modulation) follow the paper's model family,
dimensions follow the benchmark configurations.
"""

from __future__ import annotations

from dataclasses import dataclass, field

import torch

SEED_BASE = 20818 * 1000


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    d: int
    blocks: int
    K: int
    lr: float
    grad_std: float
    heavy_tail_rows: bool = False
    io_dtype: str = "bf16"         # "bf16" (bf16 params/grads) or "fp32"
    beta: float = 0.95
    nesterov: bool = True
    wd: float = 0.01
    gamma: float = 0.15
    shapes: tuple = field(default=())


def block_shapes(d: int):
    """Stored (rows, cols) of the five 2-D matrices of one transformer block:
    qkv, attention output, MLP up, MLP down (tall), adaLN modulation."""
    return [(d, 3 * d), (d, d), (d, 4 * d), (4 * d, d), (d, 6 * d)]


def dit_shapes(d: int, blocks: int):
    """Block-major list of stored shapes for a DiT-class shape set."""
    out = []
    for _ in range(blocks):
        out.extend(block_shapes(d))
    return out


def workload(config_id: int, blocks: int | None = None) -> Workload:
    """The benchmark configurations.  `blocks` overrides the block count (the
    blocks are identical and independent, so a reduced count is a strict
    subset of the same workload)."""
    if config_id == 1:
        return Workload("single-256x1024", 1, 0, 0, K=4, lr=5e-3, grad_std=1.0,
                        io_dtype="fp32", shapes=((256, 1024),))
    table = {
        2: ("dit-1.3b-class", 2048, 24, 5, 5e-3),
        3: ("dit-4b-class", 3072, 36, 5, 3e-3),
        4: ("dit-9b-class", 4096, 42, 5, 2.4e-3),
        5: ("dit-15b-class", 5120, 48, 5, 2.0e-3),
    }
    name, d, nb, K, lr = table[config_id]
    if blocks is not None:
        nb = blocks
    return Workload(name, config_id, d, nb, K=K, lr=lr, grad_std=1e-3,
                    heavy_tail_rows=(config_id == 5),
                    shapes=tuple(dit_shapes(d, nb)))


# Memory sizing of a shape set (no optimizer arithmetic): what the caller keeps
# resident per transformer block, and how many blocks a GPU can hold.
RESERVE_BYTES = 8 << 30          # workspace of the optimizer, the caching allocator's slack, test scratch
NS_WORKSPACE_BYTES_WHEN_FULL = 2 << 30   # NS5 workspace cap used when the set nearly fills the GPU


def block_resident_bytes(d: int, io_dtype: str = "bf16") -> int:
    """Bytes of parameters, gradients (I/O dtype) and fp32 momentum of one block (18 d^2 elements)."""
    io = 4 if io_dtype == "fp32" else 2
    return 18 * d * d * (2 * io + 4)


def blocks_that_fit(config_id: int, free_bytes: int, reserve_bytes: int = RESERVE_BYTES) -> int:
    """The largest block count of configuration `config_id` (at most its stated
    count) whose resident tensors fit `free_bytes` of device memory with
    `reserve_bytes` left over.  The test at full size and the benchmark both
    call this with the figure torch.cuda.mem_get_info() reports, so they run the
    same subset.  Blocks are identical and independent: time is linear in their
    number."""
    wl = workload(config_id)
    if wl.blocks == 0:
        return 0
    per = block_resident_bytes(wl.d, wl.io_dtype)
    return int(max(1, min(wl.blocks, (int(free_bytes) - int(reserve_bytes)) // per)))


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _release_temporaries(device):
    """Hand the generators' fp32 temporaries back to the driver at once.  Left in
    torch's cache, such a block is later split by a smaller persistent tensor and
    can then never be released: on a shape set that nearly fills the device that
    fragmentation costs several GiB."""
    if torch.device(device).type == "cuda":
        torch.cuda.empty_cache()


def make_param(wl: Workload, idx: int, device="cpu"):
    """Initial parameter W ~ N(0, 0.02^2), rounded to bf16.  In fp32-I/O
    workloads the bf16 values are widened back to fp32 so the same data can
    be run in either storage mode."""
    m, n = wl.shapes[idx]
    g = _gen(device, SEED_BASE + 100 * wl.config_id + 7919 * idx + 1)
    w = torch.empty(m, n, dtype=torch.float32, device=device).normal_(0.0, 0.02, generator=g)
    out = w.to(torch.bfloat16)
    if wl.io_dtype == "fp32":
        out = out.float()
    del w
    _release_temporaries(device)
    return out


def make_grad(wl: Workload, idx: int, step: int, device="cpu"):
    """Gradient for matrix `idx` at step `step`: N(0, grad_std^2), fresh per
    step; optionally with a log-normal (sigma = 1) scale per stored row."""
    m, n = wl.shapes[idx]
    g = _gen(device, SEED_BASE + 100 * wl.config_id + 7919 * idx + 104729 * (step + 1) + 2)
    x = torch.empty(m, n, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g)
    if wl.heavy_tail_rows:
        z = torch.empty(m, 1, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g)
        x.mul_(torch.exp(z))
    x.mul_(wl.grad_std)
    if wl.io_dtype == "fp32":
        return x
    out = x.to(torch.bfloat16)
    del x
    _release_temporaries(device)
    return out


def make_momentum(wl: Workload, idx: int, device="cpu"):
    """Zero-initialised fp32 momentum."""
    m, n = wl.shapes[idx]
    return torch.zeros(m, n, dtype=torch.float32, device=device)
