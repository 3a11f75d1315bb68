"""Row step over dim-0 shards (the non-refresh branch of the paper's
Algorithm 2): local column statistics of the tall matrices, one packed sum
all-reduce, the wide matrices' row steps while it is in flight, then the tall
matrices finished with the global norms.

Only orchestration lives here: the arithmetic runs in the CUDA library
(`prm_tall_shard_stats`, `prm_tall_shard_apply`, `prm_step`), the exchange is
`torch.distributed.all_reduce`.  The backend object is injectable so that the
ordering and the packing can be exercised on CPU ranks.
"""

from __future__ import annotations

import math

import torch

from . import binding as B


def pack_offsets(cols_list):
    """Offsets of each tall matrix's `cols` statistics in the packed buffer."""
    offs, total = [], 0
    for c in cols_list:
        offs.append(total)
        total += int(c)
    return offs, total


class CudaTallBackend:
    """Marshals one tall shard to the library's two entry points."""

    def __init__(self, beta, nesterov, lr, wd, gamma, eps_row):
        self.hp = dict(beta=beta, nesterov=nesterov, lr=lr, wd=wd, gamma=gamma, eps_row=eps_row)
        self._scratch = None

    def stats(self, grad, mom, out, stream):
        rows, cols = grad.shape
        need = B.lib().prm_tall_shard_scratch_bytes(rows, cols)
        if self._scratch is None or self._scratch.numel() * 4 < need:
            self._scratch = torch.empty((need + 3) // 4, dtype=torch.float32, device=grad.device)
        code = B.lib().prm_tall_shard_stats(grad.data_ptr(), mom.data_ptr(), rows, cols,
                                            1 if grad.dtype == torch.float32 else 0, self.hp["beta"],
                                            int(bool(self.hp["nesterov"])), out.data_ptr(),
                                            self._scratch.data_ptr(), self._scratch.numel() * 4, stream)
        if code != B.PRM_OK:
            raise B.PrmError(code, "prm_tall_shard_stats failed")

    def apply(self, param, grad, mom, colsumsq, scale, stream):
        rows, cols = param.shape
        hp = self.hp
        code = B.lib().prm_tall_shard_apply(param.data_ptr(), grad.data_ptr(), mom.data_ptr(), rows, cols,
                                            1 if param.dtype == torch.float32 else 0, hp["beta"],
                                            int(bool(hp["nesterov"])), hp["lr"], hp["wd"], hp["gamma"],
                                            hp["eps_row"], scale, colsumsq.data_ptr(), stream)
        if code != B.PRM_OK:
            raise B.PrmError(code, "prm_tall_shard_apply failed")


def sharded_row_step(tall, wide_step, backend, group=None, stream=0, stats_dtype=torch.float32):
    """One non-refresh step over this rank's shards.

    tall       list of (param_shard, grad_shard, momentum_shard, global_rows):
               row shards of matrices that are tall GLOBALLY (global_rows > cols)
    wide_step  callable running the row step of the locally complete (wide)
               matrices, or None; it is called while the all-reduce is in flight
    backend    object with stats(grad, mom, out, stream) and
               apply(param, grad, mom, colsumsq, scale, stream)
    group      torch.distributed process group (None: default; not initialised:
               single rank, no exchange)
    stats_dtype  element type of the packed statistics (float32 for the CUDA
               backend)
    """
    import torch.distributed as td

    offs, total = pack_offsets([p.shape[1] for (p, _, _, _) in tall])
    work = None
    packed = None
    if tall:
        p0 = tall[0][0]
        packed = torch.empty(total, dtype=stats_dtype, device=p0.device)
        for (p, g, m, _), o in zip(tall, offs):                       # Algorithm 2 line 9
            backend.stats(g, m, packed[o:o + p.shape[1]], stream)
        if td.is_available() and td.is_initialized() and td.get_world_size(group) > 1:
            work = td.all_reduce(packed, op=td.ReduceOp.SUM, group=group, async_op=True)   # line 10
    if wide_step is not None:
        wide_step()                                                   # line 11
    if work is not None:
        work.wait()                                                   # line 12
    for (p, g, m, global_rows), o in zip(tall, offs):                 # lines 12-13
        cols = p.shape[1]
        backend.apply(p, g, m, packed[o:o + cols], math.sqrt(max(1.0, global_rows / cols)), stream)
    return packed
