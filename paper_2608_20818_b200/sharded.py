"""The paper's distributed execution (Section 3.3, Algorithm 2) over dim-0
row shards, one process per GPU.

Non-refresh branch (`sharded_row_step`): local column statistics of the tall
matrices, one packed sum all-reduce, the wide matrices' row steps while it is
in flight, then the tall matrices finished with the global norms.

Refresh branch (`bucketed_refresh_step`): the Muon matrices travel in
communication buckets; while the direction input of bucket l+1 is all-gathered,
the matrices of bucket l are rebuilt, run through NS5 and sliced back to the
local rows.

Only orchestration lives here: the arithmetic runs in the CUDA library
(`prm_tall_shard_stats`, `prm_tall_shard_apply`, `prm_step`,
`prm_shard_momentum_pack`, `prm_refresh_gathered`), the exchanges are
`torch.distributed` collectives (NCCL on GPUs).  The backend objects are
injectable so that ordering, packing and slicing can be exercised on CPU ranks.
"""

from __future__ import annotations

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

    def __init__(self, beta, nesterov, lr, wd, gamma, eps_row, scale_mode=1):
        self.hp = dict(beta=beta, nesterov=nesterov, lr=lr, wd=wd, gamma=gamma, eps_row=eps_row)
        self.scale_mode = int(scale_mode)
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

    def apply(self, param, grad, mom, colsumsq, global_rows, stream):
        rows, cols = param.shape
        hp = self.hp
        scale = B.prm_shape_scale(self.scale_mode, global_rows, cols)      # s(W) of the whole matrix, not of the shard
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
               apply(param, grad, mom, colsumsq, global_rows, stream); the shape
               scale s(W) is the backend's business (it knows the scale mode)
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
        backend.apply(p, g, m, packed[o:o + cols], global_rows, stream)
    return packed


# --------------------------------------------------------------------------
# Refresh branch (Algorithm 2 lines 1-7): bucketed all-gather of the direction
# input, NS5 on the rebuilt matrices while the next bucket is in flight,
# results sliced back to the local rows.


class CudaRefreshBackend:
    """Marshals to prm_bucket_plan, prm_shard_momentum_pack and
    prm_refresh_gathered.  `opt` is a PeriodicRowwiseMuon handle over the
    GLOBAL shapes (its lr, wd, scale mode and NS5 options apply)."""

    payload_dtype = torch.bfloat16

    def __init__(self, opt, beta, nesterov):
        self.opt = opt
        self.beta = beta
        self.nesterov = nesterov

    def plan(self, shapes, world, bucket_bytes):
        return B.prm_bucket_plan(shapes, world, bucket_bytes)

    def shard_rows(self, rows, world, rank):
        return B.prm_shard_rows(rows, world, rank)

    def pack(self, grad, mom, cols, reserved, out, stream):
        B.prm_shard_momentum_pack(grad, mom, cols, reserved, self.beta, self.nesterov, out.data_ptr(), stream)

    def refresh(self, mats, gathered, segment_elems, offsets, world, rank, param_shards, stream):
        ptrs = [p.data_ptr() if p.numel() else 0 for p in param_shards]
        with torch.cuda.device(gathered.device):
            B.prm_refresh_gathered(self.opt.h, mats, gathered.data_ptr(), segment_elems, offsets, world, rank, ptrs,
                                   stream)

    def refresh_segments(self, mats, segment_ptrs, segment_elems, offsets, world, rank, param_shards, stream):
        ptrs = [p.data_ptr() if p.numel() else 0 for p in param_shards]
        with torch.cuda.device(self.opt.device):
            B.prm_refresh_segments(self.opt.h, mats, segment_ptrs, segment_elems, offsets, world, rank, ptrs, stream)


class SymmetricSendBuffers:
    """Two send buffers of n_elems bf16 elements that every rank of the group
    can read: torch symmetric memory (peer-mapped device memory over NVLink).
    `ptrs(k)` are the addresses, in this process, of all ranks' k-th buffer;
    `barrier(k)` is a cross-rank barrier enqueued on the current stream."""

    def __init__(self, n_elems, device, group=None):
        import torch.distributed as td
        import torch.distributed._symmetric_memory as symm
        group = group if group is not None else td.group.WORLD
        self.n_elems = n_elems
        self.tensors = [symm.empty(n_elems, dtype=torch.bfloat16, device=device) for _ in range(2)]
        self.handles = [symm.rendezvous(t, group) for t in self.tensors]

    def ptrs(self, k):
        return [int(p) for p in self.handles[k].buffer_ptrs]

    def barrier(self, k):
        self.handles[k].barrier()


def slot_sizes(bucket_of_mat, offsets, segments):
    """Elements reserved for each matrix in its bucket's segment, read off the
    plan: a slot ends where the next slot of the same bucket starts, the last
    one at the end of the segment."""
    sizes = [0] * len(offsets)
    for l, seg in enumerate(segments):
        members = sorted((offsets[i], i) for i in range(len(offsets)) if bucket_of_mat[i] == l)
        for k, (off, i) in enumerate(members):
            end = members[k + 1][0] if k + 1 < len(members) else seg
            sizes[i] = end - off
    return sizes


def _all_gather(recv, send, group):
    import torch.distributed as td
    try:
        return td.all_gather_into_tensor(recv, send, group=group, async_op=True)
    except (RuntimeError, NotImplementedError):       # transports without the flat form
        return td.all_gather(list(recv.chunk(td.get_world_size(group))), send, group=group, async_op=True)


def bucketed_refresh_step(shapes, param_shards, grad_shards, mom_shards, backend, bucket_bytes=240 << 20,
                          group=None, world=None, rank=None, buffers=None, trace=None, exchange="allgather"):
    """One refresh step over this rank's row shards (Algorithm 2 lines 1-7).

    shapes        GLOBAL (rows, cols) of the Muon matrices, in the handle's order
    *_shards      this rank's rows of every matrix (torch.chunk split of dim 0;
                  a rank may own no row of a matrix: shape (0, cols))
    backend       object with plan / shard_rows / pack / refresh and a
                  payload_dtype (CudaRefreshBackend on GPUs)
    bucket_bytes  cap on the gathered payload of one bucket
    buffers       optional dict that keeps the two send and two receive
                  buffers between calls
    trace         optional list that receives ("gather", l) / ("refresh", l)
                  in issue order
    exchange      "allgather": torch.distributed.all_gather_into_tensor per
                  bucket into a receive buffer.  "p2p": no collective and no
                  receive buffer; every rank packs into a symmetric-memory
                  send buffer, a stream barrier follows, and the rebuild
                  reads all ranks' segments in place with peer loads
                  (prm_refresh_segments).  Two send buffers alternate, so one
                  barrier per bucket orders both the reads after the packs
                  and the next overwrite after the reads.
    Work is issued on torch's current stream; with "allgather" the gather of
    bucket l+1 is in flight while bucket l is refreshed.  Without an
    initialised process group (or with world == 1) the exchange is local.
    """
    import torch.distributed as td

    dist_on = td.is_available() and td.is_initialized() and td.get_world_size(group) > 1
    if world is None:
        world = td.get_world_size(group) if dist_on else 1
    if rank is None:
        rank = td.get_rank(group) if dist_on else 0
    if not dist_on and world != 1:
        raise ValueError("world > 1 needs an initialised torch.distributed process group")
    n = len(shapes)
    bucket_of_mat, offsets, segments = backend.plan(shapes, world, bucket_bytes)
    n_buckets = len(segments)
    members = [[i for i in range(n) if bucket_of_mat[i] == l] for l in range(n_buckets)]
    reserved = slot_sizes(bucket_of_mat, offsets, segments)
    dev = param_shards[0].device
    seg_max = max(segments)
    if buffers is None:
        buffers = {}
    key = (seg_max, world, str(dev), backend.payload_dtype)
    if buffers.get("key") != key:
        buffers["key"] = key
        buffers["send"] = [torch.empty(seg_max, dtype=backend.payload_dtype, device=dev) for _ in range(2)]
        buffers["recv"] = [torch.empty(seg_max * world, dtype=backend.payload_dtype, device=dev) for _ in range(2)]
    stream = torch.cuda.current_stream(dev).cuda_stream if dev.type == "cuda" else 0
    if exchange == "p2p":
        return _refresh_p2p(shapes, param_shards, grad_shards, mom_shards, backend, group, world, rank, buffers,
                            trace, dist_on, (bucket_of_mat, offsets, segments), members, reserved, stream)
    if exchange != "allgather":
        raise ValueError("exchange must be 'allgather' or 'p2p'")
    pending = [None, None]

    def launch(l):                                   # lines 2 and 4: pack, then gather asynchronously
        send = buffers["send"][l % 2][:segments[l]]
        recv = buffers["recv"][l % 2][:segments[l] * world]
        for i in members[l]:
            backend.pack(grad_shards[i], mom_shards[i], shapes[i][1], reserved[i],
                         send[offsets[i]:offsets[i] + reserved[i]], stream)
        if trace is not None:
            trace.append(("gather", l))
        if dist_on:
            pending[l % 2] = _all_gather(recv, send, group)
        else:
            recv.copy_(send)
            pending[l % 2] = None

    launch(0)
    for l in range(n_buckets):
        if pending[l % 2] is not None:               # line 4: wait for the current bucket ...
            pending[l % 2].wait()
            pending[l % 2] = None
        if l + 1 < n_buckets:                        # ... and launch the next all-gather
            launch(l + 1)
        if trace is not None:
            trace.append(("refresh", l))
        recv = buffers["recv"][l % 2][:segments[l] * world]
        backend.refresh(members[l], recv, segments[l], [offsets[i] for i in members[l]], world, rank,
                        [param_shards[i] for i in members[l]], stream)      # line 5
        # line 6: the buffers of bucket l are reused by bucket l + 2
    return bucket_of_mat, offsets, segments


def _refresh_p2p(shapes, param_shards, grad_shards, mom_shards, backend, group, world, rank, buffers, trace,
                 dist_on, plan, members, reserved, stream):
    """Algorithm 2 lines 1-7 with the all-gather folded into the rebuild: the
    segments stay in the send buffers of their owners."""
    bucket_of_mat, offsets, segments = plan
    dev = param_shards[0].device
    seg_max = max(segments)
    key = ("p2p", seg_max, world, str(dev))
    if buffers.get("key") != key:
        buffers["key"] = key
        if dist_on:
            buffers["symm"] = SymmetricSendBuffers(seg_max, dev, group)
            buffers["send"] = buffers["symm"].tensors
        else:
            buffers["symm"] = None
            buffers["send"] = [torch.empty(seg_max, dtype=torch.bfloat16, device=dev) for _ in range(2)]
    symm = buffers["symm"]
    for l, seg in enumerate(segments):
        send = buffers["send"][l % 2][:seg]
        for i in members[l]:
            backend.pack(grad_shards[i], mom_shards[i], shapes[i][1], reserved[i],
                         send[offsets[i]:offsets[i] + reserved[i]], stream)
        if symm is not None:
            symm.barrier(l % 2)          # every rank has packed bucket l and is done reading bucket l-2
            ptrs = symm.ptrs(l % 2)
        else:
            ptrs = [buffers["send"][l % 2].data_ptr()]
        if trace is not None:
            trace.append(("refresh", l))
        backend.refresh_segments(members[l], ptrs, seg, [offsets[i] for i in members[l]], world, rank,
                                 [param_shards[i] for i in members[l]], stream)
    if symm is not None:
        symm.barrier(0)                  # nobody still reads a buffer that the next step packs into
    return plan
