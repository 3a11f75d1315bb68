"""ctypes binding of the prm C ABI (include/prm.h).

Argument marshalling only: every arithmetic step runs in the CUDA library.
The functions carry the C names; `PeriodicRowwiseMuon` bundles a handle with
a torch-allocated workspace.  Loading fails loudly when libprm.so is missing;
there is no fallback path.
"""

from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_float, c_int, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libprm.so")

PRM_OK = 0
PRM_ERR_ARG = -1
PRM_ERR_SHAPE = -2
PRM_ERR_ALIGN = -3
PRM_ERR_WORKSPACE = -4
PRM_ERR_CUDA = -5
PRM_ERR_DEVICE_TIMEOUT = -6
PRM_ERR_STATE = -7

PRM_OPT_GAMMA = 1
PRM_OPT_EPS_ROW = 2
PRM_OPT_EPS_NS = 3
PRM_OPT_SCALE_MODE = 4
PRM_OPT_IO_DTYPE = 5
PRM_OPT_CHECK_MODE = 6
PRM_OPT_LR = 7
PRM_OPT_WD = 8
PRM_OPT_NS_WORKSPACE_BYTES = 9
PRM_OPT_GAMMA_NS = 10
PRM_OPT_NO_REFRESH = 11
PRM_OPT_NS_GRAM_SPAN = 12
PRM_OPT_TALL_KERNEL = 13
PRM_OPT_NS_SPLIT_INPUT = 14
PRM_OPT_WIDE_KERNEL = 15

EXPORTS = (
    "prm_create", "prm_set_option", "prm_workspace_bytes", "prm_set_workspace", "prm_step",
    "prm_step_h2d", "prm_plan", "prm_status", "prm_last_error", "prm_launch_count", "prm_destroy",
    "prm_profile", "prm_profile_read", "prm_rowstep_tall_noalloc", "prm_selftest_timeout", "prm_adamw_step",
    "prm_tall_shard_scratch_bytes", "prm_tall_shard_stats", "prm_tall_shard_apply", "prm_group_info",
    "prm_shard_rows", "prm_bucket_plan", "prm_shard_momentum_pack", "prm_refresh_gathered", "prm_refresh_segments", "prm_pipeline_model",
    "prm_partition_matrices", "prm_shape_scale",
)
PRM_PROF_ROW_WIDE, PRM_PROF_ROW_TALL, PRM_PROF_PREPASS, PRM_PROF_GRAM = 0, 1, 2, 3
PRM_PROF_POLY, PRM_PROF_UPDATE, PRM_PROF_UPDATE_FINAL, PRM_PROF_GRAMSPACE, PRM_PROF_COUNT = 4, 5, 6, 7, 8
PROF_NAMES = ("row_wide", "row_tall", "prepass", "gram", "poly", "update", "update_final", "gramspace")

_lib_handle = None


class PrmError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"prm error {code}: {msg}")
        self.code = code


def lib():
    """The loaded CUDA library.  Raises if it has not been built."""
    global _lib_handle
    if _lib_handle is not None:
        return _lib_handle
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} not found: build it with `python -m paper_2608_20818_b200.build` "
            "(nvcc, sm_100a). There is no CPU fallback.")
    L = ctypes.CDLL(LIB_PATH)
    L.prm_create.argtypes = [POINTER(c_void_p), POINTER(c_int64), c_int, c_int, c_float, c_int, c_float, c_float]
    L.prm_create.restype = c_int
    L.prm_set_option.argtypes = [c_void_p, c_int, c_double]
    L.prm_set_option.restype = c_int
    L.prm_workspace_bytes.argtypes = [c_void_p]
    L.prm_workspace_bytes.restype = c_size_t
    L.prm_set_workspace.argtypes = [c_void_p, c_void_p, c_size_t]
    L.prm_set_workspace.restype = c_int
    L.prm_step.argtypes = [c_void_p, POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p), c_int64, c_void_p]
    L.prm_step.restype = c_int
    L.prm_step_h2d.argtypes = [c_void_p, POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p),
                               POINTER(c_void_p), c_int64, c_void_p]
    L.prm_step_h2d.restype = c_int
    L.prm_plan.argtypes = [c_void_p, c_int64, POINTER(c_int), POINTER(c_int), POINTER(c_int), POINTER(c_int)]
    L.prm_plan.restype = c_int
    L.prm_group_info.argtypes = [c_void_p, c_int, POINTER(c_int64), POINTER(c_int64), POINTER(c_int), POINTER(c_int),
                                 POINTER(c_int), POINTER(c_double)]
    L.prm_group_info.restype = c_int
    L.prm_status.argtypes = [c_void_p]
    L.prm_status.restype = c_int
    L.prm_last_error.argtypes = [c_void_p]
    L.prm_last_error.restype = c_char_p
    L.prm_launch_count.argtypes = [c_void_p]
    L.prm_launch_count.restype = c_int64
    L.prm_destroy.argtypes = [c_void_p]
    L.prm_destroy.restype = c_int
    L.prm_profile.argtypes = [c_void_p, c_int]
    L.prm_profile.restype = c_int
    L.prm_profile_read.argtypes = [c_void_p, POINTER(c_double), POINTER(c_int64), c_int]
    L.prm_profile_read.restype = c_int
    L.prm_rowstep_tall_noalloc.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int, c_float,
                                           c_int, c_float, c_float, c_float, c_float, c_float, c_void_p,
                                           c_char_p, c_size_t]
    L.prm_rowstep_tall_noalloc.restype = c_int
    L.prm_selftest_timeout.argtypes = [c_void_p, c_double, c_void_p]
    L.prm_selftest_timeout.restype = c_int
    L.prm_adamw_step.argtypes = [c_int, POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p),
                                 POINTER(c_int64), c_int, c_float, c_float, c_float, c_float, c_float, c_int64,
                                 c_void_p]
    L.prm_adamw_step.restype = c_int
    L.prm_tall_shard_scratch_bytes.argtypes = [c_int64, c_int64]
    L.prm_tall_shard_scratch_bytes.restype = c_size_t
    L.prm_tall_shard_stats.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int, c_float, c_int, c_void_p, c_void_p,
                                       c_size_t, c_void_p]
    L.prm_tall_shard_stats.restype = c_int
    L.prm_tall_shard_apply.argtypes = [c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int, c_float, c_int, c_float,
                                       c_float, c_float, c_float, c_float, c_void_p, c_void_p]
    L.prm_tall_shard_apply.restype = c_int
    L.prm_shard_rows.argtypes = [c_int64, c_int, c_int, POINTER(c_int64), POINTER(c_int64)]
    L.prm_shard_rows.restype = c_int
    L.prm_bucket_plan.argtypes = [POINTER(c_int64), c_int, c_int, c_int64, POINTER(c_int), POINTER(c_int64),
                                  POINTER(c_int), POINTER(c_int64)]
    L.prm_bucket_plan.restype = c_int
    L.prm_shard_momentum_pack.argtypes = [c_void_p, c_void_p, c_int64, c_int64, c_int64, c_int, c_float, c_int,
                                          c_void_p, c_void_p]
    L.prm_shard_momentum_pack.restype = c_int
    L.prm_refresh_gathered.argtypes = [c_void_p, POINTER(c_int), c_int, c_void_p, c_int64, POINTER(c_int64), c_int,
                                       c_int, POINTER(c_void_p), c_void_p]
    L.prm_refresh_gathered.restype = c_int
    L.prm_refresh_segments.argtypes = [c_void_p, POINTER(c_int), c_int, POINTER(c_void_p), c_int64, POINTER(c_int64),
                                       c_int, c_int, POINTER(c_void_p), c_void_p]
    L.prm_refresh_segments.restype = c_int
    L.prm_pipeline_model.argtypes = [POINTER(c_double), POINTER(c_double), c_int, POINTER(c_double), POINTER(c_double)]
    L.prm_pipeline_model.restype = c_int
    L.prm_partition_matrices.argtypes = [POINTER(c_int64), c_int, c_int, POINTER(c_int), POINTER(c_double)]
    L.prm_partition_matrices.restype = c_int
    L.prm_shape_scale.argtypes = [c_int, c_int64, c_int64]
    L.prm_shape_scale.restype = c_double
    _lib_handle = L
    return L


def _check(code, handle=None):
    if code != PRM_OK:
        msg = lib().prm_last_error(handle)
        raise PrmError(code, msg.decode() if msg else "")


def prm_create(shapes, K, beta, nesterov, lr, wd):
    flat = []
    for (m, n) in shapes:
        flat += [int(m), int(n)]
    arr = (c_int64 * max(1, len(flat)))(*flat)
    h = c_void_p()
    _check(lib().prm_create(byref(h), arr, len(shapes), int(K), float(beta), int(bool(nesterov)), float(lr), float(wd)))
    return h


def prm_set_option(h, key, value):
    _check(lib().prm_set_option(h, int(key), float(value)), h)


def prm_workspace_bytes(h):
    return int(lib().prm_workspace_bytes(h))


def prm_set_workspace(h, dev_ptr, nbytes):
    _check(lib().prm_set_workspace(h, c_void_p(dev_ptr), nbytes), h)


def _ptr_array(tensors):
    return (c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def prm_step(h, params, grads, momentum, step_idx, stream=0):
    """params/grads/momentum: ctypes arrays of device pointers (see ptr_arrays)."""
    _check(lib().prm_step(h, params, grads, momentum, int(step_idx), c_void_p(stream)), h)


def prm_step_h2d(h, params, grads_dev, grads_host, momentum, step_idx, stream=0):
    _check(lib().prm_step_h2d(h, params, grads_dev, grads_host, momentum, int(step_idx), c_void_p(stream)), h)


def prm_plan(h, step_idx, n_mats):
    is_refresh, n_groups = c_int(), c_int()
    g = (c_int * n_mats)()
    o = (c_int * n_mats)()
    _check(lib().prm_plan(h, int(step_idx), byref(is_refresh), byref(n_groups), g, o), h)
    return bool(is_refresh.value), n_groups.value, list(g), list(o)


def prm_group_info(h, group):
    """{rows, cols, count, ns_batch, gram_iters, ns5_flop} of one shape group."""
    rows, cols = c_int64(), c_int64()
    count, ns_batch, gram_iters = c_int(), c_int(), c_int()
    flop = c_double()
    _check(lib().prm_group_info(h, int(group), byref(rows), byref(cols), byref(count), byref(ns_batch),
                                byref(gram_iters), byref(flop)), h)
    return {"rows": rows.value, "cols": cols.value, "count": count.value, "ns_batch": ns_batch.value,
            "gram_iters": gram_iters.value, "ns5_flop": flop.value}


def prm_status(h):
    return int(lib().prm_status(h))


def prm_last_error(h):
    msg = lib().prm_last_error(h)
    return msg.decode() if msg else ""


def prm_launch_count(h):
    return int(lib().prm_launch_count(h))


def prm_profile(h, enable):
    _check(lib().prm_profile(h, int(bool(enable))), h)


def prm_profile_read(h):
    ms = (c_double * PRM_PROF_COUNT)()
    n = (c_int64 * PRM_PROF_COUNT)()
    _check(lib().prm_profile_read(h, ms, n, PRM_PROF_COUNT), h)
    return {name: (ms[i], n[i]) for i, name in enumerate(PROF_NAMES)}


def prm_rowstep_tall_noalloc(param, grad, momentum, *, beta, nesterov, lr, wd, gamma, eps_row, scale,
                             stream=None):
    """Row step of one tall matrix for callers that cannot allocate device
    memory (no workspace, no handle): the scratch sits in a fixed array inside
    the library.  Tensors are updated in place; see include/prm.h for the size
    limit and the sharing rules of that array."""
    if len(param.shape) != 2:
        raise ValueError("param must be a 2-D matrix")
    rows, cols = param.shape
    if param.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("param must be float32 or bfloat16")
    if grad.dtype != param.dtype or momentum.dtype != torch.float32:
        raise TypeError(f"dtypes must be {param.dtype} (param, grad) and float32 (momentum)")
    if tuple(grad.shape) != tuple(param.shape) or tuple(momentum.shape) != tuple(param.shape):
        raise ValueError("param, grad and momentum must have the same shape")
    if not (param.is_contiguous() and grad.is_contiguous() and momentum.is_contiguous()):
        raise ValueError("param, grad and momentum must be contiguous")
    if param.device.type != "cuda" or grad.device != param.device or momentum.device != param.device:
        raise ValueError("param, grad and momentum must sit on the same CUDA device")
    io_fp32 = 1 if param.dtype == torch.float32 else 0
    s = (stream or torch.cuda.current_stream(param.device)).cuda_stream
    buf = ctypes.create_string_buffer(256)
    with torch.cuda.device(param.device):
        code = lib().prm_rowstep_tall_noalloc(
            c_void_p(param.data_ptr()), c_void_p(grad.data_ptr()), c_void_p(momentum.data_ptr()),
            int(rows), int(cols), io_fp32, float(beta), int(bool(nesterov)), float(lr), float(wd),
            float(gamma), float(eps_row), float(scale), c_void_p(s), buf, 256)
    if code != PRM_OK:
        raise PrmError(code, buf.value.decode())


def prm_selftest_timeout(h, limit_ms, stream=0):
    _check(lib().prm_selftest_timeout(h, float(limit_ms), c_void_p(stream)), h)


def prm_adamw_step(params, grads, exp_avg, exp_avg_sq, step, *, lr=1e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.01,
                   stream=None):
    """AdamW on a list of device tensors of any shape (the parameters outside
    the Muon set), in place; step is the 1-based step count."""
    n = len(params)
    if n == 0:
        return
    io_fp32 = 1 if params[0].dtype == torch.float32 else 0
    numel = (c_int64 * n)(*[p.numel() for p in params])
    s = (stream or torch.cuda.current_stream(params[0].device)).cuda_stream
    with torch.cuda.device(params[0].device):
        code = lib().prm_adamw_step(n, _ptr_array(params), _ptr_array(grads), _ptr_array(exp_avg),
                                    _ptr_array(exp_avg_sq), numel, io_fp32, float(lr), float(beta1), float(beta2),
                                    float(eps), float(wd), int(step), c_void_p(s))
    if code != PRM_OK:
        raise PrmError(code, "prm_adamw_step failed")


def prm_shard_rows(rows, world, rank):
    """(row_start, row_count) of one rank's dim-0 shard."""
    start, count = c_int64(), c_int64()
    code = lib().prm_shard_rows(int(rows), int(world), int(rank), byref(start), byref(count))
    if code != PRM_OK:
        raise PrmError(code, "prm_shard_rows: bad argument")
    return start.value, count.value


def prm_bucket_plan(shapes, world, bucket_bytes):
    """(bucket_of_mat, offset_in_segment, segment_elems per bucket)."""
    n = len(shapes)
    flat = []
    for (m, k) in shapes:
        flat += [int(m), int(k)]
    arr = (c_int64 * max(1, len(flat)))(*flat)
    bucket = (c_int * max(1, n))()
    off = (c_int64 * max(1, n))()
    seg = (c_int64 * max(1, n))()
    nb = c_int()
    code = lib().prm_bucket_plan(arr, n, int(world), int(bucket_bytes), bucket, off, byref(nb), seg)
    if code != PRM_OK:
        raise PrmError(code, "prm_bucket_plan: bad argument")
    return list(bucket)[:n], list(off)[:n], list(seg)[:nb.value]


def prm_shard_momentum_pack(grad_shard, momentum_shard, cols, reserved_elems, beta, nesterov, u_out_ptr, stream=None):
    """grad_shard, momentum_shard: (rows_local, cols) CUDA tensors (rows_local may be 0)."""
    rows_local = int(grad_shard.shape[0])
    s = stream if stream is not None else torch.cuda.current_stream(grad_shard.device).cuda_stream
    with torch.cuda.device(grad_shard.device):
        code = lib().prm_shard_momentum_pack(c_void_p(grad_shard.data_ptr()), c_void_p(momentum_shard.data_ptr()),
                                             rows_local, int(cols), int(reserved_elems),
                                             1 if grad_shard.dtype == torch.float32 else 0, float(beta),
                                             int(bool(nesterov)), c_void_p(int(u_out_ptr)), c_void_p(s))
    if code != PRM_OK:
        raise PrmError(code, "prm_shard_momentum_pack failed")


def prm_refresh_gathered(h, mats, gathered_ptr, segment_elems, offsets, world, rank, param_shard_ptrs, stream):
    n = len(mats)
    m = (c_int * max(1, n))(*[int(x) for x in mats])
    o = (c_int64 * max(1, n))(*[int(x) for x in offsets])
    p = (c_void_p * max(1, n))(*[c_void_p(int(x)) if x else None for x in param_shard_ptrs])
    _check(lib().prm_refresh_gathered(h, m, n, c_void_p(int(gathered_ptr)), int(segment_elems), o, int(world),
                                      int(rank), p, c_void_p(stream)), h)


def prm_refresh_segments(h, mats, segment_ptrs, segment_elems, offsets, world, rank, param_shard_ptrs, stream):
    """segment_ptrs: one device pointer per rank (local or peer-mapped memory)."""
    n = len(mats)
    m = (c_int * max(1, n))(*[int(x) for x in mats])
    o = (c_int64 * max(1, n))(*[int(x) for x in offsets])
    p = (c_void_p * max(1, n))(*[c_void_p(int(x)) if x else None for x in param_shard_ptrs])
    sp = (c_void_p * max(1, int(world)))(*[c_void_p(int(x)) for x in segment_ptrs])
    _check(lib().prm_refresh_segments(h, m, n, sp, int(segment_elems), o, int(world), int(rank), p,
                                      c_void_p(stream)), h)


def prm_pipeline_model(a, c):
    """(t_pipe, t_comm_exposed) of the ideal two-stage pipeline."""
    n = len(a)
    if n != len(c) or n < 1:
        raise ValueError("a and c must have the same, positive length")
    aa = (c_double * n)(*[float(x) for x in a])
    cc = (c_double * n)(*[float(x) for x in c])
    tp, te = c_double(), c_double()
    code = lib().prm_pipeline_model(aa, cc, n, byref(tp), byref(te))
    if code != PRM_OK:
        raise PrmError(code, "prm_pipeline_model: bad argument")
    return tp.value, te.value


def prm_partition_matrices(shapes, world):
    """(owner_of_mat, flop per rank): whole matrices assigned to ranks."""
    n = len(shapes)
    flat = []
    for (m, k) in shapes:
        flat += [int(m), int(k)]
    arr = (c_int64 * max(1, len(flat)))(*flat)
    owner = (c_int * max(1, n))()
    cost = (c_double * max(1, int(world)))()
    code = lib().prm_partition_matrices(arr, n, int(world), owner, cost)
    if code != PRM_OK:
        raise PrmError(code, "prm_partition_matrices: bad argument")
    return list(owner)[:n], list(cost)[:int(world)]


def prm_shape_scale(mode, rows, cols):
    """s(W) for a stored rows x cols matrix under PRM_OPT_SCALE_MODE `mode`."""
    v = float(lib().prm_shape_scale(int(mode), int(rows), int(cols)))
    if v == 0.0:
        raise PrmError(PRM_ERR_ARG, "prm_shape_scale: bad argument")
    return v


def prm_destroy(h):
    _check(lib().prm_destroy(h))


class PeriodicRowwiseMuon:
    """Handle + workspace.  Tensors stay owned by the caller; `step` only
    marshals their device pointers."""

    def __init__(self, shapes, K, beta=0.95, nesterov=False, lr=5e-3, wd=0.01, *, gamma=0.15,
                 eps_row=1e-8, eps_ns=1e-7, scale_mode=1, io_dtype="bf16", check_mode=False,
                 ns_workspace_bytes=None, gamma_ns=1.0, no_refresh=False, gram_span=2, tall_kernel=0,
                 split_input=False, wide_kernel=0, device="cuda"):
        self.shapes = [(int(m), int(n)) for (m, n) in shapes]
        self.device = torch.device(device)
        self.io_dtype = io_dtype
        self.h = None
        with torch.cuda.device(self.device):
            self.h = prm_create(self.shapes, K, beta, nesterov, lr, wd)
            prm_set_option(self.h, PRM_OPT_GAMMA, gamma)
            prm_set_option(self.h, PRM_OPT_EPS_ROW, eps_row)
            prm_set_option(self.h, PRM_OPT_EPS_NS, eps_ns)
            prm_set_option(self.h, PRM_OPT_SCALE_MODE, scale_mode)
            prm_set_option(self.h, PRM_OPT_IO_DTYPE, 1 if io_dtype == "fp32" else 0)
            prm_set_option(self.h, PRM_OPT_CHECK_MODE, 1 if check_mode else 0)
            prm_set_option(self.h, PRM_OPT_GAMMA_NS, gamma_ns)
            prm_set_option(self.h, PRM_OPT_NO_REFRESH, 1 if no_refresh else 0)
            prm_set_option(self.h, PRM_OPT_NS_GRAM_SPAN, int(gram_span))
            prm_set_option(self.h, PRM_OPT_TALL_KERNEL, int(tall_kernel))
            prm_set_option(self.h, PRM_OPT_NS_SPLIT_INPUT, 1 if split_input else 0)
            prm_set_option(self.h, PRM_OPT_WIDE_KERNEL, int(wide_kernel))
            if ns_workspace_bytes is not None:
                prm_set_option(self.h, PRM_OPT_NS_WORKSPACE_BYTES, ns_workspace_bytes)
            nbytes = prm_workspace_bytes(self.h)
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            prm_set_workspace(self.h, base, nbytes)
        self._cache_key = None
        self._arrays = None

    def ptr_arrays(self, params, grads, momentum):
        key = (tuple(t.data_ptr() for t in params), tuple(t.data_ptr() for t in grads),
               tuple(t.data_ptr() for t in momentum))
        if key != self._cache_key:
            want = torch.float32 if self.io_dtype == "fp32" else torch.bfloat16
            for i, (p, g, m) in enumerate(zip(params, grads, momentum)):
                if p.dtype != want or g.dtype != want or m.dtype != torch.float32:
                    raise TypeError(f"matrix {i}: dtypes must be {want} (params, grads) and float32 (momentum)")
                if tuple(p.shape) != self.shapes[i] or tuple(g.shape) != self.shapes[i] or tuple(m.shape) != self.shapes[i]:
                    raise ValueError(f"matrix {i}: shape mismatch")
                if not (p.is_contiguous() and g.is_contiguous() and m.is_contiguous()):
                    raise ValueError(f"matrix {i}: tensors must be contiguous")
            self._arrays = (_ptr_array(params), _ptr_array(grads), _ptr_array(momentum))
            self._cache_key = key
        return self._arrays

    def step(self, params, grads, momentum, step_idx, stream=None):
        """One optimizer step, enqueued on `stream` (default: torch's current stream)."""
        if len(params) != len(self.shapes):
            raise ValueError("wrong number of matrices")
        P, G, M = self.ptr_arrays(params, grads, momentum)
        s = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        with torch.cuda.device(self.device):
            prm_step(self.h, P, G, M, step_idx, s)

    def step_h2d(self, params, grads_dev, grads_host, momentum, step_idx, stream=None):
        """Step whose gradients are first copied from (pinned) host tensors."""
        P, G, M = self.ptr_arrays(params, grads_dev, momentum)
        H = _ptr_array(grads_host)
        s = (stream or torch.cuda.current_stream(self.device)).cuda_stream
        with torch.cuda.device(self.device):
            prm_step_h2d(self.h, P, G, H, M, step_idx, s)

    def set_lr(self, lr):
        prm_set_option(self.h, PRM_OPT_LR, lr)

    def plan(self, step_idx):
        return prm_plan(self.h, step_idx, len(self.shapes))

    def groups(self):
        """One dict per shape group (see prm_group_info)."""
        n_groups = self.plan(0)[1]
        return [prm_group_info(self.h, g) for g in range(n_groups)]

    def status(self):
        return prm_status(self.h)

    def profile(self, enable=True):
        with torch.cuda.device(self.device):
            prm_profile(self.h, enable)

    def profile_read(self):
        """{class name: (milliseconds, launches)} since the last read."""
        with torch.cuda.device(self.device):
            return prm_profile_read(self.h)

    def launch_count(self):
        return prm_launch_count(self.h)

    def close(self):
        if self.h is not None:
            prm_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
