"""Periodic Row-wise Muon optimizer step for NVIDIA B200 (sm_100a).

The compute path is a C-ABI CUDA library (csrc/, declared in include/prm.h);
`binding` is the thin ctypes layer over it.  The library is loaded on first
use and a missing or unloadable library raises: there is no CPU fallback.
"""

from .workloads import Workload, workload  # noqa: F401
