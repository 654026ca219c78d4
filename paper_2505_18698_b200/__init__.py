"""MonarchAttention forward pass for B200 (sm_100a): hand-written CUDA kernels behind
a C-ABI library, with a thin ctypes binding.  The CUDA extension is required: there
is no CPU fallback, and calls fail loudly when the shared library is missing."""
from .workloads import WORKLOADS, Workload, make_qkv, make_workload_inputs, shard_units  # noqa: F401

__all__ = ["WORKLOADS", "Workload", "make_qkv", "make_workload_inputs", "shard_units"]
