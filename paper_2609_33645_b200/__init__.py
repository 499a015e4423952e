"""Pruned-CTC head-and-loss hot path for NVIDIA B200 (sm_100a).

The package holds the CUDA sources (``csrc/``), the build step for the C-ABI
shared library (``build.py``), the thin ctypes binding (``binding.py``) and the
seeded synthetic workload generator (``workloads.py``).  Nothing here falls
back to a CPU implementation: the binding raises if the library is missing.

Submodules are imported lazily so that ``workloads`` can be used without the
compiled library.
"""

__all__ = ["binding", "build", "workloads"]
