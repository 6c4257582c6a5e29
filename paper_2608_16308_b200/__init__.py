"""DB-SpMSpV hot path for B200 (sm_100a): C-ABI CUDA library plus a thin Python binding.

Sub-modules:
  workloads -- seeded synthetic input generators (no method arithmetic; shared by tests,
               the CPU oracle's tests and the benchmark)
  binding   -- ctypes marshalling onto libdbspmspv.so (every step runs in the CUDA kernels)

Nothing is imported eagerly: ``workloads`` must stay importable on a box with no GPU and
no built library, and ``binding`` raises loudly when the shared library is missing.
"""

__all__ = ["workloads", "binding"]
