"""zip2zip dynamic-vocabulary hot path for NVIDIA B200 (sm_100a).

Sub-modules:
  synth_inputs  seeded synthetic workloads (no method arithmetic; importable without a GPU)
  build         compiles the CUDA library in-tree with nvcc
  binding       ctypes binding of the C ABI declared in include/z2z.h (argument marshalling only)

Importing this package loads nothing heavy; ``binding`` loads the shared library on first use and
raises if it has not been built.
"""

__all__ = ["synth_inputs", "build", "binding"]
