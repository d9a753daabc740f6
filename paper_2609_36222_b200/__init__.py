"""B200-native batched MoE decode layer with batch-aware expert selection (BASE).

The package holds the CUDA kernels and their C-ABI library (``csrc/``), a thin
ctypes binding with the same entry-point names (``binding``), and the seeded
synthetic workload generator (``workloads``). Importing the package loads no
native code; ``binding.lib()`` does, and raises if the library is missing.
"""

__all__ = ["binding", "workloads"]
