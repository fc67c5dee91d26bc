"""B200-native forward pass of a SwiGLU FFN restructured into a sparse MoE.

The package holds the CUDA kernels and their C-ABI library (``csrc/``), a thin
ctypes binding with the same names (``binding``), and the seeded synthetic
workload generators (``workloads``).  Importing the package loads nothing
heavy; ``binding.load()`` opens the shared library and raises if it is absent.
"""

__all__ = ["binding", "workloads", "build"]
