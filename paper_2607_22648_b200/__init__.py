"""B200-native prefix tensor store: CUDA library (csrc/), its ctypes binding and seeded workloads.

Importing the package does not load the CUDA library; `paper_2607_22648_b200.binding` does, and it
raises if the library has not been built.
"""
__all__ = ["workloads", "binding", "build"]
