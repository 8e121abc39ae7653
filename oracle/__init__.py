"""CPU oracle of the prefix tensor store: TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this package.
It never imports the CUDA package and the CUDA package never imports it.  `Oracle` is a thin ctypes
wrapper (argument marshalling of numpy arrays) around `ptstore_oracle.cpp`, which holds all of the
oracle's arithmetic.
"""
from .reference import Oracle, build_oracle, hash_parts, PIN, NO_TOUCH, S_NOSPACE, S_BOUNDS, S_STATE

__all__ = ["Oracle", "build_oracle", "hash_parts", "PIN", "NO_TOUCH", "S_NOSPACE", "S_BOUNDS", "S_STATE"]
