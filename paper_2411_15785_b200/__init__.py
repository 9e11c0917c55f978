"""Bounded-Cache Transformer attention path for NVIDIA B200 (sm_100a).

The package holds the CUDA sources of the C-ABI library (``csrc/``), its build
script, the thin ctypes binding (``binding``) and the seeded input recipes
(``workloads``).  Importing the package loads nothing; ``binding.load()`` opens
the shared library and fails loudly when it has not been built.
"""
__all__ = ["binding", "workloads", "build"]
