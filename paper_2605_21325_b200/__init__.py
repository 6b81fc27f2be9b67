"""B200 (sm_100a) chunkwise delta-rule triangular inversion.

``workloads`` draws seeded synthetic inputs; ``binding`` is the thin ctypes layer
over the C-ABI library built from ``csrc/``.  Importing the package loads
neither torch nor the CUDA library; ``binding`` does, and raises if the library
is missing (there is no CPU path).
"""
__all__ = ["workloads", "binding"]
