"""PR-SGD (Parallel Restarted SGD) hot path for NVIDIA B200: a C-ABI CUDA library
(libprsgd.so, declared in include/prsgd.h) and a thin ctypes binding.

Importing the package loads nothing heavy; `paper_1807_06629_b200.binding` loads
the shared library and raises if it has not been built.
"""
__all__ = ["synth", "binding"]
