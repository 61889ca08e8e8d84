"""Block-decomposed Jacobi relaxation on one NVIDIA B200: hand-written sm_100a kernels
behind a C ABI (``libjac.so``), with a thin ctypes binding in :mod:`.jac`.

Importing the package is cheap; the shared library is loaded on first use of :mod:`.jac`.
"""
__all__ = ["inputs", "jac"]
