"""libmipgemm: exact C(int32) += A(int8|uint8) * B(int8) on NVIDIA B200 (sm_100a).

The Python layer is a thin ctypes binding over the C-ABI shared library built
from ``csrc/``; importing the package does not load the library (``binding``
does, and fails loudly if it has not been built).
"""
__all__ = ["binding", "inputs"]
