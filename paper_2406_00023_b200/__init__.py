"""B200-native forward/backward of the Expert-Token Resonance MoE layer (arXiv 2406.00023).

`etr` is a thin ctypes binding over the C ABI in include/etr.h: it marshals arguments
only; every step of the layer runs in the library's CUDA kernels.
"""
from . import etr  # noqa: F401
