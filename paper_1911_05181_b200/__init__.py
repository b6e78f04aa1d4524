"""B200-native error-and-gradient evaluation of large fully connected networks
by single-precision matrix products (the hot path of "Ultra-Large-Scale
Neural-Network Training on a PIII Cluster").

The compute lives in a C-ABI shared library (see include/ulsnn.h) built from
csrc/; `paper_1911_05181_b200.binding` is the thin ctypes layer over it.
Importing this package does not load the library; `binding.lib()` does, and it
raises if the library has not been built.
"""
__all__ = ["binding", "flops", "buildlib", "dp", "cg"]
