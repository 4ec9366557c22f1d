"""libkop for B200: hand-written sm_100a kernels for the fused pointwise+reduction segments a
model compiler emits between vendor GEMM / convolution calls, behind a C ABI (include/kop.h).

`kop` is the ctypes binding (same names as the C entry points), `synth` the seeded input
generators, `build` the in-tree nvcc build of libkop.so.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "kop", "build"]
