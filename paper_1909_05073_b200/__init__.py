"""B200-native PCONV forward pass: pattern-sparse 3x3 convolution behind a C ABI.

`binding` holds the ctypes wrappers of libpconv.so (built by `build`), `synth` the seeded
synthetic workloads.  Importing the package loads nothing; the first call into `binding`
loads the CUDA library and raises if it is absent.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
