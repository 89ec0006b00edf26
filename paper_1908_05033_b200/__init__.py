"""B200 (sm_100a) library for the deployed form of Differentiable Soft
Quantization: 2-4 bit uniform-quantised convolution with integer contraction
on the tcgen05 tensor cores and a fused dequantise / requantise epilogue.

The product is the C-ABI shared library `libdsq_b200.so` (see include/dsq.h).
This package is its thin Python binding: argument marshalling only, every
step of the path runs in the CUDA kernels.  Importing it loads the library and
raises if it has not been built; there is no CPU fallback.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
