"""CPU oracle for the deployed DSQ low-bit convolution path.

TEST INFRASTRUCTURE ONLY.  Plain, slow and written from the paper: the hard
uniform quantiser (Eq. 2 / Algorithm 1), the soft quantiser (Eq. 3-8), the
bit-stream packing, and direct nested-loop integer convolution / depthwise /
GEMM with the dequantise-requantise epilogue.  It shares no code with the
CUDA library and never imports it.  Only the tests, the smoke check and the
CPU-baseline leg of the benchmark may use it.

`oracle.native`  - ctypes binding of dsq_oracle.c (binary32-exact sequences,
                   integer loops)
`oracle.soft`    - numpy float64 soft quantiser and its closed-form relations
`oracle.stack`   - runs a whole layer stack (a list of layer specs) through
                   the native functions, layer by layer
"""
