// Host-side pieces shared by the two tensor-core translation units
// (dsq_tc.cu, dsq_conv3.cu).  Internal to the library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "dsq_epilogue.cuh"

#define DSQ_HIDDEN __attribute__((visibility("hidden")))

// current values of the process-wide hooks (csrc/dsq_hooks.h)
struct DsqLaunchHooks {
    int pdl;                    // programmatic dependent launch on / off
    unsigned long long wait_ns; // limit of the device-side waits
    int skip_b_round;           // test hook, -1 = off
    int window3;                // dsq_set_conv3_window
    int w8;                     // dsq_set_conv3_expanded_weights
};
DSQ_HIDDEN DsqLaunchHooks dsq_launch_hooks();

typedef CUresult (*DsqEncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                     const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                     const cuuint32_t *, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion,
                                     CUtensorMapFloatOOBfill);
typedef CUresult (*DsqEncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                      const cuuint64_t *, const cuuint64_t *, const int *,
                                      const int *, cuuint32_t, cuuint32_t, const cuuint32_t *,
                                      CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// driver entry points (looked up once; nullptr when the driver lacks them)
DSQ_HIDDEN DsqEncodeTiledFn dsq_encode_tiled_fn();
DSQ_HIDDEN DsqEncodeIm2colFn dsq_encode_im2col_fn();

// epilogue variants of the convolution kernels: codes only, without / with a
// residual operand; any outputs
enum { DSQ_EPI_CODES = 1, DSQ_EPI_CODES_RES = 2, DSQ_EPI_GENERAL = 3 };

// 3x3, stride 1, pad 1 convolution on an expanded shared-memory window
// (dsq_conv3.cu).  Arguments are those of dsq_conv2d after validation.
// Returns DSQ_ERR_UNSUPPORTED without launching anything when the geometry is
// not one it handles; the caller then takes the im2col kernel.
DSQ_HIDDEN int dsq_conv3_window(const void *act_codes, const dsq_nhwc_t *shape, int bits,
                                const void *w_packed, const dsq_conv_t *conv, const DsqEpi &e,
                                int epi_kind, int small_acc, void *workspace,
                                cudaStream_t stream);

// Two-pass GEMM (dsq_gemm8.cu): every packed row is expanded to int8 once
// into caller-provided scratch, then an 8-bit GEMM reads it by TMA.
// dsq_gemm8_scratch_bytes: scratch the path needs (0: not a problem it takes;
// force: whatever the size).
// dsq_gemm8_launch: arguments as dsq_gemm after validation, `scratch`
// 1024-byte aligned and at least that large.
DSQ_HIDDEN size_t dsq_gemm8_scratch_bytes(int64_t M, int64_t N, int64_t K, int force);
DSQ_HIDDEN int dsq_gemm8_launch(const void *A_codes, const void *B_codes, int64_t M, int64_t N,
                                int64_t K, int bits, int32_t *C_i32, const float *row_scale,
                                float *D_f32, void *workspace, void *scratch,
                                cudaStream_t stream);

// Weights of 3x3 stride-1 pad-1 dense convolutions (2- and 4-bit, 64 or a
// multiple of 128 input channels) are stored twice in the blob
// dsq_pack_weights writes: the packed rows, and behind them (1024-byte
// aligned) the same rows already expanded to the int8 bytes the tensor core
// multiplies for the grid Delta (c + 1/2), laid out K step by K step in the
// order the window kernel consumes them (Cout rows of ksteps x 128 bytes).
// The kernel then copies weight tiles by TMA straight into the swizzled operand
// ring, with no expansion warps.  enabled = 0: this geometry has no such copy.
struct DsqW8Info { int enabled; size_t offset; int ksteps; size_t bytes; };
DSQ_HIDDEN DsqW8Info dsq_w8_info(const dsq_conv_t *conv, int bits);
// builds the expanded copy from the packed rows at the start of `blob`
DSQ_HIDDEN int dsq_w8_build(void *blob, const dsq_conv_t *conv, int bits, cudaStream_t stream);
