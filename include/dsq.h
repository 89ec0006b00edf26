/*
 * dsq.h - C ABI of the B200 (sm_100a) library for the deployed form of
 * Differentiable Soft Quantization (arXiv 1908.05033): 2-4 bit uniform-
 * quantised convolution with integer contraction and a fused
 * dequantise / requantise epilogue.
 *
 * Quantiser (paper Sec. 3.1 Eq. 2; Algorithm 1 feed-forward steps 1, 3, 4):
 * bit width b, clip bounds l < u, interval Delta = (u - l) / (2^b - 1).
 * A value x becomes the unsigned code
 *       q = floor((clip(x, l, u) - l) / Delta + 1/2),   0 <= q <= 2^b - 1,
 * a value on an interval midpoint taking the upper code (sgn(0) = +1, Eq. 1);
 * its dequantised value is l + q * Delta.  This is the limit the soft
 * quantiser (Eq. 3-5) reaches as alpha -> 0, and what sgn(phi(x)) yields for
 * any alpha.  Weights are stored as signed codes c = q - 2^(b-1).
 * The binary32 operation sequence is fixed:
 *       inv = (float)(2^b - 1) / (u - l);  xc = fminf(fmaxf(x, l), u);
 *       r = fmaf(xc - l, inv, 0.5f);       q = min((int)floorf(r), 2^b - 1)
 * (NaN quantises to code 0, +-inf to the nearest end).
 *
 * Packed code format ("packed rows"): each row is a little-endian dense bit
 * stream, element j in bits [j*b, j*b + b); unsigned codes in plain binary,
 * signed codes in b-bit two's complement; the row pitch is
 * dsq_row_pitch(k, b) = ceil(k*b/8) rounded up to 16 bytes; spare bits are 0.
 * An activation tensor is NHWC with one packed row per pixel (k = C).
 *
 * Conventions for every entry point
 *  - All data pointers are DEVICE pointers unless a parameter says "host".
 *    Descriptor structs (dsq_*_t) are read on the host during the call.
 *  - Every buffer is allocated and owned by the caller and must be 16-byte
 *    aligned.  The library allocates no device memory.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Work is enqueued asynchronously; no entry point synchronises
 *    except dsq_workspace_status.
 *  - Return value: DSQ_OK (0) or a negative dsq_status code.  Arguments are
 *    validated on the host before anything is launched; nothing is launched
 *    when an error is returned.  No entry point throws, aborts or prints.
 *  - `workspace`: at least dsq_workspace_bytes() bytes of device memory,
 *    cleared once with dsq_workspace_init.  The tensor-core kernels bound
 *    every wait on a barrier; a wait that runs out records DSQ_ERR_TIMEOUT
 *    in the workspace, the kernel releases its tensor memory and returns, and
 *    dsq_workspace_status reports it.  Calls that share a workspace must be
 *    ordered on one stream.
 */
#ifndef DSQ_H_
#define DSQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum dsq_status {
    DSQ_OK = 0,
    DSQ_ERR_NULL = -1,        /* a required pointer is NULL                   */
    DSQ_ERR_ALIGN = -2,       /* a buffer is not 16-byte aligned              */
    DSQ_ERR_BITS = -3,        /* bit width outside 2..4                       */
    DSQ_ERR_SHAPE = -4,       /* non-positive or inconsistent dimensions      */
    DSQ_ERR_SIZE = -5,        /* an output / workspace buffer is too small    */
    DSQ_ERR_RANGE = -6,       /* hi <= lo, or a bound is not finite           */
    DSQ_ERR_OVERFLOW = -7,    /* K * 2^7 * (2^b - 1) would exceed int32       */
    DSQ_ERR_UNSUPPORTED = -8, /* valid request this build does not implement  */
    DSQ_ERR_CUDA = -9,        /* a CUDA runtime / driver call failed          */
    DSQ_ERR_TIMEOUT = -10     /* a bounded device-side wait ran out           */
} dsq_status;

/* Quantiser parameters (b, l, u) of one tensor. */
typedef struct dsq_quant_t {
    int32_t bits;
    float lo, hi;
} dsq_quant_t;

/* Activation tensor shape, NHWC. */
typedef struct dsq_nhwc_t {
    int32_t N, H, W, C;
} dsq_nhwc_t;

/* Convolution geometry.  groups = 1: dense, weights [Cout][KH][KW][Cin].
 * groups = Cin = Cout: depthwise, weights [C][KH][KW].  Dilation is 1. */
typedef struct dsq_conv_t {
    int32_t Cout, KH, KW, Cin;
    int32_t stride, pad;
    int32_t groups;
} dsq_conv_t;

/* Epilogue applied to the int32 accumulator acc[m][co] (Algorithm 1 steps
 * 4-5 folded onto integers, then steps 1 and 3 of the next layer):
 *   w_offset = 0   : y = fmaf((float)acc, scale[co], bias[co])
 *   w_offset = 0.5 : y = fmaf((float)(2*acc + S_a), scale[co]*0.5f, bias[co])
 *                    where S_a = sum of the activation codes under the
 *                    in-image filter taps.  This is the paper's weight grid
 *                    l_w + Delta_w*q_w with a symmetric clip l_w = -u_w, for
 *                    which w^ = Delta_w * (c + 1/2); scale = Delta_a*Delta_w.
 *   any other w_offset o_w (the clip bounds l_w, u_w are learnt separately,
 *                    Sec. 3.4, so in general o_w = l_w/Delta_w + 2^(b-1)):
 *                    y = fmaf(fmaf(o_w, (float)S_a, (float)acc), scale[co], bias[co]).
 *                    S_a is summed from the input codes by the epilogue (one
 *                    extra read of the filter window per output pixel): slower
 *                    than the two forms above.
 *   residual_codes : y = y + fmaf((float)q_r, Delta_r, l_r), q_r the unsigned
 *                    code at the same output position (packed NHWC, same
 *                    shape as the output), (l_r, Delta_r) from residual_q
 *   requant.bits>0 : codes = quantise(y; requant)  (ReLU is the clip at lo=0)
 * A non-finite w_offset returns DSQ_ERR_RANGE. */
typedef struct dsq_epilogue_t {
    const float *scale;          /* [Cout], required */
    const float *bias;           /* [Cout], required */
    float w_offset;
    const void *residual_codes;  /* nullable */
    dsq_quant_t residual_q;      /* bits must equal the layer's when used */
    dsq_quant_t requant;         /* bits = 0: no code output */
} dsq_epilogue_t;

/* ---- sizes ------------------------------------------------------------- */

/* Row pitch in bytes of k codes of `bits` bits: ceil(k*bits/8) rounded up to
 * a multiple of 16.  0 on invalid arguments. */
size_t dsq_row_pitch(int64_t k, int bits);

/* rows * dsq_row_pitch(k, bits). */
size_t dsq_packed_bytes(int64_t rows, int64_t k, int bits);

/* Size of the blob dsq_pack_weights writes for this geometry. */
size_t dsq_weight_bytes(const dsq_conv_t *conv, int bits);

/* Minimum workspace size. */
size_t dsq_workspace_bytes(void);

/* ---- workspace --------------------------------------------------------- */

/* Clear a workspace (asynchronous memset on `stream`). */
int dsq_workspace_init(void *workspace, size_t ws_bytes, void *stream);

/* Synchronise `stream`, read the status word of the workspace and clear it.
 * Returns DSQ_OK, DSQ_ERR_TIMEOUT (a kernel gave up on a wait; its outputs
 * are undefined) or DSQ_ERR_RANGE (dsq_pack_weights met a bad clip range). */
int dsq_workspace_status(void *workspace, void *stream);

/* ---- Algorithm 1 steps 1, 3 for weights (offline) ---------------------- */

/* Quantise fp32 weights to signed b-bit codes and write the layout the
 * convolution kernels read.
 *   w          fp32, [Cout][KH][KW][Cin] (dense) or [C][KH][KW] (depthwise)
 *   lo, hi     device arrays of clip bounds: one element each, or Cout
 *              elements when per_channel != 0
 *   packed_out dsq_weight_bytes(conv, bits) bytes.  Dense: Cout rows, each
 *              the KH*KW filter taps in order, every tap a packed row of Cin
 *              signed codes at the activation pixel pitch
 *              dsq_row_pitch(Cin, bits).  Depthwise: KH*KW packed rows of C
 *              signed codes.  Treat as opaque; dsq_unpack can read it.
 *              For dense 3x3 stride-1 pad-1 convolutions at 2 or 4 bits with
 *              64 or a multiple of 128 input channels the buffer is larger:
 *              behind the packed rows (1024-byte aligned) it holds the same
 *              rows already expanded to the 8-bit operand bytes of the grid
 *              Delta (c + 1/2), which dsq_conv2d then copies to the tensor
 *              core's shared-memory operand without expanding them again
 *              (dsq_weight_bytes includes that copy).
 * A clip range with hi <= lo or a non-finite bound cannot be seen from the
 * host: the kernel writes code 0 for that channel and records DSQ_ERR_RANGE
 * in the workspace. */
int dsq_pack_weights(const float *w, const dsq_conv_t *conv, int bits,
                     const float *lo, const float *hi, int per_channel,
                     void *packed_out, size_t packed_bytes, void *workspace,
                     size_t ws_bytes, void *stream);

/* ---- Algorithm 1 steps 1, 3 for activations ---------------------------- */

/* fp32 NHWC -> packed unsigned codes, one packed row per pixel.
 * codes_out: dsq_packed_bytes(N*H*W, C, q->bits) bytes.  HBM-bound:
 * 4 + bits/8 bytes per element. */
int dsq_quantize_act(const float *x, const dsq_nhwc_t *shape,
                     const dsq_quant_t *q, void *codes_out, size_t bytes,
                     void *stream);

/* ---- Algorithm 1 step 5 on codes + epilogue ---------------------------- */

/* Dense convolution as an implicit GEMM on the 5th-generation tensor cores
 * (tcgen05.mma kind::i8, int32 accumulation in tensor memory):
 * M = N*Ho*Wo output pixels, N = Cout, K = KH*KW*Cin.
 *   act_codes  packed NHWC unsigned codes of `shape`, quantiser act_q.
 *              act_q->lo must be 0 when conv->pad > 0 (padding is code 0).
 *   w_packed   from dsq_pack_weights with the same geometry and bits
 *   y_f32      nullable: fp32 NHWC output [N][Ho][Wo][Cout]
 *   y_codes    nullable: packed NHWC codes of the output (needs
 *              ep->requant.bits == act_q->bits)
 *   acc_out    nullable: raw int32 accumulators [N][Ho][Wo][Cout]
 *              (2*acc + S_a when w_offset = 0.5)
 * KH = KW in {1, 3}, stride in {1, 2}; bits in {2, 3, 4} (3-bit convolution:
 * the paper's Table 8 times it on every layer shape). */
int dsq_conv2d(const void *act_codes, const dsq_nhwc_t *shape,
               const dsq_quant_t *act_q, const void *w_packed,
               const dsq_conv_t *conv, const dsq_epilogue_t *ep,
               float *y_f32, void *y_codes, int32_t *acc_out,
               void *workspace, size_t ws_bytes, void *stream);

/* Depthwise 3x3 convolution on CUDA cores (not a dense contraction; the
 * depthwise layers of the MobileNetV2 rows of the paper's Table 7, each a
 * quantised convolution in the sense of Algorithm 1 steps 1-5 with one filter
 * per channel):
 * acc[n][ho][wo][c] = sum over the 3x3 taps of q_a * c_w, then the same
 * epilogue with per-channel S_a.  Same arguments as dsq_conv2d;
 * conv->groups = Cin = Cout = shape->C, KH = KW = 3, pad = 1, bits in {2,3,4}.
 * HBM-bound: bits/8 bytes in and out per element. */
int dsq_dwconv2d(const void *act_codes, const dsq_nhwc_t *shape,
                 const dsq_quant_t *act_q, const void *w_packed,
                 const dsq_conv_t *conv, const dsq_epilogue_t *ep,
                 float *y_f32, void *y_codes, int32_t *acc_out, void *stream);

/* Plain low-bit GEMM on the tensor cores: C[m][n] = sum_k A[m][k] * B[n][k]
 * (paper Sec. 3.5: a quantised convolution is lowered to a GEMM over codes
 * whose multiply-accumulates are the core operation; Algorithm 1 step 5 on
 * codes, without the convolution's gather).
 *   A_codes   packed rows [M][K] of SIGNED codes
 *   B_codes   packed rows [N][K] of UNSIGNED codes
 *   C_i32     nullable: int32 [M][N]
 *   row_scale nullable unless D_f32 is given: fp32 [M]
 *   D_f32     nullable: D[m][n] = (float)C[m][n] * row_scale[m]
 * bits in {2, 3, 4}. */
int dsq_gemm(const void *A_codes, const void *B_codes, int64_t M, int64_t N,
             int64_t K, int bits, int32_t *C_i32, const float *row_scale,
             float *D_f32, void *workspace, size_t ws_bytes, void *stream);

/* Workspace with which dsq_gemm runs this problem fastest.  Any workspace of
 * dsq_workspace_bytes() works (one fused kernel that expands the packed codes
 * tile by tile).  Given this many bytes (the status words, then room for both
 * operands as 8-bit rows: about (M + N) * K bytes), large problems (M, N, K >=
 * 1024 and M N K >= 2^35) take two passes instead: every packed row is expanded to 8-bit lanes
 * once, then an 8-bit tensor-core GEMM reads the rows by TMA.  Same results
 * bit for bit.  The area behind the first dsq_workspace_bytes() bytes is
 * scratch: its contents after the call are unspecified, and calls that may
 * overlap on the GPU must not share it. */
size_t dsq_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits);

/* Binary GEMM (paper Eq. 1, the binary quantiser Q_B = sgn with sgn(0) = +1,
 * i.e. the 1-bit case of the uniform quantiser on a symmetric range; the 1/1
 * rows of the paper's Tables 3 and 6):
 *   C[m][n] = sum_k a[m][k] * b[n][k],  a, b in {-1, +1}
 * which equals K - 2 * popcount(A[m] xor B[n]) (the xnor-popcount form).
 *   A_bits  packed rows [M][K], 1 bit per value: bit 1 = +1, bit 0 = -1
 *           (element j in bit j & 7 of byte j / 8; row pitch
 *           dsq_row_pitch(K, 1); bits past K are ignored)
 *   B_bits  packed rows [N][K], same format
 *   C_i32, row_scale, D_f32 as in dsq_gemm.
 * On this GPU the +-1 values go through the 8-bit integer tensor-core path:
 * every row is expanded to int8 once into the workspace, then the same
 * TMA-fed 8-bit GEMM as dsq_gemm's two-pass path runs.  `workspace` must hold
 * dsq_binary_gemm_workspace_bytes(M, N, K) bytes (DSQ_ERR_SIZE otherwise),
 * its first dsq_workspace_bytes() bytes cleared with dsq_workspace_init. */
size_t dsq_binary_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K);
int dsq_binary_gemm(const void *A_bits, const void *B_bits, int64_t M, int64_t N,
                    int64_t K, int32_t *C_i32, const float *row_scale,
                    float *D_f32, void *workspace, size_t ws_bytes, void *stream);

/* Weight-only low-bit GEMM (the W-bit / 32-bit-activation rows of the paper's
 * Table 7: weights quantised by Algorithm 1 steps 1, 3, activations left in
 * floating point; here activations are bf16):
 *   Y[m][n] = fma(sum_k X[m][k] * v[n][k], col_scale[n], col_bias[n])
 * with v = 2 c + 1 when w_offset = 0.5 (the paper's grid w^ = l_w + Delta_w q
 * on a symmetric clip: w^ = (Delta_w / 2)(2 c + 1), so col_scale = Delta_w / 2)
 * and v = c when w_offset = 0 (w^ = Delta_w c, col_scale = Delta_w); c is the
 * signed code c = q - 2^(bits-1).  Other offsets: DSQ_ERR_UNSUPPORTED.
 *   X_bf16    [M][K] bfloat16, row-major, K a multiple of 8 (rows are read by
 *             TMA: 16-byte pitch), DSQ_ERR_ALIGN otherwise
 *   W_codes   packed rows [N][K] of SIGNED codes, bits in {1, 2, 3, 4}
 *   col_scale [N] fp32; col_bias [N] fp32 or NULL
 *   Y_f32     [M][N] fp32
 * Products are exact (bf16 times a small integer); they are accumulated in
 * fp32 by the tensor core in an order of its own, so Y is within
 * K * 2^-23 * sum_k |X v| * |col_scale| of the exact value.  The weights are
 * expanded to bf16 once into the workspace (dsq_wgemm_workspace_bytes(N, K)),
 * then a TMA-fed bf16 tensor-core GEMM runs. */
size_t dsq_wgemm_workspace_bytes(int64_t N, int64_t K);
int dsq_wgemm_bf16(const void *X_bf16, const void *W_codes, int64_t M, int64_t N,
                   int64_t K, int bits, float w_offset, const float *col_scale,
                   const float *col_bias, float *Y_f32, void *workspace,
                   size_t ws_bytes, void *stream);

/* dsq_gemm for callers that cannot allocate device memory.  (The paper has
 * no counterpart: this is a deployment convenience of the library.)
 *
 * dsq_gemm needs a small device workspace from its caller.  Some callers have
 * no way to provide one: code running inside a host framework whose memory
 * pool they may not touch, plug-ins loaded after the application has handed
 * all device memory to its own allocator, or real-time loops in which
 * cudaMalloc (which synchronises the device) is forbidden.  This variant
 * takes the same operands and outputs but no workspace: it uses a 256-byte
 * array that is part of the library image on every GPU that loads it (held
 * until the process exits).  It calls no allocator of any kind.
 *
 *  - Limits: M, N, K <= 65536 each; larger problems return DSQ_ERR_SIZE
 *    (use dsq_gemm with your own workspace).  The scratch itself does not
 *    grow with the problem.
 *  - The first call on a device looks up the array's device address.  Make
 *    that first call with the device current and before starting any stream
 *    capture on it.
 *  - The array is shared by every call on the device and keeps the last
 *    call's contents; each call clears it on `stream` before launching.  Two
 *    calls that can overlap on the GPU (different streams, no dependency
 *    between them) race on it: order them, or use dsq_gemm.
 *  - wait_and_check != 0: the call synchronises `stream` and returns the
 *    device-side status (DSQ_OK or DSQ_ERR_TIMEOUT), like
 *    dsq_workspace_status.  With 0 it returns after enqueueing, and a later
 *    call with wait_and_check reports only its own launch.
 * Results are identical to dsq_gemm's. */
int dsq_gemm_static_ws(const void *A_codes, const void *B_codes, int64_t M,
                       int64_t N, int64_t K, int bits, int32_t *C_i32,
                       const float *row_scale, float *D_f32,
                       int wait_and_check, void *stream);

/* 2x2 stride-2 max-pool on packed unsigned codes.  Exact on codes: the hard
 * quantiser of Eq. 2 is monotone non-decreasing, so the maximum of the codes
 * is the code of the maximum (pooling then Algorithm 1 steps 1, 3 equals
 * steps 1, 3 then pooling).  H and W must be even. */
int dsq_maxpool2x2(const void *codes_in, const dsq_nhwc_t *shape, int bits,
                   void *codes_out, size_t bytes, void *stream);

/* ---- training side: the soft quantiser and its gradients ---------------- */

/* Forward of DSQ's differentiable soft quantiser (paper Sec. 3.2-3.3,
 * Eq. 3-8; Algorithm 1 feed-forward step 2 composed with step 4):
 *   y = l (x < l);  u (x > u);  l + Delta (i + (phi(x) + 1)/2) for x in P_i,
 *   phi(x) = s tanh(k (x - m_i)),  m_i = l + (i + 1/2) Delta,
 *   s = 1/(1 - alpha),  k = log(2/alpha - 1)/Delta,  Delta = (u - l)/(2^b - 1),
 *   P_i = [l + i Delta, l + (i+1) Delta), i = 0 .. 2^b - 2.
 * x, y: fp32 device arrays of n elements (16-byte aligned); q->bits in 1..8
 * (1 = the binary case, one interval); 0 < alpha < 1 (the paper keeps it in
 * (0, 0.5)), else DSQ_ERR_RANGE.  Arithmetic is binary32; NaN stays NaN.
 * HBM-bound: 8 bytes per element. */
int dsq_soft_quantize_fwd(const float *x, int64_t n, const dsq_quant_t *q,
                          float alpha, float *y, void *stream);

/* Back-propagation through y = Q_S(x) (paper Eq. 10-13 and the
 * back-propagation lines of Algorithm 1), the interval index taken as
 * piecewise constant:
 *   grad_x[j] = grad_y[j] * dQ_S/dx            (0 outside [l, u])
 *   grad_params[0] = sum_j grad_y[j] * dQ_S/dalpha            (Eq. 10)
 *   grad_params[1] = sum_j grad_y[j] * dQ_S/dl   (1 for x < l; Eq. 11)
 *   grad_params[2] = sum_j grad_y[j] * dQ_S/du   (1 for x > u; Eq. 12)
 * grad_params: three doubles in device memory (8-byte aligned), overwritten
 * (cleared on `stream`, then accumulated with double-precision atomic adds:
 * the order of the additions, and so the last bits, may differ from run to
 * run).  Element terms are binary32.  HBM-bound: 12 bytes per element. */
int dsq_soft_quantize_bwd(const float *x, const float *grad_y, int64_t n,
                          const dsq_quant_t *q, float alpha, float *grad_x,
                          double *grad_params, void *stream);

/* ---- format helpers (tests, tooling) ----------------------------------- */

/* int8 codes [rows][k] (dense) -> packed rows.  Values are truncated to
 * their low `bits` bits.  bits in {1, 2, 3, 4} (1: the operands of
 * dsq_binary_gemm and 1-bit weights of dsq_wgemm_bf16). */
int dsq_pack_codes(const int8_t *codes, int64_t rows, int64_t k, int bits,
                   void *packed_out, size_t bytes, void *stream);

/* packed rows -> int8 codes [rows][k] (dense), sign-extended if is_signed. */
int dsq_unpack(const void *packed, int64_t rows, int64_t k, int bits,
               int is_signed, int8_t *codes_out, void *stream);

/* ---- measurement ------------------------------------------------------- */

/* Tensor-core rate probe: every SM issues `iters` back-to-back
 * tcgen05.mma kind::i8 128x256x32 instructions on operands resident in
 * shared memory.  Synchronises; writes the elapsed milliseconds (CUDA
 * events) to *ms_out (host) and the number of multiply-accumulates performed
 * to *macs_out (host).  Gives the denominator "measured INT8 peak". */
int dsq_probe_i8_mma_rate(int iters, float *ms_out, double *macs_out,
                          void *workspace, size_t ws_bytes, void *stream);

/* ---- misc --------------------------------------------------------------- */
const char *dsq_status_string(int status);
int dsq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DSQ_H_ */
