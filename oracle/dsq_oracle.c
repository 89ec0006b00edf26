/*
 * CPU oracle for the deployed DSQ low-bit convolution path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * GPU library must compute.  It shares no code with the CUDA path and is
 * called only by the tests, the smoke check and the CPU-baseline leg of the
 * benchmark.  Every loop is the definition written out: no blocking, no
 * im2col, no vector intrinsics.  OpenMP is used on the outermost loop only.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (no fast-math), so
 * that every float operation below is a single IEEE-754 binary32 operation in
 * the order written, and fmaf() is one fused multiply-add.
 *
 * Notation (paper Sec. 3.1, Eq. 2; Algorithm 1, feed-forward steps):
 *   b      bit width, 2..4 (1..8 accepted here)
 *   l, u   clip bounds, Delta = (u - l) / (2^b - 1)
 *   q      unsigned code 0 .. 2^b-1, dequantised value l + q*Delta
 *   c      signed storage of a weight code, c = q - 2^(b-1)
 *
 * Code arrays are int8_t; accumulators int32_t; activations NHWC; weights
 * [Cout][KH][KW][Cin]; GEMM operands A[M][K], B[N][K].
 *
 * Parity status: every function here is pinned by tests/test_oracle_*.py
 * (closed forms, exact rational arithmetic, brute force written separately,
 * hand-computed byte strings).  Nothing is "parity unpinned" except the
 * paper's ARM timing tables, which no code here reproduces.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int dsqo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------ */
/* Hard uniform quantiser: Eq. 2 with the offset l of Algorithm 1 step 4,    */
/* clipping of step 1, and the tie rule sgn(0) = +1 of Eq. 1 (a value on an  */
/* interval midpoint takes the upper code).                                  */
/*                                                                           */
/* Pinned binary32 sequence:                                                 */
/*     inv = (float)(2^b - 1) / (u - l)                                      */
/*     xc  = fminf(fmaxf(x, l), u)          NaN -> l (fmaxf returns non-NaN) */
/*     r   = fmaf(xc - l, inv, 0.5f)                                         */
/*     q   = min((int)floorf(r), 2^b - 1)                                    */
/* ------------------------------------------------------------------------ */
int32_t dsqo_quantize_code(float x, int bits, float lo, float hi)
{
    const int32_t qmax = (1 << bits) - 1;
    const float inv = (float)qmax / (hi - lo);
    const float xc = fminf(fmaxf(x, lo), hi);
    const float r = fmaf(xc - lo, inv, 0.5f);
    int32_t q = (int32_t)floorf(r);
    if (q > qmax) q = qmax;
    if (q < 0) q = 0;
    return q;
}

/* x[n] -> unsigned codes q[n] (int8), same clip range for all elements. */
void dsqo_quantize(const float *x, int64_t n, int bits, float lo, float hi,
                   int8_t *q)
{
    for (int64_t i = 0; i < n; ++i)
        q[i] = (int8_t)dsqo_quantize_code(x[i], bits, lo, hi);
}

/* Weights [rows][k]: per-row (per output channel) or scalar clip range,
 * signed storage c = q - 2^(b-1). */
void dsqo_quantize_weights(const float *w, int64_t rows, int64_t k, int bits,
                           const float *lo, const float *hi, int per_row,
                           int8_t *c)
{
    const int32_t half = 1 << (bits - 1);
    for (int64_t r = 0; r < rows; ++r) {
        const float l = per_row ? lo[r] : lo[0];
        const float u = per_row ? hi[r] : hi[0];
        for (int64_t j = 0; j < k; ++j)
            c[r * k + j] =
                (int8_t)(dsqo_quantize_code(w[r * k + j], bits, l, u) - half);
    }
}

/* Dequantise unsigned codes: x^ = l + q*Delta, in binary64 (Algorithm 1
 * step 4). */
void dsqo_dequantize(const int8_t *q, int64_t n, int bits, double lo,
                     double hi, double *out)
{
    const double delta = (hi - lo) / (double)((1 << bits) - 1);
    for (int64_t i = 0; i < n; ++i)
        out[i] = lo + (double)q[i] * delta;
}

/* ------------------------------------------------------------------------ */
/* External packed format: per row a little-endian dense bit stream, element */
/* j in bits [j*b, j*b+b); unsigned codes plain binary, signed codes b-bit   */
/* two's complement; row pitch given by the caller; unused bits zero.        */
/* ------------------------------------------------------------------------ */
int64_t dsqo_row_pitch(int64_t k, int bits)
{
    int64_t bytes = (k * bits + 7) / 8;
    return (bytes + 15) / 16 * 16;
}

void dsqo_pack_rows(const int8_t *codes, int64_t rows, int64_t k, int bits,
                    uint8_t *out, int64_t pitch)
{
    const uint32_t mask = (1u << bits) - 1u;
    memset(out, 0, (size_t)(rows * pitch));
    for (int64_t r = 0; r < rows; ++r) {
        uint8_t *row = out + r * pitch;
        for (int64_t j = 0; j < k; ++j) {
            const uint32_t v = (uint32_t)(int32_t)codes[r * k + j] & mask;
            for (int t = 0; t < bits; ++t) {
                const int64_t bit = j * bits + t;
                if ((v >> t) & 1u) row[bit >> 3] |= (uint8_t)(1u << (bit & 7));
            }
        }
    }
}

void dsqo_unpack_rows(const uint8_t *packed, int64_t rows, int64_t k, int bits,
                      int is_signed, int64_t pitch, int8_t *codes)
{
    for (int64_t r = 0; r < rows; ++r) {
        const uint8_t *row = packed + r * pitch;
        for (int64_t j = 0; j < k; ++j) {
            int32_t v = 0;
            for (int t = 0; t < bits; ++t) {
                const int64_t bit = j * bits + t;
                v |= ((row[bit >> 3] >> (bit & 7)) & 1) << t;
            }
            if (is_signed && (v >> (bits - 1))) v -= (1 << bits);
            codes[r * k + j] = (int8_t)v;
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Integer contraction (Algorithm 1 step 5 on codes).                        */
/* ------------------------------------------------------------------------ */

/* C[m][n] = sum_k A[m][k] * B[n][k], int32. */
void dsqo_gemm(const int8_t *A, const int8_t *B, int64_t M, int64_t N,
               int64_t K, int32_t *C)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int32_t acc = 0;
            for (int64_t k = 0; k < K; ++k)
                acc += (int32_t)A[m * K + k] * (int32_t)B[n * K + k];
            C[m * N + n] = acc;
        }
}

/* Direct convolution.  act [N][H][W][Cin] unsigned codes, wgt
 * [Cout][KH][KW][Cin] signed codes, acc [N][Ho][Wo][Cout];
 * sa [N][Ho][Wo] = sum of activation codes over the in-image taps (nullable).
 * Taps outside the image contribute nothing (zero padding, which is code 0 =
 * real 0 when l_a = 0). */
void dsqo_conv2d(const int8_t *act, int64_t N, int64_t H, int64_t W,
                 int64_t Cin, const int8_t *wgt, int64_t Cout, int64_t KH,
                 int64_t KW, int64_t stride, int64_t pad, int32_t *acc,
                 int32_t *sa)
{
    const int64_t Ho = (H + 2 * pad - KH) / stride + 1;
    const int64_t Wo = (W + 2 * pad - KW) / stride + 1;
#pragma omp parallel for schedule(static) collapse(2)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t ho = 0; ho < Ho; ++ho)
            for (int64_t wo = 0; wo < Wo; ++wo) {
                const int64_t m = (n * Ho + ho) * Wo + wo;
                if (sa) {
                    int32_t s = 0;
                    for (int64_t kh = 0; kh < KH; ++kh)
                        for (int64_t kw = 0; kw < KW; ++kw) {
                            const int64_t hi = ho * stride - pad + kh;
                            const int64_t wi = wo * stride - pad + kw;
                            if (hi < 0 || hi >= H || wi < 0 || wi >= W)
                                continue;
                            for (int64_t ci = 0; ci < Cin; ++ci)
                                s += act[((n * H + hi) * W + wi) * Cin + ci];
                        }
                    sa[m] = s;
                }
                for (int64_t co = 0; co < Cout; ++co) {
                    int32_t a = 0;
                    for (int64_t kh = 0; kh < KH; ++kh)
                        for (int64_t kw = 0; kw < KW; ++kw) {
                            const int64_t hi = ho * stride - pad + kh;
                            const int64_t wi = wo * stride - pad + kw;
                            if (hi < 0 || hi >= H || wi < 0 || wi >= W)
                                continue;
                            for (int64_t ci = 0; ci < Cin; ++ci)
                                a += (int32_t)wgt[((co * KH + kh) * KW + kw) *
                                                      Cin + ci] *
                                     (int32_t)act[((n * H + hi) * W + wi) *
                                                      Cin + ci];
                        }
                    acc[m * Cout + co] = a;
                }
            }
}

/* Depthwise convolution.  act [N][H][W][C] unsigned, wgt [C][KH][KW] signed,
 * acc [N][Ho][Wo][C]; sa [N][Ho][Wo][C] = per-channel sum of in-image
 * activation codes (nullable). */
void dsqo_dwconv2d(const int8_t *act, int64_t N, int64_t H, int64_t W,
                   int64_t C, const int8_t *wgt, int64_t KH, int64_t KW,
                   int64_t stride, int64_t pad, int32_t *acc, int32_t *sa)
{
    const int64_t Ho = (H + 2 * pad - KH) / stride + 1;
    const int64_t Wo = (W + 2 * pad - KW) / stride + 1;
#pragma omp parallel for schedule(static) collapse(2)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t ho = 0; ho < Ho; ++ho)
            for (int64_t wo = 0; wo < Wo; ++wo)
                for (int64_t c = 0; c < C; ++c) {
                    int32_t a = 0, s = 0;
                    for (int64_t kh = 0; kh < KH; ++kh)
                        for (int64_t kw = 0; kw < KW; ++kw) {
                            const int64_t hi = ho * stride - pad + kh;
                            const int64_t wi = wo * stride - pad + kw;
                            if (hi < 0 || hi >= H || wi < 0 || wi >= W)
                                continue;
                            const int32_t q =
                                act[((n * H + hi) * W + wi) * C + c];
                            a += (int32_t)wgt[(c * KH + kh) * KW + kw] * q;
                            s += q;
                        }
                    const int64_t o = ((n * Ho + ho) * Wo + wo) * C + c;
                    acc[o] = a;
                    if (sa) sa[o] = s;
                }
}

/* ------------------------------------------------------------------------ */
/* Dequantise epilogue (Algorithm 1 steps 4-5 folded onto the accumulator).  */
/*                                                                           */
/* acc [rows][cout]; sa: NULL, [rows] (sa_per_channel = 0) or [rows][cout]   */
/* (sa_per_channel = 1, depthwise).  Pinned binary32 sequences:              */
/*   w_offset == 0   : y = fmaf((float)acc, scale, bias)                     */
/*   w_offset == 0.5 : y = fmaf((float)(2*acc + sa), scale*0.5f, bias)       */
/*   otherwise       : y = fmaf(fmaf(w_offset,(float)sa,(float)acc),         */
/*                              scale, bias)                                 */
/*   residual        : y = y + fmaf((float)q_r, delta_r, lo_r)               */
/* with w_offset = l_w/Delta_w + 2^(b-1), the offset of the signed storage   */
/* from the weight grid l_w + Delta_w * q_w.                                 */
/* ------------------------------------------------------------------------ */
void dsqo_epilogue(const int32_t *acc, const int32_t *sa, int sa_per_channel,
                   int64_t rows, int64_t cout, const float *scale,
                   const float *bias, float w_offset, const int8_t *residual,
                   float res_lo, float res_delta, float *y)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m)
        for (int64_t co = 0; co < cout; ++co) {
            const int32_t a = acc[m * cout + co];
            const int32_t s =
                sa ? (sa_per_channel ? sa[m * cout + co] : sa[m]) : 0;
            float v;
            if (w_offset == 0.0f)
                v = fmaf((float)a, scale[co], bias[co]);
            else if (w_offset == 0.5f)
                v = fmaf((float)(2 * a + s), scale[co] * 0.5f, bias[co]);
            else
                v = fmaf(fmaf(w_offset, (float)s, (float)a), scale[co],
                         bias[co]);
            if (residual)
                v = v + fmaf((float)residual[m * cout + co], res_delta,
                             res_lo);
            y[m * cout + co] = v;
        }
}

/* GEMM dequantisation: D[m][n] = (float)C[m][n] * row_scale[m] (one fmul). */
void dsqo_gemm_dequant(const int32_t *C, int64_t M, int64_t N,
                       const float *row_scale, float *D)
{
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n)
            D[m * N + n] = (float)C[m * N + n] * row_scale[m];
}

/* 2x2 max-pool, stride 2, on codes [N][H][W][C] (H, W even). */
void dsqo_maxpool2x2(const int8_t *q, int64_t N, int64_t H, int64_t W,
                     int64_t C, int8_t *out)
{
    const int64_t Ho = H / 2, Wo = W / 2;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t ho = 0; ho < Ho; ++ho)
            for (int64_t wo = 0; wo < Wo; ++wo)
                for (int64_t c = 0; c < C; ++c) {
                    int8_t m = q[((n * H + 2 * ho) * W + 2 * wo) * C + c];
                    for (int dy = 0; dy < 2; ++dy)
                        for (int dx = 0; dx < 2; ++dx) {
                            const int8_t v = q[((n * H + 2 * ho + dy) * W +
                                                2 * wo + dx) * C + c];
                            if (v > m) m = v;
                        }
                    out[((n * Ho + ho) * Wo + wo) * C + c] = m;
                }
}

/* The paper's Table 1: how many 8-bit multiply-accumulates of two b-bit
 * signed numbers fit before the 8-bit accumulator must be widened:
 * floor((2^7 - 1) / (2^(b-1))^2).  Harness sanity value only. */
int32_t dsqo_mla_per_saddw(int bits)
{
    const int32_t m = 1 << (bits - 1);
    return 127 / (m * m);
}
