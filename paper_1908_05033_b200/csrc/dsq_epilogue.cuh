// Dequantise / requantise epilogue shared by the depthwise and tensor-core
// kernels (Algorithm 1 steps 4-5 folded onto the integer accumulator, then
// steps 1 and 3 of the next layer).  The binary32 operation order is fixed.
#pragma once

#include "dsq_common.cuh"

struct DsqEpi {
    const float *scale;       // [Cout]
    const float *bias;        // [Cout]
    int half_offset;          // 1: accumulator is 2*acc + S_a, scale halved
    // general weight-grid offset o_w = l_w/Delta_w + 2^(b-1) (an asymmetric
    // learnt clip): y = fma(fma(o_w, (float)S_a, (float)acc), scale, bias), S_a
    // summed by the epilogue thread from the input codes under the filter
    int general_offset;
    float w_offset;
    const uint8_t *residual;  // packed NHWC codes of the output shape, or null
    float res_lo, res_delta;  // l_r and Delta_r = (hi_r - lo_r)/(2^b - 1)
    int has_requant;
    DsqQ rq;
    float *y_f32;             // nullable
    uint8_t *y_codes;         // nullable
    int32_t *acc_out;         // nullable
};

static inline int dsq_make_epi(const dsq_epilogue_t *ep, int bits, float *y_f32,
                               void *y_codes, int32_t *acc_out, DsqEpi *out)
{
    if (!ep || !ep->scale || !ep->bias) return DSQ_ERR_NULL;
    if (!y_f32 && !y_codes && !acc_out) return DSQ_ERR_NULL;
    if (!dsq_finite(ep->w_offset)) return DSQ_ERR_RANGE;
    DsqEpi e;
    e.scale = ep->scale;
    e.bias = ep->bias;
    e.half_offset = ep->w_offset == 0.5f ? 1 : 0;
    e.general_offset = ep->w_offset != 0.0f && ep->w_offset != 0.5f;
    e.w_offset = ep->w_offset;
    e.residual = (const uint8_t *)ep->residual_codes;
    e.res_lo = 0.f;
    e.res_delta = 0.f;
    if (e.residual) {
        int st = dsq_check_quant(&ep->residual_q);
        if (st) return st;
        if (ep->residual_q.bits != bits) return DSQ_ERR_BITS;
        if (!dsq_aligned16(e.residual)) return DSQ_ERR_ALIGN;
        e.res_lo = ep->residual_q.lo;
        e.res_delta = (ep->residual_q.hi - ep->residual_q.lo) /
                      (float)((1 << bits) - 1);
    }
    e.has_requant = 0;
    e.rq = DsqQ{0.f, 1.f, 1.f, 1};
    if (y_codes) {
        int st = dsq_check_quant(&ep->requant);
        if (st) return st;
        if (ep->requant.bits != bits) return DSQ_ERR_BITS;
        if (!dsq_aligned16(y_codes)) return DSQ_ERR_ALIGN;
        e.has_requant = 1;
        e.rq = dsq_make_q(ep->requant);
    }
    if (y_f32 && !dsq_aligned16(y_f32)) return DSQ_ERR_ALIGN;
    if (acc_out && !dsq_aligned16(acc_out)) return DSQ_ERR_ALIGN;
    e.y_f32 = y_f32;
    e.y_codes = (uint8_t *)y_codes;
    e.acc_out = acc_out;
    *out = e;
    return DSQ_OK;
}

#ifdef __CUDACC__
// v is acc (half_offset = 0) or 2*acc + S_a (half_offset = 1, with `scale`
// already multiplied by 0.5f by the caller of this function).
__device__ __forceinline__ float dsq_epi_y(int v, float scale, float bias)
{
    return __fmaf_rn((float)v, scale, bias);
}

// general weight-grid offset: v = acc, s_a = sum of the activation codes
// under the in-image filter taps
__device__ __forceinline__ float dsq_epi_y_offset(int v, int s_a, float w_offset, float scale,
                                                  float bias)
{
    return __fmaf_rn(__fmaf_rn(w_offset, (float)s_a, (float)v), scale, bias);
}

// Sum of the `bits`-bit fields of `nwords` 32-bit words of a packed row that
// starts at `row` (16-byte aligned, nwords a multiple of 4; spare bits are 0).
template <int BITS>
__device__ __forceinline__ int dsq_codes_sum(const uint8_t *row, int nwords)
{
    int s = 0;
    const uint4 *r4 = reinterpret_cast<const uint4 *>(row);
    for (int i = 0; i < nwords / 4; ++i) {
        const uint4 v = __ldg(r4 + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (BITS == 4) {
                const uint32_t t = (w[j] & 0x0F0F0F0Fu) + ((w[j] >> 4) & 0x0F0F0F0Fu);
                s = (int)__dp4a(t, 0x01010101u, (unsigned)s);
            } else if (BITS == 2) {
                uint32_t t = (w[j] & 0x33333333u) + ((w[j] >> 2) & 0x33333333u);
                t = (t & 0x0F0F0F0Fu) + ((t >> 4) & 0x0F0F0F0Fu);
                s = (int)__dp4a(t, 0x01010101u, (unsigned)s);
            } else {
                // 3-bit fields run across word boundaries: bit k of every field
                // sits at the row's bit positions = k (mod 3); word index mod 3
                // gives the phase of that pattern inside the word
                const int ph = (4 * i + j) % 3;
                const uint32_t m0 = ph == 0 ? 0x49249249u : ph == 1 ? 0x92492492u : 0x24924924u;
                const uint32_t m1 = ph == 0 ? 0x92492492u : ph == 1 ? 0x24924924u : 0x49249249u;
                const uint32_t m2 = ph == 0 ? 0x24924924u : ph == 1 ? 0x49249249u : 0x92492492u;
                s += __popc(w[j] & m0) + 2 * __popc(w[j] & m1) + 4 * __popc(w[j] & m2);
            }
        }
    }
    return s;
}

// S_a of one output pixel of a dense convolution: the codes of all channels
// of every in-image pixel under the k x k window (Algorithm 1 step 5 with the
// weight grid l_w + Delta_w q_w needs it next to the integer accumulator).
template <int BITS>
__device__ __forceinline__ int dsq_window_sa(const uint8_t *act, int n, int ho, int wo, int H,
                                             int W, int ksize, int stride, int pad, int P)
{
    int s = 0;
    for (int kh = 0; kh < ksize; ++kh)
        for (int kw = 0; kw < ksize; ++kw) {
            const int hi = ho * stride - pad + kh, wi = wo * stride - pad + kw;
            if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
            s += dsq_codes_sum<BITS>(act + (((int64_t)n * H + hi) * W + wi) * P, P / 4);
        }
    return s;
}

__device__ __forceinline__ float dsq_epi_residual(float y, uint32_t q_r,
                                                  float res_delta, float res_lo)
{
    return __fadd_rn(y, __fmaf_rn((float)q_r, res_delta, res_lo));
}
#endif
