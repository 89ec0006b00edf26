// Dequantise / requantise epilogue shared by the depthwise and tensor-core
// kernels (Algorithm 1 steps 4-5 folded onto the integer accumulator, then
// steps 1 and 3 of the next layer).  The binary32 operation order is fixed.
#pragma once

#include "dsq_common.cuh"

struct DsqEpi {
    const float *scale;       // [Cout]
    const float *bias;        // [Cout]
    int half_offset;          // 1: accumulator is 2*acc + S_a, scale halved
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
    if (ep->w_offset != 0.0f && ep->w_offset != 0.5f) return DSQ_ERR_UNSUPPORTED;
    DsqEpi e;
    e.scale = ep->scale;
    e.bias = ep->bias;
    e.half_offset = ep->w_offset == 0.5f ? 1 : 0;
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

__device__ __forceinline__ float dsq_epi_residual(float y, uint32_t q_r,
                                                  float res_delta, float res_lo)
{
    return __fadd_rn(y, __fmaf_rn((float)q_r, res_delta, res_lo));
}
#endif
