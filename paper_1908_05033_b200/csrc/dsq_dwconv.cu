// Depthwise 3x3 convolution on packed codes, CUDA cores.  A depthwise
// convolution has no shared contraction dimension across channels, so it is
// not tensor-core work: each thread owns 8 channels of one output pixel (one
// 32-bit word at 4 bits, one 16-bit half-word at 2 bits), walks the 3x3 taps
// on packed words and applies the shared epilogue.  Inputs and outputs move
// as packed codes only: bits/8 bytes per element each way.
#include "dsq_epilogue.cuh"

namespace {

template <int BITS>
__device__ __forceinline__ uint32_t load_unit(const uint8_t *p)
{
    if (BITS == 4) return __ldg(reinterpret_cast<const uint32_t *>(p));
    return __ldg(reinterpret_cast<const uint16_t *>(p));
}

template <int BITS>
__global__ void __launch_bounds__(256)
dwconv3x3_kernel(const uint8_t *__restrict__ act, const uint8_t *__restrict__ wgt,
                 int N, int H, int W, int C, int Ho, int Wo, int stride,
                 int pitch, DsqEpi e)
{
    constexpr int UB = BITS;                 // bytes per 8-channel unit
    constexpr uint32_t MASK = (1u << BITS) - 1u;
    const int units = pitch / UB;
    const int64_t total = (int64_t)N * Ho * Wo * units;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int u = (int)(i % units);
        const int64_t pix = i / units;
        const int wo = (int)(pix % Wo);
        const int ho = (int)((pix / Wo) % Ho);
        const int n = (int)(pix / ((int64_t)Wo * Ho));

        int acc[8], sa[8];
#pragma unroll
        for (int f = 0; f < 8; ++f) acc[f] = sa[f] = 0;

#pragma unroll
        for (int kh = 0; kh < 3; ++kh) {
            const int hi = ho * stride - 1 + kh;
            if (hi < 0 || hi >= H) continue;
#pragma unroll
            for (int kw = 0; kw < 3; ++kw) {
                const int wi = wo * stride - 1 + kw;
                if (wi < 0 || wi >= W) continue;
                const uint32_t a = load_unit<BITS>(
                    act + (((int64_t)n * H + hi) * W + wi) * pitch + u * UB);
                const uint32_t wv =
                    load_unit<BITS>(wgt + (kh * 3 + kw) * pitch + u * UB);
#pragma unroll
                for (int f = 0; f < 8; ++f) {
                    const int q = (int)((a >> (BITS * f)) & MASK);
                    const int c = ((int)(wv << (32 - BITS * (f + 1)))) >> (32 - BITS);
                    acc[f] += q * c;
                    sa[f] += q;
                }
            }
        }

        uint32_t res = 0;
        if (e.residual) res = load_unit<BITS>(e.residual + pix * pitch + u * UB);
        uint32_t word = 0;
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            const int ch = 8 * u + f;
            if (ch >= C) continue;
            const int v = e.half_offset ? 2 * acc[f] + sa[f] : acc[f];
            float sc = __ldg(e.scale + ch);
            if (e.half_offset) sc = __fmul_rn(sc, 0.5f);
            float y = dsq_epi_y(v, sc, __ldg(e.bias + ch));
            if (e.residual)
                y = dsq_epi_residual(y, (res >> (BITS * f)) & MASK, e.res_delta,
                                     e.res_lo);
            if (e.acc_out) e.acc_out[pix * C + ch] = v;
            if (e.y_f32) e.y_f32[pix * C + ch] = y;
            if (e.has_requant) word |= dsq_code(y, e.rq) << (BITS * f);
        }
        if (e.y_codes) {
            uint8_t *dst = e.y_codes + pix * pitch + u * UB;
            if (BITS == 4) *reinterpret_cast<uint32_t *>(dst) = word;
            else *reinterpret_cast<uint16_t *>(dst) = (uint16_t)word;
        }
    }
}

}  // namespace

extern "C" int dsq_dwconv2d(const void *act_codes, const dsq_nhwc_t *shape,
                            const dsq_quant_t *act_q, const void *w_packed,
                            const dsq_conv_t *conv, const dsq_epilogue_t *ep,
                            float *y_f32, void *y_codes, int32_t *acc_out,
                            void *stream)
{
    if (!act_codes || !shape || !act_q || !w_packed || !conv || !ep)
        return DSQ_ERR_NULL;
    int st = dsq_check_quant(act_q);
    if (st) return st;
    const int bits = act_q->bits;
    if (bits == 3) return DSQ_ERR_UNSUPPORTED;
    if (shape->N <= 0 || shape->H <= 0 || shape->W <= 0 || shape->C <= 0)
        return DSQ_ERR_SHAPE;
    if (conv->groups != shape->C || conv->Cin != shape->C || conv->Cout != shape->C)
        return DSQ_ERR_SHAPE;
    if (conv->KH != 3 || conv->KW != 3 || conv->pad != 1 ||
        (conv->stride != 1 && conv->stride != 2))
        return DSQ_ERR_UNSUPPORTED;
    if (act_q->lo != 0.0f) return DSQ_ERR_UNSUPPORTED;   // padding is code 0
    if (!dsq_aligned16(act_codes) || !dsq_aligned16(w_packed)) return DSQ_ERR_ALIGN;
    DsqEpi e;
    st = dsq_make_epi(ep, bits, y_f32, y_codes, acc_out, &e);
    if (st) return st;
    const int Ho = (shape->H + 2 - 3) / conv->stride + 1;
    const int Wo = (shape->W + 2 - 3) / conv->stride + 1;
    const int pitch = (int)dsq_row_pitch(shape->C, bits);
    const int64_t total = (int64_t)shape->N * Ho * Wo * (pitch / bits);
    int64_t g = (total + 255) / 256;
    if (g > 148 * 32) g = 148 * 32;
    if (g < 1) g = 1;
    cudaStream_t s = (cudaStream_t)stream;
    if (bits == 4)
        dwconv3x3_kernel<4><<<(int)g, 256, 0, s>>>(
            (const uint8_t *)act_codes, (const uint8_t *)w_packed, shape->N,
            shape->H, shape->W, shape->C, Ho, Wo, conv->stride, pitch, e);
    else
        dwconv3x3_kernel<2><<<(int)g, 256, 0, s>>>(
            (const uint8_t *)act_codes, (const uint8_t *)w_packed, shape->N,
            shape->H, shape->W, shape->C, Ho, Wo, conv->stride, pitch, e);
    return dsq_launch_status();
}
