// Depthwise 3x3 convolution on packed codes, CUDA cores.  A depthwise
// convolution has no shared contraction dimension across channels, so it is
// not tensor-core work: each thread owns 8 channels (one 32-bit word at 4
// bits, one 16-bit half-word at 2 bits) of four adjacent output pixels, walks
// the 3x3 taps on packed words and applies the dequantise / requantise
// epilogue.  Inputs and outputs move as packed codes only: bits/8 bytes per
// element each way.
#include "dsq_epilogue.cuh"

namespace {

template <int BITS>
__device__ __forceinline__ uint32_t load_unit(const uint8_t *p)
{
    if (BITS == 4) return __ldg(reinterpret_cast<const uint32_t *>(p));
    if (BITS == 3)      // 8 codes = 3 bytes at an odd offset: byte loads
        return (uint32_t)__ldg(p) | ((uint32_t)__ldg(p + 1) << 8) | ((uint32_t)__ldg(p + 2) << 16);
    return __ldg(reinterpret_cast<const uint16_t *>(p));
}

// One thread: 8 channels (one unit) of OW = 4 horizontally adjacent output
// pixels.  The 3 x (OW-1)*stride+3 input window and the 9 weight units are
// loaded once as packed words; then channel by channel the fields are
// extracted (each activation field is used by up to three outputs) and the
// four 9-tap sums are formed.  With the symmetric weight grid the weights are
// taken as 2c+1, so the sum is 2*acc + S_a directly.  Per output element this
// is about 30 integer / fp32 instructions against 1 byte of HBM traffic.
template <int BITS, int STRIDE>
__global__ void __launch_bounds__(256)
dwconv3x3_kernel(const uint8_t *__restrict__ act, const uint8_t *__restrict__ wgt,
                 int N, int H, int W, int C, int Ho, int Wo, int pitch, DsqEpi e)
{
    // lets a tensor-core kernel queued behind this one (programmatic dependent
    // launch) set itself up while this grid runs; it still waits for this grid
    // to complete before touching global data
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int UB = BITS;                 // bytes per 8-channel unit
    constexpr uint32_t MASK = (1u << BITS) - 1u;
    constexpr int OW = 4;                    // outputs per thread along W
    constexpr int IW = (OW - 1) * STRIDE + 3;
    const int units = BITS == 3 ? (C + 7) / 8 : pitch / UB;
    const int strips = (Wo + OW - 1) / OW;
    const int64_t total = (int64_t)N * Ho * strips * units;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int u = (int)(i % units);
        int64_t t = i / units;
        const int sx = (int)(t % strips);
        t /= strips;
        const int ho = (int)(t % Ho);
        const int n = (int)(t / Ho);
        const int wo0 = sx * OW;
        const int hi0 = ho * STRIDE - 1, wi0 = wo0 * STRIDE - 1;

        uint32_t a[3][IW], wv[9];
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int hi = hi0 + r;
#pragma unroll
            for (int x = 0; x < IW; ++x) {
                const int wi = wi0 + x;
                a[r][x] = 0u;
                if (hi >= 0 && hi < H && wi >= 0 && wi < W)
                    a[r][x] = load_unit<BITS>(
                        act + (((int64_t)n * H + hi) * W + wi) * pitch + u * UB);
            }
        }
#pragma unroll
        for (int k = 0; k < 9; ++k) wv[k] = load_unit<BITS>(wgt + k * pitch + u * UB);

        const int64_t pix0 = ((int64_t)n * Ho + ho) * Wo + wo0;
        uint32_t res[OW], cw[OW];
#pragma unroll
        for (int o = 0; o < OW; ++o) {
            cw[o] = 0u;
            res[o] = 0u;
            if (e.residual && wo0 + o < Wo)
                res[o] = load_unit<BITS>(e.residual + (pix0 + o) * pitch + u * UB);
        }
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            const int ch = 8 * u + f;
            if (ch >= C) continue;
            int wq[9];
#pragma unroll
            for (int k = 0; k < 9; ++k) {
                const int c = ((int)(wv[k] << (32 - BITS * (f + 1)))) >> (32 - BITS);
                wq[k] = e.half_offset ? 2 * c + 1 : c;
            }
            int acc[OW], sa[OW];
#pragma unroll
            for (int o = 0; o < OW; ++o) acc[o] = sa[o] = 0;
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                int q[IW];
#pragma unroll
                for (int x = 0; x < IW; ++x) q[x] = (int)((a[r][x] >> (BITS * f)) & MASK);
#pragma unroll
                for (int o = 0; o < OW; ++o)
#pragma unroll
                    for (int kw = 0; kw < 3; ++kw) {
                        acc[o] += q[o * STRIDE + kw] * wq[r * 3 + kw];
                        sa[o] += q[o * STRIDE + kw];      // (dead unless the offset is general)
                    }
            }
            float sc = __ldg(e.scale + ch);
            if (e.half_offset) sc = __fmul_rn(sc, 0.5f);
            const float bi = __ldg(e.bias + ch);
#pragma unroll
            for (int o = 0; o < OW; ++o) {
                if (wo0 + o >= Wo) continue;
                // |acc| <= 9*15*17: the 1.5*2^23 bias trick converts exactly
                const float vf = __fsub_rn(__int_as_float(0x4B400000 + acc[o]), 12582912.0f);
                float y = __fmaf_rn(vf, sc, bi);
                // general weight-grid offset: per-channel S_a (taps outside the
                // image were loaded as code 0)
                if (e.general_offset) y = dsq_epi_y_offset(acc[o], sa[o], e.w_offset, sc, bi);
                if (e.residual) {
                    const uint32_t qr = (res[o] >> (BITS * f)) & MASK;
                    y = __fadd_rn(y, __fmaf_rn(__fsub_rn(__int_as_float(0x4B000000 | qr),
                                                         8388608.0f),
                                               e.res_delta, e.res_lo));
                }
                if (e.acc_out) e.acc_out[(pix0 + o) * C + ch] = acc[o];
                if (e.y_f32) e.y_f32[(pix0 + o) * C + ch] = y;
                if (e.has_requant) {
                    const float xc = fminf(fmaxf(y, e.rq.lo), e.rq.hi);
                    const float rr = __fmaf_rn(__fsub_rn(xc, e.rq.lo), e.rq.inv, 0.5f);
                    const uint32_t q = min(
                        (uint32_t)__float_as_int(__fadd_rd(rr, 8388608.0f)) - 0x4B000000u,
                        (uint32_t)e.rq.qmax);
                    cw[o] |= q << (BITS * f);
                }
            }
        }
        if (e.y_codes) {
#pragma unroll
            for (int o = 0; o < OW; ++o) {
                if (wo0 + o >= Wo) continue;
                uint8_t *dst = e.y_codes + (pix0 + o) * pitch + u * UB;
                if (BITS == 4) *reinterpret_cast<uint32_t *>(dst) = cw[o];
                else if (BITS == 3) {
                    dst[0] = (uint8_t)cw[o]; dst[1] = (uint8_t)(cw[o] >> 8);
                    dst[2] = (uint8_t)(cw[o] >> 16);
                    // the row's spare bytes behind the last unit are zero
                    if (u == units - 1)
                        for (int b = 3 * units; b < pitch; ++b) dst[b - u * UB] = 0;
                } else *reinterpret_cast<uint16_t *>(dst) = (uint16_t)cw[o];
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Fast path: 4-bit codes in, 4-bit codes out (the form the stacks use).
//
// The nine-tap sum of one channel is three 4-way byte dot products (dp4a), one
// per filter row: the activation operand of a row is the byte vector
// [q(p), q(p+1), q(p+2), q(p+3)] of ONE channel at four horizontally adjacent
// pixels, the weight operand [w0, w1, w2, 0] (signed bytes, 2c+1 for the
// symmetric grid).  The packed words hold eight channels of one pixel, so a
// thread (eight channels, four adjacent outputs) first splits each word into
// its even and odd nibbles (two words of four channel bytes) and transposes
// 4 pixels x 4 channels of bytes with byte permutes; the vectors of outputs
// 1..3 come from the first one by funnel shifts.  Per output element this is
// about 10 instructions for the sum and 9 for the dequantise / requantise
// epilogue.  A thread keeps its eight channels for all its strips, so the
// weight vectors, scales and biases are set up once.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    return __byte_perm(a, b, sel);
}

// 4 x 4 byte transpose: in[p] = bytes (c0, c1, c2, c3) of pixel p -> out[c] =
// bytes (p0, p1, p2, p3) of channel c
__device__ __forceinline__ void transpose4x4(const uint32_t (&in)[4], uint32_t (&out)[4])
{
    const uint32_t t0 = prmt(in[0], in[1], 0x5140), t1 = prmt(in[0], in[1], 0x7362);
    const uint32_t t2 = prmt(in[2], in[3], 0x5140), t3 = prmt(in[2], in[3], 0x7362);
    out[0] = prmt(t0, t2, 0x5410);
    out[1] = prmt(t0, t2, 0x7632);
    out[2] = prmt(t1, t3, 0x5410);
    out[3] = prmt(t1, t3, 0x7632);
}

struct DwFast {
    float inv, r_hi;
    int half_offset;
};

template <int STRIDE>
__global__ void __launch_bounds__(256)
dwconv3x3_b4_kernel(const uint8_t *__restrict__ act, const uint8_t *__restrict__ wgt,
                    int N, int H, int W, int C, int Ho, int Wo, int pitch,
                    const float *__restrict__ scale, const float *__restrict__ bias,
                    uint8_t *__restrict__ y_codes, DwFast f)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int OW = 4;                          // outputs per thread along W
    constexpr int NP = STRIDE == 1 ? 6 : 9;        // input pixels per row
    constexpr int NT = STRIDE == 1 ? 2 : 3;        // 4-pixel groups (the last one partial)
    const int units = pitch / 4;
    const int strips = (Wo + OW - 1) / OW;
    const int64_t gtid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t gthreads = (int64_t)gridDim.x * blockDim.x;   // a multiple of `units`
    const int u = (int)(gtid % units);
    const int64_t streams = gthreads / units;

    // weights of the unit's eight channels: channel order (0, 2, 4, 6 | 1, 3, 5, 7),
    // one register per channel and filter row, bytes (w0, w1, w2, 0)
    uint32_t wv[3][8];
    {
        uint32_t tap[9];
#pragma unroll
        for (int k = 0; k < 9; ++k) tap[k] = __ldg(reinterpret_cast<const uint32_t *>(wgt + k * pitch) + u);
#pragma unroll
        for (int r = 0; r < 3; ++r)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int ch = i < 4 ? 2 * i : 2 * (i - 4) + 1;
                uint32_t v = 0;
#pragma unroll
                for (int kw = 0; kw < 3; ++kw) {
                    int c = ((int)(tap[3 * r + kw] << (28 - 4 * ch))) >> 28;   // signed nibble
                    if (f.half_offset) c = 2 * c + 1;
                    v |= ((uint32_t)c & 0xFFu) << (8 * kw);
                }
                wv[r][i] = v;
            }
    }
    float sc[8], bi[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int ch = 8 * u + (i < 4 ? 2 * i : 2 * (i - 4) + 1);
        sc[i] = 0.f; bi[i] = 0.f;
        if (ch < C) {
            sc[i] = __ldg(scale + ch);
            if (f.half_offset) sc[i] = __fmul_rn(sc[i], 0.5f);
            bi[i] = __ldg(bias + ch);
        }
    }
    // the data below depends on the kernels before this one
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // Strips are walked with a fixed stride; the strip index is kept as
    // (image, output row, strip of the row) and advanced by the stride's own
    // decomposition with carries: no division in the loop.
    const int per_img = Ho * strips;
    int sx, ho, n;
    {
        const uint32_t s0 = (uint32_t)(gtid / units);
        n = (int)(s0 / (uint32_t)per_img);
        const uint32_t rem = s0 - (uint32_t)n * per_img;
        ho = (int)(rem / (uint32_t)strips);
        sx = (int)(rem - (uint32_t)ho * strips);
    }
    const int d_n = (int)(streams / per_img), d_rem = (int)(streams % per_img);
    const int d_ho = d_rem / strips, d_sx = d_rem - d_ho * strips;
    const int pw = pitch / 4;                      // words per pixel
    const uint32_t *act32 = reinterpret_cast<const uint32_t *>(act) + u;

    for (; n < N; ) {
        const int wo0 = sx * OW;
        const int hi0 = ho * STRIDE - 1, wi0 = wo0 * STRIDE - 1;
        // the 3 x NP window of packed words (code 0 outside the image)
        uint32_t win[3][NP];
        const uint32_t *base = act32 + ((int64_t)n * H + hi0) * W * pw + (int64_t)wi0 * pw;
        if (hi0 >= 0 && hi0 + 2 < H && wi0 >= 0 && wi0 + NP <= W) {
#pragma unroll
            for (int r = 0; r < 3; ++r)
#pragma unroll
                for (int x = 0; x < NP; ++x) win[r][x] = __ldg(base + (r * W + x) * pw);
        } else {
#pragma unroll
            for (int r = 0; r < 3; ++r)
#pragma unroll
                for (int x = 0; x < NP; ++x) {
                    const int hi = hi0 + r, wi = wi0 + x;
                    win[r][x] = (hi >= 0 && hi < H && wi >= 0 && wi < W)
                                    ? __ldg(base + (r * W + x) * pw) : 0u;
                }
        }
        int acc[OW][8];
#pragma unroll
        for (int o = 0; o < OW; ++o)
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[o][i] = 0;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            // even / odd nibbles of the row's pixels in groups of four, then per
            // channel the bytes of 4 consecutive pixels
            uint32_t tv[NT][8];
#pragma unroll
            for (int g = 0; g < NT; ++g) {
                uint32_t ev[4], od[4], a[4], b[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const uint32_t w = 4 * g + x < NP ? win[r][4 * g + x < NP ? 4 * g + x : 0] : 0u;
                    ev[x] = w & 0x0F0F0F0Fu;
                    od[x] = (w >> 4) & 0x0F0F0F0Fu;
                }
                transpose4x4(ev, a);
                transpose4x4(od, b);
#pragma unroll
                for (int i = 0; i < 4; ++i) { tv[g][i] = a[i]; tv[g][4 + i] = b[i]; }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
#pragma unroll
                for (int o = 0; o < OW; ++o) {
                    // bytes (p, p+1, p+2, .) of the channel with p = o * STRIDE
                    const int p0 = o * STRIDE, g = p0 >> 2, sh = 8 * (p0 & 3);
                    const uint32_t v = sh == 0 ? tv[g][i]
                                               : __funnelshift_r(tv[g][i], g + 1 < NT ? tv[g + 1 < NT ? g + 1 : g][i] : 0u, sh);
                    acc[o][i] = __dp4a((int)v, (int)wv[r][i], acc[o][i]);
                }
            }
        }
        // epilogue: dequantise, requantise to [0, hi] (clip after the multiply,
        // floor by the 2^23 trick, codes summed into their nibbles)
        uint32_t *out32 = reinterpret_cast<uint32_t *>(y_codes) +
                          (((int64_t)n * Ho + ho) * Wo + wo0) * pw + u;
#pragma unroll
        for (int o = 0; o < OW; ++o) {
            if (wo0 + o >= Wo) continue;
            uint32_t cw = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int ch_in_word = i < 4 ? 2 * i : 2 * (i - 4) + 1;
                const float vf = __fsub_rn(__int_as_float(0x4B400000 + acc[o][i]), 12582912.0f);
                const float y = __fmaf_rn(vf, sc[i], bi[i]);
                const float rr = fminf(__fmaf_rn(fmaxf(y, 0.0f), f.inv, 0.5f), f.r_hi);
                cw += (uint32_t)__float_as_int(__fadd_rd(rr, 8388608.0f)) << (4 * ch_in_word);
            }
            cw -= 0x4B000000u * 0x11111111u;
            out32[o * pw] = cw;
        }
        // next strip of this thread
        sx += d_sx; ho += d_ho; n += d_n;
        if (sx >= strips) { sx -= strips; ++ho; }
        if (ho >= Ho) { ho -= Ho; ++n; }
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
    cudaStream_t s = (cudaStream_t)stream;
    // fast path: 4-bit codes to 4-bit codes, requantiser range starting at 0
    if (bits == 4 && y_codes && !y_f32 && !acc_out && !e.residual && !e.general_offset &&
        e.rq.lo == 0.0f) {
        DwFast f;
        f.inv = e.rq.inv;
        f.r_hi = fmaf(e.rq.hi, e.rq.inv, 0.5f);
        f.half_offset = e.half_offset;
        if ((int)floorf(f.r_hi) == e.rq.qmax) {
            const int units = pitch / 4;
            const int sms = dsq_sm_count() > 0 ? dsq_sm_count() : 148;
            const int64_t n_strips = (int64_t)shape->N * Ho * ((Wo + 3) / 4);
            // threads: a multiple of `units` (a thread keeps its channel word) and of 256
            int64_t blocks = (n_strips * units + 255) / 256;
            if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
            blocks = (blocks + units - 1) / units * units;     // blocks * 256 is a multiple of units
            const uint8_t *a8 = (const uint8_t *)act_codes, *w8 = (const uint8_t *)w_packed;
            if (conv->stride == 1)
                dwconv3x3_b4_kernel<1><<<(int)blocks, 256, 0, s>>>(a8, w8, shape->N, shape->H, shape->W,
                                                                  shape->C, Ho, Wo, pitch, e.scale,
                                                                  e.bias, e.y_codes, f);
            else
                dwconv3x3_b4_kernel<2><<<(int)blocks, 256, 0, s>>>(a8, w8, shape->N, shape->H, shape->W,
                                                                  shape->C, Ho, Wo, pitch, e.scale,
                                                                  e.bias, e.y_codes, f);
            return dsq_launch_status();
        }
    }
    const int64_t total = (int64_t)shape->N * Ho * ((Wo + 3) / 4) *
                          (bits == 3 ? (shape->C + 7) / 8 : pitch / bits);
    int64_t g = (total + 255) / 256;
    if (g > 148 * 32) g = 148 * 32;
    if (g < 1) g = 1;
    const uint8_t *a = (const uint8_t *)act_codes, *w = (const uint8_t *)w_packed;
#define DSQ_DW_LAUNCH(B, S)                                                               \
    dwconv3x3_kernel<B, S><<<(int)g, 256, 0, s>>>(a, w, shape->N, shape->H, shape->W, shape->C, \
                                                  Ho, Wo, pitch, e)
    if (bits == 4 && conv->stride == 1) DSQ_DW_LAUNCH(4, 1);
    else if (bits == 4) DSQ_DW_LAUNCH(4, 2);
    else if (bits == 3 && conv->stride == 1) DSQ_DW_LAUNCH(3, 1);
    else if (bits == 3) DSQ_DW_LAUNCH(3, 2);
    else if (conv->stride == 1) DSQ_DW_LAUNCH(2, 1);
    else DSQ_DW_LAUNCH(2, 2);
#undef DSQ_DW_LAUNCH
    return dsq_launch_status();
}
