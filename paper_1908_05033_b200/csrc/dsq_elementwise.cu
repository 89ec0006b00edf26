// Elementwise kernels of the DSQ B200 library: activation quantise + pack
// (Algorithm 1 steps 1 and 3), weight quantise + pack, code pack / unpack,
// 2x2 max-pool on codes.  All are HBM-bound streaming kernels.
#include "dsq_common.cuh"
#include "dsq_tc_host.h"

namespace {

// ---------------------------------------------------------------------------
// 8x8 transpose of 16-bit elements across the 8 lanes of a lane group.
// Lane s holds row s as four 32-bit registers (two 16-bit columns each); on
// return lane s holds column s.  Three butterfly stages, two shuffles each.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void transpose8x8_u16(uint32_t (&r)[4], int s)
{
    {   // 4x4 blocks: lanes s and s^4
        const bool low = (s & 4) == 0;
        uint32_t x = low ? r[2] : r[0], y = low ? r[3] : r[1];
        x = __shfl_xor_sync(0xffffffffu, x, 4);
        y = __shfl_xor_sync(0xffffffffu, y, 4);
        if (low) { r[2] = x; r[3] = y; } else { r[0] = x; r[1] = y; }
    }
    {   // 2x2 blocks: lanes s and s^2
        const bool low = (s & 2) == 0;
        uint32_t x = low ? r[1] : r[0], y = low ? r[3] : r[2];
        x = __shfl_xor_sync(0xffffffffu, x, 2);
        y = __shfl_xor_sync(0xffffffffu, y, 2);
        if (low) { r[1] = x; r[3] = y; } else { r[0] = x; r[2] = y; }
    }
    {   // single elements: lanes s and s^1 trade half-words
        const bool low = (s & 1) == 0;
        uint32_t x = low ? __byte_perm(r[0], r[1], 0x7632)
                         : __byte_perm(r[0], r[1], 0x5410);
        uint32_t y = low ? __byte_perm(r[2], r[3], 0x7632)
                         : __byte_perm(r[2], r[3], 0x5410);
        x = __shfl_xor_sync(0xffffffffu, x, 1);
        y = __shfl_xor_sync(0xffffffffu, y, 1);
        if (low) {
            r[0] = __byte_perm(r[0], x, 0x5410);
            r[1] = __byte_perm(r[1], x, 0x7610);
            r[2] = __byte_perm(r[2], y, 0x5410);
            r[3] = __byte_perm(r[3], y, 0x7610);
        } else {
            r[0] = __byte_perm(r[0], x, 0x3254);
            r[1] = __byte_perm(r[1], x, 0x3276);
            r[2] = __byte_perm(r[2], y, 0x3254);
            r[3] = __byte_perm(r[3], y, 0x3276);
        }
    }
}

// Streaming 128-bit load: read-only path, no L1 allocation (every byte is used
// once), 256-byte L2 prefetch granularity.
__device__ __forceinline__ float4 ld_stream_f4(const float4 *p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

template <int BITS>
__device__ __forceinline__ uint32_t quantize4(const float4 v, const DsqQ &q)
{
    return dsq_code(v.x, q) | (dsq_code(v.y, q) << BITS) |
           (dsq_code(v.z, q) << (2 * BITS)) | (dsq_code(v.w, q) << (3 * BITS));
}

// ---------------------------------------------------------------------------
// Activation quantise, flat fast path (b = 2 or 4, rows without padding, so
// the tensor is one dense stream).  A "line" is 16 bytes of output: 32 codes
// of 4 bits = 8 float4, or 64 codes of 2 bits = 16 float4.  A warp handles 32
// lines per pass: lane group g (8 lanes) reads lines 8g..8g+7, each lane a
// 128-bit load per line (two for 2-bit), so every load instruction covers
// whole 128-byte segments; the 16-bit pieces are then transposed inside the
// lane group with shuffles so that each lane ends up with one complete line
// and the warp writes 512 contiguous bytes with 128-bit stores.
// ---------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(256)
quantize_flat_kernel(const float4 *__restrict__ x, uint4 *__restrict__ out,
                     int64_t n_lines, DsqQ q)
{
    // lets a tensor-core kernel queued behind this one (programmatic dependent
    // launch) set itself up while this grid runs; it still waits for this grid
    // to complete before touching global data
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int NF = (BITS == 4) ? 1 : 2;
    constexpr int F4_PER_LINE = 8 * NF;
    const int lane = threadIdx.x & 31;
    const int g = lane >> 3, s = lane & 7;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t n_pass = (n_lines + 31) >> 5;

    for (int64_t pass = warp; pass < n_pass; pass += nwarps) {
        const int64_t line0 = pass * 32;
        float4 v[8][NF];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int64_t line = line0 + 8 * g + j;
#pragma unroll
            for (int f = 0; f < NF; ++f) {
                v[j][f] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (line < n_lines)
                    v[j][f] = ld_stream_f4(x + line * F4_PER_LINE + 8 * f + s);
            }
        }
        uint32_t h[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t piece = quantize4<BITS>(v[j][0], q);
            if (NF == 2) piece |= quantize4<BITS>(v[j][NF - 1], q) << 8;
            h[j] = piece;
        }
        uint32_t r[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) r[t] = h[2 * t] | (h[2 * t + 1] << 16);
        transpose8x8_u16(r, s);
        if (NF == 2) {
            // pieces are (byte p, byte 8+p) pairs: separate the two halves
            const uint32_t a0 = __byte_perm(r[0], r[1], 0x6420);
            const uint32_t a1 = __byte_perm(r[2], r[3], 0x6420);
            const uint32_t b0 = __byte_perm(r[0], r[1], 0x7531);
            const uint32_t b1 = __byte_perm(r[2], r[3], 0x7531);
            r[0] = a0; r[1] = a1; r[2] = b0; r[3] = b1;
        }
        const int64_t line = line0 + lane;
        if (line < n_lines) __stcs(out + line, make_uint4(r[0], r[1], r[2], r[3]));
    }
}

// ---------------------------------------------------------------------------
// Generic word builder: the 32-bit word `wi` of a packed row of k codes of
// `bits` bits, code_of(j) giving element j (only its low `bits` bits are
// used).  Handles codes that straddle a word boundary (3-bit).
// ---------------------------------------------------------------------------
template <class F>
__device__ __forceinline__ uint32_t build_word(int wi, int k, int bits, F code_of)
{
    const int bit0 = wi * 32;
    const int j0 = bit0 / bits;
    const int j1 = min(k, (bit0 + 32 + bits - 1) / bits);
    const uint32_t mask = (1u << bits) - 1u;
    uint32_t w = 0;
    for (int j = j0; j < j1; ++j) {
        const uint32_t c = code_of(j) & mask;
        const int sh = j * bits - bit0;
        w |= sh >= 0 ? (c << sh) : (c >> (-sh));
    }
    return w;
}

// Activation quantise, generic path: one thread per output word, any bit
// width, rows with padding.
__global__ void __launch_bounds__(256)
quantize_rows_kernel(const float *__restrict__ x, uint32_t *__restrict__ out,
                     int64_t rows, int k, int pitch_words, int bits, DsqQ q)
{
    // lets a tensor-core kernel queued behind this one (programmatic dependent
    // launch) set itself up while this grid runs; it still waits for this grid
    // to complete before touching global data
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t total = rows * pitch_words;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / pitch_words;
        const int wi = (int)(i - r * pitch_words);
        const float *row = x + r * k;
        out[i] = build_word(wi, k, bits,
                            [&](int j) { return dsq_code(__ldg(row + j), q); });
    }
}

// Weight quantise + pack.  Output: `rows` packed rows of k signed codes.
// Dense layout: row = co*taps + t, element ci, source w[row*k + ci], clip
// range of channel co.  Depthwise layout: row = tap t, element c, source
// w[c*taps + t], clip range of channel c.
__global__ void __launch_bounds__(256)
pack_weights_kernel(const float *__restrict__ w, uint32_t *__restrict__ out,
                    int rows, int k, int pitch_words, int bits, int taps,
                    int depthwise, const float *__restrict__ lo,
                    const float *__restrict__ hi, int per_channel,
                    int *__restrict__ ws)
{
    const int64_t total = (int64_t)rows * pitch_words;
    const int qmax = (1 << bits) - 1, half = 1 << (bits - 1);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int r = (int)(i / pitch_words);
        const int wi = (int)(i - (int64_t)r * pitch_words);
        out[i] = build_word(wi, k, bits, [&](int j) -> uint32_t {
            const int ch = depthwise ? j : r / taps;
            const float l = __ldg(lo + (per_channel ? ch : 0));
            const float u = __ldg(hi + (per_channel ? ch : 0));
            if (!(u > l) || !(fabsf(l) <= 3.4e38f) || !(fabsf(u) <= 3.4e38f)) {
                atomicCAS(ws + DSQ_WS_STATUS, 0, (int)DSQ_ERR_RANGE);
                return 0u;
            }
            DsqQ q;
            q.lo = l; q.hi = u; q.qmax = qmax;
            q.inv = __fdiv_rn((float)qmax, __fsub_rn(u, l));
            const float v = depthwise ? __ldg(w + (int64_t)j * taps + r)
                                      : __ldg(w + (int64_t)r * k + j);
            return (uint32_t)((int)dsq_code(v, q) - half);
        });
    }
}

__global__ void __launch_bounds__(256)
pack_codes_kernel(const int8_t *__restrict__ codes, uint32_t *__restrict__ out,
                  int64_t rows, int k, int pitch_words, int bits)
{
    const int64_t total = rows * pitch_words;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / pitch_words;
        const int wi = (int)(i - r * pitch_words);
        const int8_t *row = codes + r * k;
        out[i] = build_word(wi, k, bits,
                            [&](int j) { return (uint32_t)(int)row[j]; });
    }
}

// Field j of a packed row (low `bits` bits of the result).
__device__ __forceinline__ uint32_t read_field(const uint32_t *row, int j,
                                               int bits, int pitch_words)
{
    const int bit = j * bits;
    const int w = bit >> 5, sh = bit & 31;
    uint32_t lo = __ldg(row + w);
    uint32_t hi = (sh + bits > 32 && w + 1 < pitch_words) ? __ldg(row + w + 1) : 0u;
    return __funnelshift_r(lo, hi, sh) & ((1u << bits) - 1u);
}

__global__ void __launch_bounds__(256)
unpack_kernel(const uint32_t *__restrict__ packed, int8_t *__restrict__ out,
              int64_t rows, int k, int pitch_words, int bits, int is_signed)
{
    const int64_t total = rows * k;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / k;
        const int j = (int)(i - r * k);
        int v = (int)read_field(packed + r * pitch_words, j, bits, pitch_words);
        if (is_signed && (v >> (bits - 1))) v -= (1 << bits);
        out[i] = (int8_t)v;
    }
}

// 2x2 max-pool on codes: one thread per output word; each field that touches
// the word is pooled from the four input pixels.
__global__ void __launch_bounds__(256)
maxpool_kernel(const uint32_t *__restrict__ in, uint32_t *__restrict__ out,
               int N, int H, int W, int C, int pitch_words, int bits)
{
    // lets a tensor-core kernel queued behind this one (programmatic dependent
    // launch) set itself up while this grid runs; it still waits for this grid
    // to complete before touching global data
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int Ho = H / 2, Wo = W / 2;
    const int64_t total = (int64_t)N * Ho * Wo * pitch_words;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t pix = i / pitch_words;
        const int wi = (int)(i - pix * pitch_words);
        const int wo = (int)(pix % Wo);
        const int ho = (int)((pix / Wo) % Ho);
        const int n = (int)(pix / ((int64_t)Wo * Ho));
        const uint32_t *p00 =
            in + (((int64_t)n * H + 2 * ho) * W + 2 * wo) * pitch_words;
        const uint32_t *p01 = p00 + pitch_words;
        const uint32_t *p10 = p00 + (int64_t)W * pitch_words;
        const uint32_t *p11 = p10 + pitch_words;
        uint32_t w;
        if (bits == 4 || bits == 2) {
            // fields do not straddle words: split into byte lanes and use the
            // per-byte unsigned max
            const uint32_t a = __ldg(p00 + wi), b = __ldg(p01 + wi),
                           c = __ldg(p10 + wi), d = __ldg(p11 + wi);
            w = 0;
            const uint32_t m = bits == 4 ? 0x0F0F0F0Fu : 0x03030303u;
            for (int sh = 0; sh < 8; sh += bits) {
                const uint32_t v =
                    __vmaxu4(__vmaxu4((a >> sh) & m, (b >> sh) & m),
                             __vmaxu4((c >> sh) & m, (d >> sh) & m));
                w |= v << sh;
            }
        } else {
            w = build_word(wi, C, bits, [&](int j) {
                return max(max(read_field(p00, j, bits, pitch_words),
                               read_field(p01, j, bits, pitch_words)),
                           max(read_field(p10, j, bits, pitch_words),
                               read_field(p11, j, bits, pitch_words)));
            });
        }
        out[i] = w;
    }
}

int grid_for(int64_t work_items, int block, int max_blocks = 148 * 16)
{
    int64_t g = (work_items + block - 1) / block;
    if (g < 1) g = 1;
    if (g > max_blocks) g = max_blocks;
    return (int)g;
}

}  // namespace

extern "C" {

size_t dsq_row_pitch(int64_t k, int bits)
{
    if (k <= 0 || bits < 1 || bits > 8) return 0;
    const int64_t bytes = (k * bits + 7) / 8;
    return (size_t)((bytes + 15) / 16 * 16);
}

size_t dsq_packed_bytes(int64_t rows, int64_t k, int bits)
{
    if (rows <= 0) return 0;
    return (size_t)rows * dsq_row_pitch(k, bits);
}

size_t dsq_weight_bytes(const dsq_conv_t *c, int bits)
{
    if (!c || c->Cout <= 0 || c->Cin <= 0 || c->KH <= 0 || c->KW <= 0) return 0;
    if (c->groups == 1) {
        // (some geometries carry a second, pre-expanded copy behind the packed rows)
        const DsqW8Info w8 = dsq_w8_info(c, bits);
        if (w8.enabled) return w8.offset + w8.bytes;
        return dsq_packed_bytes((int64_t)c->Cout * c->KH * c->KW, c->Cin, bits);
    }
    if (c->groups == c->Cin && c->Cin == c->Cout)
        return dsq_packed_bytes((int64_t)c->KH * c->KW, c->Cout, bits);
    return 0;
}

size_t dsq_workspace_bytes(void) { return DSQ_WS_BYTES; }

int dsq_workspace_init(void *ws, size_t ws_bytes, void *stream)
{
    if (!ws) return DSQ_ERR_NULL;
    if (!dsq_aligned16(ws)) return DSQ_ERR_ALIGN;
    if (ws_bytes < DSQ_WS_BYTES) return DSQ_ERR_SIZE;
    DSQ_CUDA_TRY(cudaMemsetAsync(ws, 0, DSQ_WS_BYTES, (cudaStream_t)stream));
    return DSQ_OK;
}

int dsq_workspace_status(void *ws, void *stream)
{
    if (!ws) return DSQ_ERR_NULL;
    int host[4] = {0, 0, 0, 0};
    DSQ_CUDA_TRY(cudaMemcpyAsync(host, ws, sizeof(host), cudaMemcpyDeviceToHost,
                                 (cudaStream_t)stream));
    DSQ_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    if (host[DSQ_WS_STATUS] != 0)
        DSQ_CUDA_TRY(cudaMemsetAsync(ws, 0, 8, (cudaStream_t)stream));
    return host[DSQ_WS_STATUS];
}

int dsq_quantize_act(const float *x, const dsq_nhwc_t *shape,
                     const dsq_quant_t *q, void *codes_out, size_t bytes,
                     void *stream)
{
    if (!x || !shape || !q || !codes_out) return DSQ_ERR_NULL;
    int st = dsq_check_quant(q);
    if (st) return st;
    if (shape->N <= 0 || shape->H <= 0 || shape->W <= 0 || shape->C <= 0)
        return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(x) || !dsq_aligned16(codes_out)) return DSQ_ERR_ALIGN;
    const int64_t rows = (int64_t)shape->N * shape->H * shape->W;
    const int k = shape->C, bits = q->bits;
    const size_t pitch = dsq_row_pitch(k, bits);
    if (bytes < (size_t)rows * pitch) return DSQ_ERR_SIZE;
    const DsqQ dq = dsq_make_q(*q);
    cudaStream_t s = (cudaStream_t)stream;
    const bool flat = (bits == 4 || bits == 2) && ((size_t)k * bits == pitch * 8);
    if (flat) {
        const int64_t n_lines = rows * (int64_t)(pitch / 16);
        // many more CTAs than SMs: at 8-16 loads per thread the memory system
        // needs the extra resident warps to stay full
        const int grid = grid_for((n_lines + 31) / 32 * 32, 256, 148 * 64);
        if (bits == 4)
            quantize_flat_kernel<4><<<grid, 256, 0, s>>>(
                (const float4 *)x, (uint4 *)codes_out, n_lines, dq);
        else
            quantize_flat_kernel<2><<<grid, 256, 0, s>>>(
                (const float4 *)x, (uint4 *)codes_out, n_lines, dq);
    } else {
        const int pw = (int)(pitch / 4);
        quantize_rows_kernel<<<grid_for(rows * pw, 256), 256, 0, s>>>(
            x, (uint32_t *)codes_out, rows, k, pw, bits, dq);
    }
    return dsq_launch_status();
}

int dsq_pack_weights(const float *w, const dsq_conv_t *c, int bits,
                     const float *lo, const float *hi, int per_channel,
                     void *packed_out, size_t packed_bytes, void *workspace,
                     size_t ws_bytes, void *stream)
{
    if (!w || !c || !lo || !hi || !packed_out || !workspace) return DSQ_ERR_NULL;
    if (bits < 2 || bits > 4) return DSQ_ERR_BITS;
    if (c->Cout <= 0 || c->Cin <= 0 || c->KH <= 0 || c->KW <= 0)
        return DSQ_ERR_SHAPE;
    const bool dense = c->groups == 1;
    const bool dw = c->groups == c->Cin && c->Cin == c->Cout && c->groups > 1;
    if (!dense && !dw) return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(w) || !dsq_aligned16(packed_out) || !dsq_aligned16(workspace))
        return DSQ_ERR_ALIGN;
    if (ws_bytes < DSQ_WS_BYTES) return DSQ_ERR_SIZE;
    const size_t need = dsq_weight_bytes(c, bits);
    if (packed_bytes < need) return DSQ_ERR_SIZE;
    const int taps = c->KH * c->KW;
    const int rows = dense ? c->Cout * taps : taps;
    const int k = dense ? c->Cin : c->Cout;
    const int pw = (int)(dsq_row_pitch(k, bits) / 4);
    pack_weights_kernel<<<grid_for((int64_t)rows * pw, 256), 256, 0,
                          (cudaStream_t)stream>>>(
        w, (uint32_t *)packed_out, rows, k, pw, bits, taps, dw ? 1 : 0, lo, hi,
        per_channel ? 1 : 0, (int *)workspace);
    int st = dsq_launch_status();
    if (st == DSQ_OK && dense) st = dsq_w8_build(packed_out, c, bits, (cudaStream_t)stream);
    return st;
}

int dsq_pack_codes(const int8_t *codes, int64_t rows, int64_t k, int bits,
                   void *packed_out, size_t bytes, void *stream)
{
    if (!codes || !packed_out) return DSQ_ERR_NULL;
    if (bits < 1 || bits > 4) return DSQ_ERR_BITS;
    if (rows <= 0 || k <= 0 || k > (1 << 28)) return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(packed_out)) return DSQ_ERR_ALIGN;
    const size_t pitch = dsq_row_pitch(k, bits);
    if (bytes < (size_t)rows * pitch) return DSQ_ERR_SIZE;
    const int pw = (int)(pitch / 4);
    pack_codes_kernel<<<grid_for(rows * pw, 256), 256, 0, (cudaStream_t)stream>>>(
        codes, (uint32_t *)packed_out, rows, (int)k, pw, bits);
    return dsq_launch_status();
}

int dsq_unpack(const void *packed, int64_t rows, int64_t k, int bits,
               int is_signed, int8_t *codes_out, void *stream)
{
    if (!packed || !codes_out) return DSQ_ERR_NULL;
    if (bits < 1 || bits > 4) return DSQ_ERR_BITS;
    if (rows <= 0 || k <= 0 || k > (1 << 28)) return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(packed)) return DSQ_ERR_ALIGN;
    const int pw = (int)(dsq_row_pitch(k, bits) / 4);
    unpack_kernel<<<grid_for(rows * k, 256), 256, 0, (cudaStream_t)stream>>>(
        (const uint32_t *)packed, codes_out, rows, (int)k, pw, bits,
        is_signed ? 1 : 0);
    return dsq_launch_status();
}

int dsq_maxpool2x2(const void *codes_in, const dsq_nhwc_t *shape, int bits,
                   void *codes_out, size_t bytes, void *stream)
{
    if (!codes_in || !shape || !codes_out) return DSQ_ERR_NULL;
    if (bits < 2 || bits > 4) return DSQ_ERR_BITS;
    if (shape->N <= 0 || shape->H <= 0 || shape->W <= 0 || shape->C <= 0 ||
        (shape->H & 1) || (shape->W & 1))
        return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(codes_in) || !dsq_aligned16(codes_out)) return DSQ_ERR_ALIGN;
    const size_t pitch = dsq_row_pitch(shape->C, bits);
    const int64_t out_rows = (int64_t)shape->N * (shape->H / 2) * (shape->W / 2);
    if (bytes < (size_t)out_rows * pitch) return DSQ_ERR_SIZE;
    const int pw = (int)(pitch / 4);
    maxpool_kernel<<<grid_for(out_rows * pw, 256), 256, 0, (cudaStream_t)stream>>>(
        (const uint32_t *)codes_in, (uint32_t *)codes_out, shape->N, shape->H,
        shape->W, shape->C, pw, bits);
    return dsq_launch_status();
}

const char *dsq_status_string(int status)
{
    switch (status) {
    case DSQ_OK: return "ok";
    case DSQ_ERR_NULL: return "required pointer is NULL";
    case DSQ_ERR_ALIGN: return "buffer is not 16-byte aligned";
    case DSQ_ERR_BITS: return "bit width outside 2..4";
    case DSQ_ERR_SHAPE: return "invalid or inconsistent shape";
    case DSQ_ERR_SIZE: return "buffer too small";
    case DSQ_ERR_RANGE: return "clip range needs finite lo < hi";
    case DSQ_ERR_OVERFLOW: return "accumulator could overflow int32";
    case DSQ_ERR_UNSUPPORTED: return "not supported by this build";
    case DSQ_ERR_CUDA: return "CUDA call failed";
    case DSQ_ERR_TIMEOUT: return "device-side wait ran out";
    default: return "unknown status";
    }
}

int dsq_version(void) { return DSQ_VERSION; }

}  // extern "C"
