// 3x3, stride 1, pad 1 low-bit convolution on the tensor cores, with the A
// operand read from an expanded WINDOW of the input in shared memory
// (Algorithm 1 step 5 on codes, plus the fused epilogue of steps 4, 1, 3).
//
// An im2col formulation expands every input pixel nine times, once per filter
// tap.  Here every input pixel of a tile is expanded ONCE:
//
//   * Output positions are numbered in a zero-padded, stacked coordinate
//     g = (n * (H+2) + ho) * (W+2) + wo.  The input pixel under filter tap
//     (kh, kw) of output g then sits at padded position g + kh*(W+2) + kw,
//     whatever g is: one constant shift per tap.  (Positions with ho >= H or
//     wo >= W are padding of the numbering; their results are dropped.)
//   * A tile is 128 consecutive positions g0 .. g0+127.  The padded input
//     pixels g0 .. g0+129+2(W+2) are fetched by TMA im2col loads whose
//     bounding box is the image grown by one pixel on every side (the loads
//     traverse W, then H, then N and fill what lies outside the image with
//     zeros = code 0), into a packed staging buffer.
//   * Four warps expand the staged codes to int8 rows of 128 bytes (128
//     channels; wider inputs take several such "planes") in the K-major
//     128-byte-swizzled layout the tensor core reads.
//   * For tap (kh, kw) the A operand of tcgen05.mma is that SAME buffer, its
//     descriptor's start address moved by (kh*(W+2) + kw) rows.  Nine taps x
//     Cin/32 instructions of 128 x BN x 32 accumulate one tile in tensor
//     memory (two accumulator buffers: the epilogue of a tile overlaps the
//     next tile's instructions).
//   * B (weights): TMA brings packed rows of one K step (128 codes of one tap)
//     into a small ring, eight warps expand them to int8, as in the im2col
//     kernel; a weight matrix of few K steps stays resident.
//   * Sixteen epilogue warps (four per tensor-memory lane quarter) take
//     16-column units of a tile: tcgen05.ld, dequantise, residual, requantise,
//     pack, store.  The epilogue is a long chain of dependent arithmetic per
//     element, so it wants many warps in flight; the per-channel scale and bias
//     of the whole layer sit in shared memory, the residual words of a tile
//     are fetched before its accumulators are waited for.
//
// Measured: with the A operand read through a shared-memory descriptor an
// instruction takes about 110-130 clocks whatever its N (the tensor core
// fetches A at roughly 32 bytes a clock), so only 256-wide N tiles run the
// tensor pipe at its full rate; a variant that copied each K step of the
// window to tensor memory (ld.shared + tcgen05.st, A taken from there) was
// slower than this one at every layer size and is not kept.
//
// Wide images (W + 2 > 139) would need a window of more than 416 pixels; they
// are staged as three bands of 136 pixels, one per filter row, instead.
//
// Every wait on a barrier is bounded, as in the im2col kernel.
#include "dsq_tc_common.cuh"
#include "dsq_tc_host.h"

// Cycle stamps of the roles of CTA 0 (profiling builds only: -DDSQ_W3_STAMPS).
#ifdef DSQ_W3_STAMPS
__device__ long long g_w3_stamps[16][64];
#define W3_STAMP(row, col)                                                          \
    do {                                                                            \
        if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && (col) < 64)               \
            g_w3_stamps[row][col] = clock64();                                      \
    } while (0)
extern "C" int dsq_w3_read_stamps(long long *out)
{
    if (cudaMemcpyFromSymbol(out, g_w3_stamps, sizeof(g_w3_stamps)) != cudaSuccess) return -9;
    void *dev = nullptr;
    if (cudaGetSymbolAddress(&dev, g_w3_stamps) != cudaSuccess) return -9;
    return cudaMemset(dev, 0, sizeof(g_w3_stamps)) == cudaSuccess ? 0 : -9;
}
#else
#define W3_STAMP(row, col) do { } while (0)
#endif

namespace {

constexpr int W3_BM = 128;
constexpr int W3_WARP_TMA_B = 0, W3_WARP_MMA = 1, W3_WARP_TMA_A = 2, W3_WARP_A0 = 3,
              W3_NUM_A_WARPS = 4, W3_WARP_B0 = 7, W3_NUM_B_WARPS = 8, W3_WARP_E0 = 15,
              W3_NUM_E_WARPS = 16, W3_NUM_WARPS = 31;
constexpr int W3_B_GROUP_WARPS = W3_NUM_B_WARPS / 2;   // two B groups take alternate K steps
constexpr int W3_EPQ = W3_NUM_E_WARPS / 4;   // epilogue warps per tensor-memory lane quarter
constexpr int W3_MAX_COUT = 1024;            // scale / bias of the layer stay in shared memory
constexpr int W3_THREADS = W3_NUM_WARPS * 32;
constexpr int W3_A_SLOTS = 2;          // expanded windows
constexpr int W3_MAX_BP = 4;           // packed B ring slots
constexpr int W3_MAX_AS = 3;           // packed A staging slots
constexpr int W3_MAX_BST = 10;         // expanded B stages (resident: all K steps)
constexpr int W3_BAND_PX = 136;        // pixels of a band (three-band staging)
constexpr int W3_MAX_WINDOW_PX = 416;

// byte offsets of the kernel's shared-memory regions (w3_layout)
struct W3Smem {
    uint32_t a_slots, b_tiles, a_stage, b_packed, epi, lut, a_tab, bars, tmem_slot, abort_flag, total;
};

struct W3Params {
    // geometry
    int N, H, W, Hp, Wp;               // Hp = H + 2, Wp = W + 2
    int m_tiles, n_tiles, BN, Ncols;
    int E;                             // int8 bytes per pixel = Cin
    int npl, kpp, ksteps;              // planes of 128 channels, K steps per plane, total
    int PB, cpp;                       // packed bytes per pixel and plane; 16-byte chunks of it
    int two_taps;                      // 64-channel rows of 2 / 4 bits: a K step is two filter taps
    int xstep;                         // bytes between two K steps of a plane in a weight row
    int apx;                           // pixels of an A slot
    int a_box, a_nload, nbands, band_px;
    int tap_stride;                    // slot rows between two filter rows
    int as_slots, bp_slots, b_stages, b_res;
    int w8;                            // weight K steps come expanded, by TMA, into the operand ring
    int dup;                           // transposed tiles, <= 64 output channels: the 128 A rows hold the
                                       // weight rows twice; lanes 64..127 of the accumulator repeat lanes
                                       // 0..63 and their epilogue warps take the other half of the columns
    int cout_pad;                      // Cout rounded up to the N tiling
    int tr;                            // transposed tiles (kernel form TR)
    int mstep;                         // M tiles between two tiles of a CTA
    int t_dn, t_dh, t_dw;              // mstep * 128 positions as images, padded rows, columns
    // start of every load of a fill, from the tile's start: images, padded rows
    // (< Hp), padded columns (< Wp)
    int ld_dn[3], ld_dh[3], ld_dw[3];
    int smem_bytes;
    unsigned long long wait_ns;
    int skip_b_round;
    int base_offset_mode;              // probe: put the row phase into the descriptor
    // epilogue
    int shift, out_pitch;
    float r_hi;                        // fmaf(hi - lo, inv, 0.5f) of the requantiser
    DsqEpi e;
    uint32_t orv;
    const uint8_t *act;                // input codes and pixel pitch (general weight offset: S_a)
    int P;
    W3Smem L;                          // shared-memory layout (host-made: w3_layout)
    int *ws;
};


__host__ __device__ inline W3Smem w3_layout(int apx, int BN, int bits, int PB, int as_slots,
                                            int b_stages, int bp_slots, int cout_pad)
{
    W3Smem L;
    uint32_t o = 0;
    L.a_slots = o;  o += W3_A_SLOTS * apx * 128;           // apx is a multiple of 8
    L.b_tiles = o;  o += b_stages * BN * 128;              // BN is a multiple of 8
    L.a_stage = o;  o += as_slots * apx * PB;
    L.b_packed = o; o += bp_slots * BN * 16 * bits;
    L.epi = o;      o += 2 * cout_pad * 4;                  // scale[cout_pad], bias[cout_pad]
    L.lut = o;      o += 16 * 4;
    L.a_tab = o;    o += 9 * 16;                            // four A offsets per K step of a plane
    o = (o + 127u) & ~127u;
    // barriers: a_full/a_empty[2], as_full/as_empty[3], bp_full/bp_empty[4],
    // b_full/b_empty[W3_MAX_BST], acc_full/acc_empty[2], drain
    L.bars = o;     o += 8 * (2 * W3_A_SLOTS + 2 * W3_MAX_AS + 2 * W3_MAX_BP + 2 * W3_MAX_BST + 4 + 1);
    L.tmem_slot = o; o += 8;
    L.abort_flag = o; o += 8;
    L.total = o;
    return L;
}

// 16 columns of one accumulator row -> BITS/2 words of codes, codes-only form
// with requantiser range [0, hi]: per element
//   v  = raw >> shift                       (the factor of the top-bit expansion)
//   vf = (float)v by the 1.5 * 2^23 trick   (|v| < 2^22, checked by the host)
//   y  = fma(vf, scale, bias) (+ lut[q_r])  (lut[q] = fma((float)q, Delta_r, l_r))
//   r  = min(fma(max(y, 0), inv, 0.5), r_hi)
// which is the pinned sequence: max(y, 0) - 0 = max(y, 0); clipping y at hi
// first or r at r_hi = fma(hi, inv, 0.5) afterwards gives the same r because
// fma is monotone; floor(r) <= qmax because floor(r_hi) = qmax (host-checked).
// floor and the packing use the 2^23 trick: the bits of r + 2^23 (rounded
// down) are 0x4B000000 + floor(r); the codes are summed into their fields and
// the constant is taken out once per word.
template <int BITS, bool RES>
__device__ __forceinline__ void w3_codes_unit(const uint32_t (&r)[16], const float *sc,
                                              const float *bi, const uint32_t (&resw)[BITS / 2],
                                              const float *lut, int shift, float inv,
                                              float r_hi, uint32_t (&cw)[BITS / 2])
{
    constexpr uint32_t MASK = (1u << BITS) - 1u;
#pragma unroll
    for (int w = 0; w < BITS / 2; ++w) cw[w] = 0u;
    const float4 *sc4 = reinterpret_cast<const float4 *>(sc);
    const float4 *bi4 = reinterpret_cast<const float4 *>(bi);
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        const float4 s4 = sc4[v], b4 = bi4[v];
        const float scs[4] = {s4.x, s4.y, s4.z, s4.w};
        const float bis[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = 4 * v + u;
            const float vf =
                __fsub_rn(__int_as_float(0x4B400000 + ((int)r[c] >> shift)), 12582912.0f);
            float y = __fmaf_rn(vf, scs[u], bis[u]);
            if (RES) {
                const uint32_t qr = (resw[(c * BITS) >> 5] >> ((c * BITS) & 31)) & MASK;
                y = __fadd_rn(y, lut[qr]);
            }
            const float rr = fminf(__fmaf_rn(fmaxf(y, 0.0f), inv, 0.5f), r_hi);
            const uint32_t rb = (uint32_t)__float_as_int(__fadd_rd(rr, 8388608.0f));
            cw[(c * BITS) >> 5] += rb << ((c * BITS) & 31);
        }
    }
    // 0x4B000000 summed over the fields of a word (mod 2^32)
    constexpr uint32_t FIELDS = BITS == 4 ? 0x11111111u : 0x55555555u;
#pragma unroll
    for (int w = 0; w < BITS / 2; ++w) cw[w] -= 0x4B000000u * FIELDS;
}

// Position in the padded, stacked numbering: image, padded row, padded column.
// Moving by a fixed number of positions is an addition of its (host-made)
// decomposition plus at most one carry per digit: no division in any loop.
struct W3Pos {
    int n, h, w;
};
__device__ __forceinline__ W3Pos w3_add(W3Pos a, int dn, int dh, int dw, int Hp, int Wp)
{
    a.w += dw;
    a.h += dh;
    a.n += dn;
    if (a.w >= Wp) { a.w -= Wp; ++a.h; }
    if (a.h >= Hp) { a.h -= Hp; ++a.n; }
    return a;
}

// Transposed tiles (template parameter TR).  An instruction whose A operand
// comes through a shared-memory descriptor takes ~130 clocks whatever its N, so
// it should carry N = 256.  With the roles swapped - A = 128 weight rows of the K
// step, B = 256 rows of the window - every instruction is 128 x 256 x 32 even
// for 64 or 128 output channels.  The accumulator then has output CHANNELS on
// the tensor-memory lanes and POSITIONS in the columns: an epilogue thread owns
// one channel, gathers its codes of 8 (16 at 2 bits) positions in a word and an
// 8 x 8 (16 x 16) transpose of bit fields across the lanes of a channel group
// (shuffles) turns that into the packed NHWC words of those positions.
template <int BITS>
__device__ __forceinline__ uint32_t w3_transpose_fields(uint32_t x, int lane)
{
    constexpr int E = 32 / BITS;                 // fields per word = lanes per group
#pragma unroll
    for (int d = E / 2; d >= 1; d >>= 1) {
        const int block = BITS * d;
        const uint32_t M = block == 16 ? 0x0000FFFFu : block == 8 ? 0x00FF00FFu
                           : block == 4 ? 0x0F0F0F0Fu : 0x33333333u;
        const uint32_t px = __shfl_xor_sync(0xffffffffu, x, d);
        x = (lane & d) ? (((px >> block) & M) | (x & ~M)) : ((x & M) | ((px << block) & ~M));
    }
    return x;
}

template <int BITS, int EPI, bool TR>
__global__ void __launch_bounds__(W3_THREADS, 1)
dsq_win3_kernel(const __grid_constant__ CUtensorMap tmap_b,
                const __grid_constant__ CUtensorMap tmap_a, const W3Params p)
{
    constexpr int CH = Chunks<BITS>::CH;       // packed 16-byte chunks per 128 codes
    constexpr int OUT = Chunks<BITS>::OUT;     // int8 chunks per packed chunk
    constexpr int TP = TR ? 256 : W3_BM;       // positions of a tile
    static_assert(!TR || BITS != 3, "transposed tiles: 2- and 4-bit codes");
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    if ((threadIdx.x >> 5) == 1) W3_STAMP(13, 0);
    uint8_t *smem = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~(uintptr_t)1023u);
    const int BN = p.BN;
    // (the layout comes ready-made: every warp's first instructions are on the
    // critical path of a launch)
    const W3Smem &L = p.L;
    if ((uint32_t)(smem - smem_raw) + L.total > (uint32_t)p.smem_bytes) {
        grid_dependency_wait();
        if (threadIdx.x == 0) atomicCAS(p.ws + DSQ_WS_STATUS, 0, (int)DSQ_ERR_UNSUPPORTED);
        return;
    }
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    // CTA c works on N tile c % n_tiles and on the M tiles m_first, m_first +
    // mstep, ... (the grid is a multiple of n_tiles)
    const int n_tile = p.n_tiles == 1 ? 0 : (int)blockIdx.x % p.n_tiles;
    const int m_first = p.n_tiles == 1 ? (int)blockIdx.x : (int)blockIdx.x / p.n_tiles;
    const int my_tiles = m_first < p.m_tiles ? (p.m_tiles - 1 - m_first) / p.mstep + 1 : 0;
    const uint32_t n_b_fills =
        my_tiles == 0 ? 0u : (p.b_res ? (uint32_t)p.ksteps : (uint32_t)my_tiles * p.ksteps);
    const uint32_t n_a_fills = (uint32_t)my_tiles * p.npl;
    const uint32_t a_slot_bytes = (uint32_t)p.apx * 128u;
    const uint32_t a_stage_bytes = (uint32_t)p.apx * p.PB;
    const uint32_t b_stage_bytes = (uint32_t)BN * 128u;
    const uint32_t b_packed_bytes = (uint32_t)BN * 16u * BITS;
    const int img_positions = p.Hp * p.Wp;

    const uint32_t bars = smem_u32(smem + L.bars);
    auto bar_a_full = [&](int s) { return bars + 8u * s; };
    auto bar_a_empty = [&](int s) { return bars + 8u * (W3_A_SLOTS + s); };
    constexpr int O_AS = 2 * W3_A_SLOTS;
    auto bar_as_full = [&](int s) { return bars + 8u * (O_AS + s); };
    auto bar_as_empty = [&](int s) { return bars + 8u * (O_AS + W3_MAX_AS + s); };
    constexpr int O_BP = O_AS + 2 * W3_MAX_AS;
    auto bar_bp_full = [&](int s) { return bars + 8u * (O_BP + s); };
    auto bar_bp_empty = [&](int s) { return bars + 8u * (O_BP + W3_MAX_BP + s); };
    constexpr int O_B = O_BP + 2 * W3_MAX_BP;
    auto bar_b_full = [&](int s) { return bars + 8u * (O_B + s); };
    auto bar_b_empty = [&](int s) { return bars + 8u * (O_B + W3_MAX_BST + s); };
    constexpr int O_ACC = O_B + 2 * W3_MAX_BST;
    auto bar_acc_full = [&](int s) { return bars + 8u * (O_ACC + s); };
    auto bar_acc_empty = [&](int s) { return bars + 8u * (O_ACC + 2 + s); };
    const uint32_t bar_drain = bars + 8u * (O_ACC + 4);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L.tmem_slot);
    Ctl ctl{reinterpret_cast<volatile int *>(smem + L.abort_flag), p.ws, p.wait_ns};

    if (warp == 0) W3_STAMP(13, 9);
    if (threadIdx.x == 0) {
        for (int s = 0; s < W3_A_SLOTS; ++s) {
            mbar_init(bar_a_full(s), W3_NUM_A_WARPS);
            mbar_init(bar_a_empty(s), 1);            // tcgen05.commit
        }
        for (int s = 0; s < W3_MAX_AS; ++s) {
            mbar_init(bar_as_full(s), 1);            // TMA producer (+ bytes)
            mbar_init(bar_as_empty(s), W3_NUM_A_WARPS);
        }
        for (int s = 0; s < W3_MAX_BP; ++s) {
            mbar_init(bar_bp_full(s), 1);            // TMA producer (+ bytes)
            mbar_init(bar_bp_empty(s), W3_B_GROUP_WARPS);
        }
        for (int s = 0; s < W3_MAX_BST; ++s) {
            mbar_init(bar_b_full(s), p.w8 ? 1 : W3_B_GROUP_WARPS);   // (w8: TMA producer + bytes)
            mbar_init(bar_b_empty(s), 1);            // tcgen05.commit
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_acc_full(s), 1);           // tcgen05.commit
            mbar_init(bar_acc_empty(s), W3_NUM_E_WARPS);
        }
        mbar_init(bar_drain, 1);
        *ctl.abort_flag = 0;
        W3_STAMP(13, 10);
        mbar_init_fence();
        W3_STAMP(13, 11);
    }
    if (warp == W3_WARP_MMA) {
        W3_STAMP(13, 5);
        tmem_alloc(smem_u32((const void *)tmem_slot), 512);
        tmem_relinquish();
        W3_STAMP(13, 6);
        // A descriptor offsets (16-byte units from the start of a slot) of the
        // four instructions of every K step of a plane; 0xFFFFFFFF = no
        // instruction (the half-empty last K step of a 64-channel input)
        uint32_t *tab = reinterpret_cast<uint32_t *>(smem + L.a_tab);
        for (int i = lane; i < 4 * p.kpp; i += 32) {
            const int kk = i >> 2, j = i & 3;
            const int tap = p.two_taps ? 2 * kk + (j >> 1) : kk;
            const int within = p.two_taps ? 32 * (j & 1) : 32 * j;
            const int kh = tap / 3, kw = tap - 3 * kh;
            tab[i] = tap < 9 && within < p.E
                         ? (uint32_t)((kh * p.tap_stride + kw) * 8 + (within >> 4))
                         : 0xFFFFFFFFu;
        }
    }
    if (warp == W3_WARP_TMA_B && lane == 0) tma_prefetch_desc(&tmap_b);
    if (warp == W3_WARP_TMA_A && lane == 0) tma_prefetch_desc(&tmap_a);
    // residual table: the 2^BITS dequantised residual values
    if (EPI != DSQ_EPI_CODES && threadIdx.x >= 64 && threadIdx.x < 64 + (1 << BITS)) {
        const int q = threadIdx.x - 64;
        reinterpret_cast<float *>(smem + L.lut)[q] = __fmaf_rn((float)q, p.e.res_delta, p.e.res_lo);
    }
    // the window producer's first position (two divisions on one lane), worked out
    // here, where the warp would otherwise only wait for the slower warps at the
    // barrier: it is on the critical path of a launch
    W3Pos a_base0 = {0, 0, 0};
    if (warp == W3_WARP_TMA_A && lane == 0) {
        const int g0 = m_first * TP;
        a_base0.n = g0 / img_positions;
        const int rem = g0 - a_base0.n * img_positions;
        a_base0.h = rem / p.Wp;
        a_base0.w = rem - a_base0.h * p.Wp;
    }
    if (warp == W3_WARP_MMA) W3_STAMP(13, 7);
    if (warp == W3_WARP_E0) W3_STAMP(13, 8);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
    // everything above touched no global data; nothing below starts before the
    // kernels ahead of this one in the stream have completed
    W3_STAMP(13, 1);
    grid_launch_dependents();
    // (the window producer first works out its coordinates, then waits)
    if (warp != W3_WARP_TMA_A) grid_dependency_wait();
    W3_STAMP(13, 2);

    if (warp == W3_WARP_TMA_B) {
        // ---------------- producer: packed B rows of one K step ------------------
        if (lane == 0 && p.w8) {
            // weights already expanded (blob's int8 copy): K step g of this CTA's
            // sequence goes straight into stage g % b_stages of the operand ring
            uint32_t issued = 0, ph = 0;
            const int BST = p.b_stages;
            const int y = n_tile * BN;
            int s = 0, x = 0;
#pragma unroll 1
            for (uint32_t g = 0; g < n_b_fills; ++g) {
                if (!wait_bar(bar_b_empty(s), ph ^ 1u, ctl, 1)) break;
                if ((int)g == p.skip_b_round) break;
                mbar_arrive_expect_tx(bar_b_full(s), b_stage_bytes);
                tma_load_2d(smem_u32(smem + L.b_tiles + s * b_stage_bytes), &tmap_b, x, y,
                            bar_b_full(s));
                if (p.dup)     // the map's box is 64 rows: the same rows again behind them
                    tma_load_2d(smem_u32(smem + L.b_tiles + s * b_stage_bytes + 64 * 128), &tmap_b,
                                x, y, bar_b_full(s));
                ++issued;
                x += 128;
                if (x == p.ksteps * 128) x = 0;
                if (++s == BST) { s = 0; ph ^= 1u; }
            }
            for (uint32_t k = (issued > (uint32_t)BST ? issued - BST : 0); k < issued; ++k)
                wait_bar_drain(bar_b_full(k % BST), (k / BST) & 1u);
        } else if (lane == 0) {
            uint32_t issued = 0, ph = 0;
            const int BP = p.bp_slots;
            const int y = n_tile * BN;
            // byte offset of a K step in a weight row of 9 taps x Cin codes: tap kk,
            // plane pl (64-channel inputs: two taps per K step)
            const int xstep = p.xstep;
            int s = 0, kk = 0, xk = 0, xpl = 0;
#pragma unroll 1
            for (uint32_t g = 0; g < n_b_fills; ++g) {
                if (!wait_bar(bar_bp_empty(s), ph ^ 1u, ctl, 1)) break;
                if ((int)g == p.skip_b_round) break;
                mbar_arrive_expect_tx(bar_bp_full(s), b_packed_bytes);
                tma_load_2d(smem_u32(smem + L.b_packed + s * b_packed_bytes), &tmap_b, xk + xpl, y,
                            bar_bp_full(s));
                ++issued;
                W3_STAMP(12, g);
                xk += xstep;
                if (++kk == p.kpp) {
                    kk = 0; xk = 0;
                    xpl += 16 * BITS;
                    if (xpl == p.npl * 16 * BITS) xpl = 0;
                }
                if (++s == BP) { s = 0; ph ^= 1u; }
            }
            for (uint32_t k = (issued > (uint32_t)BP ? issued - BP : 0); k < issued; ++k)
                wait_bar_drain(bar_bp_full(k % BP), (k / BP) & 1u);
        }
    } else if (warp == W3_WARP_TMA_A) {
        // ---------------- producer: packed window of a tile and plane ------------
        if (lane != 0) grid_dependency_wait();
        if (lane == 0) {
            uint32_t issued = 0, ph = 0;
            const int AS = p.as_slots;
            const int nld = p.nbands * p.a_nload;
            int s = 0, pl = 0;
            // The start coordinates of a fill's loads are worked out one fill ahead
            // (the first before anything can be issued), so that between the
            // moment a slot is free and the copies only the issue itself remains.
            // Loads that start behind the last image hold nothing a valid output
            // reads: they are left out (and not counted).  An im2col load must
            // start inside the map's bounding box (0 <= h < Hp, 0 <= w < Wp, n >= 0,
            // which the position arithmetic guarantees): a position outside it is
            // never issued - the roles then run into their wait limit and the
            // kernel reports the failure.
            W3Pos base = a_base0;
            W3Pos q[3];
            int nl = 0;
            bool bad = false;
            auto prepare = [&]() {
                nl = 0;
                bad = false;
#pragma unroll
                for (int i = 0; i < 3; ++i) {
                    if (i >= nld) break;
                    q[i] = w3_add(base, p.ld_dn[i], p.ld_dh[i], p.ld_dw[i], p.Hp, p.Wp);
                    if (q[i].n < p.N) {
                        ++nl;
                        bad |= q[i].n < 0 || q[i].h < 0 || q[i].h >= p.Hp || q[i].w < 0 || q[i].w >= p.Wp;
                    }
                }
            };
            prepare();
            grid_dependency_wait();
#pragma unroll 1
            for (uint32_t g = 0; g < n_a_fills; ++g) {
                if (!wait_bar(bar_as_empty(s), ph ^ 1u, ctl, 11)) break;
                if (bad) {
                    if (atomicCAS(p.ws + DSQ_WS_STATUS, 0, (int)DSQ_ERR_SHAPE) == 0)
                        p.ws[DSQ_WS_DETAIL] = 16;
                    *ctl.abort_flag = 1;
                    break;
                }
                mbar_arrive_expect_tx(bar_as_full(s), (uint32_t)(nl * p.a_box * p.PB));
                const uint32_t dst0 = smem_u32(smem + L.a_stage) + s * a_stage_bytes;
#pragma unroll
                for (int i = 0; i < 3; ++i) {
                    if (i >= nld) break;
                    if (q[i].n >= p.N) continue;
                    // bounding box = image grown by one pixel: base positions
                    // -2 .. W-1 / -2 .. H-1, filter offset (1, 1)
                    tma_load_im2col_4d(dst0 + (uint32_t)(i * p.a_box * p.PB), &tmap_a, pl * p.PB,
                                       q[i].w - 2, q[i].h - 2, q[i].n, (uint16_t)1, (uint16_t)1,
                                       bar_as_full(s));
                }
                ++issued;
                W3_STAMP(0, g);
                if (++pl == p.npl) {
                    pl = 0;
                    base = w3_add(base, p.t_dn, p.t_dh, p.t_dw, p.Hp, p.Wp);
                    prepare();
                }
                if (++s == AS) { s = 0; ph ^= 1u; }
            }
            for (uint32_t k = (issued > (uint32_t)AS ? issued - AS : 0); k < issued; ++k)
                wait_bar_drain(bar_as_full(k % AS), (k / AS) & 1u);
        }
    } else if (warp == W3_WARP_MMA) {
        // ---------------- MMA issuer (whole warp, uniform; one lane issues) --------
        // (TR: A = 128 weight rows, signed; B = 256 window rows, unsigned)
        const uint32_t idesc = TR ? idesc_i8(256, true, false, 128) : idesc_i8(BN, false, true, W3_BM);
        const uint64_t desc0 = smem_desc_sw128(0u);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32), desc_lo = (uint32_t)desc0;
        const uint32_t a_lo_base = desc_lo + (smem_u32(smem + L.a_slots) >> 4);
        const uint32_t b_lo_base = desc_lo + (smem_u32(smem + L.b_tiles) >> 4);
        const uint4 *tab = reinterpret_cast<const uint4 *>(smem + L.a_tab);
        const int BST = p.b_stages;
        int aslot = 0, st = 0;
        uint32_t aph = 0, bph = 0;
        bool ok = true;
#pragma unroll 1
        for (int it = 0; ok && it < my_tiles; ++it) {
            const int as = it & 1;
            if (!(ok = wait_bar_warp(bar_acc_empty(as), ((it >> 1) & 1) ^ 1u, ctl, 3))) break;
            W3_STAMP(4, it);
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + as * (TR ? 256 : BN);
            uint32_t first = 0u;                    // 0: the tile's first instruction overwrites
#pragma unroll 1
            for (int pl = 0; ok && pl < p.npl; ++pl) {
                if (!(ok = wait_bar_warp(bar_a_full(aslot), aph, ctl, 4))) break;
                if (pl == 0) W3_STAMP(5, it);
                tc_fence_after_sync();
                const uint32_t a_lo = a_lo_base + aslot * (a_slot_bytes >> 4);
                if (p.b_res) st = pl * p.kpp;
#pragma unroll 1
                for (int kk = 0; kk < p.kpp; ++kk) {
                    const uint4 t = tab[kk];
                    if (!p.b_res || it == 0) {
                        if (!(ok = wait_bar_warp(bar_b_full(st), bph, ctl, 10))) break;
                        tc_fence_after_sync();
                    }
                    // (a slot lies below 256 KB, so the sums stay inside the
                    // 14-bit address field; 0xFFFFFFFF marks no instruction)
                    if (TR)
                        mma_i8_ss_x4b_elect(d_tmem, b_lo_base + st * (b_stage_bytes >> 4), desc_hi,
                                            a_lo + t.x, t.y == 0xFFFFFFFFu ? t.y : a_lo + t.y,
                                            t.z == 0xFFFFFFFFu ? t.z : a_lo + t.z,
                                            t.w == 0xFFFFFFFFu ? t.w : a_lo + t.w, desc_hi, idesc,
                                            first);
                    else
                    mma_i8_ss_x4_elect(d_tmem, a_lo + t.x, t.y == 0xFFFFFFFFu ? t.y : a_lo + t.y,
                                       t.z == 0xFFFFFFFFu ? t.z : a_lo + t.z,
                                       t.w == 0xFFFFFFFFu ? t.w : a_lo + t.w, desc_hi,
                                       b_lo_base + st * (b_stage_bytes >> 4), desc_hi, idesc, first);
                    first = 1u;
                    if (!p.b_res) {
                        mma_commit_elect(bar_b_empty(st));
                        if (++st == BST) { st = 0; bph ^= 1u; }
                    } else {
                        ++st;
                    }
                }
                if (ok) mma_commit_elect(bar_a_empty(aslot));
                if (++aslot == W3_A_SLOTS) { aslot = 0; aph ^= 1u; }
            }
            if (ok) mma_commit_elect(bar_acc_full(as));
            W3_STAMP(6, it);
        }
        if (!ok) {
            // instructions already issued may still read the operands and write
            // the accumulators: let them finish before memory is given up
            mma_commit_elect(bar_drain);
            wait_bar_drain(bar_drain, 0u);
        }
    } else if (warp < W3_WARP_B0) {
        // ---------------- A: expand the staged window -------------------------------
        const int tid = threadIdx.x - W3_WARP_A0 * 32;
        const int n_tasks = p.apx * p.cpp;
        const int AS = p.as_slots;
        // task t = (pixel, packed chunk) = (t >> lcpp, t & (cpp - 1)); the staged
        // window is dense, so its address is just 16 t
        const int lcpp = p.cpp == 4 ? 2 : p.cpp == 2 ? 1 : 0;
        int ss = 0, slot = 0;
        uint32_t phs = 0, pha = 0;
        bool ok = true;
#pragma unroll 1
        for (uint32_t g = 0; ok && g < n_a_fills; ++g) {
            if (!(ok = wait_bar_warp(bar_as_full(ss), phs, ctl, 12))) break;
            if (warp == W3_WARP_A0) W3_STAMP(1, g);
            if (!(ok = wait_bar_warp(bar_a_empty(slot), pha ^ 1u, ctl, 5))) break;
            if (warp == W3_WARP_A0) W3_STAMP(2, g);
            const uint32_t src = smem_u32(smem + L.a_stage) + ss * a_stage_bytes;
            const uint32_t dst = smem_u32(smem + L.a_slots) + slot * a_slot_bytes;
            if (BITS == 3) {
                // 3-bit rows: one task per pixel (8 codes per 3 bytes from the
                // row's start): its 32 or 48 packed bytes -> 64 or 128 int8 bytes
                const int nq = p.E >= 128 ? 8 : 4;
#pragma unroll 1
                for (int px = tid; px < p.apx; px += W3_NUM_A_WARPS * 32) {
                    uint32_t w[12];
#pragma unroll
                    for (int l = 0; l < 3; ++l) {
                        uint4 v = make_uint4(0u, 0u, 0u, 0u);
                        if (l < p.cpp) v = lds_128(src + (uint32_t)(px * p.PB + 16 * l));
                        w[4 * l] = v.x; w[4 * l + 1] = v.y; w[4 * l + 2] = v.z; w[4 * l + 3] = v.w;
                    }
                    const uint32_t row = dst + (uint32_t)px * 128u;
                    const int sw = px & 7;
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        if (q < nq) {
                            const uint4 c = expand3_chunk<false>(w, q, 0u);
                            sts_128(row + (uint32_t)((q ^ sw) << 4), c.x, c.y, c.z, c.w);
                        }
                }
            } else
#pragma unroll 4
            for (int t = tid; t < n_tasks; t += W3_NUM_A_WARPS * 32) {
                const int px = t >> lcpp, ch = t & (p.cpp - 1);
                const uint4 v = lds_128(src + 16u * t);
                const uint32_t row = dst + (uint32_t)px * 128u;
                const int sw = px & 7;
#pragma unroll
                for (int c = 0; c < OUT; ++c)
                    sts_128(row + (uint32_t)(((ch * OUT + c) ^ sw) << 4),
                            expand_word<BITS, false>(v.x, c, 0u), expand_word<BITS, false>(v.y, c, 0u),
                            expand_word<BITS, false>(v.z, c, 0u), expand_word<BITS, false>(v.w, c, 0u));
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_a_full(slot));
                mbar_arrive(bar_as_empty(ss));
            }
            if (warp == W3_WARP_A0) W3_STAMP(3, g);
            if (++ss == AS) { ss = 0; phs ^= 1u; }
            if (++slot == W3_A_SLOTS) { slot = 0; pha ^= 1u; }
        }
    } else if (warp < W3_WARP_E0) {
        // ---------------- B: expand packed weight rows --------------------------------
        // Two groups of four warps take alternate K steps, so that the latency
        // chains of two steps (barrier, loads, stores, fence, arrival) overlap.
        const int group = (warp - W3_WARP_B0) / W3_B_GROUP_WARPS;
        const int tid = threadIdx.x - (W3_WARP_B0 + group * W3_B_GROUP_WARPS) * 32;
        constexpr int BT = W3_B_GROUP_WARPS * 32;
        constexpr int ROWS_PER_IT = BT / CH;       // a multiple of 8: (row & 7) is the same in every pass
        constexpr int HALF_IT = (128 * CH) / BT;   // passes over 128 rows
        const int row0 = tid / CH, j = tid % CH;
        const int sw = row0 & 7;
        const int BP = p.bp_slots, BST = p.b_stages;
        // own fills: g = group, group + 2, ...
        int sp = group % BP, st = p.b_res ? group : group % BST;
        uint32_t php = (uint32_t)(group / BP) & 1u, phu = p.b_res ? 0u : (uint32_t)(group / BST) & 1u;
        bool ok = !p.w8;                           // (w8: nothing to expand)
#pragma unroll 1
        for (uint32_t g = group; ok && g < n_b_fills; g += 2) {
            if (!(ok = wait_bar_warp(bar_bp_full(sp), php, ctl, 6))) break;
            if (warp == W3_WARP_B0) W3_STAMP(10, g >> 1);
            const uint4 *src = reinterpret_cast<const uint4 *>(smem + L.b_packed + sp * b_packed_bytes);
            uint8_t *rowp = smem + L.b_tiles + st * b_stage_bytes + row0 * 128;
            bool waited = p.b_res != 0;
            if (BITS == 3) {
                // 3-bit rows: one thread per row of 48 packed bytes
                uint32_t w[2][12];
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    if (tid + i * BT < BN) {
                        const uint4 *r4 = reinterpret_cast<const uint4 *>(
                            smem + L.b_packed + sp * b_packed_bytes + (tid + i * BT) * 48);
#pragma unroll
                        for (int l = 0; l < 3; ++l) {
                            const uint4 v = r4[l];
                            w[i][4 * l] = v.x; w[i][4 * l + 1] = v.y;
                            w[i][4 * l + 2] = v.z; w[i][4 * l + 3] = v.w;
                        }
                    }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_bp_empty(sp));
                if (!waited && !(ok = wait_bar_warp(bar_b_empty(st), phu ^ 1u, ctl, 7))) break;
#pragma unroll
                for (int i = 0; i < 2; ++i)
                    if (tid + i * BT < BN) {
                        uint8_t *rp = smem + L.b_tiles + st * b_stage_bytes + (tid + i * BT) * 128;
                        const int sw3 = (tid + i * BT) & 7;
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            *reinterpret_cast<uint4 *>(rp + ((q ^ sw3) << 4)) =
                                expand3_chunk<true>(w[i], q, p.orv);
                    }
            } else
            // 128 rows at a time (register budget)
#pragma unroll 1
            for (int r0 = 0; r0 < BN; r0 += 128) {
                uint4 v[HALF_IT];
#pragma unroll
                for (int i = 0; i < HALF_IT; ++i)
                    if (r0 + row0 + i * ROWS_PER_IT < BN)
                        v[i] = src[(r0 + row0 + i * ROWS_PER_IT) * CH + j];
                if (r0 + 128 >= BN) {
                    // the packed slot is free as soon as every lane holds its chunks
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_bp_empty(sp));
                }
                if (!waited) {
                    if (!(ok = wait_bar_warp(bar_b_empty(st), phu ^ 1u, ctl, 7))) break;
                    waited = true;
                }
#pragma unroll
                for (int i = 0; i < HALF_IT; ++i)
                    if (r0 + row0 + i * ROWS_PER_IT < BN) {
#pragma unroll
                        for (int c = 0; c < OUT; ++c)
                            *reinterpret_cast<uint4 *>(rowp + (r0 + i * ROWS_PER_IT) * 128 +
                                                       (((j * OUT + c) ^ sw) << 4)) =
                                make_uint4(expand_word<BITS, true>(v[i].x, c, p.orv),
                                           expand_word<BITS, true>(v[i].y, c, p.orv),
                                           expand_word<BITS, true>(v[i].z, c, p.orv),
                                           expand_word<BITS, true>(v[i].w, c, p.orv));
                    }
            }
            if (!ok) break;
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_b_full(st));
            if (warp == W3_WARP_B0) W3_STAMP(11, g >> 1);
            sp += 2;
            if (sp >= BP) { sp -= BP; php ^= 1u; }
            if (p.b_res) {
                st += 2;
            } else {
                st += 2;
                if (st >= BST) { st -= BST; phu ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue: four warps per tensor-memory lane quarter -----------
        const int quarter = warp & 3;
        const int k = (warp - W3_WARP_E0) >> 2;              // which of the quarter's warps
        if constexpr (TR) {
            // thread = output channel (tensor-memory lane), columns = positions;
            // warp k of a quarter takes columns 64 k .. 64 k + 63 in units of 16
            constexpr int E = 32 / BITS;                     // positions per code word
            constexpr int CWU = 16 / E;                      // code words per unit: 2 (4-bit), 1 (2-bit)
            constexpr uint32_t MASK = (1u << BITS) - 1u;
            const DsqEpi &e = p.e;
            const float *lut = reinterpret_cast<const float *>(smem + L.lut);
            // (dup: lanes 64..127 repeat channels 0..63; quarters 2, 3 take columns 128..255)
            const int chq = p.dup ? (quarter & 1) * 32 : quarter * 32;
            const int colbase = p.dup ? 128 * (quarter >> 1) + 32 * k : 64 * k;
            const int units = p.dup ? 2 : 4;
            const int ch = n_tile * 128 + chq + lane;
            // a warp has work while its first code word lies inside the output row:
            // channels past Cout are padding lanes of the packed row and get zeros
            // (warp-uniform)
            const bool warp_live = (n_tile * 128 + chq) * BITS / 8 < p.out_pitch;
            float sc = 0.f, bi = 0.f;
            if (ch < p.Ncols) {
                sc = __ldg(e.scale + ch);
                if (e.half_offset) sc = __fmul_rn(sc, 0.5f);
                bi = __ldg(e.bias + ch);
            }
            const int pw = p.out_pitch / 4;                  // words of an output pixel
            const int cg = (n_tile * 128 + chq + (lane & ~(E - 1))) / E;   // this lane group's word
            const uint32_t *res32 = reinterpret_cast<const uint32_t *>(e.residual);
            uint32_t *y32 = reinterpret_cast<uint32_t *>(e.y_codes);
            // output pixel (or -1) of the warp's columns: lane L follows columns
            // colbase + 2 L and colbase + 2 L + 1; the others get them by shuffle
            // (dup: a warp has 32 columns and only asks lanes 0..15)
            W3Pos pos0, pos1;
            {
                const int g0 = m_first * TP + colbase + 2 * lane;
                pos0.n = g0 / img_positions;
                const int rem = g0 - pos0.n * img_positions;
                pos0.h = rem / p.Wp;
                pos0.w = rem - pos0.h * p.Wp;
                pos1 = w3_add(pos0, 0, 0, 1, p.Hp, p.Wp);
            }
            bool ok = true;
#pragma unroll 1
            for (int it = 0; ok && it < my_tiles; ++it) {
                const int as = it & 1;
                const int m0 = (pos0.n < p.N && pos0.h < p.H && pos0.w < p.W)
                                   ? (pos0.n * p.H + pos0.h) * p.W + pos0.w : -1;
                const int m1 = (pos1.n < p.N && pos1.h < p.H && pos1.w < p.W)
                                   ? (pos1.n * p.H + pos1.h) * p.W + pos1.w : -1;
                pos0 = w3_add(pos0, p.t_dn, p.t_dh, p.t_dw, p.Hp, p.Wp);
                pos1 = w3_add(pos1, p.t_dn, p.t_dh, p.t_dw, p.Hp, p.Wp);
                // Word w of a unit covers E positions; lane i of a channel group owns
                // position i of them: it stores that position's word at the end, and it
                // fetches that position's residual word - one unit ahead, the first
                // unit's before the wait for the accumulator, so that the loads'
                // latency is off the path.  The same transpose that turns "E positions
                // of my channel" into "E channels of my position" is its own inverse,
                // so it also turns the fetched words into "residual codes of my channel
                // at E positions".
                int mpn[CWU];
                uint32_t wordn[CWU];
                auto fetch = [&](int u) {
#pragma unroll
                    for (int w = 0; w < CWU; ++w) {
                        const int cpos = 16 * u + w * E + (lane & (E - 1));   // column of the warp
                        const int mp_a = __shfl_sync(0xffffffffu, m0, cpos >> 1);
                        const int mp_b = __shfl_sync(0xffffffffu, m1, cpos >> 1);
                        mpn[w] = (cpos & 1) ? mp_b : mp_a;
                        wordn[w] = 0u;
                        if (EPI != DSQ_EPI_CODES && e.residual && mpn[w] >= 0 && 4 * cg < p.out_pitch)
                            wordn[w] = __ldg(res32 + (int64_t)mpn[w] * pw + cg);
                    }
                };
                if (warp_live) fetch(0);
                if (warp == W3_WARP_E0) W3_STAMP(7, it);
                if (!(ok = wait_bar_warp(bar_acc_full(as), (it >> 1) & 1u, ctl, 8))) break;
                if (warp == W3_WARP_E0) W3_STAMP(8, it);
                tc_fence_after_sync();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + as * 256;
#pragma unroll 1
                for (int u = 0; warp_live && u < units; ++u) {
                    const int col0 = colbase + 16 * u;
                    uint32_t r[16], cw[CWU], resT[CWU];
                    int mp[CWU];
                    __syncwarp();
                    tmem_ld_32x16(taddr + col0, r);
                    uint32_t word[CWU];
#pragma unroll
                    for (int w = 0; w < CWU; ++w) { mp[w] = mpn[w]; word[w] = wordn[w]; }
                    if (u + 1 < units) fetch(u + 1);
#pragma unroll
                    for (int w = 0; w < CWU; ++w) {
                        resT[w] = 0u;
                        if (EPI != DSQ_EPI_CODES) resT[w] = w3_transpose_fields<BITS>(word[w], lane);
                        cw[w] = 0u;
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        // column 16 u + j of the warp: held by lane 8 u + j / 2
                        const int mj = __shfl_sync(0xffffffffu, (j & 1) ? m1 : m0, 8 * u + (j >> 1));
                        const int vi = (int)r[j] >> p.shift;
                        if constexpr (EPI == DSQ_EPI_CODES || EPI == DSQ_EPI_CODES_RES) {
                            const float vf = __fsub_rn(__int_as_float(0x4B400000 + vi), 12582912.0f);
                            float y = __fmaf_rn(vf, sc, bi);
                            if (EPI == DSQ_EPI_CODES_RES) {
                                // (positions without an output and channels past Cout
                                // carry no residual: their codes are not stored / are 0)
                                const uint32_t qr = (resT[(j * BITS) >> 5] >> ((j * BITS) & 31)) & MASK;
                                y = __fadd_rn(y, ch < p.Ncols ? lut[qr] : 0.0f);
                            }
                            const float rr = fminf(__fmaf_rn(fmaxf(y, 0.0f), e.rq.inv, 0.5f), p.r_hi);
                            cw[(j * BITS) >> 5] +=
                                (uint32_t)__float_as_int(__fadd_rd(rr, 8388608.0f)) << ((j * BITS) & 31);
                        } else {
                            if (mj >= 0 && ch < p.Ncols) {
                                if (e.acc_out) e.acc_out[(int64_t)mj * p.Ncols + ch] = vi;
                                float y;
                                if (e.general_offset) {
                                    // S_a of the position (recomputed by every channel's
                                    // thread: this form is not a fast path)
                                    const int wo = mj % p.W, t2 = mj / p.W;
                                    const int s_a = dsq_window_sa<BITS>(p.act, t2 / p.H, t2 % p.H, wo,
                                                                        p.H, p.W, 3, 1, 1, p.P);
                                    y = dsq_epi_y_offset(vi, s_a, e.w_offset, sc, bi);
                                } else {
                                    y = dsq_epi_y(vi, sc, bi);
                                }
                                if (e.residual) {
                                    const uint32_t qr = (resT[(j * BITS) >> 5] >> ((j * BITS) & 31)) & MASK;
                                    y = dsq_epi_residual(y, qr, e.res_delta, e.res_lo);
                                }
                                if (e.has_requant)
                                    cw[(j * BITS) >> 5] |= dsq_code(y, e.rq) << ((j * BITS) & 31);
                                if (e.y_f32) e.y_f32[(int64_t)mj * p.Ncols + ch] = y;
                            }
                        }
                    }
                    if constexpr (EPI == DSQ_EPI_CODES || EPI == DSQ_EPI_CODES_RES) {
                        constexpr uint32_t FIELDS = BITS == 4 ? 0x11111111u : 0x55555555u;
#pragma unroll
                        for (int w = 0; w < CWU; ++w) cw[w] -= 0x4B000000u * FIELDS;
                    }
                    if (e.y_codes) {
                        // fields of E positions of one channel -> fields of the E
                        // channels of this lane group at one position
#pragma unroll
                        for (int w = 0; w < CWU; ++w) {
                            const uint32_t word = w3_transpose_fields<BITS>(cw[w], lane);
                            if (mp[w] >= 0 && 4 * cg < p.out_pitch) y32[(int64_t)mp[w] * pw + cg] = word;
                        }
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty(as));
                if (warp == W3_WARP_E0) W3_STAMP(9, it);
            }
        } else {
        const int row_in_tile = quarter * 32 + lane;
        float *sm_scale = reinterpret_cast<float *>(smem + L.epi);
        float *sm_bias = sm_scale + p.cout_pad;
        const float *lut = reinterpret_cast<const float *>(smem + L.lut);
        const DsqEpi &e = p.e;
        // a unit = the columns whose codes fill whole 32-bit words: 16 columns
        // (32 for 3-bit codes, where 16 would be 6 bytes)
        constexpr int UW = BITS == 3 ? 32 : 16;
        constexpr int CWU = UW * BITS / 32;                  // code words per unit
        // scale (halved for the symmetric weight grid) and bias of every output
        // channel, once per CTA; columns past Cout get 0
        for (int c = threadIdx.x - W3_WARP_E0 * 32; c < p.cout_pad; c += W3_NUM_E_WARPS * 32) {
            float sc = 0.f, bi = 0.f;
            if (c < p.Ncols) {
                sc = __ldg(e.scale + c);
                if (e.half_offset) sc = __fmul_rn(sc, 0.5f);
                bi = __ldg(e.bias + c);
            }
            sm_scale[c] = sc;
            sm_bias[c] = bi;
        }
        named_barrier_sync(1, W3_NUM_E_WARPS * 32);
        const int units = BN / UW;
        // this thread's row of the CTA's first tile: image, row, column in the
        // padded stacked numbering (positions in its padding have no output)
        W3Pos pos;
        {
            const int g0 = m_first * W3_BM + row_in_tile;
            pos.n = g0 / img_positions;
            const int rem = g0 - pos.n * img_positions;
            pos.h = rem / p.Wp;
            pos.w = rem - pos.h * p.Wp;
        }
        bool ok = true;
#pragma unroll 1
        for (int it = 0; ok && it < my_tiles; ++it) {
            const int as = it & 1;
            const bool row_ok = pos.n < p.N && pos.h < p.H && pos.w < p.W;
            const int64_t m = ((int64_t)pos.n * p.H + pos.h) * p.W + pos.w;
            // general weight-grid offset: S_a of this output pixel, summed from
            // the input codes under its 3 x 3 window
            int s_a = 0;
            if (EPI == DSQ_EPI_GENERAL && e.general_offset && row_ok)
                s_a = dsq_window_sa<BITS>(p.act, pos.n, pos.h, pos.w, p.H, p.W, 3, 1, 1, p.P);
            pos = w3_add(pos, p.t_dn, p.t_dh, p.t_dw, p.Hp, p.Wp);
            // residual codes of a unit of this row are fetched one unit ahead (the
            // first unit's while the tile's instructions are still running); the
            // unit loop is not unrolled: the kernel's roles share the instruction
            // caches, and every role runs faster when the whole kernel is small
            uint32_t res_nx[CWU];
            auto fetch_res = [&](int u) {
#pragma unroll
                for (int w = 0; w < CWU; ++w) res_nx[w] = 0u;
                const int byte0 = (n_tile * BN + u * UW) * BITS / 8;
                if (EPI != DSQ_EPI_CODES && e.residual && row_ok && u < units &&
                    byte0 < p.out_pitch) {
                    const uint32_t *rp =
                        reinterpret_cast<const uint32_t *>(e.residual + m * p.out_pitch + byte0);
                    // (a unit of 3-bit codes may reach past the end of the row)
#pragma unroll
                    for (int w = 0; w < CWU; ++w)
                        if (BITS != 3 || byte0 + 4 * w < p.out_pitch) res_nx[w] = __ldg(rp + w);
                }
            };
            fetch_res(k);
            if (warp == W3_WARP_E0) W3_STAMP(7, it);
            if (!(ok = wait_bar_warp(bar_acc_full(as), (it >> 1) & 1u, ctl, 8))) break;
            if (warp == W3_WARP_E0) W3_STAMP(8, it);
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + as * BN;
#pragma unroll 1
            for (int u = k; u < units; u += W3_EPQ) {
                uint32_t r[UW], resw[CWU];
#pragma unroll
                for (int w = 0; w < CWU; ++w) resw[w] = res_nx[w];
                __syncwarp();
                if constexpr (UW == 32) tmem_ld_32x32(taddr + u * UW, r);
                else tmem_ld_32x16(taddr + u * UW, r);
                fetch_res(u + W3_EPQ);
                tmem_ld_wait();
                const int n0 = n_tile * BN + u * UW;
                const int byte0 = n0 * BITS / 8;
                if (!row_ok) continue;
                uint32_t cw[CWU];
                if constexpr (BITS != 3 && (EPI == DSQ_EPI_CODES || EPI == DSQ_EPI_CODES_RES)) {
                    if (byte0 >= p.out_pitch) continue;
                    w3_codes_unit<BITS, EPI == DSQ_EPI_CODES_RES>(
                        r, sm_scale + n0, sm_bias + n0, resw, lut, p.shift, e.rq.inv, p.r_hi, cw);
                } else {
                    constexpr uint32_t MASK = (1u << BITS) - 1u;
#pragma unroll
                    for (int w = 0; w < CWU; ++w) cw[w] = 0u;
#pragma unroll
                    for (int c = 0; c < UW; ++c) {
                        const int v = (int)r[c] >> p.shift;
                        // field c of the unit: word fw, bit fs (a 3-bit field may
                        // straddle two words; never the last word)
                        const int fw = (c * BITS) >> 5, fs = (c * BITS) & 31;
                        const int fw1 = fw + 1 < CWU ? fw + 1 : fw;
                        if (n0 + c < p.Ncols) {
                            if (e.acc_out) e.acc_out[m * p.Ncols + n0 + c] = v;
                            float y = e.general_offset
                                          ? dsq_epi_y_offset(v, s_a, e.w_offset, sm_scale[n0 + c],
                                                             sm_bias[n0 + c])
                                          : dsq_epi_y(v, sm_scale[n0 + c], sm_bias[n0 + c]);
                            if (e.residual) {
                                const uint32_t qr =
                                    __funnelshift_r(resw[fw], fw + 1 < CWU ? resw[fw1] : 0u, fs) & MASK;
                                y = dsq_epi_residual(y, qr, e.res_delta, e.res_lo);
                            }
                            if (e.has_requant) {
                                const uint32_t q = dsq_code(y, e.rq);
                                cw[fw] |= q << fs;
                                if (BITS == 3 && fs > 29) cw[fw1] |= q >> (32 - fs);
                            }
                            if (e.y_f32) e.y_f32[m * p.Ncols + n0 + c] = y;
                        }
                    }
                    if (!e.y_codes || byte0 >= p.out_pitch) continue;
                }
                // columns past Cout are padding lanes of the packed row: zero
                const int nvalid_bits = min(UW, max(0, p.Ncols - n0)) * BITS;
#pragma unroll
                for (int w = 0; w < CWU; ++w) {
                    const int nb = nvalid_bits - 32 * w;
                    cw[w] &= nb >= 32 ? 0xFFFFFFFFu : nb <= 0 ? 0u : ((1u << nb) - 1u);
                }
                uint32_t *dst = reinterpret_cast<uint32_t *>(e.y_codes + m * p.out_pitch + byte0);
                if (CWU == 2)
                    *reinterpret_cast<uint2 *>(dst) = make_uint2(cw[0], cw[CWU - 1]);
                else if (CWU == 3) {
                    // 12 bytes, as far as the row goes
                    dst[0] = cw[0];
                    if (byte0 + 4 < p.out_pitch) dst[1] = cw[1];
                    if (byte0 + 8 < p.out_pitch) dst[2] = cw[CWU - 1];
                    // 3-bit rows: the N tiles may end before the row's pitch does
                    // (64 columns = 24 bytes, pitch 32); the spare bytes are zero
                    if (n_tile == p.n_tiles - 1 && u == units - 1)
                        for (int b = p.cout_pad * BITS / 8; b < p.out_pitch; b += 4)
                            *reinterpret_cast<uint32_t *>(e.y_codes + m * p.out_pitch + b) = 0u;
                } else
                    *dst = cw[0];
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty(as));
            if (warp == W3_WARP_E0) W3_STAMP(9, it);
        }
        }   // !TR
    }

    // ---------------- teardown ------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) W3_STAMP(13, 3);
    if (warp == W3_WARP_MMA) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
        W3_STAMP(13, 4);
    }
}

template <int BITS, int EPI, bool TR = false>
int w3_launch(const CUtensorMap &tb, const CUtensorMap &ta, const W3Params &p, cudaStream_t s,
              int pdl)
{
    static std::atomic<unsigned long long> configured{0ull};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return DSQ_ERR_CUDA;
    const unsigned long long dev_bit = dev < 64 ? 1ull << dev : 0ull;
    if (!(configured.load(std::memory_order_acquire) & dev_bit)) {
        if (cudaFuncSetAttribute(dsq_win3_kernel<BITS, EPI, TR>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 227 * 1024) != cudaSuccess)
            return DSQ_ERR_CUDA;
        configured.fetch_or(dev_bit, std::memory_order_release);
    }
    const int grid = p.mstep * p.n_tiles;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(W3_THREADS);
    cfg.dynamicSmemBytes = (size_t)p.smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    int na = 0;
    if (pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, dsq_win3_kernel<BITS, EPI, TR>, tb, ta, p) != cudaSuccess) {
        cudaGetLastError();
        return DSQ_ERR_CUDA;
    }
    return dsq_launch_status();
}

template <int BITS>
int w3_dispatch(int epi, const CUtensorMap &tb, const CUtensorMap &ta, const W3Params &p,
                cudaStream_t s, int pdl)
{
    if (p.tr) {
        switch (epi) {
        case DSQ_EPI_CODES: return w3_launch<BITS, DSQ_EPI_CODES, true>(tb, ta, p, s, pdl);
        case DSQ_EPI_CODES_RES: return w3_launch<BITS, DSQ_EPI_CODES_RES, true>(tb, ta, p, s, pdl);
        default: return w3_launch<BITS, DSQ_EPI_GENERAL, true>(tb, ta, p, s, pdl);
        }
    }
    switch (epi) {
    case DSQ_EPI_CODES: return w3_launch<BITS, DSQ_EPI_CODES>(tb, ta, p, s, pdl);
    case DSQ_EPI_CODES_RES: return w3_launch<BITS, DSQ_EPI_CODES_RES>(tb, ta, p, s, pdl);
    default: return w3_launch<BITS, DSQ_EPI_GENERAL>(tb, ta, p, s, pdl);
    }
}

}  // namespace

// ---------------------------------------------------------------------------
// pre-expanded weights
// ---------------------------------------------------------------------------
namespace {

// One thread per (row, K step, packed 16-byte chunk): the chunk's OUT int8
// chunks, in the operand's logical order (TMA applies the 128-byte swizzle when
// it copies a tile).  Same expansion as the kernel's own (expand_word), for the
// grid Delta (c + 1/2); bytes past the end of a weight row read as packed
// zeros, as the kernel's TMA loads of the packed rows do.
template <int BITS>
__global__ void __launch_bounds__(256)
w8_build_kernel(const uint8_t *__restrict__ packed, uint8_t *__restrict__ out, int Cout,
                int row_bytes, int ksteps, int kpp, int xstep)
{
    constexpr int CH = Chunks<BITS>::CH, OUT = Chunks<BITS>::OUT;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int j = (int)(idx % CH);
    const int ks = (int)((idx / CH) % ksteps);
    const int64_t row = idx / ((int64_t)CH * ksteps);
    if (row >= Cout) return;
    const int pl = ks / kpp, kk = ks - pl * kpp;
    const int x = kk * xstep + pl * 16 * BITS + 16 * j;        // byte offset in the packed row
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (x < row_bytes) v = *reinterpret_cast<const uint4 *>(packed + row * row_bytes + x);
    const uint32_t orv = 0x01010101u << (7 - BITS);
    uint8_t *dst = out + (row * ksteps + ks) * 128;
#pragma unroll
    for (int c = 0; c < OUT; ++c)
        *reinterpret_cast<uint4 *>(dst + 16 * (j * OUT + c)) =
            make_uint4(expand_word<BITS, true>(v.x, c, orv), expand_word<BITS, true>(v.y, c, orv),
                       expand_word<BITS, true>(v.z, c, orv), expand_word<BITS, true>(v.w, c, orv));
}

}  // namespace

DsqW8Info dsq_w8_info(const dsq_conv_t *conv, int bits)
{
    DsqW8Info w = {0, 0, 0, 0};
    if (!conv || conv->groups != 1 || conv->KH != 3 || conv->KW != 3 || conv->stride != 1 ||
        conv->pad != 1 || (bits != 2 && bits != 4))
        return w;
    const int Cin = conv->Cin;
    if (!(Cin == 64 || (Cin % 128 == 0 && Cin <= 1024))) return w;
    const int npl = Cin == 64 ? 1 : Cin / 128;
    w.enabled = 1;
    w.ksteps = npl * (Cin == 64 ? 5 : 9);
    const size_t packed = (size_t)conv->Cout * 9 * dsq_row_pitch(Cin, bits);
    w.offset = (packed + 1023) / 1024 * 1024;
    w.bytes = (size_t)conv->Cout * w.ksteps * 128;
    return w;
}

int dsq_w8_build(void *blob, const dsq_conv_t *conv, int bits, cudaStream_t stream)
{
    const DsqW8Info w = dsq_w8_info(conv, bits);
    if (!w.enabled) return DSQ_OK;
    const int Cin = conv->Cin;
    const int P = (int)dsq_row_pitch(Cin, bits);
    const int kpp = Cin == 64 ? 5 : 9;
    const int xstep = Cin == 64 ? 16 * bits : P;
    const int64_t threads = (int64_t)conv->Cout * w.ksteps * bits;       // CH = bits
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    const uint8_t *packed = (const uint8_t *)blob;
    uint8_t *out = (uint8_t *)blob + w.offset;
    if (bits == 4)
        w8_build_kernel<4><<<blocks, 256, 0, stream>>>(packed, out, conv->Cout, 9 * P, w.ksteps, kpp, xstep);
    else
        w8_build_kernel<2><<<blocks, 256, 0, stream>>>(packed, out, conv->Cout, 9 * P, w.ksteps, kpp, xstep);
    return cudaGetLastError() == cudaSuccess ? DSQ_OK : DSQ_ERR_CUDA;
}

int dsq_conv3_window(const void *act_codes, const dsq_nhwc_t *shape, int bits,
                     const void *w_packed, const dsq_conv_t *conv, const DsqEpi &e,
                     int epi_kind, int small_acc, void *workspace, cudaStream_t stream)
{
    const DsqLaunchHooks hooks = dsq_launch_hooks();
    if (!hooks.window3) return DSQ_ERR_UNSUPPORTED;
    if (conv->KH != 3 || conv->KW != 3 || conv->stride != 1 || conv->pad != 1)
        return DSQ_ERR_UNSUPPORTED;
    if (bits < 2 || bits > 4) return DSQ_ERR_UNSUPPORTED;
    if (bits == 3) epi_kind = DSQ_EPI_GENERAL;   // the lean codes epilogue packs whole nibbles / pairs
    if (e.general_offset) epi_kind = DSQ_EPI_GENERAL;
    const int Cin = conv->Cin, Cout = conv->Cout;
    if (!(Cin == 64 || (Cin % 128 == 0 && Cin <= 1024))) return DSQ_ERR_UNSUPPORTED;
    if (shape->W + 2 > 32000 || shape->H + 2 > 32000) return DSQ_ERR_UNSUPPORTED;
    // Which kernel (hook value 1 = automatic; measured on the ResNet-18- and
    // VGG-16-shaped layers, per layer, 20 launches back to back):
    //  * transposed tiles wherever they fit, except 7x7-sized images with >= 512
    //    input channels (a handful of tiles with very long K loops, where the
    //    im2col kernel is as fast or faster).  With up to 64 output channels the
    //    transposed form needs the weight rows twice in its A operand (`dup`),
    //    which it only gets from the blob's expanded copy: 64->64 at 56x56 runs
    //    in 18 us against 22.5 us on plain tiles;
    //  * otherwise plain tiles.
    const bool tiny_deep = shape->H * shape->W <= 64 && Cin >= 512;
    if (hooks.window3 == 1 && tiny_deep) return DSQ_ERR_UNSUPPORTED;
    // the lean codes epilogue wants the requantiser range to start at 0, the
    // accumulator to fit the 2^22 conversion trick and floor(r_hi) = qmax
    float r_hi = 0.f;
    if (epi_kind != DSQ_EPI_GENERAL) {
        r_hi = fmaf(e.rq.hi - e.rq.lo, e.rq.inv, 0.5f);
        if (e.rq.lo != 0.0f || !small_acc || (int)floorf(r_hi) != e.rq.qmax)
            epi_kind = DSQ_EPI_GENERAL;
    }
    W3Params p = {};
    p.N = shape->N; p.H = shape->H; p.W = shape->W;
    p.Hp = p.H + 2; p.Wp = p.W + 2;
    const int64_t G = ((int64_t)p.N - 1) * p.Hp * p.Wp + (int64_t)p.H * p.Wp;
    if (G > (1ll << 30)) return DSQ_ERR_UNSUPPORTED;
    p.Ncols = Cout;
    p.E = Cin;
    p.two_taps = Cin == 64 && bits != 3;
    p.npl = Cin == 64 ? 1 : Cin / 128;
    p.kpp = p.two_taps ? 5 : 9;
    p.ksteps = p.npl * p.kpp;
    const int P = (int)dsq_row_pitch(Cin, bits);           // packed bytes per pixel
    p.PB = Cin == 64 ? P : 16 * bits;
    p.cpp = p.PB / 16;
    p.xstep = p.two_taps ? 16 * bits : P;
    // Tiling, window and shared memory for one of the two kernel forms.
    // Transposed (tr): tiles of 256 positions x 128 output channels, A = weights.
    // Plain: 128 positions x up to 256 channels, A = window.
    const DsqW8Info w8 = dsq_w8_info(conv, bits);
    // (plain tiles with up to 64 output channels keep the expanded weights resident in
    // shared memory for the whole CTA anyway: nothing to gain, measured slightly slower)
    const bool w8_ok = hooks.w8 && w8.enabled && e.half_offset && bits != 3;
    auto configure = [&](int tr) -> int {
        p.tr = tr;
        // transposed tiles for <= 64 output channels: the weight rows twice in the
        // A operand (two TMA boxes of the expanded copy), so that all 128 lanes of
        // the accumulator, and all epilogue warps, carry data
        p.dup = tr && Cout <= 64;
        if (p.dup && !w8_ok) return 0;
        p.w8 = w8_ok && (Cout > 64 || p.dup);
        const int tile_pos = tr ? 256 : W3_BM;
        p.m_tiles = (int)((G + tile_pos - 1) / tile_pos);
        p.BN = tr ? 128 : (Cout >= 256 ? 256 : ((Cout + 63) / 64) * 64);
        p.n_tiles = (Cout + p.BN - 1) / p.BN;
        p.cout_pad = p.n_tiles * p.BN;
        if (p.cout_pad > W3_MAX_COUT) return 0;
        const int need = tile_pos + 2 + 2 * p.Wp;
        if (need <= (tr ? 768 : W3_MAX_WINDOW_PX)) {
            p.nbands = 1;
            p.a_nload = (need + 255) / 256;
            p.a_box = (((need + p.a_nload - 1) / p.a_nload) + 7) / 8 * 8;
            p.band_px = p.a_nload * p.a_box;
            p.apx = p.band_px;
            p.tap_stride = p.Wp;
        } else if (!tr) {
            p.nbands = 3;
            p.a_nload = 1;
            p.a_box = W3_BAND_PX;
            p.band_px = W3_BAND_PX;
            p.apx = 3 * W3_BAND_PX;
            p.tap_stride = W3_BAND_PX;
        } else {
            return 0;
        }
        // shared memory: resident B where one N tile's K steps all fit, else rings
        p.b_res = 0;
        if (p.ksteps <= W3_MAX_BST) {
            for (int as = W3_MAX_AS; as >= 2; --as) {
                const int bp = p.w8 ? 0 : 2;
                const W3Smem L = w3_layout(p.apx, p.BN, bits, p.PB, as, p.ksteps, bp, p.cout_pad);
                if (L.total + 1024 <= 227u * 1024u) {
                    p.b_res = 1; p.b_stages = p.ksteps; p.as_slots = as; p.bp_slots = bp;
                    return 1;
                }
            }
        }
        // {A staging slots, expanded B stages, packed B slots}: the packed ring is
        // what hides the latency of the weight loads, so it goes first
        if (p.w8) {
            // no packed ring: the operand ring itself hides the latency of the loads
            for (int as = W3_MAX_AS; as >= 1; --as)
                for (int bst = 6; bst >= 2; --bst) {
                    const W3Smem L = w3_layout(p.apx, p.BN, bits, p.PB, as, bst, 0, p.cout_pad);
                    if (L.total + 1024 <= 227u * 1024u) {
                        p.as_slots = as; p.b_stages = bst; p.bp_slots = 0;
                        return 1;
                    }
                }
            return 0;
        }
        const int tries[6][3] = {{3, 3, 4}, {2, 3, 4}, {2, 2, 4}, {2, 2, 3}, {2, 2, 2}, {1, 2, 2}};
        for (int t = 0; t < 6; ++t) {
            const W3Smem L = w3_layout(p.apx, p.BN, bits, p.PB, tries[t][0], tries[t][1],
                                       tries[t][2], p.cout_pad);
            if (L.total + 1024 <= 227u * 1024u) {
                p.as_slots = tries[t][0]; p.b_stages = tries[t][1]; p.bp_slots = tries[t][2];
                return 1;
            }
        }
        return 0;
    };
    int found = 0;
    const bool want_tr = hooks.window3 == 3 || hooks.window3 == 1;
    if (bits != 3 && want_tr) found = configure(1);
    if (!found) found = configure(0);
    if (!found) return DSQ_ERR_UNSUPPORTED;
    p.L = w3_layout(p.apx, p.BN, bits, p.PB, p.as_slots, p.b_stages, p.bp_slots, p.cout_pad);
    p.smem_bytes = (int)p.L.total + 1024;
    // grid: a multiple of n_tiles; CTA c takes N tile c % n_tiles and every
    // mstep-th M tile
    const int sms = dsq_sm_count();
    if (sms <= 0) return DSQ_ERR_CUDA;
    p.mstep = sms / p.n_tiles;
    if (p.mstep > p.m_tiles) p.mstep = p.m_tiles;
    if (p.mstep < 1) return DSQ_ERR_UNSUPPORTED;
    {
        const int64_t d = (int64_t)p.mstep * (p.tr ? 256 : W3_BM), img = (int64_t)p.Hp * p.Wp;
        p.t_dn = (int)(d / img);
        p.t_dh = (int)((d % img) / p.Wp);
        p.t_dw = (int)((d % img) % p.Wp);
        for (int b = 0; b < p.nbands; ++b)
            for (int i = 0; i < p.a_nload; ++i) {
                // (every digit below its base, so that one carry per digit is
                // enough when the kernel adds them to a position)
                const int off = p.nbands > 1 ? b * p.Wp : i * p.a_box;
                p.ld_dn[b * p.a_nload + i] = (int)(off / img);
                p.ld_dh[b * p.a_nload + i] = (int)((off % img) / p.Wp);
                p.ld_dw[b * p.a_nload + i] = (int)((off % img) % p.Wp);
            }
    }
    p.wait_ns = hooks.wait_ns;
    p.skip_b_round = hooks.skip_b_round;
    p.base_offset_mode = hooks.window3 == 2;   // (probe)
    p.e = e;
    p.r_hi = r_hi;
    p.out_pitch = (int)dsq_row_pitch(Cout, bits);
    if (e.half_offset) {
        p.shift = 7 - bits;
        p.orv = 0x01010101u << (7 - bits);
    } else {
        p.shift = 8 - bits;
        p.orv = 0;
    }
    p.ws = (int *)workspace;
    p.act = (const uint8_t *)act_codes;
    p.P = P;

    // weights: Cout rows of 9 taps x P bytes; one box = BN rows x one K step
    DsqEncodeTiledFn enc = dsq_encode_tiled_fn();
    DsqEncodeIm2colFn enc_i2c = dsq_encode_im2col_fn();
    if (!enc || !enc_i2c) return DSQ_ERR_CUDA;
    CUtensorMap tb, ta;
    if (p.w8) {
        // the blob's expanded copy: Cout rows of ksteps x 128 bytes; one box = BN
        // rows x one K step, swizzled on the way in
        cuuint64_t dims[2] = {(cuuint64_t)p.ksteps * 128, (cuuint64_t)Cout};
        cuuint64_t strides[1] = {(cuuint64_t)p.ksteps * 128};
        cuuint32_t box[2] = {128u, (cuuint32_t)(p.dup ? 64 : p.BN)};
        cuuint32_t estr[2] = {1, 1};
        if (enc(&tb, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                const_cast<uint8_t *>((const uint8_t *)w_packed + w8.offset), dims, strides, box,
                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DSQ_ERR_CUDA;
    } else {
        cuuint64_t dims[2] = {(cuuint64_t)9 * P, (cuuint64_t)Cout};
        cuuint64_t strides[1] = {(cuuint64_t)9 * P};
        cuuint32_t box[2] = {(cuuint32_t)(16 * bits), (cuuint32_t)p.BN};
        cuuint32_t estr[2] = {1, 1};
        if (enc(&tb, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(w_packed), dims, strides,
                box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DSQ_ERR_CUDA;
    }
    {
        // im2col map over the NHWC codes: the bounding box of base positions is
        // [-2, W-1] x [-2, H-1] (lower corner -2, upper corner 0) and every load
        // uses filter offset (1, 1): pixels -1 .. W / -1 .. H, the image grown by
        // its zero padding
        cuuint64_t dims[4] = {(cuuint64_t)P, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.N};
        cuuint64_t strides[3] = {(cuuint64_t)P, (cuuint64_t)P * p.W, (cuuint64_t)P * p.W * p.H};
        int lower[2] = {-2, -2};
        int upper[2] = {0, 0};
        cuuint32_t estr[4] = {1, 1, 1, 1};
        if (enc_i2c(&ta, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(act_codes), dims,
                    strides, lower, upper, (cuuint32_t)p.PB, (cuuint32_t)p.a_box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DSQ_ERR_UNSUPPORTED;
    }
    if (bits == 4) return w3_dispatch<4>(epi_kind, tb, ta, p, stream, hooks.pdl);
    if (bits == 3) return w3_launch<3, DSQ_EPI_GENERAL>(tb, ta, p, stream, hooks.pdl);
    return w3_dispatch<2>(epi_kind, tb, ta, p, stream, hooks.pdl);
}
