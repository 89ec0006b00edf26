// Large low-bit GEMMs in two passes (paper Sec. 3.5: the quantised layer as a
// GEMM over codes; Algorithm 1 step 5 on codes).
//
// The fused kernel (dsq_tc.cu) expands the packed codes of BOTH operands to
// 8-bit lanes again for every output tile: a 4096^3 problem expands each A row
// 16 times and each B row 16 times, and that expansion (shared-memory
// bandwidth, cluster-scope hand-over of the expanded halves) is what bounds it.
// Here every row is expanded ONCE:
//   pass 1  expand_rows_kernel: packed codes -> int8 rows in a scratch area
//           the caller provides (M*Kp + N*Kp bytes, Kp = K rounded up to 16;
//           HBM / L2-bound, a few microseconds);
//   pass 2  gemm8_kernel: an 8-bit integer GEMM whose operands go from that
//           scratch straight into swizzled shared memory by TMA - no thread
//           touches an operand byte.  CTA pairs on 256 x 256 tiles
//           (tcgen05.mma cta_group::2, kind::i8, both operands through
//           shared-memory descriptors: at N = 256 a descriptor-fed instruction
//           runs at the pipe's full rate), a ring of seven 32 KB stages per CTA,
//           and TWO 256-column accumulators in tensor memory, so the epilogue
//           of a tile (eight warps per CTA) overlaps the next tile's
//           instructions.
// The scratch for 4096^3 is 33.5 MB and stays in the 126 MB L2 between the
// passes.
//
// Every mbarrier wait is bounded (see dsq_tc_common.cuh).
#include <algorithm>
#include <atomic>
#include <cstdint>

#include "dsq_common.cuh"
#include "dsq_tc_common.cuh"
#include "dsq_tc_host.h"

namespace {

constexpr int G8_ROWS = 128;                 // operand rows per CTA and stage (A and B alike)
constexpr int G8_BN = 256;                   // tile width (both CTAs' B halves)
constexpr int G8_BM = 256;                   // tile height of a pair
constexpr int G8_KB = 128;                   // bytes of K per stage
constexpr int G8_STAGES = 7;
constexpr int G8_OP_BYTES = G8_ROWS * G8_KB;             // 16 KB
constexpr int G8_STAGE_BYTES = 2 * G8_OP_BYTES;          // A then B
constexpr int G8_WARP_TMA = 0, G8_WARP_MMA = 1, G8_WARP_TMEM = 2, G8_WARP_E0 = 4;
constexpr int G8_E_WARPS = 8;                // per CTA: two per tensor-memory lane quarter
constexpr int G8_THREADS = 32 * (G8_WARP_E0 + G8_E_WARPS);
constexpr int G8_BARS = 2 * G8_STAGES + 4 + 1;
constexpr int G8_SMEM = G8_STAGES * G8_STAGE_BYTES + 1024 /* alignment */ + 256 /* barriers */;

struct G8Params {
    int M, N;
    int m_tiles, n_tiles, kblocks;
    uint32_t idesc;          // instruction descriptor (operand types, M = 256, N = 256)
    // integer problems: C = acc, D = (float)acc * row_scale[m]
    int32_t *C_i32;
    const float *row_scale;
    float *D_f32;
    // floating-point problems: Y = fma(acc, col_scale[n], col_bias[n])
    const float *col_scale;
    const float *col_bias;   // nullable
    float *Y_f32;
    int *ws;
    unsigned long long wait_ns;
};

// ---------------------------------------------------------------------------
// pass 1: packed codes -> int8.  One thread per 16 codes (16 output bytes).
// ---------------------------------------------------------------------------
// bytes (each < 2^BITS) -> two's-complement int8 of the BITS-bit signed code
template <int BITS>
__device__ __forceinline__ uint32_t sign_extend_bytes(uint32_t x)
{
    constexpr uint32_t HALF = 0x01010101u * (1u << (BITS - 1));
    // per byte (x ^ half) - half without borrows between bytes
    return (((x ^ HALF) | 0x80808080u) - HALF) ^ 0x80808080u;
}

// 16 codes (2 BITS bytes at `src`) -> 16 bytes
template <int BITS>
__device__ __forceinline__ uint4 expand_chunk(const uint8_t *src, int bytes_left, bool is_signed)
{
    uint32_t o[4];
    if (BITS == 4) {
        const uint2 v = __ldcs(reinterpret_cast<const uint2 *>(src));
        const uint32_t w[2] = {v.x, v.y};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t lo = w[h] & 0x0F0F0F0Fu, hi = (w[h] >> 4) & 0x0F0F0F0Fu;
            o[2 * h] = __byte_perm(lo, hi, 0x5140);       // codes 0..3 of the word
            o[2 * h + 1] = __byte_perm(lo, hi, 0x7362);   // codes 4..7
        }
    } else if (BITS == 2) {
        const uint32_t v = __ldcs(reinterpret_cast<const uint32_t *>(src));
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t x = (v >> (8 * j)) & 0xFFu;    // four codes
            o[j] = (x | (x << 6) | (x << 12) | (x << 18)) & 0x03030303u;
        }
    } else {
        // 16 codes of 3 bits = 6 bytes at an even offset; a row's last chunk may
        // reach past the row pitch: those bytes are not read
        uint64_t v = 0;
#pragma unroll
        for (int j = 0; j < 3; ++j)
            if (2 * j < bytes_left)
                v |= (uint64_t) * reinterpret_cast<const uint16_t *>(src + 2 * j) << (16 * j);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t x = 0;
#pragma unroll
            for (int t = 0; t < 4; ++t)
                x |= (uint32_t)((v >> (3 * (4 * j + t))) & 7u) << (8 * t);
            o[j] = x;
        }
    }
    if (is_signed) {
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = sign_extend_bytes<BITS>(o[j]);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// One thread per four consecutive chunks of a row (64 output bytes).  Codes
// past K inside a row's last chunk are spare bits of the packed row: zero.
template <int BITS>
__global__ void __launch_bounds__(256)
expand_rows_kernel(const uint8_t *__restrict__ A, const uint8_t *__restrict__ B, int64_t M,
                   int64_t N, int pitch_in, int pitch_out, uint8_t *__restrict__ A8,
                   uint8_t *__restrict__ B8)
{
    // lets the second pass (queued behind with programmatic dependent launch)
    // set itself up while this grid runs; it waits for this grid to complete
    // before its first copy
    grid_launch_dependents();
    const int cpr = pitch_out >> 4;                       // 16-byte chunks per output row
    const int qpr = (cpr + 3) >> 2;                       // work items per row
    const int64_t total = (M + N) * qpr;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = idx / qpr;
        const int c0 = (int)(idx - row * qpr) * 4;
        const bool is_a = row < M;                        // A: signed codes, B: unsigned
        const uint8_t *src = is_a ? A + row * pitch_in : B + (row - M) * pitch_in;
        uint8_t *dst = is_a ? A8 + row * pitch_out : B8 + (row - M) * pitch_out;
        uint4 o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (c0 + j < cpr)
                o[j] = expand_chunk<BITS>(src + (c0 + j) * (2 * BITS),
                                          pitch_in - (c0 + j) * (2 * BITS), is_a);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (c0 + j < cpr) *reinterpret_cast<uint4 *>(dst + (c0 + j) * 16) = o[j];
    }
}

// Binary operands (Eq. 1): bit 1 -> +1, bit 0 -> -1; positions past K -> 0, so
// the row tail adds nothing.  One thread per 16 codes of either operand.
__global__ void __launch_bounds__(256)
expand_binary_kernel(const uint8_t *__restrict__ A, const uint8_t *__restrict__ B, int64_t M,
                     int64_t N, int K, int pitch_in, int pitch_out, uint8_t *__restrict__ A8,
                     uint8_t *__restrict__ B8)
{
    const int cpr = pitch_out >> 4;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t row = idx / cpr;
    const int c = (int)(idx - row * cpr);
    if (row >= M + N) return;
    const bool is_a = row < M;
    const uint8_t *src = (is_a ? A + row * pitch_in : B + (row - M) * pitch_in) + 2 * c;
    const uint32_t v = *reinterpret_cast<const uint16_t *>(src);
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        // four bits -> the low bits of four bytes, then 2 x - 1 per byte
        const uint32_t x = (((v >> (4 * j)) & 0xFu) * 0x00204081u) & 0x01010101u;
        uint32_t y = (((x << 1) | 0x80808080u) - 0x01010101u) ^ 0x80808080u;
        const int left = K - (16 * c + 4 * j);            // codes of this word inside the row
        if (left < 4) y = left <= 0 ? 0u : (y & (0xFFFFFFFFu >> (8 * (4 - left))));
        o[j] = y;
    }
    uint8_t *dst = (is_a ? A8 + row * pitch_out : B8 + (row - M) * pitch_out) + c * 16;
    *reinterpret_cast<uint4 *>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
}

// Weight codes -> bf16: value 2c + 1 (grid Delta (c + 1/2), `odd` != 0) or c, c
// the signed BITS-bit code; positions past K -> 0.  One thread per 8 codes
// (BITS input bytes, 16 output bytes).
template <int BITS>
__global__ void __launch_bounds__(256)
expand_w_bf16_kernel(const uint8_t *__restrict__ W, int64_t N, int K, int pitch_in, int pitch_out,
                     int odd, uint8_t *__restrict__ W16)
{
    const int cpr = pitch_out >> 4;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t row = idx / cpr;
    const int c = (int)(idx - row * cpr);
    if (row >= N) return;
    const uint8_t *src = W + row * pitch_in + c * BITS;
    uint32_t v = 0;
#pragma unroll
    for (int j = 0; j < BITS; ++j)
        if (c * BITS + j < pitch_in) v |= (uint32_t)src[j] << (8 * j);
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t pair = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int k = 8 * c + 2 * j + t;
            int code = (int)((v >> (BITS * (2 * j + t))) & ((1u << BITS) - 1u));
            if (code >> (BITS - 1)) code -= 1 << BITS;
            const float f = k < K ? (float)(odd ? 2 * code + 1 : code) : 0.0f;
            pair |= (__float_as_uint(f) >> 16) << (16 * t);    // small integers: exact in bf16
        }
        o[j] = pair;
    }
    *reinterpret_cast<uint4 *>(W16 + row * pitch_out + c * 16) = make_uint4(o[0], o[1], o[2], o[3]);
}

// ---------------------------------------------------------------------------
// pass 2: int8 GEMM, CTA pairs
// ---------------------------------------------------------------------------
// F16 = false: 8-bit integer operands, s32 accumulators (kind::i8);
// F16 = true: bf16 operands, f32 accumulators (kind::f16).  A stage row is 128
// bytes of K either way (128 or 64 elements), four instructions per stage.
template <bool F16>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(G8_THREADS, 1)
gemm8_kernel(const __grid_constant__ CUtensorMap tmap_a,
             const __grid_constant__ CUtensorMap tmap_b, const G8Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~(uintptr_t)1023u);
    uint8_t *tail = smem + G8_STAGES * G8_STAGE_BYTES;
    const uint32_t bars = smem_u32(tail);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(tail + 8 * G8_BARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tail + 8 * G8_BARS + 8);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    Ctl ctl{abort_flag, p.ws, p.wait_ns};

    // full: operand bytes of BOTH CTAs' stage s have landed (counted on the
    //       leader's barrier only: the leader's producer expects 64 KB, both
    //       producers' copies complete on it);
    // empty: the pair's instructions on stage s are done (tcgen05.commit,
    //       signalled in both CTAs);
    // acc_full[b]: the tile in accumulator b is complete (both CTAs);
    // acc_empty[b]: (leader) all epilogue warps of both CTAs have read it.
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (G8_STAGES + s); };
    auto bar_acc_full = [&](int b) { return bars + 8u * (2 * G8_STAGES + b); };
    auto bar_acc_empty = [&](int b) { return bars + 8u * (2 * G8_STAGES + 2 + b); };
    const uint32_t bar_drain = bars + 8u * (2 * G8_STAGES + 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < G8_STAGES; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full(b), 1);
            mbar_init(bar_acc_empty(b), 2 * G8_E_WARPS);
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == G8_WARP_TMEM) {
        tmem_alloc<2>(smem_u32((const void *)tmem_slot), 512);
        tmem_relinquish<2>();
    }
    if (warp == G8_WARP_TMA && lane == 0) {
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    tc_fence_before_sync();
    __syncthreads();
    // the peer's barriers must be initialised before anything signals them
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int total_tiles = p.m_tiles * p.n_tiles;
    grid_dependency_wait();

    if (warp == G8_WARP_TMA) {
        // ---------------- TMA producer (one thread per CTA) -----------------
        if (lane == 0) {
            uint32_t g = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < total_tiles; tile += npairs) {
                const int m0 = (tile / p.n_tiles) * G8_BM + (int)rank * G8_ROWS;
                const int n0 = (tile % p.n_tiles) * G8_BN + (int)rank * G8_ROWS;
                for (int kb = 0; kb < p.kblocks; ++kb, ++g) {
                    const int s = g % G8_STAGES;
                    if (!(ok = wait_bar(bar_empty(s), ((g / G8_STAGES) & 1u) ^ 1u, ctl, 21))) break;
                    const uint32_t full0 = map_to_cta(bar_full(s), 0u);
                    if (rank == 0) mbar_arrive_expect_tx(bar_full(s), 2 * G8_STAGE_BYTES);
                    const uint32_t dst = smem_u32(smem + s * G8_STAGE_BYTES);
                    tma_load_2d_pair(dst, &tmap_a, kb * G8_KB, m0, full0);
                    tma_load_2d_pair(dst + G8_OP_BYTES, &tmap_b, kb * G8_KB, n0, full0);
                }
            }
            if (!ok) {
                // copies in flight write this CTA's shared memory: give them time
                const uint64_t t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) { }
            }
        }
    } else if (warp == G8_WARP_MMA) {
        // ---------------- MMA issuer (leader CTA; whole warp, elected lane) ---
        if (rank == 0) {
            const uint32_t idesc = p.idesc;
            uint32_t g = 0, it = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < total_tiles; tile += npairs, ++it) {
                const int b = it & 1;
                if (!(ok = wait_bar_warp<true>(bar_acc_empty(b), ((it >> 1) & 1u) ^ 1u, ctl, 22)))
                    break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + b * G8_BN;
                for (int kb = 0; kb < p.kblocks; ++kb, ++g) {
                    const int s = g % G8_STAGES;
                    if (!(ok = wait_bar_warp<true>(bar_full(s), (g / G8_STAGES) & 1u, ctl, 23)))
                        break;
                    tc_fence_after_sync();
                    const uint64_t ad = smem_desc_sw128(smem_u32(smem + s * G8_STAGE_BYTES));
                    const uint64_t bd =
                        smem_desc_sw128(smem_u32(smem + s * G8_STAGE_BYTES + G8_OP_BYTES));
                    if (F16)
                        mma_f16_ss_pair_x4_elect(d_tmem, (uint32_t)ad, (uint32_t)(ad >> 32),
                                                 (uint32_t)bd, (uint32_t)(bd >> 32), idesc,
                                                 (uint32_t)kb);
                    else
                        mma_i8_ss_pair_x4_elect(d_tmem, (uint32_t)ad, (uint32_t)(ad >> 32),
                                                (uint32_t)bd, (uint32_t)(bd >> 32), idesc,
                                                (uint32_t)kb);
                    mma_commit_pair_elect(bar_empty(s), (uint16_t)3);
                }
                if (ok) mma_commit_pair_elect(bar_acc_full(b), (uint16_t)3);
            }
            if (!ok) {
                // instructions already issued still read shared memory and write
                // the accumulators: they finish before either is given up
                mma_commit_elect(bar_drain);
                wait_bar_drain(bar_drain, 0u);
            }
        }
    } else if (warp >= G8_WARP_E0) {
        // ---------------- epilogue: eight warps per CTA ----------------------
        const int quarter = warp & 3;                      // tensor-memory lane quarter
        const int half = (warp - G8_WARP_E0) >> 2;         // columns [128 half, 128 half + 128)
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; ok && tile < total_tiles; tile += npairs, ++it) {
            const int b = it & 1;
            const int m = (tile / p.n_tiles) * G8_BM + (int)rank * G8_ROWS + quarter * 32 + lane;
            const int n0 = (tile % p.n_tiles) * G8_BN + half * 128;
            if (!(ok = wait_bar_warp(bar_acc_full(b), (it >> 1) & 1u, ctl, 24))) break;
            tc_fence_after_sync();
            const float rs = (!F16 && p.D_f32 && m < p.M) ? __ldg(p.row_scale + m) : 0.0f;
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + b * G8_BN +
                                  half * 128 + c0,
                              r);
                tmem_ld_wait();
                if (c0 == 96) {
                    // the accumulator is in registers: hand it back
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) {
                        if (rank != 0) mbar_arrive_cluster(map_to_cta(bar_acc_empty(b), 0u));
                        else mbar_arrive(bar_acc_empty(b));
                    }
                }
                const int n = n0 + c0;
                if (m >= p.M || n >= p.N) continue;
                const int64_t at = (int64_t)m * p.N + n;
                if (F16) {
                    // Y = fma(acc, col_scale[n], col_bias[n])
                    const bool vec = n + 32 <= p.N &&
                                     (reinterpret_cast<uintptr_t>(p.Y_f32 + at) & 31u) == 0;
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        uint32_t f[8];
#pragma unroll
                        for (int t = 0; t < 8; ++t) {
                            const int nn = min(n + j + t, p.N - 1);
                            const float cb = p.col_bias ? __ldg(p.col_bias + nn) : 0.0f;
                            f[t] = __float_as_uint(
                                __fmaf_rn(__uint_as_float(r[j + t]), __ldg(p.col_scale + nn), cb));
                        }
                        if (vec)
                            stg_256(p.Y_f32 + at + j, f[0], f[1], f[2], f[3], f[4], f[5], f[6], f[7]);
                        else
                            for (int t = 0; t < 8 && n + j + t < p.N; ++t)
                                p.Y_f32[at + j + t] = __uint_as_float(f[t]);
                    }
                    continue;
                }
                const bool vec =
                    n + 32 <= p.N &&
                    (!p.C_i32 || (reinterpret_cast<uintptr_t>(p.C_i32 + at) & 31u) == 0) &&
                    (!p.D_f32 || (reinterpret_cast<uintptr_t>(p.D_f32 + at) & 31u) == 0);
                if (vec) {
                    if (p.C_i32) {
                        int32_t *dst = p.C_i32 + at;
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            stg_256(dst + j, r[j], r[j + 1], r[j + 2], r[j + 3], r[j + 4], r[j + 5],
                                    r[j + 6], r[j + 7]);
                    }
                    if (p.D_f32) {
                        float *dst = p.D_f32 + at;
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            uint32_t f[8];
#pragma unroll
                            for (int t = 0; t < 8; ++t)
                                f[t] = __float_as_uint(__fmul_rn((float)(int)r[j + t], rs));
                            stg_256(dst + j, f[0], f[1], f[2], f[3], f[4], f[5], f[6], f[7]);
                        }
                    }
                } else {
                    for (int j = 0; j < 32 && n + j < p.N; ++j) {
                        if (p.C_i32) p.C_i32[at + j] = (int)r[j];
                        if (p.D_f32) p.D_f32[at + j] = __fmul_rn((float)(int)r[j], rs);
                    }
                }
            }
        }
    }

    // ---------------- teardown ---------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    // a CTA stays until its peer has stopped signalling its barriers and reading
    // operands from its shared memory
    cluster_sync_all();
    if (warp == G8_WARP_TMEM) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc<2>(tmem_base, 512);
    }
}

int make_rows128_tmap(CUtensorMap *map, const void *base, uint64_t k_bytes, uint64_t rows,
                      uint64_t pitch)
{
    DsqEncodeTiledFn fn = dsq_encode_tiled_fn();
    if (!fn) return DSQ_ERR_CUDA;
    cuuint64_t dims[2] = {k_bytes, rows};
    cuuint64_t strides[1] = {pitch};
    cuuint32_t box[2] = {G8_KB, G8_ROWS};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DSQ_OK : DSQ_ERR_CUDA;
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Pass 2 over operands that are rows of k_bytes bytes of K (byte maps: the
// kernel never looks at an element, only the tensor core does).
template <bool F16>
int launch_pass2(const void *A, size_t a_pitch, const void *B, size_t b_pitch, size_t k_bytes,
                 int64_t M, int64_t N, G8Params p, cudaStream_t stream)
{
    p.M = (int)M; p.N = (int)N;
    p.m_tiles = (int)((M + G8_BM - 1) / G8_BM);
    p.n_tiles = (int)((N + G8_BN - 1) / G8_BN);
    p.kblocks = (int)((k_bytes + G8_KB - 1) / G8_KB);
    p.wait_ns = dsq_launch_hooks().wait_ns;
    CUtensorMap ta, tb;
    int st = make_rows128_tmap(&ta, A, k_bytes, (uint64_t)M, a_pitch);
    if (st) return st;
    st = make_rows128_tmap(&tb, B, k_bytes, (uint64_t)N, b_pitch);
    if (st) return st;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= DSQ_MAX_DEVICES) return DSQ_ERR_CUDA;
    static std::atomic<unsigned long long> configured{0};
    if (!(configured.load() >> dev & 1ull)) {
        if (cudaFuncSetAttribute(gemm8_kernel<F16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 G8_SMEM) != cudaSuccess)
            return DSQ_ERR_CUDA;
        configured.fetch_or(1ull << dev);
    }
    const int sms = dsq_sm_count() > 0 ? dsq_sm_count() : 148;
    const int pairs = std::min(sms / 2, p.m_tiles * p.n_tiles);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(G8_THREADS);
    cfg.dynamicSmemBytes = G8_SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    int na = 0;
    if (dsq_launch_hooks().pdl) {
        // set-up overlaps the tail of pass 1; the kernel waits for it itself
        // (griddepcontrol.wait) before the first copy
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, gemm8_kernel<F16>, ta, tb, p) != cudaSuccess) {
        cudaGetLastError();
        return DSQ_ERR_CUDA;
    }
    return DSQ_OK;
}

// first 1024-byte boundary behind the status words of a caller workspace
inline uint8_t *scratch_of(void *workspace)
{
    const uintptr_t w0 = reinterpret_cast<uintptr_t>(workspace);
    return reinterpret_cast<uint8_t *>((w0 + DSQ_WS_BYTES + 1023u) & ~(uintptr_t)1023u);
}

}  // namespace

// Scratch the two-pass path needs behind the status words (0: the problem is
// one the fused kernel keeps).
size_t dsq_gemm8_scratch_bytes(int64_t M, int64_t N, int64_t K, int force)
{
    // below this the fused kernel's single launch wins (measured: 2048^3 takes
    // 22.5 us fused and 25.6 us in two passes, 4096^3 85 and 71 us)
    if (!force && (M < 1024 || N < 1024 || K < 1024 ||
                   (double)M * (double)N * (double)K < 34359738368.0 /* 2^35 */))
        return 0;
    const size_t kp = round_up((size_t)K, 16);
    return round_up((size_t)M * kp, 1024) + round_up((size_t)N * kp, 1024);
}

// Arguments as dsq_gemm after validation; `scratch` 1024-byte aligned.
int dsq_gemm8_launch(const void *A_codes, const void *B_codes, int64_t M, int64_t N, int64_t K,
                     int bits, int32_t *C_i32, const float *row_scale, float *D_f32,
                     void *workspace, void *scratch, cudaStream_t stream)
{
    const size_t kp = round_up((size_t)K, 16);
    uint8_t *A8 = (uint8_t *)scratch;
    uint8_t *B8 = A8 + round_up((size_t)M * kp, 1024);
    const int pitch_in = (int)dsq_row_pitch(K, bits);
    const int64_t threads = (M + N) * (int64_t)((kp / 16 + 3) / 4);
    const int sms = dsq_sm_count() > 0 ? dsq_sm_count() : 148;
    // whole waves of resident blocks (8 per SM), a few items per thread
    const unsigned blocks = (unsigned)std::min<int64_t>((threads + 255) / 256, (int64_t)sms * 8);
    const uint8_t *A = (const uint8_t *)A_codes, *B = (const uint8_t *)B_codes;
    switch (bits) {
    case 2: expand_rows_kernel<2><<<blocks, 256, 0, stream>>>(A, B, M, N, pitch_in, (int)kp, A8, B8); break;
    case 3: expand_rows_kernel<3><<<blocks, 256, 0, stream>>>(A, B, M, N, pitch_in, (int)kp, A8, B8); break;
    default: expand_rows_kernel<4><<<blocks, 256, 0, stream>>>(A, B, M, N, pitch_in, (int)kp, A8, B8); break;
    }
    if (cudaGetLastError() != cudaSuccess) return DSQ_ERR_CUDA;
    G8Params p = {};
    p.idesc = idesc_i8(G8_BN, true, false, G8_BM);
    p.C_i32 = C_i32; p.row_scale = row_scale; p.D_f32 = D_f32;
    p.ws = (int *)workspace;
    return launch_pass2<false>(A8, kp, B8, kp, (size_t)K, M, N, p, stream);
}

// ---------------------------------------------------------------------------
// binary GEMM (both operands 1 bit, values -1 / +1)
// ---------------------------------------------------------------------------
size_t dsq_binary_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K)
{
    if (M <= 0 || N <= 0 || K <= 0) return DSQ_WS_BYTES;
    const size_t kp = round_up((size_t)K, 16);
    return DSQ_WS_BYTES + 1024 + round_up((size_t)M * kp, 1024) + round_up((size_t)N * kp, 1024);
}

int dsq_binary_gemm(const void *A_bits, const void *B_bits, int64_t M, int64_t N, int64_t K,
                    int32_t *C_i32, const float *row_scale, float *D_f32, void *workspace,
                    size_t ws_bytes, void *stream)
{
    if (!A_bits || !B_bits || !workspace) return DSQ_ERR_NULL;
    if (!C_i32 && !D_f32) return DSQ_ERR_NULL;
    if (D_f32 && !row_scale) return DSQ_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || M > (1 << 24) || N > (1 << 24) || K > (1 << 24))
        return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(A_bits) || !dsq_aligned16(B_bits) || !dsq_aligned16(workspace) ||
        (C_i32 && !dsq_aligned16(C_i32)) || (D_f32 && !dsq_aligned16(D_f32)))
        return DSQ_ERR_ALIGN;
    uint8_t *scratch = scratch_of(workspace);
    const size_t kp = round_up((size_t)K, 16);
    const size_t need = round_up((size_t)M * kp, 1024) + round_up((size_t)N * kp, 1024);
    if (ws_bytes < (size_t)(scratch - (uint8_t *)workspace) + need) return DSQ_ERR_SIZE;
    uint8_t *A8 = scratch, *B8 = scratch + round_up((size_t)M * kp, 1024);
    const int64_t threads = (M + N) * (int64_t)(kp / 16);
    expand_binary_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
        (const uint8_t *)A_bits, (const uint8_t *)B_bits, M, N, (int)K,
        (int)dsq_row_pitch(K, 1), (int)kp, A8, B8);
    if (cudaGetLastError() != cudaSuccess) return DSQ_ERR_CUDA;
    G8Params p = {};
    p.idesc = idesc_i8(G8_BN, true, true, G8_BM);
    p.C_i32 = C_i32; p.row_scale = row_scale; p.D_f32 = D_f32;
    p.ws = (int *)workspace;
    return launch_pass2<false>(A8, kp, B8, kp, (size_t)K, M, N, p, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------
// weight-only low-bit GEMM: bf16 activations x b-bit weights
// ---------------------------------------------------------------------------
size_t dsq_wgemm_workspace_bytes(int64_t N, int64_t K)
{
    if (N <= 0 || K <= 0) return DSQ_WS_BYTES;
    return DSQ_WS_BYTES + 1024 + round_up((size_t)N * round_up((size_t)K, 8) * 2, 1024);
}

int dsq_wgemm_bf16(const void *X_bf16, const void *W_codes, int64_t M, int64_t N, int64_t K,
                   int bits, float w_offset, const float *col_scale, const float *col_bias,
                   float *Y_f32, void *workspace, size_t ws_bytes, void *stream)
{
    if (!X_bf16 || !W_codes || !col_scale || !Y_f32 || !workspace) return DSQ_ERR_NULL;
    if (bits < 1 || bits > 4) return DSQ_ERR_BITS;
    if (M <= 0 || N <= 0 || K <= 0 || M > (1 << 24) || N > (1 << 24) || K > (1 << 24))
        return DSQ_ERR_SHAPE;
    if (w_offset != 0.0f && w_offset != 0.5f) return DSQ_ERR_UNSUPPORTED;
    // rows of X are read by TMA: 16-byte pitch
    if ((K % 8) != 0 || !dsq_aligned16(X_bf16) || !dsq_aligned16(W_codes) ||
        !dsq_aligned16(Y_f32) || !dsq_aligned16(workspace))
        return DSQ_ERR_ALIGN;
    uint8_t *W16 = scratch_of(workspace);
    const size_t wp = round_up((size_t)K, 8) * 2;          // scratch row pitch in bytes
    if (ws_bytes < (size_t)(W16 - (uint8_t *)workspace) + round_up((size_t)N * wp, 1024))
        return DSQ_ERR_SIZE;
    const int pitch_in = (int)dsq_row_pitch(K, bits);
    const int64_t threads = N * (int64_t)(wp / 16);
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    const int odd = w_offset == 0.5f;
    const uint8_t *W = (const uint8_t *)W_codes;
    cudaStream_t s = (cudaStream_t)stream;
    switch (bits) {
    case 1: expand_w_bf16_kernel<1><<<blocks, 256, 0, s>>>(W, N, (int)K, pitch_in, (int)wp, odd, W16); break;
    case 2: expand_w_bf16_kernel<2><<<blocks, 256, 0, s>>>(W, N, (int)K, pitch_in, (int)wp, odd, W16); break;
    case 3: expand_w_bf16_kernel<3><<<blocks, 256, 0, s>>>(W, N, (int)K, pitch_in, (int)wp, odd, W16); break;
    default: expand_w_bf16_kernel<4><<<blocks, 256, 0, s>>>(W, N, (int)K, pitch_in, (int)wp, odd, W16); break;
    }
    if (cudaGetLastError() != cudaSuccess) return DSQ_ERR_CUDA;
    G8Params p = {};
    p.idesc = idesc_bf16(G8_BN, G8_BM);
    p.col_scale = col_scale; p.col_bias = col_bias; p.Y_f32 = Y_f32;
    p.ws = (int *)workspace;
    return launch_pass2<true>(X_bf16, (size_t)K * 2, W16, wp, (size_t)K * 2, M, N, p, s);
}
