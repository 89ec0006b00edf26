// Device helpers shared by the tensor-core kernels (dsq_tc.cu: GEMM and
// im2col convolution; dsq_conv3.cu: 3x3 convolution on a shared-memory
// window): bounded barrier waits and the packed -> int8 expansion.
#pragma once

#include <cuda.h>

#include "dsq_epilogue.cuh"
#include "dsq_hooks.h"
#include "dsq_ptx.cuh"

using namespace dsq_ptx;

namespace {

constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // default: a wait gives up after 2 s
// once a CTA has given up, copies and MMAs already in flight get this long to land
constexpr unsigned long long DRAIN_LIMIT_NS = 20000000ull;

// ---------------------------------------------------------------------------
// bounded wait
// ---------------------------------------------------------------------------
struct Ctl {
    volatile int *abort_flag;   // shared memory
    int *ws;
    unsigned long long limit_ns;
};

// Slow path of a wait.  Not inlined on purpose: the kernel has a dozen wait
// sites and its code must stay small enough for the instruction caches.
// CLUSTER: acquire at cluster scope (the barrier also collects arrivals that
// threads of the peer CTA released at cluster scope).
template <bool CLUSTER>
__device__ __noinline__ bool wait_bar_slow(uint32_t bar, uint32_t parity, const Ctl &c, int tag)
{
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 1;; ++it) {
        if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0u) {
            if (*c.abort_flag) return false;
            if (global_timer_ns() - t0 > c.limit_ns) break;
        }
    }
    if (atomicCAS(c.ws + DSQ_WS_STATUS, 0, (int)DSQ_ERR_TIMEOUT) == 0)
        c.ws[DSQ_WS_DETAIL] = tag;
    *c.abort_flag = 1;
    return false;
}

// Bounded wait of ONE thread (the TMA producer threads).
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const Ctl &c, int tag)
{
    if (mbar_try_wait(bar, parity)) return true;
    return wait_bar_slow<false>(bar, parity, c, tag);
}

// Bounded wait of a whole converged warp.  All 32 lanes get the same answer:
// the code behind a wait holds warp-wide instructions (tcgen05.ld / st,
// __syncwarp), so the lanes must not part ways when one of them sees the phase
// complete and another the abort flag.
template <bool CLUSTER = false>
__device__ __forceinline__ bool wait_bar_warp(uint32_t bar, uint32_t parity, const Ctl &c, int tag)
{
    bool ok = CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity);
    if (!ok) ok = wait_bar_slow<CLUSTER>(bar, parity, c, tag);
    return __all_sync(0xffffffffu, ok);
}

// Wait used while leaving after a failure: ignores the abort flag (what is in
// flight must still land before shared or tensor memory is given up), bounded
// by DRAIN_LIMIT_NS.
__device__ __noinline__ void wait_bar_drain(uint32_t bar, uint32_t parity)
{
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if ((it & 15u) == 0u && global_timer_ns() - t0 > DRAIN_LIMIT_NS) return;
    }
}

// ---------------------------------------------------------------------------
// packed -> int8 expansion.  One 128-code K step of a row is CH packed
// 16-byte chunks and 32 words (128 bytes) of int8.  Word order (the same for
// both operands): 4-bit chunk j gives words 8j..8j+3 from the even nibbles of
// its four words and 8j+4..8j+7 from the odd nibbles; 2-bit chunk j gives
// words 16j+4c..16j+4c+3 from bit pair c of every byte; 3-bit rows keep the
// natural order.
// ---------------------------------------------------------------------------
template <int BITS, bool SIGNED>
__device__ __forceinline__ uint32_t expand_word(uint32_t w, int c, uint32_t orv)
{
    if (BITS == 4) {
        if (!SIGNED) return (c == 0 ? w : (w >> 4)) & 0x0F0F0F0Fu;
        return ((c == 0 ? (w << 4) : w) & 0xF0F0F0F0u) | orv;
    } else {
        if (!SIGNED) return (w >> (2 * c)) & 0x03030303u;
        return ((c == 3 ? w : (w << (6 - 2 * c))) & 0xC0C0C0C0u) | orv;
    }
}

// words 4q..4q+3 of a 3-bit row step held in w[12]
template <bool SIGNED>
__device__ __forceinline__ uint4 expand3_chunk(const uint32_t (&w)[12], int q, uint32_t orv)
{
    uint32_t o[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const int bit = (16 * q + 4 * t) * 3;
        const int wi = bit >> 5, sh = bit & 31;
        const uint32_t hi = wi + 1 < 12 ? w[wi + 1] : 0u;
        const uint32_t x = __funnelshift_r(w[wi], hi, sh);
        uint32_t b = (x & 7u) | ((x & 0x38u) << 5) | ((x & 0x1C0u) << 10) |
                     ((x & 0xE00u) << 15);
        if (SIGNED) b = (b << 5) | orv;
        o[t] = b;
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

template <int BITS>
struct Chunks {
    static constexpr int CH = BITS;              // packed 16-byte chunks per row step
    static constexpr int OUT = (BITS == 4) ? 2 : 4;   // int8 chunks per packed chunk (2/4-bit)
};

// whole row step in registers: v[CH] -> o[32]
template <int BITS, bool SIGNED>
__device__ __forceinline__ void expand_row_regs(const uint4 (&v)[Chunks<BITS>::CH],
                                                uint32_t orv, uint32_t (&o)[32])
{
    if (BITS == 3) {
        uint32_t w[12];
#pragma unroll
        for (int l = 0; l < 3; ++l) {
            w[4 * l] = v[l].x; w[4 * l + 1] = v[l].y;
            w[4 * l + 2] = v[l].z; w[4 * l + 3] = v[l].w;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint4 c = expand3_chunk<SIGNED>(w, q, orv);
            o[4 * q] = c.x; o[4 * q + 1] = c.y; o[4 * q + 2] = c.z; o[4 * q + 3] = c.w;
        }
    } else {
        constexpr int OUT = Chunks<BITS>::OUT;
#pragma unroll
        for (int j = 0; j < Chunks<BITS>::CH; ++j)
#pragma unroll
            for (int c = 0; c < OUT; ++c) {
                const int b = (j * OUT + c) * 4;
                o[b] = expand_word<BITS, SIGNED>(v[j].x, c, orv);
                o[b + 1] = expand_word<BITS, SIGNED>(v[j].y, c, orv);
                o[b + 2] = expand_word<BITS, SIGNED>(v[j].z, c, orv);
                o[b + 3] = expand_word<BITS, SIGNED>(v[j].w, c, orv);
            }
    }
}


}  // namespace
