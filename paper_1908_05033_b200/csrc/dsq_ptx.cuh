// Thin inline-PTX wrappers for sm_100a: mbarrier, TMA (cp.async.bulk.tensor),
// tcgen05 (alloc / mma / commit / ld) and the proxy fences between them.
#pragma once

#include <cuda.h>
#include <stdint.h>

namespace dsq_ptx {

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

// ---- mbarrier --------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count)
                 : "memory");
}
__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                 "r"(bytes)
                 : "memory");
}
// One bounded attempt: the thread may be suspended by the hardware for up to
// `hint_ns` while the phase is incomplete, and is woken when it completes.
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity,
                                                  uint32_t hint_ns = 2000u)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// ---- programmatic dependent launch --------------------------------------------
// launch_dependents: the grids queued behind this one with the programmatic
// serialisation attribute may start being scheduled once every CTA of this
// grid has executed it (or exited).  wait: blocks until all grids this one
// depends on have completed and their memory is visible; a no-op for a grid
// launched without the attribute.
__device__ __forceinline__ void grid_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---- thread-block clusters (CTA pairs) ---------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Barrier over all threads of all CTAs of the cluster (every thread calls it).
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\t"
                 "barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of this CTA's shared-memory location `addr` as seen in CTA `rank` of
// the cluster (shared::cluster window).
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// One bounded attempt with acquire semantics at cluster scope (pairs with an
// arrival released at cluster scope by a thread of the peer CTA).
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity,
                                                          uint32_t hint_ns = 2000u)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok;
}
// Arrive on an mbarrier of any CTA of the cluster (shared::cluster address)
// with the default semantics of mbarrier.arrive (release at CTA scope).  For
// arrivals that publish no memory the waiting CTA reads: the signal itself is
// an atomic update of the barrier object in its home shared memory and is
// seen by the waiter whatever the scope.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Arrival on this CTA's own barrier, released at cluster scope: what the
// arriving thread wrote (and what it has observed of its warp-mates' writes)
// to shared memory is in place before a thread that waits with acquire at
// cluster scope sees the arrival - and therefore before the tensor core of
// the peer SM, started by that thread, reads it.
__device__ __forceinline__ void mbar_arrive_release_cluster(uint32_t bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Same on a barrier of any CTA of the cluster (shared::cluster address).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr)
                 : "memory");
}

// ---- cp.async (16-byte, L2 only); src_bytes = 0 writes zeros -----------------
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src),
                 "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds_128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr)
                 : "memory");
    return v;
}
__device__ __forceinline__ void sts_128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c),
                 "r"(d)
                 : "memory");
}
// 256-bit global store (one full 32-byte sector per lane); dst 32-byte aligned
__device__ __forceinline__ void stg_256(void *dst, uint32_t a, uint32_t b, uint32_t c, uint32_t d,
                                        uint32_t e, uint32_t f, uint32_t g, uint32_t h)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(a),
                 "r"(b), "r"(c), "r"(d), "r"(e), "r"(f), "r"(g), "r"(h)
                 : "memory");
}

// Barrier among `nthreads` threads (a multiple of 32) of the CTA on hardware
// barrier `id` (1..15; 0 is __syncthreads).
__device__ __forceinline__ void named_barrier_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// ---- proxy / tcgen05 fences ------------------------------------------------
// Make generic-proxy shared-memory writes visible to the async proxy (TMA,
// tcgen05.mma operand reads).
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before_sync()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// ---- TMA -------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *m)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
// 2-D tiled load, completion counted in bytes on an mbarrier.  x is the inner
// (contiguous) coordinate; x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *m,
                                            int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(m), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// Same for a CTA pair (cta_group::2): the copy lands in THIS CTA's shared
// memory, its bytes are counted on an mbarrier of either CTA of the pair
// (`bar` is a shared::cluster address, e.g. the leader's barrier through
// map_to_cta).  No multicast: every CTA fetches its own tile.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *m,
                                                 int x, int y, uint32_t bar_cluster)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(m), "r"(x), "r"(y), "r"(bar_cluster)
        : "memory");
}

// 4-D im2col load over an NHWC tensor (dims C, W, H, N): `pixelsPerColumn`
// pixels x `channelsPerPixel` bytes.  (w, h) is the position of the filter
// window's corner for the first pixel (output position * stride - pad); the
// pixels that follow are the next window positions in W, then H, then N order
// inside the map's bounding box.  (off_w, off_h) selects the filter tap; a
// pixel outside the image is filled with zeros.  c * element size must be a
// multiple of 16 bytes.
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap *m, int c,
                                                   int w, int h, int n, uint16_t off_w,
                                                   uint16_t off_h, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};" ::"r"(dst),
        "l"(m), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(off_w), "h"(off_h)
        : "memory");
}

// ---- tensor memory ---------------------------------------------------------
// Executed by one full warp.  ncols: power of two, 32..512.  CG = 2: the
// same warp of both CTAs of a pair executes it, and both get the same columns.
template <int CG = 1>
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols)
{
    if (CG == 1)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         dst_smem),
                     "r"(ncols)
                     : "memory");
    else
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         dst_smem),
                     "r"(ncols)
                     : "memory");
}
template <int CG = 1>
__device__ __forceinline__ void tmem_relinquish()
{
    if (CG == 1)
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::
                         : "memory");
    else
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::
                         : "memory");
}
template <int CG = 1>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    if (CG == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr),
                     "r"(ncols)
                     : "memory");
    else
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr),
                     "r"(ncols)
                     : "memory");
}

// ---- tcgen05.mma kind::i8 --------------------------------------------------
// D[tmem] (+)= A[smem desc] * B[smem desc]; 8-bit integer operands, s32
// accumulate, M = 128, K = 32 per instruction, N from the descriptor.
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t a_desc,
                                       uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once all previously issued tcgen05.mma of this thread
// have completed (implies tcgen05.fence::before_thread_sync).
// CG = 2: tracks the pair's instructions; `bar` may be a shared::cluster
// address of either CTA.
template <int CG = 1>
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    if (CG == 1)
        asm volatile(
            "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                bar)
            : "memory");
    else
        asm volatile(
            "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                bar)
            : "memory");
}

// Same for a CTA pair: one instruction signals the barrier at this shared-memory
// offset in every CTA of `cta_mask` (bit r = CTA rank r of the cluster).
__device__ __forceinline__ void mma_commit_pair(uint32_t bar, uint16_t cta_mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 "
        "[%0], %1;" ::"r"(bar),
        "h"(cta_mask)
        : "memory");
}

// Same with the A operand read from tensor memory: 128 lanes (rows) x 8
// columns (32 bytes of K) per instruction.
__device__ __forceinline__ void mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem,
                                          uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Four consecutive K=32 instructions of one 128-byte K step in a single block:
// A advances 8 tensor-memory columns and the B descriptor 32 bytes (2 units of
// 16 bytes in its low word) per instruction.  Only the first one takes the
// caller's accumulate flag.
//
// Called by ALL lanes of a converged warp with warp-uniform arguments; one
// elected lane issues.  Keeping the issuing code in uniform control flow lets
// the compiler hold the descriptors in uniform registers, which is where the
// instruction takes them from: issued from a divergent single-lane branch,
// every instruction first pays for moving its operands there.
#define DSQ_MMA_X4_BODY(CGS)                                                              \
    asm volatile(                                                                         \
        "{\n\t.reg .pred p0, p1, pe;\n\t.reg .b64 d0, d1, d2, d3;\n\t"                   \
        ".reg .b32 l1, l2, l3, a1, a2, a3;\n\t"                                           \
        "setp.ne.b32 p0, %5, 0;\n\tsetp.eq.b32 p1, %5, %5;\n\t"                           \
        "add.u32 l1, %2, 2;\n\tadd.u32 l2, %2, 4;\n\tadd.u32 l3, %2, 6;\n\t"              \
        "add.u32 a1, %1, 8;\n\tadd.u32 a2, %1, 16;\n\tadd.u32 a3, %1, 24;\n\t"            \
        "mov.b64 d0, {%2, %3};\n\tmov.b64 d1, {l1, %3};\n\t"                              \
        "mov.b64 d2, {l2, %3};\n\tmov.b64 d3, {l3, %3};\n\t"                              \
        "elect.sync _|pe, 0xffffffff;\n\t"                                                \
        "@pe tcgen05.mma.cta_group::" CGS ".kind::i8 [%0], [%1], d0, %4, p0;\n\t"          \
        "@pe tcgen05.mma.cta_group::" CGS ".kind::i8 [%0], [a1], d1, %4, p1;\n\t"          \
        "@pe tcgen05.mma.cta_group::" CGS ".kind::i8 [%0], [a2], d2, %4, p1;\n\t"          \
        "@pe tcgen05.mma.cta_group::" CGS ".kind::i8 [%0], [a3], d3, %4, p1;\n\t}" ::"r"(  \
            d_tmem),                                                                      \
        "r"(a_tmem), "r"(b_desc_lo), "r"(b_desc_hi), "r"(idesc), "r"(accumulate_first)    \
        : "memory")
template <int CG = 1>
__device__ __forceinline__ void mma_i8_ts_x4(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_desc_lo,
                                             uint32_t b_desc_hi, uint32_t idesc,
                                             uint32_t accumulate_first)
{
    if (CG == 1) DSQ_MMA_X4_BODY("1");
    else DSQ_MMA_X4_BODY("2");
}
#undef DSQ_MMA_X4_BODY

// One tcgen05.mma kind::i8 with BOTH operands read through shared-memory
// descriptors (given as their two 32-bit halves), issued by one elected lane
// of a converged warp; all lanes call with warp-uniform arguments.
__device__ __forceinline__ void mma_i8_ss_elect(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi,
                                                uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p, pe;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %5, p;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Four such instructions in one block (one K step of 128 bytes): the B
// descriptor advances 32 bytes (2 units of 16 bytes in its low word) per
// instruction, the low words of the four A descriptors are given one by one
// (0xFFFFFFFF = leave this instruction out); the first instruction takes the
// caller's accumulate flag, the others accumulate.  a_lo0 must be valid.
__device__ __forceinline__ void mma_i8_ss_x4_elect(uint32_t d_tmem, uint32_t a_lo0, uint32_t a_lo1,
                                                   uint32_t a_lo2, uint32_t a_lo3, uint32_t a_hi,
                                                   uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                                   uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t.reg .pred p0, p1, pe, v1, v2, v3;\n\t"
        ".reg .b64 da0, da1, da2, da3, db0, db1, db2, db3;\n\t.reg .b32 l1, l2, l3;\n\t"
        "setp.ne.b32 p0, %9, 0;\n\tsetp.eq.b32 p1, %9, %9;\n\t"
        "add.u32 l1, %6, 2;\n\tadd.u32 l2, %6, 4;\n\tadd.u32 l3, %6, 6;\n\t"
        "mov.b64 da0, {%1, %5};\n\tmov.b64 da1, {%2, %5};\n\t"
        "mov.b64 da2, {%3, %5};\n\tmov.b64 da3, {%4, %5};\n\t"
        "mov.b64 db0, {%6, %7};\n\tmov.b64 db1, {l1, %7};\n\t"
        "mov.b64 db2, {l2, %7};\n\tmov.b64 db3, {l3, %7};\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "setp.ne.b32 v1, %2, 0xFFFFFFFF;\n\tsetp.ne.b32 v2, %3, 0xFFFFFFFF;\n\t"
        "setp.ne.b32 v3, %4, 0xFFFFFFFF;\n\t"
        "and.pred v1, v1, pe;\n\tand.pred v2, v2, pe;\n\tand.pred v3, v3, pe;\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::i8 [%0], da0, db0, %8, p0;\n\t"
        "@v1 tcgen05.mma.cta_group::1.kind::i8 [%0], da1, db1, %8, p1;\n\t"
        "@v2 tcgen05.mma.cta_group::1.kind::i8 [%0], da2, db2, %8, p1;\n\t"
        "@v3 tcgen05.mma.cta_group::1.kind::i8 [%0], da3, db3, %8, p1;\n\t}" ::"r"(d_tmem),
        "r"(a_lo0), "r"(a_lo1), "r"(a_lo2), "r"(a_lo3), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc),
        "r"(accumulate_first)
        : "memory");
}

// Same with the roles swapped: the A descriptor advances 32 bytes per
// instruction, the four B descriptors' low words are given one by one
// (0xFFFFFFFF = leave this instruction out).
__device__ __forceinline__ void mma_i8_ss_x4b_elect(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi,
                                                    uint32_t b_lo0, uint32_t b_lo1, uint32_t b_lo2,
                                                    uint32_t b_lo3, uint32_t b_hi, uint32_t idesc,
                                                    uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t.reg .pred p0, p1, pe, v1, v2, v3;\n\t"
        ".reg .b64 da0, da1, da2, da3, db0, db1, db2, db3;\n\t.reg .b32 l1, l2, l3;\n\t"
        "setp.ne.b32 p0, %9, 0;\n\tsetp.eq.b32 p1, %9, %9;\n\t"
        "add.u32 l1, %1, 2;\n\tadd.u32 l2, %1, 4;\n\tadd.u32 l3, %1, 6;\n\t"
        "mov.b64 da0, {%1, %2};\n\tmov.b64 da1, {l1, %2};\n\t"
        "mov.b64 da2, {l2, %2};\n\tmov.b64 da3, {l3, %2};\n\t"
        "mov.b64 db0, {%3, %7};\n\tmov.b64 db1, {%4, %7};\n\t"
        "mov.b64 db2, {%5, %7};\n\tmov.b64 db3, {%6, %7};\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "setp.ne.b32 v1, %4, 0xFFFFFFFF;\n\tsetp.ne.b32 v2, %5, 0xFFFFFFFF;\n\t"
        "setp.ne.b32 v3, %6, 0xFFFFFFFF;\n\t"
        "and.pred v1, v1, pe;\n\tand.pred v2, v2, pe;\n\tand.pred v3, v3, pe;\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::i8 [%0], da0, db0, %8, p0;\n\t"
        "@v1 tcgen05.mma.cta_group::1.kind::i8 [%0], da1, db1, %8, p1;\n\t"
        "@v2 tcgen05.mma.cta_group::1.kind::i8 [%0], da2, db2, %8, p1;\n\t"
        "@v3 tcgen05.mma.cta_group::1.kind::i8 [%0], da3, db3, %8, p1;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(a_hi), "r"(b_lo0), "r"(b_lo1), "r"(b_lo2), "r"(b_lo3), "r"(b_hi), "r"(idesc),
        "r"(accumulate_first)
        : "memory");
}

// One 128-byte K step of a CTA pair's tile with both operands in shared
// memory (cta_group::2: M = 256, each CTA holds 128 rows of A and half of the
// B rows at the same shared-memory offsets): four K = 32 instructions, the
// descriptors advancing 32 bytes each; issued by one elected lane of the
// converged warp of the pair's leader CTA.
__device__ __forceinline__ void mma_i8_ss_pair_x4_elect(uint32_t d_tmem, uint32_t a_lo,
                                                        uint32_t a_hi, uint32_t b_lo,
                                                        uint32_t b_hi, uint32_t idesc,
                                                        uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t.reg .pred p0, p1, pe;\n\t"
        ".reg .b64 da0, da1, da2, da3, db0, db1, db2, db3;\n\t.reg .b32 x1, x2, x3, y1, y2, y3;\n\t"
        "setp.ne.b32 p0, %6, 0;\n\tsetp.eq.b32 p1, %6, %6;\n\t"
        "add.u32 x1, %1, 2;\n\tadd.u32 x2, %1, 4;\n\tadd.u32 x3, %1, 6;\n\t"
        "add.u32 y1, %3, 2;\n\tadd.u32 y2, %3, 4;\n\tadd.u32 y3, %3, 6;\n\t"
        "mov.b64 da0, {%1, %2};\n\tmov.b64 da1, {x1, %2};\n\t"
        "mov.b64 da2, {x2, %2};\n\tmov.b64 da3, {x3, %2};\n\t"
        "mov.b64 db0, {%3, %4};\n\tmov.b64 db1, {y1, %4};\n\t"
        "mov.b64 db2, {y2, %4};\n\tmov.b64 db3, {y3, %4};\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::i8 [%0], da0, db0, %5, p0;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::i8 [%0], da1, db1, %5, p1;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::i8 [%0], da2, db2, %5, p1;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::i8 [%0], da3, db3, %5, p1;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate_first)
        : "memory");
}

// Same for 16-bit floating-point operands (kind::f16: f16 or bf16 per the
// instruction descriptor, K = 16 elements = 32 bytes per instruction, f32
// accumulate).
__device__ __forceinline__ void mma_f16_ss_pair_x4_elect(uint32_t d_tmem, uint32_t a_lo,
                                                        uint32_t a_hi, uint32_t b_lo,
                                                        uint32_t b_hi, uint32_t idesc,
                                                        uint32_t accumulate_first)
{
    asm volatile(
        "{\n\t.reg .pred p0, p1, pe;\n\t"
        ".reg .b64 da0, da1, da2, da3, db0, db1, db2, db3;\n\t.reg .b32 x1, x2, x3, y1, y2, y3;\n\t"
        "setp.ne.b32 p0, %6, 0;\n\tsetp.eq.b32 p1, %6, %6;\n\t"
        "add.u32 x1, %1, 2;\n\tadd.u32 x2, %1, 4;\n\tadd.u32 x3, %1, 6;\n\t"
        "add.u32 y1, %3, 2;\n\tadd.u32 y2, %3, 4;\n\tadd.u32 y3, %3, 6;\n\t"
        "mov.b64 da0, {%1, %2};\n\tmov.b64 da1, {x1, %2};\n\t"
        "mov.b64 da2, {x2, %2};\n\tmov.b64 da3, {x3, %2};\n\t"
        "mov.b64 db0, {%3, %4};\n\tmov.b64 db1, {y1, %4};\n\t"
        "mov.b64 db2, {y2, %4};\n\tmov.b64 db3, {y3, %4};\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], da0, db0, %5, p0;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], da1, db1, %5, p1;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], da2, db2, %5, p1;\n\t"
        "@pe tcgen05.mma.cta_group::2.kind::f16 [%0], da3, db3, %5, p1;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate_first)
        : "memory");
}

// tcgen05.commit by one elected lane of a converged warp (all lanes call).
__device__ __forceinline__ void mma_commit_elect(uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(
            bar)
        : "memory");
}
__device__ __forceinline__ void mma_commit_pair_elect(uint32_t bar, uint16_t cta_mask)
{
    asm volatile(
        "{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 "
        "[%0], %1;\n\t}" ::"r"(bar),
        "h"(cta_mask)
        : "memory");
}

// 32 lanes x 32 columns store: thread t of the warp writes lane (base + t),
// columns col .. col+31.
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]),
        "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]),
        "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
        "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
// 32 lanes x 16 columns store.
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]),
        "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]),
        "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait()
{
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// 32 lanes x 32 columns of 32-bit: thread t of the warp receives lane
// (base lane + t), columns col .. col+31.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, "
        "[%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]),
          "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]),
          "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]),
          "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]),
          "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// 32 lanes x 16 columns.
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]),
          "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]),
          "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---- descriptors -----------------------------------------------------------
// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows of
// 128 bytes, 8-row groups 1024 bytes apart (stride byte offset), tile base
// 1024-byte aligned.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);   // start address
    d |= (uint64_t)1 << 16;                       // leading byte offset (unused)
    d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset
    d |= (uint64_t)1 << 46;                       // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                       // SWIZZLE_128B
    return d;
}

// Instruction descriptor for kind::i8: s32 accumulator, K-major A and B.
__host__ __device__ inline uint32_t idesc_i8(int n, bool a_signed, bool b_signed, int m = 128)
{
    uint32_t d = 0;
    d |= 2u << 4;                              // D format: S32
    d |= (a_signed ? 1u : 0u) << 7;            // A: 0 = u8, 1 = s8
    d |= (b_signed ? 1u : 0u) << 10;           // B
    d |= (uint32_t)(n >> 3) << 17;             // N / 8
    d |= (uint32_t)(m >> 4) << 24;             // M / 16 (256: both CTAs of a pair)
    return d;
}

// Instruction descriptor for kind::f16 with bf16 operands and an f32
// accumulator, K-major A and B.
__host__ __device__ inline uint32_t idesc_bf16(int n, int m = 128)
{
    uint32_t d = 0;
    d |= 1u << 4;                              // D format: F32
    d |= 1u << 7;                              // A: BF16
    d |= 1u << 10;                             // B: BF16
    d |= (uint32_t)(n >> 3) << 17;             // N / 8
    d |= (uint32_t)(m >> 4) << 24;             // M / 16
    return d;
}

}  // namespace dsq_ptx
