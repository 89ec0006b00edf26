// Low-bit implicit GEMM on the 5th-generation tensor cores (sm_100a).
//
//   acc[m][n] = sum_k A[m][k] * B[n][k]       (Algorithm 1 step 5 on codes)
//
// A rows are output pixels (or GEMM rows) gathered from packed NHWC codes, B
// rows are output channels (packed weights, or the GEMM's B).  Both operands
// live in HBM as packed b-bit codes; the tensor core wants 8-bit integers, so
// each 128-code K step is expanded on the way through the SM:
//
//   B: TMA (cp.async.bulk.tensor.2d) packed tile -> shared ring ->
//      unpack warps -> int8 tile in the K-major 128B-swizzled layout
//   A: TMA brings the packed rows of a tile into a second shared ring: plain
//      2-D boxes for a GEMM or a 1x1 stride-1 convolution, im2col boxes
//      (cp.async.bulk.tensor.4d...im2col: 128 consecutive output pixels x one
//      run of one filter tap, zero fill outside the image) for every other
//      convolution.  One thread per tile row reads its row's 16-byte chunks,
//      expands them in registers and stores them to TENSOR MEMORY
//      (tcgen05.st): the expanded A operand never touches shared memory,
//      whose bandwidth is what bounds this kernel.  (3-bit GEMM rows are
//      gathered with cp.async instead.)
//   one warp issues tcgen05.mma.kind::i8 (128 x BN x 32 per instruction, or
//      256 x BN x 32 for a CTA pair; A from tensor memory, B from shared
//      memory), accumulating int32 in tensor memory (two accumulator buffers
//      where they fit beside the A stages)
//   epilogue warps read tensor memory (tcgen05.ld), apply the dequantise /
//      requantise epilogue and write codes / fp32 / int32 with vector stores;
//      on a CTA's last tile the A and B warps join them.
//
// Each role's loop is a chain of hand-offs (barrier wait, expect, TMA or MMA
// issue, commit); one hand-off costs a few hundred cycles while the unpack
// warps keep the shared-memory pipeline busy, whatever amount of data is
// behind it.  Hence: rounds of several K steps, A and B boxes issued by
// threads of two different warps, MMA issue in uniform control flow.
//
// Signed codes are expanded into the TOP b bits of the byte (value * 2^(8-b)):
// this costs no sign-extension arithmetic, and the exact factor is shifted out
// of the int32 accumulator in the epilogue.  With the paper's symmetric weight
// grid (w^ = Delta_w (c + 1/2)) the bit below is set as well, which makes the
// byte 2^(7-b) (2c + 1) and the accumulator 2^(7-b) (2 acc + S_a).
//
// The order of the codes inside a 128-code K step is permuted by the unpack
// (even / odd nibbles land in different 16-byte chunks); A and B use the same
// permutation, and a sum over k does not depend on the order.
//
// Every wait on an mbarrier is bounded; a wait that runs out records
// DSQ_ERR_TIMEOUT in the workspace, all roles leave their loops, tensor memory
// is released and the kernel returns.
#include <cuda.h>

#include "dsq_tc_common.cuh"
#include "dsq_tc_host.h"

// Scratch of dsq_gemm_static_ws: the workspace (status word, failure detail)
// that dsq_gemm normally receives from its caller, held by the library
// itself.  One copy lives on every GPU that loads the library, until exit.
#define DSQ_STATIC_WS_BYTES 256
#define DSQ_STATIC_WS_MAX_DIM 65536
static __device__ __align__(256) unsigned char g_static_ws[DSQ_STATIC_WS_BYTES];

namespace {

constexpr int BM = 128;               // tile rows = MMA M
constexpr int BK_BYTES = 128;         // int8 bytes per row per K step (128 codes)
// Pipeline modes (template parameter PM).  A barrier round covers KS K steps of
// 128 codes: with the fixed cost of a round (barrier hand-offs, MMA issue) near
// a thousand cycles, two K steps per round pay whenever they fit.
//   PM 1: KS = 1, 4 stages, two A groups          (any N tile, 3-bit rows)
//   PM 2: KS = 2, 3 stages, two A groups          (N tile <= 128)
//   PM 3: KS = 2, 2 stages, one A group ("wide")  (N tile 192 / 256: shared memory
//         holds two double stages of B only; the second A group's warps help
//         the epilogue instead)
//   PM 4: KS = 2, 3 stages, two A groups, CTA PAIR: the two CTAs of a cluster
//         work on one 256 x 256 tile with tcgen05.mma.cta_group::2.  Each CTA
//         gathers and expands its 128 A rows and HALF of the B rows (128 output
//         channels), the even CTA issues the instructions for both, and each
//         keeps the accumulators of its own 128 rows.  Per tensor-core clock
//         every SM then expands half as much B, which is what bounds the
//         single-CTA modes at wide N tiles.
//   PM 5: KS = 5, 2 stages, two A groups, ONE round per tile ("whole K"): small
//         convolutions (K <= 640 codes, e.g. 3x3 over 64 channels) with a
//         resident B tile.  Every hand-off between the roles (a barrier wait, an
//         expect, a TMA issue, a commit) costs a few hundred cycles whatever the
//         amount of data behind it, so a tile pays for them once instead of
//         once per K step; the two A groups take alternate tiles.
constexpr int SU_MAX = 4;
template <int PM> struct Pipe {
    static constexpr int KS = PM == 1 ? 1 : PM == 5 ? 5 : 2;
    static constexpr bool WIDE = PM == 3;
    static constexpr bool PAIR = PM == 4;
    static constexpr bool WHOLE_K = PM == 5;
    // stages of expanded operands
    static constexpr int SU = PM == 1 ? 4 : (PM == 3 || PM == 5) ? 2 : 3;
    static constexpr int GROUPS = WIDE ? 1 : 2;              // A groups in use
    static constexpr int A_D = PM == 1 ? 2 : 1;              // own A rounds in flight per thread
    static constexpr int A_RING = A_D + 1;                   // packed A ring slots per group
    static constexpr int A_COL0 = 512 - SU * 32 * KS;        // A stages: top TMEM columns
    static constexpr int S_P = WHOLE_K ? 1 : WIDE ? 2 : 3;   // packed B ring slots
    // coalesced A gather (adjacent lanes fetch one row's contiguous chunks): fewer
    // memory requests, more instructions in the A threads; pays where the A
    // threads have slack
    static constexpr bool COAL = PAIR;
    // B warps: one group of eight expands every round, or (pair mode, where a
    // round is only 128 rows per CTA) two groups of four take alternate rounds,
    // so that two rounds' latency chains (barrier, shared loads, stores, fence,
    // arrival) overlap
    static constexpr int B_GROUPS = PAIR ? 2 : 1;
};
constexpr int TMEM_COLS = 512;

constexpr int WARP_TMA = 0, WARP_MMA = 1, WARP_A0 = 2, WARP_B0 = 10, WARP_E0 = 18,
              WARP_TMA_A = 22;
// two groups of four A warps take alternate K steps
constexpr int NUM_A_GROUPS = 2, NUM_A_WARPS = 4 * NUM_A_GROUPS, NUM_B_WARPS = 8, NUM_E_WARPS = 4;
constexpr int NUM_B_THREADS = NUM_B_WARPS * 32;
constexpr int NUM_WARPS = 23;
static_assert(WARP_A0 + NUM_A_WARPS == WARP_B0 && WARP_B0 + NUM_B_WARPS == WARP_E0 &&
                  WARP_E0 + NUM_E_WARPS == WARP_TMA_A && WARP_TMA_A + 1 == NUM_WARPS,
              "warp roles");
constexpr int NUM_THREADS = NUM_WARPS * 32;

enum { MODE_CONV = 0, MODE_GEMM = 1 };
// epilogue variants (template parameter): GEMM; convolution writing codes
// only, without / with a residual operand; convolution with any outputs
enum { EPI_GEMM = 0, EPI_CODES = 1, EPI_CODES_RES = 2, EPI_GENERAL = 3 };

struct TcParams {
    // problem
    int M, Ncols, ksteps, rounds, BN, m_tiles, n_tiles, n_acc, s_p;
    // b_res = 1: the whole expanded B tile (all K steps) stays in shared memory
    // for the life of the CTA (one N tile, few K steps: small weight matrices)
    int b_res, b_stages;
    int epw;                          // epilogue warps per TMEM lane quarter (1..3)
    // join = 1: on the CTA's last tile the A and B warps join the epilogue (needs
    // a scale / bias staging slot for each of the 20 warps in shared memory)
    int join;
    int smem_bytes;                   // dynamic shared memory given to the launch
    // every wait on a barrier gives up after this many nanoseconds
    unsigned long long wait_ns;
    // test hook (dsq_set_test_skip_b_round): the B producer leaves out the copy
    // of this round (counted over the CTA's rounds; -1 = none) and stops, so
    // that the wait on it runs out
    int skip_b_round;
    // A gather geometry (a GEMM is a 1x1 convolution over an M x 1 image)
    const uint8_t *act;
    int H, W, Ho, Wo, stride, pad, KW, taps, P;
    int a_lcr;                        // log2 of the A gather's run length in 16-byte chunks
    // a_tma != 0: TMA brings each round's 128 rows of packed A into the A ring and
    // the A threads only read their rows.  A round is a_nsub boxes of 128 rows x
    // a_sub bytes (a_sub = 16 << a_lc <= 128, one swizzle span), stored one after
    // the other.
    //   1: the rows are rows of a plain 2-D matrix (GEMM, 1x1 stride-1
    //      convolution): one box per round
    //   2: im2col over the NHWC tensor: a box is one run of a_sub bytes of one
    //      filter tap of 128 consecutive output pixels (a_sub divides the pixel
    //      pitch, so a box never straddles two taps); K columns past the last
    //      tap are not loaded, the A threads put zeros there (a_kchunks = 16-byte
    //      chunks of a row that exist)
    //   3: whole image rows (3x3, stride 1, pad 1 over 64 channels, whole-K
    //      rounds): the tile's output pixels lie in a few consecutive image rows
    //      and all their taps in those rows plus one above and one below.  a_nr
    //      rows of the (N*H) x (W*P bytes) matrix are fetched once per tile as ONE
    //      box, and every A thread picks its pixel's 3 x 3P bytes out of them,
    //      zeroing the taps outside the image: a third of the im2col bytes, in
    //      rows of up to 2 KB instead of one pixel's P bytes (the TMA unit spends
    //      a few cycles per row whatever its length).  a_bw = W*P.
    int a_tma, a_lc, a_nsub, a_kchunks, a_nr, a_bw;
    // 3-bit convolution: a pixel's packed row (P bytes, 8 codes per 3 bytes
    // from the row's start) is not a whole number of 48-byte K steps unless
    // Cin is a multiple of 128, so every filter tap starts a K step of its
    // own: Pk = P rounded up to 48 bytes, the A gather fills the rest of a
    // tap's last K step with zeros, and B's K step (tap, s) lies at byte
    // tap * P + 48 s of a weight row (spt K steps per tap; 0 = dense rows).
    int Pk, spt;
    // epilogue
    int mode, shift, out_pitch, small_acc;
    float r_hi;                       // fmaf(hi - lo, inv, 0.5f) of the requantiser
    DsqEpi e;
    int32_t *C_i32;
    const float *row_scale;
    float *D_f32;
    uint32_t orv;                     // OR-ed into every signed byte
    int *ws;
};

// ---------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------
struct SmemLayout {
    uint32_t b_tiles, b_packed, a_ring, epi, lut, bars, tmem_slot, abort_flag, total;
};

constexpr int MAX_S_P = 4;
constexpr int MAX_A_SLOTS = 6;
constexpr int MAX_B_STAGES = 16;

constexpr int JOIN_CNT = 5;               // warps per lane quarter in a joined epilogue
// 256-byte slots behind the rings: scale / bias staging of the epilogue warps
__host__ __device__ inline int epi_slots(int join, int epw)
{
    return join ? 4 * JOIN_CNT : 4 * epw;
}

__host__ __device__ inline SmemLayout smem_layout(int BN, int bits, int s_p, int b_stages, int ks,
                                                int a_slots, int epi_slots)
{
    SmemLayout L;
    uint32_t o = 0;
    L.b_tiles = o;  o += b_stages * ks * BN * BK_BYTES;
    L.b_packed = o; o += s_p * ks * BN * 16 * bits;
    L.a_ring = o;   o += a_slots * ks * BM * 16 * bits;
    // per-warp scale / bias staging (any warp may take part in an epilogue)
    L.epi = o;      o += epi_slots * 64 * 4;
    L.lut = o;      o += 16 * 4;             // dequantised residual values (codes epilogue)
    o = (o + 127u) & ~127u;
    L.bars = o;     o += 8 * (2 * SU_MAX + MAX_B_STAGES + 2 * MAX_S_P + 4 + 2 * MAX_A_SLOTS + 2);
    L.tmem_slot = o; o += 8;
    L.abort_flag = o; o += 8;
    L.total = o;
    return L;
}

// A_TMA: 0 = A gathered with cp.async, 1 = TMA boxes (2-D or im2col), 3 = whole
// image rows (TcParams::a_tma); a template parameter so that the A threads' loop
// carries one fetch path (the kernel is sensitive to its code size)
template <int BITS, bool A_SIGNED, int EPI, int PM, int A_TMA>
__global__ void __launch_bounds__(NUM_THREADS, 1)
dsq_tc_kernel(const __grid_constant__ CUtensorMap tmap_b,
              const __grid_constant__ CUtensorMap tmap_a, const TcParams p)
{
    constexpr bool B_SIGNED = !A_SIGNED;
    constexpr int CH = Chunks<BITS>::CH;
    constexpr int KS = Pipe<PM>::KS, GROUPS = Pipe<PM>::GROUPS;
    constexpr bool WIDE = Pipe<PM>::WIDE, PAIR = Pipe<PM>::PAIR;
    constexpr int B_GROUPS = Pipe<PM>::B_GROUPS;
    constexpr int CG = PAIR ? 2 : 1;          // CTAs per tcgen05 instruction
    constexpr int BMT = BM * CG;              // tile rows
    constexpr int S_U = Pipe<PM>::SU, A_D = Pipe<PM>::A_D, A_RING = Pipe<PM>::A_RING;
    constexpr int A_COL0 = Pipe<PM>::A_COL0;
    constexpr int A_SLOTS = GROUPS * A_RING;                // packed A ring slots
    constexpr int A_SLOT_BYTES = KS * CH * BM * 16;         // one round of 128 rows
    static_assert(A_SLOTS <= MAX_A_SLOTS, "A ring barriers");
    static_assert(KS == 1 || BITS != 3, "3-bit rows use single K steps");
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~(uintptr_t)1023u);
    const int BN = p.BN;
    const int BNL = BN / CG;                  // B rows this CTA expands
    const SmemLayout L =
        smem_layout(BNL, BITS, p.s_p, p.b_stages, KS, GROUPS * A_RING,
                    epi_slots(p.join, p.epw));
    // the layout must fit behind the 1024-byte aligned base (the host adds
    // slack only while it stays within the 227 KB limit); same answer in every
    // thread of every CTA, taken before any barrier exists
    if ((uint32_t)(smem - smem_raw) + L.total > (uint32_t)p.smem_bytes) {
        // (global memory, the workspace included, is touched only once the
        // kernels before this one have completed)
        grid_dependency_wait();
        if (threadIdx.x == 0) atomicCAS(p.ws + DSQ_WS_STATUS, 0, (int)DSQ_ERR_UNSUPPORTED);
        return;
    }
    const int S_P = p.s_p;
    // (the shuffle tells the compiler that the warp index is the same in all
    // lanes, so the role branches below are uniform control flow)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    // a pair is the two CTAs of a cluster; rank 0 issues the MMAs
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const int tile0 = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int tstep = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int row_base = (int)rank * BM;      // first tile row of this CTA
    const int total_tiles = p.m_tiles * p.n_tiles;
    const uint32_t b_sub_bytes = BNL * BK_BYTES;             // one K step of the (half) tile
    const uint32_t b_tile_bytes = KS * b_sub_bytes;          // one round
    const uint32_t b_packed_bytes = KS * BNL * 16 * BITS;
    int my_tiles_all = 0;
    for (int t = tile0; t < total_tiles; t += tstep) ++my_tiles_all;
    // B is produced for every step of every tile, or once (resident mode)
    const uint32_t n_b_steps =
        my_tiles_all == 0 ? 0u : (p.b_res ? (uint32_t)p.rounds : (uint32_t)my_tiles_all * p.rounds);

    const uint32_t bars = smem_u32(smem + L.bars);
    auto bar_a_full = [&](int s) { return bars + 8u * s; };
    auto bar_u_empty = [&](int s) { return bars + 8u * (SU_MAX + s); };
    auto bar_b_full = [&](int s) { return bars + 8u * (2 * SU_MAX + s); };
    constexpr int BAR_P = 2 * SU_MAX + MAX_B_STAGES;
    auto bar_p_full = [&](int s) { return bars + 8u * (BAR_P + s); };
    auto bar_p_empty = [&](int s) { return bars + 8u * (BAR_P + MAX_S_P + s); };
    auto bar_acc_full = [&](int s) { return bars + 8u * (BAR_P + 2 * MAX_S_P + s); };
    auto bar_acc_empty = [&](int s) { return bars + 8u * (BAR_P + 2 * MAX_S_P + 2 + s); };
    auto bar_ar_full = [&](int s) { return bars + 8u * (BAR_P + 2 * MAX_S_P + 4 + s); };
    auto bar_ar_empty = [&](int s) {
        return bars + 8u * (BAR_P + 2 * MAX_S_P + 4 + MAX_A_SLOTS + s);
    };
    // completes once, when the accumulators of this CTA's last tile are final
    const uint32_t bar_last_full = bars + 8u * (BAR_P + 2 * MAX_S_P + 4 + 2 * MAX_A_SLOTS);
    // used once, by an MMA warp that gives up: completion of what it had issued
    const uint32_t bar_drain = bar_last_full + 8u;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + L.tmem_slot);
    Ctl ctl{reinterpret_cast<volatile int *>(smem + L.abort_flag), p.ws, p.wait_ns};
    // The consumer of a_full / b_full / acc_empty is the MMA thread of rank 0:
    // in a pair both CTAs arrive on rank 0's barriers.
    // Memory ordering in a pair.  The expanded B halves in shared memory are read
    // by the tensor cores of BOTH SMs, so the B warps of both CTAs release their
    // arrivals at cluster scope and rank 0's MMA warp spins on the barrier with
    // acquire at cluster scope (wait_bar_warp<true>).  (With CTA-scope arrivals,
    // one 8192^3 GEMM launch in about 150 returned a wrong block of 128
    // columns.)  The A operand sits in each SM's own tensor memory, is complete
    // there before its arrival (tcgen05.wait::st) and is read by that SM's
    // tensor core only: those arrivals publish no memory and keep the default
    // scope.  The epilogue warps' arrivals (accumulator handed back) cross with
    // a cluster-scope release as well.
    auto arrive_leader = [&](uint32_t bar) {
        if (PAIR && rank != 0) mbar_arrive_cluster(map_to_cta(bar, 0u));
        else mbar_arrive(bar);
    };
    // completion of the issued MMAs, signalled to this barrier in both CTAs
    // (called by all lanes of the MMA warp; one elected lane issues)
    auto commit_all = [&](uint32_t bar) {
        if (PAIR) mma_commit_pair_elect(bar, (uint16_t)3);
        else mma_commit_elect(bar);
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < S_U; ++s) {
            // operands of a round: the four warps of one A group and (unless the
            // expanded B tile is resident) the B warps, of every CTA of the pair
            mbar_init(bar_a_full(s), (4 + (p.b_res ? 0 : NUM_B_WARPS / B_GROUPS)) * CG);
            mbar_init(bar_u_empty(s), 1);    // tcgen05.commit
        }
        for (int s = 0; s < MAX_B_STAGES; ++s) mbar_init(bar_b_full(s), NUM_B_WARPS * CG);
        for (int s = 0; s < S_P; ++s) {
            mbar_init(bar_p_full(s), 1);     // TMA producer (+ transaction bytes)
            mbar_init(bar_p_empty(s), NUM_B_WARPS / B_GROUPS);
        }
        for (int s = 0; s < A_SLOTS; ++s) {
            mbar_init(bar_ar_full(s), 1);    // TMA producer (+ transaction bytes)
            mbar_init(bar_ar_empty(s), 4);   // the four warps of the slot's A group
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_acc_full(s), 1);   // tcgen05.commit
            mbar_init(bar_acc_empty(s), 4 * p.epw * CG);
        }
        mbar_init(bar_last_full, 1);         // tcgen05.commit
        mbar_init(bar_drain, 1);             // tcgen05.commit
        *ctl.abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == WARP_MMA) {
        tmem_alloc<CG>(smem_u32((const void *)tmem_slot), TMEM_COLS);
        tmem_relinquish<CG>();
    }
    if (warp == WARP_TMA && lane == 0) {
        tma_prefetch_desc(&tmap_b);
        if (A_TMA) tma_prefetch_desc(&tmap_a);
    }
    // the 2^BITS dequantised values of a residual code
    if (EPI == EPI_CODES_RES && warp == WARP_TMA_A && lane < (1 << BITS))
        reinterpret_cast<float *>(smem + L.lut)[lane] =
            __fmaf_rn((float)lane, p.e.res_delta, p.e.res_lo);
    tc_fence_before_sync();
    __syncthreads();
    // no arrival may reach the peer before its barriers exist
    if (PAIR) cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
    // Programmatic dependent launch: everything above (barriers, tensor memory,
    // descriptor prefetch) touched no global data, so it may run while the
    // kernel before this one is still finishing; nothing below starts before
    // that kernel has completed.  The kernel behind this one may set up likewise.
    grid_launch_dependents();
    grid_dependency_wait();

    // Epilogue roles.  epi_idx >= 0: the warp takes part in the epilogue of every
    // tile (p.epw warps per TMEM lane quarter).  join_idx >= 0: it takes part in
    // the epilogue of the CTA's LAST tile, where nothing is left to overlap with,
    // so the A and B warps, done with their rounds, help out (JOIN_CNT warps per
    // quarter: a lone warp issues an instruction every few cycles at best).
    int epi_idx = -1, join_idx = -1;
    int epi_slot = warp - WARP_A0;         // joined: one slot per A / B / epilogue warp
    if (warp == WARP_TMA) {
        // ---------------- producer: TMA packed B tiles -----------------------
        // (the A boxes have a producer thread of their own in another warp: every
        // wait / expect / issue of one thread is a chain of shared-memory
        // pipeline round trips, a few hundred cycles each while the unpack warps
        // keep that pipeline busy)
        if (lane == 0) {
            uint32_t g = 0, ph = 0, issued_b = 0;
            int s = 0, ks = 0, tile = tile0, btap = 0, bsub = 0;
#pragma unroll 1
            for (; g < n_b_steps; ++g) {
                if (!wait_bar(bar_p_empty(s), ph ^ 1u, ctl, 1)) break;
                if ((int)g == p.skip_b_round) break;
                mbar_arrive_expect_tx(bar_p_full(s), b_packed_bytes);
                if (Pipe<PM>::WHOLE_K) {
                    // a box is at most 256 bytes wide: one box per K step, stored
                    // [K step][row][16 * BITS bytes]
                    for (int h = 0; h < KS; ++h)
                        tma_load_2d(smem_u32(smem + L.b_packed + s * b_packed_bytes) +
                                        h * (BNL * 16 * BITS),
                                    &tmap_b, (ks * KS + h) * (16 * BITS),
                                    (tile % p.n_tiles) * BN + (int)rank * BNL, bar_p_full(s));
                } else
                tma_load_2d(smem_u32(smem + L.b_packed + s * b_packed_bytes), &tmap_b,
                            p.spt ? btap * p.P + bsub * (16 * BITS) : ks * (KS * 16 * BITS),
                            (tile % p.n_tiles) * BN + (int)rank * BNL, bar_p_full(s));
                ++issued_b;
                if (++s == S_P) { s = 0; ph ^= 1u; }
                if (p.spt && ++bsub == p.spt) { bsub = 0; ++btap; }
                if (++ks == p.rounds) { ks = 0; tile += tstep; btap = bsub = 0; }
            }
            // let outstanding copies land before the CTA can exit
            for (uint32_t k = (issued_b > (uint32_t)S_P ? issued_b - S_P : 0); k < issued_b; ++k)
                wait_bar_drain(bar_p_full(k % S_P), (k / S_P) & 1u);
        }
    } else if (warp == WARP_TMA_A) {
        // ---------------- producer: TMA packed A boxes -----------------------
        if (A_TMA && lane == 0) {
            const int a_steps_tile = p.rounds;                   // A steps per tile
            const uint32_t n_a_steps = (uint32_t)my_tiles_all * a_steps_tile;
            const uint32_t ring = smem_u32(smem + L.a_ring);
            uint32_t g = 0, issued_a = 0;
            int ka = 0, tile_a = tile0;
            int i2c_w = 0, i2c_h = 0, i2c_n = 0, i2c_c = 0, i2c_kw = 0, i2c_kh = 0;
#pragma unroll 1
            for (; g < n_a_steps; ++g) {
                const int sl = (int)(g % A_SLOTS);
                if (!wait_bar(bar_ar_empty(sl), ((g / A_SLOTS) & 1u) ^ 1u, ctl, 11)) break;
                const int m0 = (tile_a / p.n_tiles) * BMT + row_base;
                if (A_TMA == 3) {
                    // rows R0-1 .. R0-2+a_nr of the row matrix (R = n*H + h); rows
                    // outside it are filled with zeros (and masked by the readers)
                    mbar_arrive_expect_tx(bar_ar_full(sl), (uint32_t)(p.a_nr * p.a_bw));
                    tma_load_2d(ring + sl * A_SLOT_BYTES, &tmap_a, 0, m0 / p.W - 1,
                                bar_ar_full(sl));
                } else if (p.a_tma == 1) {
                    mbar_arrive_expect_tx(bar_ar_full(sl), A_SLOT_BYTES);
                    tma_load_2d(ring + sl * A_SLOT_BYTES, &tmap_a, ka * (KS * 16 * BITS), m0,
                                bar_ar_full(sl));
                } else {
                    if (ka == 0) {                 // first pixel of the tile, first tap
                        const int wo = m0 % p.Wo, t = m0 / p.Wo;
                        i2c_w = wo * p.stride - p.pad;
                        i2c_h = (t % p.Ho) * p.stride - p.pad;
                        i2c_n = t / p.Ho;
                        i2c_c = 0; i2c_kw = 0; i2c_kh = 0;
                    }
                    const int sub = 16 << p.a_lc;
                    const int left = (p.a_kchunks * 16 - ka * (KS * 16 * BITS)) / sub;
                    const int nb = left < p.a_nsub ? left : p.a_nsub;
                    mbar_arrive_expect_tx(bar_ar_full(sl), (uint32_t)(nb * BM * sub));
                    for (int i = 0; i < nb; ++i) {
                        tma_load_im2col_4d(ring + sl * A_SLOT_BYTES + i * (BM * sub), &tmap_a,
                                           i2c_c, i2c_w, i2c_h, i2c_n, (uint16_t)i2c_kw,
                                           (uint16_t)i2c_kh, bar_ar_full(sl));
                        i2c_c += sub;
                        if (i2c_c == p.P) {
                            i2c_c = 0;
                            if (++i2c_kw == p.KW) { i2c_kw = 0; ++i2c_kh; }
                        }
                    }
                }
                ++issued_a;
                if (++ka == a_steps_tile) { ka = 0; tile_a += tstep; }
            }
            for (uint32_t k = (issued_a > (uint32_t)A_SLOTS ? issued_a - A_SLOTS : 0);
                 k < issued_a; ++k)
                wait_bar_drain(bar_ar_full(k % A_SLOTS), (k / A_SLOTS) & 1u);
        }
    } else if (warp == WARP_MMA) {
        // ---------------- MMA issuer ---------------------------------------
        // The whole warp runs the loop in uniform control flow (waits included);
        // the issue wrappers elect one lane.
        if (rank == 0) {
            const uint32_t idesc = idesc_i8(BN, A_SIGNED, B_SIGNED, BMT);
            const uint64_t b_desc0 = smem_desc_sw128(smem_u32(smem + L.b_tiles));
            const uint32_t b_desc_lo0 = (uint32_t)b_desc0, b_desc_hi = (uint32_t)(b_desc0 >> 32);
            uint32_t g = 0, it = 0;
            bool ok = true;
#pragma unroll 1
            for (int tile = tile0; ok && tile < total_tiles; tile += tstep, ++it) {
                const int as = p.n_acc == 2 ? (it & 1) : 0;
                const uint32_t aph = (p.n_acc == 2 ? (it >> 1) : it) & 1u;
                // (in a pair the peer CTA's arrivals were released at cluster scope)
                if (!(ok = wait_bar_warp<PAIR>(bar_acc_empty(as), aph ^ 1u, ctl, 3))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + as * BN;
#pragma unroll 1
                for (int ks = 0; ks < p.rounds; ++ks, ++g) {
                    const int s = g % S_U;
                    const uint32_t ph = (g / S_U) & 1u;
                    const int bs = p.b_res ? ks : s;
                    if (p.b_res && it == 0)
                        if (!(ok = wait_bar_warp<PAIR>(bar_b_full(bs), 0u, ctl, 10))) break;
                    if (!(ok = wait_bar_warp<PAIR>(bar_a_full(s), ph, ctl, 4))) break;
                    tc_fence_after_sync();
                    // per K step 4 instructions, 32 bytes of K each
#pragma unroll
                    for (int h = 0; h < KS; ++h)
                        mma_i8_ts_x4<CG>(d_tmem, tmem_base + A_COL0 + (s * KS + h) * 32,
                                     b_desc_lo0 + (bs * KS + h) * (b_sub_bytes >> 4), b_desc_hi,
                                     idesc, (uint32_t)(ks | h));
                    commit_all(bar_u_empty(s));
                }
                if (ok) {
                    commit_all(bar_acc_full(as));
                    if (tile + tstep >= total_tiles) commit_all(bar_last_full);
                }
            }
            if (!ok) {
                // giving up: instructions already issued may still be reading the
                // operands and writing the accumulators; they must have finished
                // before shared and tensor memory are given up
                commit_all(bar_drain);
                wait_bar_drain(bar_drain, 0u);
            }
        }
    } else if (warp < WARP_B0) {
        // ---------------- A: one thread per tile row, two groups ---------------
        // Group k (four warps, one per TMEM lane quarter) handles the K steps with
        // step index = k (mod 2), so two steps are in flight at once and the
        // per-step latency chain of one group overlaps the other's.  Per step:
        // global --cp.async--> 16-byte cells of a shared ring (A_D own steps in
        // flight) -> registers -> expand -> tensor memory (tcgen05.st),
        // completed and published at once.
        //
        // The copies are issued coalesced: a row's codes of one filter tap are
        // contiguous, so a run of 2^a_lcr chunks is fetched by that many adjacent
        // lanes (the row's owner hands the run's address over by shuffle), and a
        // warp instruction covers a few rows x up to 128 contiguous bytes instead
        // of 32 rows x 16 bytes: an eighth of the L1 requests and of the
        // shared-memory write cycles.  Each thread then reads its own row.
        const int group = (warp - WARP_A0) >> 2;
        if (group < GROUPS) {
        const int quarter = warp & 3;              // TMEM lane quarter of this warp
        const int row = quarter * 32 + lane;
        constexpr int SLOT_BYTES = A_SLOT_BYTES;   // ring slot = KS*CH planes x 128 rows x 16 B
        const uint32_t cell0 =
            smem_u32(smem + L.a_ring) + group * (A_RING * SLOT_BYTES) + row * 16;
        // walk position over the flattened (tile, K step) sequence; starts one
        // tile back with ld_ks at its end, so that the first step advances
        int ld_tile = tile0 - tstep, ld_ks = p.rounds, ld_slot = 0;
        int tap = 0, kw = 0, off = 0;
        const int lcr = p.a_lcr, crm = (1 << lcr) - 1;
        const int lane_row = lane >> lcr, lane_c = lane & crm;
        const uint32_t ring0 = smem_u32(smem + L.a_ring) + group * (A_RING * SLOT_BYTES) +
                               quarter * (32 * 16);
        uint32_t tap_mask = 0;                     // bit t: filter tap t is inside the image
        const uint8_t *src = p.act;
        const int64_t row_jump = (int64_t)(p.W - p.KW) * p.P;
        auto set_tile = [&](int t) {
            tap = kw = off = 0;
            tap_mask = 0;
            if (t >= total_tiles) return;
            const int m = (t / p.n_tiles) * BMT + row_base + row;
            if (m < p.M) {
                const int wo = m % p.Wo;
                const int ho = (m / p.Wo) % p.Ho;
                const int n = m / (p.Wo * p.Ho);
                const int hb = ho * p.stride - p.pad, wb = wo * p.stride - p.pad;
                for (int tt = 0, th = 0, tw = 0; tt < p.taps; ++tt) {
                    const int hi = hb + th, wi = wb + tw;
                    if (hi >= 0 && hi < p.H && wi >= 0 && wi < p.W) tap_mask |= 1u << tt;
                    if (++tw == p.KW) { tw = 0; ++th; }
                }
                src = p.act + (((int64_t)n * p.H + hb) * p.W + wb) * p.P;
            }
        };
        // one K step of the walk: with `load`, its CH chunks go to the ring
        auto walk_step = [&](bool load) {
            if (ld_ks == p.rounds) {
                ld_ks = 0;
                ld_tile += tstep;
                set_tile(ld_tile);
            }
            if (ld_tile < total_tiles) {
                const uint32_t dst = ring0 + ld_slot * SLOT_BYTES;
                // The walk advances run by run (2^lcr chunks that are contiguous in
                // memory and lie in one filter tap), which keeps its dependent chain
                // of address / tap updates short.
                unsigned long long run = 0ull;     // this row's current run (0: zero fill)
#pragma unroll
                for (int j = 0; j < KS * CH; ++j) {
                    if ((j & crm) == 0) {          // a new run starts
                        // (chunks past the pixel's P bytes, 3-bit rows only, are zeros)
                        const bool real = off < p.P;
                        const bool ok = real && tap < 32 && ((tap_mask >> tap) & 1u);
                        run = ok ? (unsigned long long)reinterpret_cast<uintptr_t>(src) : 0ull;
                        off += 16 << lcr;
                        if (real) src += 16 << lcr;
                        if (off == p.Pk) {
                            off = 0;
                            ++tap;
                            if (++kw == p.KW) { kw = 0; src += row_jump; }
                        }
                    }
                    if (!load) continue;
                    if (Pipe<PM>::COAL) {
                        // lane -> (row of this warp, chunk of the run)
                        const int rsel = ((j & crm) << (5 - lcr)) + lane_row;
                        const unsigned long long ptr = __shfl_sync(0xffffffffu, run, rsel);
                        const int cj = (j & ~crm) + lane_c;
                        cp_async_16(dst + cj * (BM * 16) + rsel * 16,
                                    ptr ? reinterpret_cast<const uint8_t *>((uintptr_t)ptr) +
                                              16 * lane_c
                                        : p.act,
                                    ptr ? 16u : 0u);
                    } else {
                        // every thread fetches its own row
                        cp_async_16(dst + lane * 16 + j * (BM * 16),
                                    run ? reinterpret_cast<const uint8_t *>((uintptr_t)run) +
                                              16 * (j & crm)
                                        : p.act,
                                    run ? 16u : 0u);
                    }
                }
                ++ld_ks;
                if (load && ++ld_slot == A_RING) ld_slot = 0;
            }
        };
        const uint32_t n_steps = (uint32_t)my_tiles_all * p.rounds;
        // own steps: g = group, group + GROUPS, ...
        const uint32_t n_own =
            GROUPS == 1 ? n_steps : (n_steps > (uint32_t)group ? (n_steps - group + 1) / 2 : 0u);
        int rd_slot = 0, pend_s = -1;
        bool ok = true;
        auto publish = [&]() {
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            // The A operand sits in this SM's tensor memory and only this SM's
            // tensor core reads it.  tcgen05.wait::st above returns once the
            // stores have COMPLETED (the data is in tensor memory; completion
            // of a tcgen05 operation carries no scope), and
            // tcgen05.fence::before_thread_sync orders it before the arrival:
            // the crossing arrival publishes no memory of its own, so it needs
            // no cluster-scope release.
            if (lane == 0) {
                if (PAIR && rank != 0) mbar_arrive_remote(map_to_cta(bar_a_full(pend_s), 0u));
                else mbar_arrive(bar_a_full(pend_s));
            }
            pend_s = -1;
        };
        // TMA mode: slot = 128 rows of KS*CH chunks, chunk index XOR-swizzled
        constexpr bool a_tma = A_TMA != 0;
        // chunk jj of the round lies in box jj >> a_lc, at chunk (jj ^ swizzle) of
        // this thread's row of that box
        const int lc = p.a_lc;
        const uint32_t tma_row = smem_u32(smem + L.a_ring) + ((uint32_t)row << (4 + lc));
        const int swz = (row >> (3 - lc)) & ((1 << lc) - 1);
        auto tma_chunk = [&](int jj) {
            return tma_row + ((uint32_t)(jj >> lc) << (11 + lc)) +
                   (uint32_t)((((jj & ((1 << lc) - 1)) ^ swz)) << 4);
        };
        int kr = group % p.rounds;                 // K round of the step being consumed
        if (!a_tma && GROUPS == 2 && group == 1) walk_step(false);   // step 0 belongs to group 0
        // iteration i issues own step i and consumes own step i - A_D
#pragma unroll 1
        for (uint32_t i = 0; ok && i < n_own + A_D; ++i) {
            if (!a_tma) {
                walk_step(true);                   // own step (no-op past the end)
                cp_async_commit();                 // one group per own step
                if (GROUPS == 2) walk_step(false); // the other group's step
            }
            if (i < (uint32_t)A_D) continue;
            const uint32_t g = GROUPS * (i - A_D) + group;
            const int aslot = (int)(g % A_SLOTS);
            if (a_tma) {
                if (!(ok = wait_bar_warp(bar_ar_full(aslot), (g / A_SLOTS) & 1u, ctl, 12))) break;
            } else {
                cp_async_wait<A_D>();              // own step i - A_D has landed
                if (Pipe<PM>::COAL) __syncwarp();  // ... the other lanes' copies of my row too
            }
            const int s = g % S_U;
            const uint32_t ph = (g / S_U) & 1u;
            // chunks of this round that exist (im2col: nothing is loaded past the
            // last filter tap)
            int kvalid = KS * CH;
            // rows mode: where this thread's pixel lies in the staged image rows
            constexpr int CPP = BITS / 2;              // 16-byte chunks per pixel (64 channels)
            constexpr bool rows_mode = Pipe<PM>::WHOLE_K && BITS != 3 && A_TMA == 3;
            uint32_t rows_base = 0, rowmask = 0, colmask = 0, sw16 = 0;
            if (Pipe<PM>::WHOLE_K && rows_mode) {
                const int tile = tile0 + (int)g * tstep;       // one round per tile
                const int m0 = (tile / p.n_tiles) * BMT + row_base;
                const int m = m0 + row;
                const int R = m / p.W, wo = m - R * p.W, ho = R % p.H;
                // bit kh / kw: that row / column of the 3x3 window is inside the image
                rowmask = m < p.M ? (uint32_t)((ho > 0) | 2 | ((ho < p.H - 1) << 2)) : 0u;
                colmask = (uint32_t)((wo > 0) | 2 | ((wo < p.W - 1) << 2));
                rows_base = smem_u32(smem + L.a_ring) + aslot * SLOT_BYTES +
                            (uint32_t)((R - m0 / p.W) * p.a_bw + (wo - 1) * p.P);
                // two chunks per pixel: adjacent lanes are 32 bytes apart, so lanes
                // 4..7 of a quarter warp fetch each pair of chunks in the other
                // order (and swap afterwards): conflict-free 128-bit loads
                sw16 = CPP == 2 ? (uint32_t)((lane >> 2) & 1) << 4 : 0u;
            }
            if (a_tma) {
                if (p.a_tma == 2) kvalid = p.a_kchunks - kr * (KS * CH);
                kr += GROUPS;
                if (kr >= p.rounds) kr -= p.rounds;
                if (kr >= p.rounds) kr -= p.rounds;
            }
#pragma unroll
            for (int h = 0; h < KS; ++h) {
                uint32_t o[32];
                {
                    uint4 cur[CH];
#pragma unroll
                    for (int j = 0; j < CH; ++j) {
                        if (Pipe<PM>::WHOLE_K && BITS != 3 && rows_mode) {
                            // chunk jj of the K row: window row jj / (3 CPP), then
                            // 3 CPP consecutive chunks.  Always loaded (the address
                            // stays inside shared memory), zeroed when outside
                            const int kk = h * CH + j;
                            const int kh = kk / (3 * CPP), q = kk % (3 * CPP);
                            const uint32_t keep =
                                ((rowmask >> kh) & (colmask >> (q / CPP)) & 1u) ? 0xFFFFFFFFu : 0u;
                            uint4 v = lds_128(rows_base + (uint32_t)(kh * p.a_bw) +
                                              ((uint32_t)(q * 16) ^ sw16));
                            v.x &= keep; v.y &= keep; v.z &= keep; v.w &= keep;
                            cur[j] = v;
                        } else if (a_tma) {
                            cur[j] = (h * CH + j < kvalid)
                                         ? lds_128(tma_chunk(h * CH + j) + aslot * SLOT_BYTES)
                                         : make_uint4(0u, 0u, 0u, 0u);
                        } else {
                            cur[j] = lds_128(cell0 + rd_slot * SLOT_BYTES +
                                             (h * CH + j) * (BM * 16));
                        }
                    }
                    if (rows_mode && CPP == 2 && sw16) {
#pragma unroll
                        for (int j = 0; j + 1 < CH; j += 2) {
                            const uint4 t = cur[j];
                            cur[j] = cur[j + 1];
                            cur[j + 1] = t;
                        }
                    }
                    expand_row_regs<BITS, A_SIGNED>(cur, p.orv, o);
                }
                if (h == 0) {
                    if (!(ok = wait_bar_warp(bar_u_empty(s), ph ^ 1u, ctl, 5))) break;
                    tc_fence_after_sync();
                }
                __syncwarp();
                tmem_st_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + A_COL0 +
                                  (s * KS + h) * 32, o);
            }
            if (!ok) break;
            if (++rd_slot == A_RING) rd_slot = 0;
            if (a_tma) {                           // the slot may be refilled
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_ar_empty(aslot));
            }
            pend_s = s;
            publish();                             // the other group's step overlaps this
        }
        cp_async_wait<0>();
        if (ok && p.join) join_idx = 1 + group;
        } else if (WIDE) {
            // the unused second A group helps the epilogue
            epi_idx = 1;
            join_idx = 2;
            if (!p.join) epi_slot = NUM_E_WARPS + (warp - WARP_A0 - 4);
        }
    } else if (warp < WARP_E0) {
        // ---------------- B: expand packed shared tiles ---------------------
        constexpr int BT = NUM_B_THREADS / B_GROUPS;      // threads expanding one round
        const int bgroup = B_GROUPS == 1 ? 0 : (warp - WARP_B0) / (NUM_B_WARPS / B_GROUPS);
        const int tid = threadIdx.x - WARP_B0 * 32 - bgroup * BT;
        // a packed row of the round holds CHK = KS*CH chunks.  Thread (row0, j)
        // owns chunk j of every K step of rows row0 + i*ROWS_PER_IT: the eight
        // lanes of a 128-bit store phase then cover two rows x four chunks of
        // one K step, i.e. eight different 16-byte bank groups of the swizzled
        // tile (lanes split over two K steps would collide pairwise, the K steps
        // being a multiple of 128 bytes apart); (row & 7) does not depend on i
        constexpr int CHK = KS * CH;
        constexpr int ROWS_PER_IT = (BITS == 3) ? BT : BT / CH;
        // (pairs expand half of a tile's B rows)
        constexpr int MAX_IT = (BITS == 3) ? 1 : ((PAIR ? 128 : 256) * CH) / BT;
        const int row0 = (BITS == 3) ? tid : tid / CH;
        const int j = (BITS == 3) ? 0 : tid % CH;
        const int sw = row0 & 7;
        const int n_it = (BNL + ROWS_PER_IT - 1) / ROWS_PER_IT;
        uint32_t php = 0;
        int sp = bgroup - B_GROUPS;
        bool ok = true;
        {
#pragma unroll 1
            for (uint32_t g = bgroup; g < n_b_steps; g += B_GROUPS) {
                sp += B_GROUPS;                      // sp = g % S_P, php = (g / S_P) & 1
                if (sp >= S_P) { sp -= S_P; php ^= 1u; }
                const int su = p.b_res ? (int)g : (int)(g % S_U);
                const uint32_t phu = (g / S_U) & 1u;
                if (!(ok = wait_bar_warp(bar_p_full(sp), php, ctl, 6))) break;
                const uint8_t *src = smem + L.b_packed + sp * b_packed_bytes;
                uint8_t *dst = smem + L.b_tiles + su * b_tile_bytes;
                if (BITS == 3) {
                    uint32_t w[12];
                    if (row0 < BNL) {
                        const uint4 *r4 = reinterpret_cast<const uint4 *>(src + row0 * 48);
#pragma unroll
                        for (int l = 0; l < 3; ++l) {
                            const uint4 v = r4[l];
                            w[4 * l] = v.x; w[4 * l + 1] = v.y;
                            w[4 * l + 2] = v.z; w[4 * l + 3] = v.w;
                        }
                    }
                    if (!p.b_res && !(ok = wait_bar_warp(bar_u_empty(su), phu ^ 1u, ctl, 7))) break;
                    if (row0 < BNL) {
                        uint8_t *rowp = dst + row0 * BK_BYTES;
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            *reinterpret_cast<uint4 *>(rowp + ((q ^ sw) << 4)) =
                                expand3_chunk<B_SIGNED>(w, q, p.orv);
                    }
                } else if (Pipe<PM>::WHOLE_K) {
                    // whole-K mode (resident tile, expanded once per CTA): K step
                    // by K step, packed layout [K step][row][CH chunks]
                    constexpr int OUT = Chunks<BITS>::OUT;
#pragma unroll 1
                    for (int h = 0; h < KS; ++h)
#pragma unroll 1
                        for (int r = row0; r < BNL; r += ROWS_PER_IT) {
                            const uint4 v = reinterpret_cast<const uint4 *>(
                                src)[(h * BNL + r) * CH + j];
                            uint8_t *rowp = dst + h * b_sub_bytes + r * BK_BYTES;
#pragma unroll
                            for (int c = 0; c < OUT; ++c)
                                *reinterpret_cast<uint4 *>(rowp + (((j * OUT + c) ^ sw) << 4)) =
                                    make_uint4(expand_word<BITS, B_SIGNED>(v.x, c, p.orv),
                                               expand_word<BITS, B_SIGNED>(v.y, c, p.orv),
                                               expand_word<BITS, B_SIGNED>(v.z, c, p.orv),
                                               expand_word<BITS, B_SIGNED>(v.w, c, p.orv));
                        }
                } else {
                    constexpr int OUT = Chunks<BITS>::OUT;
                    constexpr int KSV = Pipe<PM>::WHOLE_K ? 1 : KS;   // (whole-K never gets here)
                    uint4 v[MAX_IT][KSV];
                    // The packed tile is row-major, so the rows of a quarter warp
                    // (two with 4-bit codes, four with 2-bit codes) would fetch the
                    // same 16-byte bank groups: each row starts at another K step
                    // (register slot h holds K step (h + rot) mod KS)
                    const int rot = BITS == 4 ? (row0 & 1) : KSV == 4 ? (row0 & 3) : ((row0 >> 1) & 1);
#pragma unroll
                    for (int i = 0; i < MAX_IT; ++i)
                        if (i < n_it && row0 + i * ROWS_PER_IT < BNL) {
#pragma unroll
                            for (int h = 0; h < KSV; ++h)
                                v[i][h] = reinterpret_cast<const uint4 *>(
                                    src)[(row0 + i * ROWS_PER_IT) * CHK +
                                         ((h + rot) & (KSV - 1)) * CH + j];
                        }
                    if (!p.b_res && !(ok = wait_bar_warp(bar_u_empty(su), phu ^ 1u, ctl, 7))) break;
                    uint8_t *rowp = dst + row0 * BK_BYTES;
#pragma unroll
                    for (int i = 0; i < MAX_IT; ++i) {
                        if (i < n_it && row0 + i * ROWS_PER_IT < BNL) {
#pragma unroll
                            for (int h = 0; h < KSV; ++h)
#pragma unroll
                                for (int c = 0; c < OUT; ++c) {
                                    const uint4 o = make_uint4(
                                        expand_word<BITS, B_SIGNED>(v[i][h].x, c, p.orv),
                                        expand_word<BITS, B_SIGNED>(v[i][h].y, c, p.orv),
                                        expand_word<BITS, B_SIGNED>(v[i][h].z, c, p.orv),
                                        expand_word<BITS, B_SIGNED>(v[i][h].w, c, p.orv));
                                    *reinterpret_cast<uint4 *>(
                                        rowp + ((h + rot) & (KSV - 1)) * b_sub_bytes +
                                        i * ROWS_PER_IT * BK_BYTES +
                                        (((j * OUT + c) ^ sw) << 4)) = o;
                                }
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    // (a pair's B halves are read by the tensor cores of BOTH SMs)
                    if (PAIR && rank == 0) mbar_arrive_release_cluster(bar_a_full(su));
                    else arrive_leader(p.b_res ? bar_b_full(su) : bar_a_full(su));
                    mbar_arrive(bar_p_empty(sp));
                }
            }
        }
        // with a resident B tile these eight warps are done after the first
        // rounds: they join the epilogue (two more warps per TMEM lane quarter)
        if (p.b_res && ok) {
            epi_idx = 1 + ((warp - WARP_B0) >> 2);
            if (!p.join) epi_slot = NUM_E_WARPS + (warp - WARP_B0);
        }
        if (ok && p.join) join_idx = 3 + ((warp - WARP_B0) >> 2);
    } else {
        epi_idx = 0;
        join_idx = 0;
        if (!p.join) epi_slot = warp - WARP_E0;
    }

    if (epi_idx >= 0 || join_idx >= 0) {
        // ---------------- epilogue -------------------------------------------
        // epi_cnt warps share a lane quarter and take the 32-column chunks of a
        // tile in turn
        const int quarter = warp & 3;                 // TMEM lanes 32q .. 32q+31
        const int row_in_tile = quarter * 32 + lane;
        uint32_t it = 0;
        bool ok = true;
#pragma unroll 1
        for (int tile = tile0; ok && tile < total_tiles; tile += tstep, ++it) {
            const bool last = tile + tstep >= total_tiles;
            const bool joined = last && p.join;
            const int my_idx = joined ? join_idx : epi_idx;
            const int epi_cnt = joined ? JOIN_CNT : p.epw;
            if (my_idx < 0) continue;
            const int as = p.n_acc == 2 ? (it & 1) : 0;
            const uint32_t aph = (p.n_acc == 2 ? (it >> 1) : it) & 1u;
            const int m_tile = tile / p.n_tiles, n_tile = tile % p.n_tiles;
            const int64_t m = (int64_t)m_tile * BMT + row_base + row_in_tile;
            const bool row_ok = m < p.M;
            // helpers have not followed the accumulator barriers' phases: they wait
            // on the single-use barrier of the last tile
            if (!(ok = epi_idx >= 0 ? wait_bar_warp(bar_acc_full(as), aph, ctl, 8)
                                    : wait_bar_warp(bar_last_full, 0u, ctl, 13)))
                break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + as * BN;
            float rs = 0.f;
            if (EPI == EPI_GEMM && p.row_scale && row_ok) rs = __ldg(p.row_scale + m);
            // general weight-grid offset: S_a of this output pixel, summed from
            // the input codes under its filter window
            int s_a = 0;
            if (EPI == EPI_GENERAL && p.e.general_offset && row_ok) {
                const int wo = (int)(m % p.Wo), t = (int)(m / p.Wo);
                s_a = dsq_window_sa<BITS>(p.act, t / p.Ho, t % p.Ho, wo, p.H, p.W, p.KW, p.stride,
                                          p.pad, p.P);
            }
            // per-warp staging of the chunk's 32 scale / bias values: lane i fetches
            // column i (prefetched one chunk ahead), the warp reads them back as
            // broadcast 128-bit shared loads
            float *epi_scale = reinterpret_cast<float *>(smem + L.epi) + epi_slot * 64;
            float *epi_bias = epi_scale + 32;
            float sc_nx = 0.f, bi_nx = 0.f;
            auto fetch_cols = [&](int c0) {
                const int n = n_tile * BN + c0 + lane;
                sc_nx = 0.f; bi_nx = 0.f;
                if (EPI != EPI_GEMM && c0 < BN && n < p.Ncols) {
                    sc_nx = __ldg(p.e.scale + n);
                    if (p.e.half_offset) sc_nx = __fmul_rn(sc_nx, 0.5f);
                    bi_nx = __ldg(p.e.bias + n);
                }
            };
            fetch_cols(my_idx * 32);
#pragma unroll 1
            for (int c0 = my_idx * 32; c0 < BN; c0 += 32 * epi_cnt) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_32x32(taddr + c0, r);
                if (EPI != EPI_GEMM) {
                    epi_scale[lane] = sc_nx;
                    epi_bias[lane] = bi_nx;
                    fetch_cols(c0 + 32 * epi_cnt);
                    __syncwarp();
                }
                tmem_ld_wait();
                const int n0 = n_tile * BN + c0;
                if (!row_ok) continue;
                if (EPI == EPI_GEMM || EPI == EPI_GENERAL) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) r[c] = (uint32_t)((int)r[c] >> p.shift);
                }
                const bool full = n0 + 32 <= p.Ncols && (p.Ncols & 3) == 0;
                if (EPI == EPI_GEMM) {
                    if (n0 >= p.Ncols) continue;
                    if (p.C_i32) {
                        int32_t *dst = p.C_i32 + m * p.Ncols + n0;
                        if (full && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
                            // one full 32-byte sector per lane and store
#pragma unroll
                            for (int v = 0; v < 4; ++v)
                                stg_256(dst + 8 * v, r[8 * v], r[8 * v + 1], r[8 * v + 2],
                                        r[8 * v + 3], r[8 * v + 4], r[8 * v + 5], r[8 * v + 6],
                                        r[8 * v + 7]);
                        } else if (full) {
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                reinterpret_cast<int4 *>(dst)[v] =
                                    make_int4((int)r[4 * v], (int)r[4 * v + 1],
                                              (int)r[4 * v + 2], (int)r[4 * v + 3]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (n0 + c < p.Ncols) dst[c] = (int)r[c];
                        }
                    }
                    if (p.D_f32) {
                        float *dst = p.D_f32 + m * p.Ncols + n0;
                        if (full && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
#pragma unroll
                            for (int v = 0; v < 4; ++v) {
                                uint32_t f[8];
#pragma unroll
                                for (int u = 0; u < 8; ++u)
                                    f[u] = __float_as_uint(
                                        __fmul_rn((float)(int)r[8 * v + u], rs));
                                stg_256(dst + 8 * v, f[0], f[1], f[2], f[3], f[4], f[5], f[6],
                                        f[7]);
                            }
                        } else if (full) {
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                reinterpret_cast<float4 *>(dst)[v] =
                                    make_float4(__fmul_rn((float)(int)r[4 * v], rs),
                                                __fmul_rn((float)(int)r[4 * v + 1], rs),
                                                __fmul_rn((float)(int)r[4 * v + 2], rs),
                                                __fmul_rn((float)(int)r[4 * v + 3], rs));
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (n0 + c < p.Ncols)
                                    dst[c] = __fmul_rn((float)(int)r[c], rs);
                        }
                    }
                } else if (EPI == EPI_CODES || EPI == EPI_CODES_RES) {
                    // codes-only convolution epilogue (the form the stacks use).
                    // Per element, bit-identical to the pinned sequence:
                    //   v  = raw >> shift; vf = (float)v (1.5 * 2^23 trick where the
                    //        accumulator is below 2^22)
                    //   y  = fma(vf, scale, bias) (+ lut[q_r]: lut[q] = fma(q, Delta_r, l_r))
                    //   r  = min(fma(max(y, lo) - lo, inv, 0.5), r_hi)
                    // (clipping y at hi first, or r at r_hi = fma(hi - lo, inv, 0.5)
                    // afterwards, gives the same r: fma is monotone; floor(r) <= qmax
                    // because floor(r_hi) = qmax, checked by the host).  The bits of
                    // r + 2^23 rounded down are 0x4B000000 + floor(r): the codes are
                    // summed into their fields, the constant leaves once per word.
                    const DsqEpi &e = p.e;
                    constexpr uint32_t MASK = (1u << BITS) - 1u;
                    constexpr int CW = BITS;                 // code words per 32 columns
                    const int byte0 = n0 * BITS / 8;
                    if (byte0 >= p.out_pitch) continue;
                    uint32_t resw[CW];
#pragma unroll
                    for (int w = 0; w < CW; ++w) resw[w] = 0u;
                    if (EPI == EPI_CODES_RES) {
                        const uint32_t *rp = reinterpret_cast<const uint32_t *>(
                            e.residual + m * p.out_pitch + byte0);
#pragma unroll
                        for (int w = 0; w < CW; ++w) resw[w] = __ldg(rp + w);
                    }
                    uint32_t cw[CW];
#pragma unroll
                    for (int w = 0; w < CW; ++w) cw[w] = 0u;
                    const float *lut = reinterpret_cast<const float *>(smem + L.lut);
                    const float4 *sc4 = reinterpret_cast<const float4 *>(epi_scale);
                    const float4 *bi4 = reinterpret_cast<const float4 *>(epi_bias);
                    float4 s_nx = sc4[0], b_nx = bi4[0];
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const float4 s_cur = s_nx, b_cur = b_nx;
                        if (v < 7) { s_nx = sc4[v + 1]; b_nx = bi4[v + 1]; }
                        const float scs[4] = {s_cur.x, s_cur.y, s_cur.z, s_cur.w};
                        const float bis[4] = {b_cur.x, b_cur.y, b_cur.z, b_cur.w};
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int c = 4 * v + u;
                            const int vi = (int)r[c] >> p.shift;
                            const float vf = p.small_acc
                                ? __fsub_rn(__int_as_float(0x4B400000 + vi), 12582912.0f)
                                : (float)vi;
                            float y = __fmaf_rn(vf, scs[u], bis[u]);
                            if (EPI == EPI_CODES_RES) {
                                const uint32_t qr =
                                    (resw[(c * BITS) >> 5] >> ((c * BITS) & 31)) & MASK;
                                y = __fadd_rn(y, lut[qr]);
                            }
                            const float d = __fsub_rn(fmaxf(y, e.rq.lo), e.rq.lo);
                            const float rr = fminf(__fmaf_rn(d, e.rq.inv, 0.5f), p.r_hi);
                            cw[(c * BITS) >> 5] +=
                                (uint32_t)__float_as_int(__fadd_rd(rr, 8388608.0f)) << ((c * BITS) & 31);
                        }
                    }
                    {
                        // 0x4B000000 summed over the fields of a word (mod 2^32)
                        constexpr uint32_t FIELDS = BITS == 4 ? 0x11111111u : 0x55555555u;
#pragma unroll
                        for (int w = 0; w < CW; ++w) cw[w] -= 0x4B000000u * FIELDS;
                    }
                    // columns past Cout are padding lanes of the packed row: zero
                    const int nvalid_bits = min(32, max(0, p.Ncols - n0)) * BITS;
#pragma unroll
                    for (int w = 0; w < CW; ++w) {
                        const int nb = nvalid_bits - 32 * w;
                        cw[w] &= nb >= 32 ? 0xFFFFFFFFu : nb <= 0 ? 0u : ((1u << nb) - 1u);
                    }
                    uint32_t *dst =
                        reinterpret_cast<uint32_t *>(e.y_codes + m * p.out_pitch + byte0);
                    if (CW == 4)
                        *reinterpret_cast<uint4 *>(dst) = make_uint4(cw[0], cw[1], cw[2], cw[CW - 1]);
                    else
                        *reinterpret_cast<uint2 *>(dst) = make_uint2(cw[0], cw[CW - 1]);
                } else {
                    const DsqEpi &e = p.e;
                    constexpr uint32_t MASK = (1u << BITS) - 1u;
                    constexpr int CW = BITS;                 // code words per 32 columns
                    const int byte0 = n0 * BITS / 8;
                    uint32_t resw[CW];
#pragma unroll
                    for (int w = 0; w < CW; ++w) resw[w] = 0u;
                    if (e.residual && byte0 < p.out_pitch) {
                        const uint32_t *rp = reinterpret_cast<const uint32_t *>(
                            e.residual + m * p.out_pitch + byte0);
                        // (a block of 3-bit codes may reach past the end of the row)
#pragma unroll
                        for (int w = 0; w < CW; ++w)
                            if (BITS != 3 || byte0 + 4 * w < p.out_pitch) resw[w] = __ldg(rp + w);
                    }
                    uint32_t cw[CW];
#pragma unroll
                    for (int w = 0; w < CW; ++w) cw[w] = 0u;
                    if (e.acc_out && n0 < p.Ncols) {
                        int32_t *dst = e.acc_out + m * p.Ncols + n0;
                        if (full) {
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                reinterpret_cast<int4 *>(dst)[v] =
                                    make_int4((int)r[4 * v], (int)r[4 * v + 1],
                                              (int)r[4 * v + 2], (int)r[4 * v + 3]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (n0 + c < p.Ncols) dst[c] = (int)r[c];
                        }
                    }
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        float y4[4];
                        const float4 sc4 = *reinterpret_cast<const float4 *>(epi_scale + 4 * v);
                        const float4 bi4 = *reinterpret_cast<const float4 *>(epi_bias + 4 * v);
                        const float scs[4] = {sc4.x, sc4.y, sc4.z, sc4.w};
                        const float bis[4] = {bi4.x, bi4.y, bi4.z, bi4.w};
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int c = 4 * v + u;
                            const int n = n0 + c;
                            float y = 0.f;
                            if (n < p.Ncols) {
                                y = e.general_offset
                                        ? dsq_epi_y_offset((int)r[c], s_a, e.w_offset, scs[u], bis[u])
                                        : dsq_epi_y((int)r[c], scs[u], bis[u]);
                                // field c of the 32-column block: word fw, bit fs (a
                                // 3-bit field may straddle two words; never the last)
                                const int fw = (c * BITS) >> 5, fs = (c * BITS) & 31;
                                const int fw1 = fw + 1 < CW ? fw + 1 : fw;
                                if (e.residual) {
                                    const uint32_t qr =
                                        __funnelshift_r(resw[fw], fw + 1 < CW ? resw[fw1] : 0u, fs) & MASK;
                                    y = dsq_epi_residual(y, qr, e.res_delta, e.res_lo);
                                }
                                if (e.has_requant) {
                                    const uint32_t q = dsq_code(y, e.rq);
                                    cw[fw] |= q << fs;
                                    if (BITS == 3 && fs > 29) cw[fw1] |= q >> (32 - fs);
                                }
                            }
                            y4[u] = y;
                        }
                        if (e.y_f32 && n0 + 4 * v < p.Ncols) {
                            float *dst = e.y_f32 + m * p.Ncols + n0 + 4 * v;
                            if (full) {
                                *reinterpret_cast<float4 *>(dst) =
                                    make_float4(y4[0], y4[1], y4[2], y4[3]);
                            } else {
#pragma unroll
                                for (int u = 0; u < 4; ++u)
                                    if (n0 + 4 * v + u < p.Ncols) dst[u] = y4[u];
                            }
                        }
                    }
                    if (e.y_codes && byte0 < p.out_pitch) {
                        uint32_t *dst = reinterpret_cast<uint32_t *>(
                            e.y_codes + m * p.out_pitch + byte0);
                        if (CW == 4)
                            *reinterpret_cast<uint4 *>(dst) =
                                make_uint4(cw[0], cw[1], cw[2], cw[CW - 1]);
                        else if (CW == 3) {
                            // 12 bytes, as far as the row goes
                            dst[0] = cw[0];
                            if (byte0 + 4 < p.out_pitch) dst[1] = cw[1];
                            if (byte0 + 8 < p.out_pitch) dst[2] = cw[CW - 1];
                            // 3-bit rows: the N tiles may end before the row's pitch
                            // does (64 columns = 24 bytes, pitch 32): spare bytes are zero
                            if (n_tile == p.n_tiles - 1 && c0 + 32 >= BN)
                                for (int b = p.n_tiles * BN * BITS / 8; b < p.out_pitch; b += 4)
                                    *reinterpret_cast<uint32_t *>(e.y_codes + m * p.out_pitch + b) = 0u;
                        } else
                            *reinterpret_cast<uint2 *>(dst) = make_uint2(cw[0], cw[CW - 1]);
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0 && epi_idx >= 0) arrive_leader(bar_acc_empty(as));
        }
    }

    // ---------------- teardown ---------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    // a CTA of a pair stays until its peer has stopped signalling its barriers
    // and reading operands from its shared and tensor memory
    if (PAIR) cluster_sync_all();
    if (warp == WARP_MMA) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc<CG>(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------
// tensor-core rate probe: MMAs only, operands resident in shared memory
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int iters, int *ws)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~(uintptr_t)1023u);
    __shared__ uint64_t bar_storage[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5;
    // A: 128 rows x 128 B, B: 256 rows x 128 B, filled with varied bytes
    for (int i = threadIdx.x; i < (128 + 256) * 128 / 4; i += blockDim.x)
        reinterpret_cast<uint32_t *>(smem)[i] = 0x9E3779B9u * (uint32_t)(i + 1);
    const uint32_t bar = smem_u32(&bar_storage[0]);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_init(bar + 8, 1);
        abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 256);
        tmem_relinquish();
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    if (threadIdx.x == 0) {
        Ctl ctl{&abort_flag, ws, WAIT_LIMIT_NS};
        const uint32_t idesc = idesc_i8(256, true, false);
        const uint64_t ad = smem_desc_sw128(smem_u32(smem));
        const uint64_t bd = smem_desc_sw128(smem_u32(smem + 128 * 128));
        // batches of 64 instructions, two in flight: wait for batch b-1 only
        // after batch b has been issued, so the pipe never drains
        const int batches = (iters + 63) / 64;
        bool ok = true;
        for (int b = 0; ok && b < batches; ++b) {
            const int n = min(64, iters - 64 * b);
            for (int k = 0; k < n; ++k)
                mma_i8(tmem, ad + 2 * (k & 3), bd + 2 * (k & 3), idesc, 1u);
            mma_commit(bar + 8 * (b & 1));
            if (b > 0)
                ok = wait_bar(bar + 8 * ((b - 1) & 1), ((b - 1) >> 1) & 1u, ctl, 9);
        }
        if (ok && batches > 0)
            wait_bar(bar + 8 * ((batches - 1) & 1), ((batches - 1) >> 1) & 1u, ctl, 9);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem, 256);
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
typedef DsqEncodeTiledFn EncodeTiledFn;
EncodeTiledFn get_encode_fn() { return dsq_encode_tiled_fn(); }

// 2-D byte map over packed rows: inner dimension = row bytes, outer = rows.
struct TcMaps { CUtensorMap b, a; };   // the two operands

int make_rows_tmap(CUtensorMap *map, const void *base, uint64_t row_bytes, uint64_t rows,
                   uint64_t pitch, uint32_t box_bytes, uint32_t box_rows,
                   CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return DSQ_ERR_CUDA;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {pitch};
    cuuint32_t box[2] = {box_bytes, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DSQ_OK : DSQ_ERR_CUDA;
}

// Resident B: one N tile and few K steps, so the expanded B tile of every K
// step fits in shared memory next to the rings; it is then expanded once per
// CTA instead of once per M tile.
struct PipeInfo { int ks, su, a_slots, a_col0, s_p, wide, pair, whole_k; };
PipeInfo pipe_info(int pm)
{
    switch (pm) {
    case 5: return {Pipe<5>::KS, Pipe<5>::SU, Pipe<5>::GROUPS * Pipe<5>::A_RING, Pipe<5>::A_COL0, Pipe<5>::S_P, 0, 0, 1};
    case 4: return {Pipe<4>::KS, Pipe<4>::SU, Pipe<4>::GROUPS * Pipe<4>::A_RING, Pipe<4>::A_COL0, Pipe<4>::S_P, 0, 1};
    case 1: return {Pipe<1>::KS, Pipe<1>::SU, Pipe<1>::GROUPS * Pipe<1>::A_RING, Pipe<1>::A_COL0, Pipe<1>::S_P, 0};
    case 2: return {Pipe<2>::KS, Pipe<2>::SU, Pipe<2>::GROUPS * Pipe<2>::A_RING, Pipe<2>::A_COL0, Pipe<2>::S_P, 0};
    default: return {Pipe<3>::KS, Pipe<3>::SU, Pipe<3>::GROUPS * Pipe<3>::A_RING, Pipe<3>::A_COL0, Pipe<3>::S_P, 1};
    }
}

// Fills the fields that depend on the pipeline mode; picks resident B where it
// fits (one N tile, few rounds, more M tiles than SMs).
void choose_b_mode(TcParams *p, int bits, int pm)
{
    const PipeInfo pi = pipe_info(pm);
    p->rounds = (p->ksteps + pi.ks - 1) / pi.ks;
    p->n_acc = 2 * p->BN <= pi.a_col0 ? 2 : 1;
    p->s_p = pi.s_p;
    p->b_res = 0;
    p->b_stages = pi.su;
    p->epw = pi.wide ? 2 : 1;
    if (!pi.wide && !pi.pair && p->n_tiles == 1 && p->rounds <= MAX_B_STAGES && p->m_tiles > dsq_sm_count()) {
        const SmemLayout L = smem_layout(p->BN, bits, p->s_p, p->rounds, pi.ks, pi.a_slots,
                                         epi_slots(1, 3));
        if (L.total + 1024 <= 227u * 1024u) {
            p->b_res = 1;
            p->b_stages = p->rounds;
            p->epw = 3;
        }
    }
    if (pi.whole_k && !p->b_res) p->rounds = -1;     // the caller falls back to another mode
    const SmemLayout Lj = smem_layout(pi.pair ? p->BN / 2 : p->BN, bits, p->s_p, p->b_stages, pi.ks,
                                      pi.a_slots, epi_slots(1, p->epw));
    p->join = Lj.total + 1024 <= 227u * 1024u;
}

// Run length of the coalesced A gather: the largest power of two of 16-byte
// chunks that divides both a pixel's packed row (so a run never straddles two
// filter taps) and the chunks of a round.
int a_run_log2(int P, int bits, int ks)
{
    if (bits == 3) return 0;
    const int chk = ks * bits, q = P / 16;
    int l = 0;
    while (l < 3 && (2 << l) <= chk && q % (2 << l) == 0) ++l;
    return l;
}

typedef DsqEncodeIm2colFn EncodeIm2colFn;
EncodeIm2colFn get_encode_im2col_fn() { return dsq_encode_im2col_fn(); }

CUtensorMapSwizzle swizzle_for_span(int bytes)
{
    return bytes == 128  ? CU_TENSOR_MAP_SWIZZLE_128B
           : bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
           : bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                         : CU_TENSOR_MAP_SWIZZLE_NONE;
}

// TMA-fed A ring.  A round of a row (32, 64 or 128 packed bytes) is cut into
// boxes of 128 rows x `sub` bytes, sub a power of two between 16 and 128 (one
// swizzle span, so that the row-per-thread reads of the ring are free of bank
// conflicts).  Plain rows (GEMM, 1x1 stride-1 unpadded convolution): one 2-D
// box per round.  Any other convolution: im2col boxes over the NHWC tensor,
// `sub` the largest such power of two that divides the pixel pitch.
int setup_a_tma(TcParams *p, CUtensorMap *map, const void *A, int64_t rows, int bits, int ks,
                bool plain_rows, const dsq_nhwc_t *shape, int ksize, bool whole_k)
{
    p->a_tma = 0;
    p->a_lc = 0;
    p->a_nsub = 1;
    p->a_kchunks = 0;
    p->a_nr = p->a_bw = 0;
    const int round_bytes = ks * bits * 16;
    if (bits == 3) return DSQ_OK;
    // whole image rows (TcParams::a_tma == 3): 3x3, stride 1, pad 1, 64 channels
    if (whole_k && !plain_rows && ksize == 3 && p->stride == 1 && p->pad == 1 &&
        p->P == 8 * bits) {
        const int64_t row_bytes = (int64_t)shape->W * p->P;
        const int nr = (BM - 1 + shape->W - 1) / shape->W + 3;
        if (row_bytes <= 2048 && row_bytes % 16 == 0 && nr <= 256 &&
            nr * row_bytes <= (int64_t)round_bytes * BM) {
            EncodeTiledFn fn = get_encode_fn();
            if (!fn) return DSQ_ERR_CUDA;
            // 8-byte elements, so that a box may span a whole row of up to 2 KB
            cuuint64_t dims[2] = {(cuuint64_t)(row_bytes / 8),
                                  (cuuint64_t)shape->N * (cuuint64_t)shape->H};
            cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
            cuuint32_t box[2] = {(cuuint32_t)(row_bytes / 8), (cuuint32_t)nr};
            cuuint32_t estr[2] = {1, 1};
            const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void *>(A),
                                  dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return DSQ_ERR_CUDA;
            p->a_tma = 3;
            p->a_nr = nr;
            p->a_bw = (int)row_bytes;
            return DSQ_OK;
        }
    }
    if (plain_rows) {
        const int st = make_rows_tmap(map, A, (uint64_t)p->P, (uint64_t)rows, (uint64_t)p->P,
                                      (uint32_t)round_bytes, BM, swizzle_for_span(round_bytes));
        if (st) return st;
        p->a_tma = 1;
        p->a_lc = round_bytes == 128 ? 3 : round_bytes == 64 ? 2 : 1;
        return DSQ_OK;
    }
    int sub = 128;
    while (sub > 16 && (p->P % sub != 0 || round_bytes % sub != 0)) sub >>= 1;
    EncodeIm2colFn fn = get_encode_im2col_fn();
    if (!fn) return DSQ_ERR_CUDA;
    const cuuint64_t P = (cuuint64_t)p->P;
    cuuint64_t dims[4] = {P, (cuuint64_t)shape->W, (cuuint64_t)shape->H, (cuuint64_t)shape->N};
    cuuint64_t strides[3] = {P, P * shape->W, P * shape->W * shape->H};
    // window-corner positions run from -pad to (extent - 1) + pad - (ksize - 1)
    int lower[2] = {-p->pad, -p->pad};
    int upper[2] = {p->pad - (ksize - 1), p->pad - (ksize - 1)};
    cuuint32_t estr[4] = {1, (cuuint32_t)p->stride, (cuuint32_t)p->stride, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(A), dims,
                          strides, lower, upper, (cuuint32_t)sub, BM, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for_span(sub),
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DSQ_ERR_CUDA;
    p->a_tma = 2;
    p->a_lc = sub == 128 ? 3 : sub == 64 ? 2 : sub == 32 ? 1 : 0;
    p->a_nsub = round_bytes / sub;
    p->a_kchunks = p->taps * (p->P / 16);
    return DSQ_OK;
}

// process-wide hooks (csrc/dsq_hooks.h)
std::atomic<int> g_forced_bn{0};      // dsq_set_tile_n
std::atomic<int> g_pdl{1};            // dsq_set_dependent_launch
std::atomic<int> g_forced_ks{0};      // dsq_set_round_k_steps: 0 automatic, 1 single K steps, 2 double
std::atomic<int> g_pair_mode{0};      // dsq_set_cta_pairs: 0 automatic, 1 never, 2 wherever possible
std::atomic<unsigned long long> g_wait_ns{WAIT_LIMIT_NS};   // dsq_set_wait_limit_ns
std::atomic<int> g_skip_b_round{-1};  // dsq_set_test_skip_b_round
std::atomic<int> g_window3{1};        // dsq_set_conv3_window
std::atomic<int> g_two_pass{1};       // dsq_set_gemm_two_pass
std::atomic<int> g_w8{1};             // dsq_set_conv3_expanded_weights

int pick_bn(int m_tiles, int ncols, int bits)
{
    const int forced = g_forced_bn.load();
    if (forced) return (bits == 2 && forced < 64) ? 64 : forced;
    const int sms = dsq_sm_count() > 0 ? dsq_sm_count() : 148;
    const int cands[5] = {256, 192, 128, 64, 32};
    int best = 0;
    double best_cost = 1e30;
    for (int i = 0; i < 5; ++i) {
        const int bn = cands[i];
        if (bits == 2 && bn < 64) continue;
        const int n_tiles = (ncols + bn - 1) / bn;
        const int64_t tiles = (int64_t)m_tiles * n_tiles;
        const int64_t waves = (tiles + sms - 1) / sms;
        const double cost = (double)waves * (100.0 + bn);
        if (cost < best_cost) { best_cost = cost; best = bn; }
    }
    return best;
}

template <int BITS, bool A_SIGNED, int EPI, int PM, int A_TMA>
int launch_tc(const TcMaps &tmap, const TcParams &p, cudaStream_t s)
{
    if ((p.a_tma == 3 ? 3 : p.a_tma != 0) != A_TMA) return DSQ_ERR_UNSUPPORTED;
    constexpr bool PAIR = Pipe<PM>::PAIR;
    const SmemLayout L = smem_layout(PAIR ? p.BN / 2 : p.BN, BITS, p.s_p, p.b_stages,
                                     Pipe<PM>::KS,
                                     Pipe<PM>::GROUPS * Pipe<PM>::A_RING,
                                     epi_slots(p.join, p.epw));
    if (L.total > 227u * 1024u) return DSQ_ERR_UNSUPPORTED;
    int smem_bytes = (int)L.total + 1024;            // slack for the 1024-byte alignment
    if (smem_bytes > 227 * 1024) smem_bytes = 227 * 1024;
    // The opt-in to large dynamic shared memory is a per-device attribute of
    // the function: one bit per device ordinal for this instantiation.
    static std::atomic<unsigned long long> configured{0ull};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return DSQ_ERR_CUDA;
    const unsigned long long dev_bit = dev < 64 ? 1ull << dev : 0ull;
    if (!(configured.load(std::memory_order_acquire) & dev_bit)) {
        if (cudaFuncSetAttribute(dsq_tc_kernel<BITS, A_SIGNED, EPI, PM, A_TMA>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 227 * 1024) != cudaSuccess)
            return DSQ_ERR_CUDA;
        configured.fetch_or(dev_bit, std::memory_order_release);
    }
    const int sms = dsq_sm_count();
    if (sms <= 0) return DSQ_ERR_CUDA;
    int grid = p.m_tiles * p.n_tiles;
    if (grid > sms) grid = sms;
    if (p.BN * p.n_acc > Pipe<PM>::A_COL0) return DSQ_ERR_UNSUPPORTED;
    TcParams q = p;
    q.smem_bytes = smem_bytes;
    q.wait_ns = g_wait_ns.load();
    q.skip_b_round = g_skip_b_round.load();
    // one cluster of two CTAs (the two SMs of a TPC) per tile in flight
    if (PAIR && grid > sms / 2) grid = sms / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(PAIR ? 2 * grid : grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (PAIR) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 2;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (g_pdl.load()) {
        // the kernel waits for its predecessors itself (griddepcontrol.wait)
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, dsq_tc_kernel<BITS, A_SIGNED, EPI, PM, A_TMA>, tmap.b, tmap.a,
                           q) != cudaSuccess) {
        cudaGetLastError();
        return DSQ_ERR_CUDA;
    }
    return dsq_launch_status();
}

template <int BITS, int PM>
int launch_conv(int epi, const TcMaps &tmap, const TcParams &p, cudaStream_t s)
{
    if (p.a_tma) {
        switch (epi) {
        case EPI_CODES: return launch_tc<BITS, false, EPI_CODES, PM, 1>(tmap, p, s);
        case EPI_CODES_RES: return launch_tc<BITS, false, EPI_CODES_RES, PM, 1>(tmap, p, s);
        default: return launch_tc<BITS, false, EPI_GENERAL, PM, 1>(tmap, p, s);
        }
    }
    switch (epi) {
    case EPI_CODES: return launch_tc<BITS, false, EPI_CODES, PM, 0>(tmap, p, s);
    case EPI_CODES_RES: return launch_tc<BITS, false, EPI_CODES_RES, PM, 0>(tmap, p, s);
    default: return launch_tc<BITS, false, EPI_GENERAL, PM, 0>(tmap, p, s);
    }
}

template <int BITS>
int launch_bits(int epi, int pm, const TcMaps &tmap, const TcParams &p, cudaStream_t s)
{
    if (epi == EPI_GEMM) {
        // 2- and 4-bit GEMMs always fetch A with TMA
        if (pm == 4) return launch_tc<BITS, true, EPI_GEMM, 4, 1>(tmap, p, s);
        if (pm == 3) return launch_tc<BITS, true, EPI_GEMM, 3, 1>(tmap, p, s);
        if (pm == 2) return launch_tc<BITS, true, EPI_GEMM, 2, 1>(tmap, p, s);
        return launch_tc<BITS, true, EPI_GEMM, 1, 1>(tmap, p, s);
    }
    if (pm == 5 && p.a_tma == 3) {
        switch (epi) {
        case EPI_CODES: return launch_tc<BITS, false, EPI_CODES, 5, 3>(tmap, p, s);
        case EPI_CODES_RES: return launch_tc<BITS, false, EPI_CODES_RES, 5, 3>(tmap, p, s);
        default: return launch_tc<BITS, false, EPI_GENERAL, 5, 3>(tmap, p, s);
        }
    }
    if (pm == 5) {
        switch (epi) {
        case EPI_CODES: return launch_tc<BITS, false, EPI_CODES, 5, 1>(tmap, p, s);
        case EPI_CODES_RES: return launch_tc<BITS, false, EPI_CODES_RES, 5, 1>(tmap, p, s);
        default: return launch_tc<BITS, false, EPI_GENERAL, 5, 1>(tmap, p, s);
        }
    }
    if (pm == 4) return launch_conv<BITS, 4>(epi, tmap, p, s);
    if (pm == 3) return launch_conv<BITS, 3>(epi, tmap, p, s);
    if (pm == 2) return launch_conv<BITS, 2>(epi, tmap, p, s);
    return launch_conv<BITS, 1>(epi, tmap, p, s);
}

int dispatch_tc(int bits, int epi, int pm, const TcMaps &tmap, const TcParams &p,
                cudaStream_t s)
{
    if (bits == 4) return launch_bits<4>(epi, pm, tmap, p, s);
    if (bits == 2) return launch_bits<2>(epi, pm, tmap, p, s);
    if (bits == 3 && epi == EPI_GEMM) return launch_tc<3, true, EPI_GEMM, 1, 0>(tmap, p, s);
    // 3-bit convolutions: single K steps, rows gathered with cp.async, the
    // epilogue that handles fields straddling two words
    if (bits == 3) return launch_tc<3, false, EPI_GENERAL, 1, 0>(tmap, p, s);
    return DSQ_ERR_UNSUPPORTED;
}

// Pipeline mode for a problem (see Pipe<PM>).
int pick_pm(const TcParams &p, int bits, bool im2col)
{
    const int forced_ks = g_forced_ks.load();
    if (bits == 3 || p.ksteps < 2 || forced_ks == 1) return 1;
    // whole-K rounds: a small convolution whose B tile can stay resident
    if (im2col && forced_ks == 0 && p.ksteps >= 3 && p.ksteps <= Pipe<5>::KS &&
        2 * p.BN <= Pipe<5>::A_COL0) {
        TcParams q = p;
        choose_b_mode(&q, bits, 5);
        if (q.rounds == 1 && q.b_res) return 5;
    }
    // CTA pairs: 256-wide N tiles and at least two 128-row tiles to put together
    if (p.BN == 256 && p.M > BM && g_pair_mode.load() != 1) return 4;
    if (p.BN > 128) return p.ksteps >= 4 ? 3 : 1;
    // two K steps per round: a round costs about the same whatever it carries
    // (measured faster than single steps even where those would keep the
    // expanded B tile resident)
    return 2;
}

}  // namespace

// ---- shared with the other tensor-core translation unit (dsq_tc_host.h) -------
DsqLaunchHooks dsq_launch_hooks()
{
    DsqLaunchHooks h;
    h.pdl = g_pdl.load();
    h.wait_ns = g_wait_ns.load();
    h.skip_b_round = g_skip_b_round.load();
    h.window3 = g_window3.load();
    h.w8 = g_w8.load();
    return h;
}

static void *driver_entry_point(const char *name)
{
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint(name, &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    return sym;
}

DsqEncodeTiledFn dsq_encode_tiled_fn()
{
    static std::atomic<void *> fn{nullptr};
    void *f = fn.load(std::memory_order_acquire);
    if (!f) {
        f = driver_entry_point("cuTensorMapEncodeTiled");
        fn.store(f, std::memory_order_release);
    }
    return reinterpret_cast<DsqEncodeTiledFn>(f);
}

DsqEncodeIm2colFn dsq_encode_im2col_fn()
{
    static std::atomic<void *> fn{nullptr};
    void *f = fn.load(std::memory_order_acquire);
    if (!f) {
        f = driver_entry_point("cuTensorMapEncodeIm2col");
        fn.store(f, std::memory_order_release);
    }
    return reinterpret_cast<DsqEncodeIm2colFn>(f);
}

extern "C" {

int dsq_set_round_k_steps(int ks)
{
    if (ks != 0 && ks != 1 && ks != 2) return DSQ_ERR_SHAPE;
    g_forced_ks = ks;
    return DSQ_OK;
}

int dsq_set_cta_pairs(int mode)
{
    if (mode < 0 || mode > 2) return DSQ_ERR_SHAPE;
    g_pair_mode = mode;
    return DSQ_OK;
}

int dsq_set_dependent_launch(int on)
{
    if (on != 0 && on != 1) return DSQ_ERR_SHAPE;
    g_pdl = on;
    return DSQ_OK;
}

int dsq_set_test_skip_b_round(int round)
{
    g_skip_b_round = round < 0 ? -1 : round;
    return DSQ_OK;
}

int dsq_set_conv3_window(int mode)
{
    if (mode < 0 || mode > 4) return DSQ_ERR_SHAPE;
    g_window3 = mode;
    return DSQ_OK;
}

int dsq_set_wait_limit_ns(long long ns)
{
    if (ns < 0) return DSQ_ERR_SHAPE;
    g_wait_ns = ns == 0 ? WAIT_LIMIT_NS : (unsigned long long)ns;
    return DSQ_OK;
}

int dsq_set_tile_n(int bn)
{
    if (bn != 0 && bn != 32 && bn != 64 && bn != 128 && bn != 192 && bn != 256)
        return DSQ_ERR_SHAPE;
    g_forced_bn = bn;
    return DSQ_OK;
}

// Argument checks of dsq_gemm (everything that can be seen from the host).
static int gemm_check_args(const void *A_codes, const void *B_codes, int64_t M, int64_t N,
                           int64_t K, int bits, const int32_t *C_i32, const float *row_scale,
                           const float *D_f32)
{
    if (!A_codes || !B_codes) return DSQ_ERR_NULL;
    if (!C_i32 && !D_f32) return DSQ_ERR_NULL;
    if (D_f32 && !row_scale) return DSQ_ERR_NULL;
    if (bits < 2 || bits > 4) return DSQ_ERR_BITS;
    if (M <= 0 || N <= 0 || K <= 0 || M > (1 << 24) || N > (1 << 24) || K > (1 << 24))
        return DSQ_ERR_SHAPE;
    if ((double)K * 128.0 * (double)((1 << bits) - 1) > 2147483647.0) return DSQ_ERR_OVERFLOW;
    if (!dsq_aligned16(A_codes) || !dsq_aligned16(B_codes) ||
        (C_i32 && !dsq_aligned16(C_i32)) || (D_f32 && !dsq_aligned16(D_f32)))
        return DSQ_ERR_ALIGN;
    return DSQ_OK;
}

size_t dsq_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits)
{
    if (bits < 2 || bits > 4 || M <= 0 || N <= 0 || K <= 0) return DSQ_WS_BYTES;
    const int mode = g_two_pass.load();
    const size_t need = mode ? dsq_gemm8_scratch_bytes(M, N, K, mode == 2) : 0;
    return need ? DSQ_WS_BYTES + 1024 + need : DSQ_WS_BYTES;
}

int dsq_set_conv3_expanded_weights(int on)
{
    g_w8 = on ? 1 : 0;
    return DSQ_OK;
}

int dsq_set_gemm_two_pass(int on)
{
    if (on < 0 || on > 2) return DSQ_ERR_SHAPE;
    g_two_pass = on;
    return DSQ_OK;
}

int dsq_gemm(const void *A_codes, const void *B_codes, int64_t M, int64_t N, int64_t K,
             int bits, int32_t *C_i32, const float *row_scale, float *D_f32, void *workspace,
             size_t ws_bytes, void *stream)
{
    if (!workspace) return DSQ_ERR_NULL;
    int st = gemm_check_args(A_codes, B_codes, M, N, K, bits, C_i32, row_scale, D_f32);
    if (st) return st;
    if (!dsq_aligned16(workspace)) return DSQ_ERR_ALIGN;
    if (ws_bytes < DSQ_WS_BYTES) return DSQ_ERR_SIZE;

    // large problems, when the caller's workspace has room for the expanded
    // operands (dsq_gemm_workspace_bytes): expand every row once, then an
    // 8-bit GEMM fed by TMA alone
    const int two_pass = g_two_pass.load();
    const size_t scratch_need = two_pass ? dsq_gemm8_scratch_bytes(M, N, K, two_pass == 2) : 0;
    if (scratch_need) {
        const uintptr_t w0 = reinterpret_cast<uintptr_t>(workspace);
        const uintptr_t s0 = (w0 + DSQ_WS_BYTES + 1023u) & ~(uintptr_t)1023u;
        if (ws_bytes >= (s0 - w0) + scratch_need)
            return dsq_gemm8_launch(A_codes, B_codes, M, N, K, bits, C_i32, row_scale, D_f32,
                                    workspace, reinterpret_cast<void *>(s0),
                                    (cudaStream_t)stream);
    }

    const size_t pitch = dsq_row_pitch(K, bits);
    TcParams p = {};
    p.M = (int)M;
    p.Ncols = (int)N;
    p.ksteps = (int)((pitch + 16 * bits - 1) / (16 * bits));
    p.m_tiles = (int)((M + BM - 1) / BM);
    p.BN = pick_bn(p.m_tiles, (int)N, bits);
    if (bits == 2 && p.BN < 64) p.BN = 64;
    p.n_tiles = (int)((N + p.BN - 1) / p.BN);
    const int pm = pick_pm(p, bits, false);
    const int ks = pipe_info(pm).ks;
    const bool pair = pipe_info(pm).pair != 0;
    if (pair) p.m_tiles = (int)((M + 2 * BM - 1) / (2 * BM));
    choose_b_mode(&p, bits, pm);
    p.act = (const uint8_t *)A_codes;
    p.H = 1; p.W = (int)M; p.Ho = 1; p.Wo = (int)M;
    p.stride = 1; p.pad = 0; p.KW = 1; p.taps = 1; p.P = (int)pitch;
    p.Pk = p.P;
    p.a_lcr = a_run_log2(p.P, bits, ks);
    p.mode = MODE_GEMM;
    p.shift = 8 - bits;
    p.orv = 0;
    p.C_i32 = C_i32;
    p.row_scale = row_scale;
    p.D_f32 = D_f32;
    p.ws = (int *)workspace;
    TcMaps tmap;
    st = make_rows_tmap(&tmap.b, B_codes, pitch, (uint64_t)N, pitch, ks * 16 * bits,
                        pair ? p.BN / 2 : p.BN);
    if (st) return st;
    tmap.a = tmap.b;
    st = setup_a_tma(&p, &tmap.a, A_codes, M, bits, ks, true, nullptr, 1, false);
    if (st) return st;
    return dispatch_tc(bits, EPI_GEMM, pm, tmap, p, (cudaStream_t)stream);
}

int dsq_conv2d(const void *act_codes, const dsq_nhwc_t *shape, const dsq_quant_t *act_q,
               const void *w_packed, const dsq_conv_t *conv, const dsq_epilogue_t *ep,
               float *y_f32, void *y_codes, int32_t *acc_out, void *workspace,
               size_t ws_bytes, void *stream)
{
    if (!act_codes || !shape || !act_q || !w_packed || !conv || !ep || !workspace)
        return DSQ_ERR_NULL;
    int st = dsq_check_quant(act_q);
    if (st) return st;
    const int bits = act_q->bits;
    if (shape->N <= 0 || shape->H <= 0 || shape->W <= 0 || shape->C <= 0 || conv->Cout <= 0)
        return DSQ_ERR_SHAPE;
    if (conv->groups != 1 || conv->Cin != shape->C) return DSQ_ERR_SHAPE;
    if (conv->KH != conv->KW || (conv->KH != 1 && conv->KH != 3) ||
        (conv->stride != 1 && conv->stride != 2) || conv->pad < 0 || conv->pad > conv->KH / 2)
        return DSQ_ERR_UNSUPPORTED;
    if (conv->pad > 0 && act_q->lo != 0.0f) return DSQ_ERR_UNSUPPORTED;
    const int Ho = (shape->H + 2 * conv->pad - conv->KH) / conv->stride + 1;
    const int Wo = (shape->W + 2 * conv->pad - conv->KW) / conv->stride + 1;
    if (Ho <= 0 || Wo <= 0) return DSQ_ERR_SHAPE;
    const int64_t M = (int64_t)shape->N * Ho * Wo;
    if (M > (1 << 30)) return DSQ_ERR_SHAPE;
    const int taps = conv->KH * conv->KW;
    if ((double)taps * conv->Cin * 128.0 * (double)((1 << bits) - 1) > 2147483647.0)
        return DSQ_ERR_OVERFLOW;
    if (!dsq_aligned16(act_codes) || !dsq_aligned16(w_packed) || !dsq_aligned16(workspace))
        return DSQ_ERR_ALIGN;
    if (ws_bytes < DSQ_WS_BYTES) return DSQ_ERR_SIZE;
    DsqEpi e;
    st = dsq_make_epi(ep, bits, y_f32, y_codes, acc_out, &e);
    if (st) return st;

    // largest |2*acc + S_a| below 2^22: the epilogue may convert integers to
    // float through the 1.5 * 2^23 bias trick, which is exact there
    const int small_acc = (double)taps * conv->Cin * (double)((1 << bits) - 1) *
                              (2.0 * (double)(1 << (bits - 1)) + 1.0) < 4194304.0;
    const int epi = (y_f32 || acc_out || !y_codes || e.general_offset)
                        ? EPI_GENERAL
                        : (e.residual ? EPI_CODES_RES : EPI_CODES);
    // 3x3 stride-1 convolutions: every input pixel expanded once (dsq_conv3.cu)
    st = dsq_conv3_window(act_codes, shape, bits, w_packed, conv, e, epi, small_acc, workspace,
                          (cudaStream_t)stream);
    if (st != DSQ_ERR_UNSUPPORTED) return st;

    const size_t P = dsq_row_pitch(conv->Cin, bits);
    const size_t row_bytes = (size_t)taps * P;
    TcParams p = {};
    p.M = (int)M;
    p.Ncols = conv->Cout;
    p.ksteps = (int)((row_bytes + 16 * bits - 1) / (16 * bits));
    p.Pk = (int)P;
    if (bits == 3) {
        // every tap starts a K step of its own (see TcParams::Pk)
        p.spt = (int)((P + 47) / 48);
        p.Pk = p.spt * 48;
        p.ksteps = taps * p.spt;
    }
    p.m_tiles = (int)((M + BM - 1) / BM);
    p.BN = pick_bn(p.m_tiles, conv->Cout, bits);
    p.n_tiles = (conv->Cout + p.BN - 1) / p.BN;
    const bool plain_rows = conv->KH == 1 && conv->stride == 1 && conv->pad == 0;
    const int pm = pick_pm(p, bits, !plain_rows);
    const int ks = pipe_info(pm).ks;
    if (pm == 4) p.m_tiles = (int)((M + 2 * BM - 1) / (2 * BM));
    choose_b_mode(&p, bits, pm);
    p.act = (const uint8_t *)act_codes;
    p.H = shape->H; p.W = shape->W; p.Ho = Ho; p.Wo = Wo;
    p.stride = conv->stride; p.pad = conv->pad; p.KW = conv->KW; p.taps = taps; p.P = (int)P;
    p.a_lcr = a_run_log2(p.P, bits, ks);
    p.mode = MODE_CONV;
    p.e = e;
    p.out_pitch = (int)dsq_row_pitch(conv->Cout, bits);
    if (e.half_offset) {
        p.shift = 7 - bits;
        p.orv = 0x01010101u << (7 - bits);
    } else {
        p.shift = 8 - bits;
        p.orv = 0;
    }
    p.ws = (int *)workspace;
    TcMaps tmap;
    // (whole-K rounds fetch B one K step per box)
    st = make_rows_tmap(&tmap.b, w_packed, row_bytes, (uint64_t)conv->Cout, row_bytes,
                        (pm == 5 ? 1 : ks) * 16 * bits, pm == 4 ? p.BN / 2 : p.BN);
    if (st) return st;
    tmap.a = tmap.b;
    // a 1x1 stride-1 unpadded convolution reads the pixel rows as they lie
    st = setup_a_tma(&p, &tmap.a, act_codes, M, bits, ks, plain_rows, shape, conv->KH, pm == 5);
    if (st) return st;
    p.small_acc = small_acc;
    int epi_im2col = epi;
    if (epi != EPI_GENERAL) {
        // the codes epilogue clips after the requantiser's multiply: it needs
        // floor(fma(hi - lo, inv, 0.5)) = qmax (true for every sane range)
        p.r_hi = fmaf(e.rq.hi - e.rq.lo, e.rq.inv, 0.5f);
        if ((int)floorf(p.r_hi) != e.rq.qmax) epi_im2col = EPI_GENERAL;
    }
    return dispatch_tc(bits, epi_im2col, pm, tmap, p, (cudaStream_t)stream);
}

int dsq_probe_i8_mma_rate(int iters, float *ms_out, double *macs_out, void *workspace,
                          size_t ws_bytes, void *stream)
{
    if (!ms_out || !macs_out || !workspace) return DSQ_ERR_NULL;
    if (iters <= 0 || iters > (1 << 24)) return DSQ_ERR_SHAPE;
    if (ws_bytes < DSQ_WS_BYTES) return DSQ_ERR_SIZE;
    cudaStream_t s = (cudaStream_t)stream;
    const int smem_bytes = (128 + 256) * 128 + 1024;
    DSQ_CUDA_TRY(cudaFuncSetAttribute(mma_rate_kernel,
                                      cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
    int dev = 0, sms = 0;
    DSQ_CUDA_TRY(cudaGetDevice(&dev));
    DSQ_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    cudaEvent_t e0, e1;
    DSQ_CUDA_TRY(cudaEventCreate(&e0));
    DSQ_CUDA_TRY(cudaEventCreate(&e1));
    mma_rate_kernel<<<sms, 128, smem_bytes, s>>>(iters < 64 ? iters : 64, (int *)workspace);
    DSQ_CUDA_TRY(cudaEventRecord(e0, s));
    mma_rate_kernel<<<sms, 128, smem_bytes, s>>>(iters, (int *)workspace);
    DSQ_CUDA_TRY(cudaEventRecord(e1, s));
    DSQ_CUDA_TRY(cudaEventSynchronize(e1));
    DSQ_CUDA_TRY(cudaEventElapsedTime(ms_out, e0, e1));
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *macs_out = (double)sms * (double)iters * 128.0 * 256.0 * 32.0;
    return dsq_launch_status();
}

int dsq_gemm_static_ws(const void *A_codes, const void *B_codes, int64_t M, int64_t N,
                       int64_t K, int bits, int32_t *C_i32, const float *row_scale,
                       float *D_f32, int wait_and_check, void *stream)
{
    static_assert(DSQ_STATIC_WS_BYTES >= DSQ_WS_BYTES, "static workspace too small");
    // everything that can fail on the host fails here, before the symbol
    // lookup and before anything is enqueued on the caller's stream
    const int bad = gemm_check_args(A_codes, B_codes, M, N, K, bits, C_i32, row_scale, D_f32);
    if (bad) return bad;
    if (M > DSQ_STATIC_WS_MAX_DIM || N > DSQ_STATIC_WS_MAX_DIM || K > DSQ_STATIC_WS_MAX_DIM)
        return DSQ_ERR_SIZE;
    // In host code `g_static_ws` is only a handle for the symbol, not a device
    // address.  The address on the current device is looked up once per device
    // (no allocation happens: the array is part of the loaded module).
    static std::atomic<void *> dev_ptr[DSQ_MAX_DEVICES];
    int dev = -1;
    DSQ_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= DSQ_MAX_DEVICES) return DSQ_ERR_UNSUPPORTED;
    void *ws = dev_ptr[dev].load(std::memory_order_acquire);
    if (!ws) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_ws) != cudaSuccess || !ptr) return DSQ_ERR_CUDA;
        dev_ptr[dev].store(ptr, std::memory_order_release);
        ws = ptr;
    }
    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps what the previous call left: the status words start at 0
    DSQ_CUDA_TRY(cudaMemsetAsync(ws, 0, DSQ_STATIC_WS_BYTES, s));
    const int st = dsq_gemm(A_codes, B_codes, M, N, K, bits, C_i32, row_scale, D_f32, ws,
                            DSQ_STATIC_WS_BYTES, stream);
    if (st != DSQ_OK || !wait_and_check) return st;
    int host[2] = {0, 0};
    DSQ_CUDA_TRY(cudaMemcpyAsync(host, ws, sizeof(host), cudaMemcpyDeviceToHost, s));
    DSQ_CUDA_TRY(cudaStreamSynchronize(s));
    return host[DSQ_WS_STATUS];
}

}  // extern "C"
