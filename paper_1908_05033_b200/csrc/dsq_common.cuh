// Shared host/device helpers of the DSQ B200 library: status codes, argument
// checks, the pinned quantiser sequence, workspace layout.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/dsq.h"

#define DSQ_VERSION 100

// Workspace layout (device memory owned by the caller).
//   word 0 : status (0 = ok, else a dsq_status code written by a kernel)
//   word 1 : detail of the first failure (which wait ran out)
#define DSQ_WS_BYTES 256
#define DSQ_WS_STATUS 0
#define DSQ_WS_DETAIL 1

#define DSQ_CUDA_TRY(expr)                          \
    do {                                            \
        cudaError_t e__ = (expr);                   \
        if (e__ != cudaSuccess) return DSQ_ERR_CUDA; \
    } while (0)

static inline bool dsq_aligned16(const void *p)
{
    return (reinterpret_cast<uintptr_t>(p) & 15u) == 0;
}

static inline bool dsq_finite(float v) { return v == v && v - v == 0.0f; }

static inline int dsq_check_quant(const dsq_quant_t *q)
{
    if (!q) return DSQ_ERR_NULL;
    if (q->bits < 2 || q->bits > 4) return DSQ_ERR_BITS;
    if (!dsq_finite(q->lo) || !dsq_finite(q->hi) || !(q->hi > q->lo))
        return DSQ_ERR_RANGE;
    return DSQ_OK;
}

// Number of SMs of the current device (looked up once per device; 0 if the
// runtime cannot tell).  Grids are sized from it.
#define DSQ_MAX_DEVICES 64
inline int dsq_sm_count()
{
    static std::atomic<int> cached[DSQ_MAX_DEVICES];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return 0;
    if (dev < DSQ_MAX_DEVICES) {
        const int c = cached[dev].load(std::memory_order_relaxed);
        if (c > 0) return c;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (dev < DSQ_MAX_DEVICES) cached[dev].store(sms, std::memory_order_relaxed);
    return sms;
}

static inline int dsq_launch_status()
{
    return cudaGetLastError() == cudaSuccess ? DSQ_OK : DSQ_ERR_CUDA;
}

// Quantiser parameters as the kernels take them.  inv is formed on the host
// in binary32: (float)(2^b - 1) / (hi - lo).
struct DsqQ {
    float lo, hi, inv;
    int qmax;
};

static inline DsqQ dsq_make_q(const dsq_quant_t &q)
{
    DsqQ r;
    r.lo = q.lo;
    r.hi = q.hi;
    r.qmax = (1 << q.bits) - 1;
    r.inv = (float)r.qmax / (q.hi - q.lo);
    return r;
}

#ifdef __CUDACC__
// Hard quantiser (Eq. 2 with Algorithm 1's clip and offset, midpoint up).
// Returns the unsigned code.  Every operation is a single round-to-nearest
// binary32 operation; the intrinsics keep the compiler from contracting
// the subtraction into the fused multiply-add.
__device__ __forceinline__ uint32_t dsq_code(float x, const DsqQ &q)
{
    const float xc = fminf(fmaxf(x, q.lo), q.hi);
    const float r = __fmaf_rn(__fsub_rn(xc, q.lo), q.inv, 0.5f);
    return (uint32_t)min(__float2int_rd(r), q.qmax);
}
#endif
