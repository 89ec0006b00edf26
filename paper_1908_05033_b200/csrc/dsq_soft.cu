// Training-side elementwise kernels of DSQ: the soft quantiser Q_S (Eq. 3-8)
// and its back-propagation (Eq. 10-13, Algorithm 1).  HBM-bound streaming
// kernels: 8 bytes per element forward (fp32 in, fp32 out), 12 bytes per
// element backward (x and dL/dy in, dL/dx out) plus three scalar reductions.
#include "dsq_common.cuh"

namespace {

// Everything that depends on (b, l, u, alpha) only, formed on the host in
// binary64 and rounded once to binary32.
struct SoftP {
    float lo, hi, delta, inv_delta, k, s;
    float half_ds;        // Delta/2 * s
    float half_dsk;       // Delta/2 * s * k
    float ds_da;          // ds/dalpha = 1/(1-alpha)^2
    float dk_da;          // dk/dalpha = -2/(Delta alpha (2-alpha))
    float dd_dl, dd_du;   // -1/(2^b-1), +1/(2^b-1)
    float k_over_delta;
    int imax;             // 2^b - 2
};

__device__ __forceinline__ float4 ld_stream(const float4 *p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::256B.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

// interval index i, tanh(k (x - m_i)) and x - m_i of a value inside [l, u]
__device__ __forceinline__ void soft_core(float x, const SoftP &p, float &fi, float &t, float &xm)
{
    const float xc = fminf(fmaxf(x, p.lo), p.hi);
    fi = fminf(fmaxf(floorf((xc - p.lo) * p.inv_delta), 0.0f), (float)p.imax);
    const float m = fmaf(fi + 0.5f, p.delta, p.lo);
    xm = xc - m;
    t = tanhf(p.k * xm);
}

__device__ __forceinline__ float soft_fwd_one(float x, const SoftP &p)
{
    float fi, t, xm;
    soft_core(x, p, fi, t, xm);
    // l + Delta (i + (phi + 1)/2) = l + Delta i + Delta/2 + (Delta/2) s tanh
    float y = fmaf(p.half_ds, t, fmaf(fi + 0.5f, p.delta, p.lo));
    y = x < p.lo ? p.lo : y;
    y = x > p.hi ? p.hi : y;
    return x != x ? x : y;        // NaN stays NaN
}

__global__ void __launch_bounds__(256) soft_fwd_kernel(const float *__restrict__ x,
                                                       float *__restrict__ y, int64_t n, SoftP p)
{
    const int64_t n4 = n >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = tid; i < n4; i += stride) {
        const float4 v = ld_stream(reinterpret_cast<const float4 *>(x) + i);
        float4 o;
        o.x = soft_fwd_one(v.x, p); o.y = soft_fwd_one(v.y, p);
        o.z = soft_fwd_one(v.z, p); o.w = soft_fwd_one(v.w, p);
        __stcs(reinterpret_cast<float4 *>(y) + i, o);
    }
    for (int64_t i = 4 * n4 + tid; i < n; i += stride) y[i] = soft_fwd_one(x[i], p);
}

// tanh(z) and sech^2(z) from one exponential and one reciprocal (the special
// function unit's ex2 and rcp, each good to about 2^-22 relative):
//   e = exp(2 z), r = 1/(e + 1):  tanh = 1 - 2 r,  sech^2 = 4 e r^2
// sech^2 has no cancellation (relative error ~1e-6); tanh is good to ~1e-6
// absolute, and it only enters sums next to terms of order one.  z -> +inf:
// e = inf, r = 0, tanh = 1 and sech^2 is forced to 0; z -> -inf: e = 0.
__device__ __forceinline__ void tanh_sech2(float z, float &t, float &sech2)
{
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(z * 2.885390081777927f));   // 2 log2(e)
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(e + 1.0f));
    t = fmaf(-2.0f, r, 1.0f);
    sech2 = r == 0.0f ? 0.0f : 4.0f * e * r * r;
}

// one element of the backward pass: returns dL/dx, adds this element's terms
// of dL/dalpha, dL/dl, dL/du (times g) to the accumulators (binary32 partial
// sums of a few elements; the caller folds them into binary64)
__device__ __forceinline__ float soft_bwd_one(float x, float g, const SoftP &p, float &aa,
                                              float &al, float &au)
{
    if (x != x) return x;
    if (x < p.lo) { al += g; return 0.0f; }
    if (x > p.hi) { au += g; return 0.0f; }
    const float xc = x;
    const float fi = fminf(fmaxf(floorf((xc - p.lo) * p.inv_delta), 0.0f), (float)p.imax);
    const float xm = xc - fmaf(fi + 0.5f, p.delta, p.lo);
    float t, sech2;
    tanh_sech2(p.k * xm, t, sech2);
    const float q = fi + fmaf(0.5f * p.s, t, 0.5f);                  // Eq. 13
    // Eq. 10: (Delta/2) (ds/da tanh + s sech^2 (x - m) dk/da)
    const float da = 0.5f * p.delta * fmaf(p.ds_da, t, p.s * sech2 * xm * p.dk_da);
    // Eq. 11, 12: dphi/dp = s sech^2 (dk/dp (x - m) - k dm/dp), dk/dp = -(k/Delta) dDelta/dp
    const float ssech = p.s * sech2;
    const float dm_dl = fmaf(fi + 0.5f, p.dd_dl, 1.0f), dm_du = (fi + 0.5f) * p.dd_du;
    const float dphi_dl = ssech * (-p.k_over_delta * p.dd_dl * xm - p.k * dm_dl);
    const float dphi_du = ssech * (-p.k_over_delta * p.dd_du * xm - p.k * dm_du);
    const float dl = 1.0f + fmaf(q, p.dd_dl, 0.5f * p.delta * dphi_dl);
    const float du = fmaf(q, p.dd_du, 0.5f * p.delta * dphi_du);
    aa = fmaf(g, da, aa);
    al = fmaf(g, dl, al);
    au = fmaf(g, du, au);
    return g * p.half_dsk * sech2;
}

__global__ void __launch_bounds__(256) soft_bwd_kernel(const float *__restrict__ x,
                                                       const float *__restrict__ gy,
                                                       float *__restrict__ gx, int64_t n, SoftP p,
                                                       double *__restrict__ sums)
{
    double aa = 0.0, al = 0.0, au = 0.0;
    const int64_t n4 = n >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (int64_t i = tid; i < n4; i += stride) {
        const float4 v = ld_stream(reinterpret_cast<const float4 *>(x) + i);
        const float4 g = ld_stream(reinterpret_cast<const float4 *>(gy) + i);
        float4 o;
        float fa = 0.0f, fl = 0.0f, fu = 0.0f;          // this vector's four terms
        o.x = soft_bwd_one(v.x, g.x, p, fa, fl, fu);
        o.y = soft_bwd_one(v.y, g.y, p, fa, fl, fu);
        o.z = soft_bwd_one(v.z, g.z, p, fa, fl, fu);
        o.w = soft_bwd_one(v.w, g.w, p, fa, fl, fu);
        aa += (double)fa; al += (double)fl; au += (double)fu;
        __stcs(reinterpret_cast<float4 *>(gx) + i, o);
    }
    for (int64_t i = 4 * n4 + tid; i < n; i += stride) {
        float fa = 0.0f, fl = 0.0f, fu = 0.0f;
        gx[i] = soft_bwd_one(x[i], gy[i], p, fa, fl, fu);
        aa += (double)fa; al += (double)fl; au += (double)fu;
    }
    // the three sums: warp shuffles, one shared-memory pass per block, one
    // double-precision atomic add per block and sum
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        aa += __shfl_xor_sync(0xffffffffu, aa, o);
        al += __shfl_xor_sync(0xffffffffu, al, o);
        au += __shfl_xor_sync(0xffffffffu, au, o);
    }
    __shared__ double part[3][8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { part[0][warp] = aa; part[1][warp] = al; part[2][warp] = au; }
    __syncthreads();
    if (threadIdx.x < 3) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += part[threadIdx.x][w];
        atomicAdd(sums + threadIdx.x, s);
    }
}

int make_soft_params(const dsq_quant_t *q, float alpha, SoftP *out)
{
    if (!q) return DSQ_ERR_NULL;
    if (q->bits < 1 || q->bits > 8) return DSQ_ERR_BITS;
    if (!dsq_finite(q->lo) || !dsq_finite(q->hi) || !(q->hi > q->lo)) return DSQ_ERR_RANGE;
    if (!(alpha > 0.0f && alpha < 1.0f)) return DSQ_ERR_RANGE;
    const double lo = q->lo, hi = q->hi, a = alpha;
    const double n = (double)((1 << q->bits) - 1);
    const double delta = (hi - lo) / n;
    const double k = log(2.0 / a - 1.0) / delta;          // Eq. 8
    const double s = 1.0 / (1.0 - a);                     // Eq. 7
    SoftP p;
    p.lo = q->lo; p.hi = q->hi;
    p.delta = (float)delta; p.inv_delta = (float)(1.0 / delta);
    p.k = (float)k; p.s = (float)s;
    p.half_ds = (float)(0.5 * delta * s);
    p.half_dsk = (float)(0.5 * delta * s * k);
    p.ds_da = (float)(1.0 / ((1.0 - a) * (1.0 - a)));
    p.dk_da = (float)(-2.0 / (delta * a * (2.0 - a)));
    p.dd_dl = (float)(-1.0 / n); p.dd_du = (float)(1.0 / n);
    p.k_over_delta = (float)(k / delta);
    p.imax = (1 << q->bits) - 2;
    *out = p;
    return DSQ_OK;
}

int soft_grid(int64_t n)
{
    const int sms = dsq_sm_count() > 0 ? dsq_sm_count() : 148;
    int64_t g = (n / 4 + 255) / 256;
    if (g > (int64_t)sms * 16) g = (int64_t)sms * 16;
    return g < 1 ? 1 : (int)g;
}

}  // namespace

extern "C" int dsq_soft_quantize_fwd(const float *x, int64_t n, const dsq_quant_t *q, float alpha,
                                     float *y, void *stream)
{
    if (!x || !y) return DSQ_ERR_NULL;
    SoftP p;
    const int st = make_soft_params(q, alpha, &p);
    if (st) return st;
    if (n <= 0) return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(x) || !dsq_aligned16(y)) return DSQ_ERR_ALIGN;
    soft_fwd_kernel<<<soft_grid(n), 256, 0, (cudaStream_t)stream>>>(x, y, n, p);
    return dsq_launch_status();
}

extern "C" int dsq_soft_quantize_bwd(const float *x, const float *grad_y, int64_t n,
                                     const dsq_quant_t *q, float alpha, float *grad_x,
                                     double *grad_params, void *stream)
{
    if (!x || !grad_y || !grad_x || !grad_params) return DSQ_ERR_NULL;
    SoftP p;
    const int st = make_soft_params(q, alpha, &p);
    if (st) return st;
    if (n <= 0) return DSQ_ERR_SHAPE;
    if (!dsq_aligned16(x) || !dsq_aligned16(grad_y) || !dsq_aligned16(grad_x) ||
        (reinterpret_cast<uintptr_t>(grad_params) & 7u))
        return DSQ_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    DSQ_CUDA_TRY(cudaMemsetAsync(grad_params, 0, 3 * sizeof(double), s));
    soft_bwd_kernel<<<soft_grid(n), 256, 0, s>>>(x, grad_y, grad_x, n, p, grad_params);
    return dsq_launch_status();
}
