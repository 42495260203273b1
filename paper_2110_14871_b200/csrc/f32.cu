// fp32 kernels (NCHW or NHWC through explicit strides).  Plain FFMA on both stages:
// the tensor cores have no full-fp32 mode and TF32 would miss the 1e-4 parity bound.
#include "gdws_internal.h"

namespace gdws {

struct F32Shape {
    int N, C, H, W, D, G, k, stride, pad, Ho, Wo, relu;
    // element strides of x (xn, xc, xh, xw), of z / y (channel count G / D) in the same layout
    long long xn, xc, xh, xw;
    long long zn, zc, zh, zw;
    long long yn, yc, yh, yw;
};

static F32Shape make_shape(const gdws_plan_s *p, gdws_layout_t layout, int N, int H, int W)
{
    F32Shape s;
    s.N = N; s.C = p->C; s.H = H; s.W = W; s.D = p->D; s.G = p->G; s.k = p->k; s.stride = p->stride; s.pad = p->pad;
    s.Ho = gdws_out_dim(H, p->k, p->stride, p->pad);
    s.Wo = gdws_out_dim(W, p->k, p->stride, p->pad);
    s.relu = p->opt_relu;
    if (layout == GDWS_NCHW) {
        s.xw = 1; s.xh = W; s.xc = (long long)H * W; s.xn = s.xc * s.C;
        s.zw = 1; s.zh = s.Wo; s.zc = (long long)s.Ho * s.Wo; s.zn = s.zc * s.G;
        s.yw = 1; s.yh = s.Wo; s.yc = (long long)s.Ho * s.Wo; s.yn = s.yc * s.D;
    } else {
        s.xc = 1; s.xw = s.C; s.xh = (long long)W * s.C; s.xn = s.xh * H;
        s.zc = 1; s.zw = s.G; s.zh = (long long)s.Wo * s.G; s.zn = s.zh * s.Ho;
        s.yc = 1; s.yw = s.D; s.yh = (long long)s.Wo * s.D; s.yn = s.yh * s.Ho;
    }
    return s;
}

// One depthwise output: sum over the k x k window of channel c at output (ho, wo), zero padding.
__device__ __forceinline__ float dw_point(const F32Shape &s, const float *__restrict__ xc,
                                          const float *__restrict__ ker, int ho, int wo)
{
    float acc = 0.f;
    for (int u = 0; u < s.k; ++u) {
        const int hi = ho * s.stride + u - s.pad;
        if (hi < 0 || hi >= s.H) continue;
        for (int v = 0; v < s.k; ++v) {
            const int wi = wo * s.stride + v - s.pad;
            if (wi < 0 || wi >= s.W) continue;
            acc = fmaf(__ldg(ker + u * s.k + v), __ldg(xc + hi * s.xh + wi * s.xw), acc);
        }
    }
    return acc;
}

// z[n,i,ho,wo]: one thread per element; threads run along wo (NCHW) so reads of x coalesce.
__global__ void gdw_f32_kernel(F32Shape s, const float *__restrict__ x, const float *__restrict__ dw,
                               const int32_t *__restrict__ chan, float *__restrict__ z)
{
    const long long total = (long long)s.N * s.G * s.Ho * s.Wo;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const int wo = (int)(t % s.Wo);
        long long r = t / s.Wo;
        const int ho = (int)(r % s.Ho);
        r /= s.Ho;
        const int i = (int)(r % s.G);
        const int n = (int)(r / s.G);
        const int c = chan[i];
        const float v = dw_point(s, x + n * s.xn + c * s.xc, dw + (size_t)i * s.k * s.k, ho, wo);
        z[n * s.zn + i * s.zc + ho * s.zh + wo * s.zw] = v;
    }
}

// y[n,d,ho,wo] = bias[d] + sum_i P[d,i] z[n,i,ho,wo]: one thread per element.
__global__ void pw_f32_kernel(F32Shape s, const float *__restrict__ z, const float *__restrict__ pw,
                              const float *__restrict__ bias, float *__restrict__ y)
{
    const long long total = (long long)s.N * s.D * s.Ho * s.Wo;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const int wo = (int)(t % s.Wo);
        long long r = t / s.Wo;
        const int ho = (int)(r % s.Ho);
        r /= s.Ho;
        const int d = (int)(r % s.D);
        const int n = (int)(r / s.D);
        const float *zp = z + n * s.zn + ho * s.zh + wo * s.zw;
        const float *pp = pw + (size_t)d * s.G;
        float acc = 0.f;
        for (int i = 0; i < s.G; ++i) acc = fmaf(__ldg(pp + i), __ldg(zp + i * s.zc), acc);
        acc += bias ? __ldg(bias + d) : 0.f;
        if (s.relu) acc = fmaxf(acc, 0.f);
        y[n * s.yn + d * s.yc + ho * s.yh + wo * s.yw] = acc;
    }
}

// Fused fp32 forward.  A block owns 32 consecutive output pixels.  The intermediate channels
// are produced 128 at a time into shared memory (z never reaches global memory) and consumed
// by 8 warps that each hold 16 output channels of the 32 pixels in registers.  Layers with
// more than 128 output channels repeat the depthwise work once per group of 128.
constexpr int kF32Pix = 32, kF32GC = 128, kF32DPerWarp = 16, kF32Threads = 256;

__global__ void __launch_bounds__(kF32Threads)
fused_f32_kernel(F32Shape s, const float *__restrict__ x, const float *__restrict__ dw,
                 const float *__restrict__ pw, const float *__restrict__ bias,
                 const int32_t *__restrict__ chan, float *__restrict__ y)
{
    __shared__ float zs[kF32GC][kF32Pix];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long npix = (long long)s.N * s.Ho * s.Wo;
    const long long p = (long long)blockIdx.x * kF32Pix + lane;
    const bool live = p < npix;
    int n = 0, ho = 0, wo = 0;
    if (live) {
        wo = (int)(p % s.Wo);
        const long long r = p / s.Wo;
        ho = (int)(r % s.Ho);
        n = (int)(r / s.Ho);
    }
    for (int d0 = 0; d0 < s.D; d0 += 8 * kF32DPerWarp) {
        float acc[kF32DPerWarp];
#pragma unroll
        for (int j = 0; j < kF32DPerWarp; ++j) acc[j] = 0.f;
        const int dbase = d0 + warp * kF32DPerWarp;
        for (int i0 = 0; i0 < s.G; i0 += kF32GC) {
            const int ni = min(kF32GC, s.G - i0);
            __syncthreads();
            for (int ic = warp; ic < ni; ic += kF32Threads / 32) {
                const int i = i0 + ic;
                float v = 0.f;
                if (live) v = dw_point(s, x + n * s.xn + chan[i] * s.xc, dw + (size_t)i * s.k * s.k, ho, wo);
                zs[ic][lane] = v;
            }
            __syncthreads();
            if (dbase < s.D) {
                for (int ic = 0; ic < ni; ++ic) {
                    const float zv = zs[ic][lane];
#pragma unroll
                    for (int j = 0; j < kF32DPerWarp; ++j) {
                        const int d = min(dbase + j, s.D - 1);
                        acc[j] = fmaf(__ldg(pw + (size_t)d * s.G + i0 + ic), zv, acc[j]);
                    }
                }
            }
        }
        if (live) {
#pragma unroll
            for (int j = 0; j < kF32DPerWarp; ++j) {
                const int d = dbase + j;
                if (d < s.D) {
                    float v = acc[j] + (bias ? __ldg(bias + d) : 0.f);
                    if (s.relu) v = fmaxf(v, 0.f);
                    y[n * s.yn + d * s.yc + ho * s.yh + wo * s.yw] = v;
                }
            }
        }
    }
}

static int grid_for(const gdws_plan_s *p, long long total, int block)
{
    long long b = (total + block - 1) / block;
    const long long cap = (long long)sm_count_of(p) * 16;
    return (int)(b < 1 ? 1 : (b > cap ? cap : b));
}

gdws_status_t f32_depthwise(gdws_plan_s *p, const gdws_tensor_t *x, const float *dw_w, float *z, cudaStream_t st)
{
    const F32Shape s = make_shape(p, x->layout, x->n, x->h, x->w);
    const long long total = (long long)s.N * s.G * s.Ho * s.Wo;
    gdw_f32_kernel<<<grid_for(p, total, 256), 256, 0, st>>>(s, (const float *)x->ptr, dw_w, p->d_chan, z);
    p->launches++;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "gdw_f32_kernel launch");
}

gdws_status_t f32_pointwise(gdws_plan_s *p, const float *z, const float *pw_w, const float *bias,
                            gdws_tensor_t *y, cudaStream_t st)
{
    F32Shape s = make_shape(p, y->layout, y->n, 1, 1);
    s.Ho = y->h; s.Wo = y->w;
    // strides of z and y depend only on the output extents
    if (y->layout == GDWS_NCHW) {
        s.zw = 1; s.zh = s.Wo; s.zc = (long long)s.Ho * s.Wo; s.zn = s.zc * s.G;
        s.yw = 1; s.yh = s.Wo; s.yc = (long long)s.Ho * s.Wo; s.yn = s.yc * s.D;
    } else {
        s.zc = 1; s.zw = s.G; s.zh = (long long)s.Wo * s.G; s.zn = s.zh * s.Ho;
        s.yc = 1; s.yw = s.D; s.yh = (long long)s.Wo * s.D; s.yn = s.yh * s.Ho;
    }
    const long long total = (long long)s.N * s.D * s.Ho * s.Wo;
    pw_f32_kernel<<<grid_for(p, total, 256), 256, 0, st>>>(s, z, pw_w, bias, (float *)y->ptr);
    p->launches++;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "pw_f32_kernel launch");
}

gdws_status_t f32_fused(gdws_plan_s *p, const gdws_tensor_t *x, const float *dw_w, const float *pw_w,
                        const float *bias, gdws_tensor_t *y, cudaStream_t st)
{
    const F32Shape s = make_shape(p, x->layout, x->n, x->h, x->w);
    const long long npix = (long long)s.N * s.Ho * s.Wo;
    const long long blocks = (npix + kF32Pix - 1) / kF32Pix;
    if (blocks > 0x7fffffffLL) return fail(GDWS_ERR_UNSUPPORTED, "too many pixels for the fp32 fused kernel");
    fused_f32_kernel<<<(int)blocks, kF32Threads, 0, st>>>(s, (const float *)x->ptr, dw_w, pw_w, bias, p->d_chan,
                                                         (float *)y->ptr);
    p->launches++;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "fused_f32_kernel launch");
}

}  // namespace gdws
