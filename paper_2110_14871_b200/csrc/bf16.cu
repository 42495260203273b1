// bf16 NHWC kernels for sm_100a: weight packing, the unfused GDW kernel and the pointwise
// 1x1 convolution as a tcgen05/TMEM GEMM.
#include "sm100.cuh"

namespace gdws {

// ------------------------------------------------------------------------------------------
// Weight packing
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float load_weight(const void *w, size_t idx, int is_bf16)
{
    return is_bf16 ? bf16_bits_to_float(((const uint16_t *)w)[idx]) : ((const float *)w)[idx];
}

// pw_w[D][G] -> one operand image per 64-wide K chunk: rows d (zero rows up to Dpad), 64 bf16
// of K per 128-byte row, 128-byte swizzle; columns beyond G are zero.
__global__ void pack_pw_kernel(const void *__restrict__ pw, int is_bf16, int D, int Dpad, int G, int nchunks,
                               uint16_t *__restrict__ img)
{
    const long long total = (long long)nchunks * Dpad * kChunk;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const int kk = (int)(t % kChunk);
        const long long r = t / kChunk;
        const int d = (int)(r % Dpad);
        const int q = (int)(r / Dpad);
        const int i = q * kChunk + kk;
        float v = 0.f;
        if (d < D && i < G) v = load_weight(pw, (size_t)d * G + i, is_bf16);
        const uint32_t off = (uint32_t)(d >> 3) * 1024u + (uint32_t)(d & 7) * 128u +
                             (uint32_t)(((kk >> 3) ^ (d & 7)) << 4) + (uint32_t)(kk & 7) * 2u;
        img[(size_t)q * Dpad * kChunk + (off >> 1)] = float_to_bf16_bits(v);
    }
}

// dw_w[G][k][k] -> (1) fp32 taps [Gpad][k*k] (zero rows for the padding) for the unfused kernel,
// (2) [Gpad][wstride] words for the fused kernel: the taps, then the index of the channel inside the
// input box staged for its K chunk (chan[i] - first channel of that box).
__global__ void pack_dw_kernel(const void *__restrict__ dw, int is_bf16, int G, int Gpad, int k2, int wstride,
                               const int32_t *__restrict__ chan, const int32_t *__restrict__ chunk_meta,
                               float *__restrict__ out, uint32_t *__restrict__ outp)
{
    const int total = Gpad * wstride;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
        const int i = t / wstride, j = t - i * wstride;
        uint32_t word = 0;
        if (j < k2) {
            float v = 0.f;
            if (i < G) v = load_weight(dw, (size_t)i * k2 + j, is_bf16);
            v = bf16_bits_to_float(float_to_bf16_bits(v));
            out[(size_t)i * k2 + j] = v;
            word = __float_as_uint(v);
        } else if (j == k2 && i < G) {
            word = (uint32_t)(chan[i] - chunk_meta[4 * (i / kChunk) + 2]);
        }
        outp[t] = word;
    }
}

__global__ void pack_bias_kernel(const float *__restrict__ bias, int D, int Dpad, float *__restrict__ out)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t < Dpad) out[t] = (bias && t < D) ? bias[t] : 0.f;
}

gdws_status_t bf16_pack(gdws_plan_s *p, const void *dw_w, const void *pw_w, const float *bias, gdws_dtype_t dtype,
                        cudaStream_t st)
{
    const int is_bf16 = dtype == GDWS_BF16;
    const int k2 = p->k * p->k;
    const long long tot_pw = (long long)p->nchunks * p->Dpad * kChunk;
    int blocks = (int)((tot_pw + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    pack_pw_kernel<<<blocks, 256, 0, st>>>(pw_w, is_bf16, p->D, p->Dpad, p->G, p->nchunks, p->d_pw_img);
    int blocks2 = (p->Gpad * p->wstride + 255) / 256;
    pack_dw_kernel<<<blocks2, 256, 0, st>>>(dw_w, is_bf16, p->G, p->Gpad, k2, p->wstride, p->d_chan, p->d_chunk_meta,
                                            p->d_dw, p->d_dwpack);
    pack_bias_kernel<<<(p->Dpad + 255) / 256, 256, 0, st>>>(bias, p->D, p->Dpad, p->d_bias);
    p->launches += 3;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "weight pack launch");
    p->packed = true;
    return GDWS_OK;
}

// ------------------------------------------------------------------------------------------
// Unfused GDW kernel: z[pixel][Gpad] (bf16), one thread per pixel and group of 8 intermediate
// channels, one 16-byte store each; the padding columns are written as zeros.
// ------------------------------------------------------------------------------------------
struct DwShape {
    int N, H, W, C, Ho, Wo, G, Gpad, k, stride, pad;
};

__global__ void gdw_bf16_kernel(DwShape s, const uint16_t *__restrict__ x, const float *__restrict__ dw,
                                const int32_t *__restrict__ chan, uint16_t *__restrict__ z)
{
    const int groups = s.Gpad / 8;
    const long long total = (long long)s.N * s.Ho * s.Wo * groups;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const int ig = (int)(t % groups);
        const long long p = t / groups;
        const int wo = (int)(p % s.Wo);
        const long long r = p / s.Wo;
        const int ho = (int)(r % s.Ho);
        const int n = (int)(r / s.Ho);
        float out[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int i = ig * 8 + e;
            const int c = __ldg(chan + i);
            float acc = 0.f;
            if (c >= 0) {
                const float *ker = dw + (size_t)i * s.k * s.k;
                for (int u = 0; u < s.k; ++u) {
                    const int hi = ho * s.stride + u - s.pad;
                    if (hi < 0 || hi >= s.H) continue;
                    for (int v = 0; v < s.k; ++v) {
                        const int wi = wo * s.stride + v - s.pad;
                        if (wi < 0 || wi >= s.W) continue;
                        const uint16_t xb = __ldg(x + (((size_t)n * s.H + hi) * s.W + wi) * s.C + c);
                        acc = fmaf(__ldg(ker + u * s.k + v), bf16_bits_to_float(xb), acc);
                    }
                }
            }
            out[e] = acc;
        }
        uint4 v4;
        v4.x = pack_bf16x2(out[0], out[1]);
        v4.y = pack_bf16x2(out[2], out[3]);
        v4.z = pack_bf16x2(out[4], out[5]);
        v4.w = pack_bf16x2(out[6], out[7]);
        *reinterpret_cast<uint4 *>(z + (size_t)p * s.Gpad + ig * 8) = v4;
    }
}

gdws_status_t bf16_depthwise(gdws_plan_s *p, const gdws_tensor_t *x, void *z, cudaStream_t st)
{
    if (p->C % 8 == 0) {   // tiled pipeline first; shapes it cannot tile fall through to the simple kernel
        const gdws_status_t rc = bf16_depthwise_tiled(p, x, z, st);
        if (rc != GDWS_ERR_UNSUPPORTED) return rc;
    }
    DwShape s;
    s.N = x->n; s.H = x->h; s.W = x->w; s.C = p->C; s.G = p->G; s.Gpad = p->Gpad; s.k = p->k; s.stride = p->stride; s.pad = p->pad;
    s.Ho = gdws_out_dim(x->h, p->k, p->stride, p->pad);
    s.Wo = gdws_out_dim(x->w, p->k, p->stride, p->pad);
    const long long total = (long long)s.N * s.Ho * s.Wo * (s.Gpad / 8);
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    gdw_bf16_kernel<<<(int)blocks, 256, 0, st>>>(s, (const uint16_t *)x->ptr, p->d_dw, p->d_chan, (uint16_t *)z);
    p->launches++;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "gdw_bf16_kernel launch");
}

// ------------------------------------------------------------------------------------------
// Pointwise 1x1 convolution as a GEMM: y[pixel][d] = bias[d] + sum_i z[pixel][i] * P[d][i].
// One block = 128 pixels x all D; K loop over 64-wide chunks with two shared-memory stages.
// ------------------------------------------------------------------------------------------
constexpr int kPwThreads = 128;

__global__ void __launch_bounds__(kPwThreads)
pw_bf16_tc_kernel(const uint16_t *__restrict__ z, const uint16_t *__restrict__ pw_img, const float *__restrict__ bias,
                  uint16_t *__restrict__ y, long long npix, int Gpad, int D, int Dpad, int relu, int tmem_cols,
                  int *status)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[4];     // b_full[2], mma_done[2]
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_s = smem_u32(base);
    const uint32_t b_bytes = (uint32_t)Dpad * kChunk * 2;
    const uint32_t b_s = a_s + 2 * 16384;
    const uint32_t bar_bfull = smem_u32(&bars[0]), bar_done = smem_u32(&bars[2]);
    const int nchunks = Gpad / kChunk;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < 2; ++i) { mbar_init(bar_bfull + 8 * i, 1); mbar_init(bar_done + 8 * i, 1); }
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), (uint32_t)tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const long long p0 = (long long)blockIdx.x * kTileRows;

    for (int q = 0; q < nchunks; ++q) {
        const int s = q & 1;
        if (q >= 2) mbar_wait(bar_done + 8 * s, ((q >> 1) - 1) & 1, &abort_flag, status, kStatusWaitStage);
        if (tid == 0) {
            mbar_expect_tx(bar_bfull + 8 * s, b_bytes);
            bulk_g2s(b_s + s * b_bytes, pw_img + (size_t)q * Dpad * kChunk, b_bytes, bar_bfull + 8 * s);
        }
        // A chunk: 128 rows x 128 bytes, 16-byte pieces into the swizzled K-major layout
        for (int t = tid; t < kTileRows * 8; t += kPwThreads) {
            const int row = t >> 3, ch = t & 7;
            const long long p = p0 + row;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (p < npix) v = __ldg(reinterpret_cast<const uint4 *>(z + (size_t)p * Gpad + q * kChunk + ch * 8));
            sts128(a_s + s * 16384 + row * 128 + ((ch ^ (row & 7)) << 4), v);
        }
        fence_proxy_async();
        __syncthreads();
        if (tid == 0) {
            mbar_wait(bar_bfull + 8 * s, (q >> 1) & 1, &abort_flag, status, kStatusWaitOperand);
            tc_fence_after();
            issue_chunk(tmem, a_s + s * 16384, b_s + s * b_bytes, Dpad, false, q == 0);
            umma_commit(bar_done + 8 * s);
        }
    }
    {
        const int ql = nchunks - 1;
        mbar_wait(bar_done + 8 * (ql & 1), (ql >> 1) & 1, &abort_flag, status, kStatusWaitMma);
        if (nchunks >= 2) {   // the other stage's last commit, so that no arrival is pending at exit
            const int qo = nchunks - 2;
            mbar_wait(bar_done + 8 * (qo & 1), (qo >> 1) & 1, &abort_flag, status, kStatusWaitMma);
        }
    }
    tc_fence_after();
    {
        const long long p = p0 + warp * 32 + lane;
        for (int d0 = 0; d0 < Dpad; d0 += 16) {
            uint32_t acc[16];
            tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)d0, acc);
            tmem_ld_wait();
            if (p < npix) store_row16(acc, bias, d0, D, relu, y + (size_t)p * D);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)tmem_cols);
}

gdws_status_t bf16_pointwise(gdws_plan_s *p, const void *z, gdws_tensor_t *y, cudaStream_t st)
{
    if (p->Dpad > 512) return fail(GDWS_ERR_UNSUPPORTED, "bf16 pointwise kernel supports D <= 512 (got %d)", p->D);
    if (p->D % 8) return fail(GDWS_ERR_UNSUPPORTED, "bf16 kernels need D %% 8 == 0 (got %d)", p->D);
    const long long npix = (long long)y->n * y->h * y->w;
    const int cols = tmem_cols_for(p->Dpad);
    size_t smem = 1024 + 2 * 16384 + 2 * (size_t)p->Dpad * kChunk * 2;
    smem = smem_for_tmem(smem, cols);
    cudaError_t e = cudaSuccess;
    static bool attr_set[64] = {};
    if (!attr_set[p->device & 63]) {   // once per device: allow the full dynamic shared memory
        e = cudaFuncSetAttribute(pw_bf16_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(pw_bf16_tc_kernel)");
        attr_set[p->device & 63] = true;
    }
    const long long blocks = (npix + kTileRows - 1) / kTileRows;
    pw_bf16_tc_kernel<<<(int)blocks, kPwThreads, smem, st>>>((const uint16_t *)z, p->d_pw_img, p->d_bias,
                                                             (uint16_t *)y->ptr, npix, p->Gpad, p->D, p->Dpad,
                                                             p->opt_relu, cols, p->d_status);
    p->launches++;
    e = cudaGetLastError();
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "pw_bf16_tc_kernel launch");
}

}  // namespace gdws
