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
    if (blocks > sm_count_of(p) * 8) blocks = sm_count_of(p) * 8;
    pack_pw_kernel<<<blocks, 256, 0, st>>>(pw_w, is_bf16, p->D, p->Dpad, p->G, p->nchunks, p->d_pw_img);
    int blocks2 = (p->Gpad * p->wstride + 255) / 256;
    pack_dw_kernel<<<blocks2, 256, 0, st>>>(dw_w, is_bf16, p->G, p->Gpad, k2, p->wstride, p->d_chan, p->d_chunk_meta,
                                            p->d_dw, p->d_dwpack);
    pack_bias_kernel<<<(p->Dpad + 255) / 256, 256, 0, st>>>(bias, p->D, p->Dpad, p->d_bias);
    p->launches += 3;
    tc_pack(p, dw_w, pw_w, is_bf16, st);
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
    grid_launch_dependents();
    grid_dependency_wait();
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
    if (blocks > (long long)sm_count_of(p) * 32) blocks = (long long)sm_count_of(p) * 32;
    cudaError_t e = launch_overlapped(gdw_bf16_kernel, (unsigned)blocks, 256u, 0, st, s, (const uint16_t *)x->ptr, (const float *)p->d_dw,
                                      (const int32_t *)p->d_chan, (uint16_t *)z);
    p->launches++;
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "gdw_bf16_kernel launch");
}

// ------------------------------------------------------------------------------------------
// Pointwise 1x1 convolution as a GEMM: y[pixel][d] = bias[d] + sum_i z[pixel][i] * P[d][i].
// Persistent blocks walk over tiles of 128 pixels (all D).  One thread loads (TMA tiled loads of the
// 128 x 64 piece of z with the 128-byte swizzle the tensor cores expect, bulk copies of the packed
// weight chunk), one thread issues tcgen05.mma into TMEM (two accumulators when D <= 256), four
// warps run the epilogue of the previous tile meanwhile.  A ring of `ns` stages (z piece + weights).
// ------------------------------------------------------------------------------------------
struct alignas(64) PwParams {
    CUtensorMap tmap;            // z as (Gpad, pixels) bf16, box (64, 128), SWIZZLE_128B
    const uint16_t *pw_img;
    const float *bias;
    uint16_t *y;
    int *status;
    long long npix;
    int ntiles, nchunks, D, Dpad, relu, ns, stage_bytes, nacc, acc_cols;
};

constexpr int kPwThreads = 6 * 32;      // warp 0 loader, warp 1 MMA issue, warps 2-5 epilogue
constexpr int kPwMaxStages = 8;

__global__ void __launch_bounds__(kPwThreads, 1) pw_bf16_tc_kernel(const __grid_constant__ PwParams P)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[2 * kPwMaxStages + 4 + 1];   // full[8] free[8] acc_full[2] acc_free[2] drain
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t st_s = smem_u32(base);
    const uint32_t bar_full = smem_u32(&bars[0]), bar_free = smem_u32(&bars[kPwMaxStages]);
    const uint32_t bar_accfull = smem_u32(&bars[2 * kPwMaxStages]), bar_accfree = bar_accfull + 16;
    const uint32_t bar_drain = bar_accfull + 32;
    volatile int *const vabort = &abort_flag;
    const uint32_t b_bytes = (uint32_t)P.Dpad * kChunk * 2;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < kPwMaxStages; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_free + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_accfull + 8 * i, 1); mbar_init(bar_accfree + 8 * i, 4); }
        mbar_init(bar_drain, 1);
        fence_mbar_init();
    }
    __syncwarp();
    grid_launch_dependents();
    if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), (uint32_t)(P.nacc * P.acc_cols));
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    grid_dependency_wait();      // z comes from the kernel before this one in the stream
    const uint32_t tmem = tmem_slot;
    const int my_tiles = (P.ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp == 0) {
        if (lane == 0) {        // ---------------- loader ----------------
            uint32_t s = 0, par = 1;
            int it = 0;
            bool stop = false;
            for (int tl = 0; tl < my_tiles && !stop; ++tl) {
                const int row0 = ((int)blockIdx.x + tl * (int)gridDim.x) * kTileRows;
                for (int q = 0; q < P.nchunks; ++q, ++it) {
                    if (it >= P.ns) mbar_wait(bar_free + 8 * s, par, &abort_flag, P.status, kStatusWaitStage);
                    if (*vabort) { stop = true; break; }      // a wait ran out somewhere: no new copies
                    const uint32_t dst = st_s + s * (uint32_t)P.stage_bytes;
                    mbar_expect_tx(bar_full + 8 * s, 16384u + b_bytes);
                    tma_load_2d(dst, &P.tmap, q * kChunk, row0, bar_full + 8 * s);
                    bulk_g2s(dst + 16384u, P.pw_img + (size_t)q * P.Dpad * kChunk, b_bytes, bar_full + 8 * s);
                    if (++s == (uint32_t)P.ns) { s = 0; par ^= 1; }
                }
            }
            // Teardown: no copy into this block's shared memory may be in flight when it ends.  The last phase armed
            // on each stage completes when its copies have landed.
            for (int j = 0; j < P.ns && j < it; ++j) mbar_wait_drain(bar_full + 8 * j, (uint32_t)((it - 1 - j) / P.ns) & 1u);
        }
    } else if (warp == 1) {
        if (lane == 0) {        // ---------------- MMA issue ----------------
            uint32_t s = 0, par = 0;
            for (int tl = 0; tl < my_tiles; ++tl) {
                const int buf = tl % P.nacc;
                if (tl >= P.nacc)
                    mbar_wait(bar_accfree + 8 * buf, ((tl / P.nacc) - 1) & 1, &abort_flag, P.status, kStatusWaitStage);
                tc_fence_after();
                for (int q = 0; q < P.nchunks; ++q) {
                    mbar_wait(bar_full + 8 * s, par, &abort_flag, P.status, kStatusWaitOperand);
                    tc_fence_after();
                    const uint32_t a_addr = st_s + s * (uint32_t)P.stage_bytes;
                    issue_chunk(tmem + (uint32_t)(buf * P.acc_cols), a_addr, a_addr + 16384u, P.Dpad, false, q == 0);
                    umma_commit(bar_free + 8 * s);
                    if (++s == (uint32_t)P.ns) { s = 0; par ^= 1; }
                }
                umma_commit(bar_accfull + 8 * buf);
            }
            // Teardown: all issued products complete before the tensor memory is freed (bounded, ignores the abort flag).
            umma_commit(bar_drain);
            mbar_wait_drain(bar_drain, 0);
        }
    } else {
        // ---------------- epilogue warps ----------------
        const int lg = warp & 3;
        for (int tl = 0; tl < my_tiles; ++tl) {
            const long long p = ((long long)blockIdx.x + (long long)tl * gridDim.x) * kTileRows + lg * 32 + lane;
            const int buf = tl % P.nacc;
            if (lane == 0) mbar_wait(bar_accfull + 8 * buf, (tl / P.nacc) & 1, &abort_flag, P.status, kStatusWaitMma);
            __syncwarp();
            tc_fence_after();
            const uint32_t t_base = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * P.acc_cols);
            for (int d0 = 0; d0 < P.Dpad; d0 += 16) {
                uint32_t acc[16];
                tmem_ld16(t_base + (uint32_t)d0, acc);
                tmem_ld_wait();
                if (p < P.npix) store_row16(acc, P.bias, d0, P.D, P.relu, P.y, (size_t)p * P.D);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_accfree + 8 * buf);
        }
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (warp == 1) tmem_dealloc(tmem, (uint32_t)(P.nacc * P.acc_cols));
}

gdws_status_t bf16_pointwise(gdws_plan_s *p, const void *z, gdws_tensor_t *y, cudaStream_t st)
{
    if (p->Dpad > 512) return fail(GDWS_ERR_UNSUPPORTED, "bf16 pointwise kernel supports D <= 512 (got %d)", p->D);
    if (p->D % 8) return fail(GDWS_ERR_UNSUPPORTED, "bf16 kernels need D %% 8 == 0 (got %d)", p->D);
    const long long npix = (long long)y->n * y->h * y->w;
    const long long tiles = (npix + kTileRows - 1) / kTileRows;
    if (tiles > 0x7fffffffLL / kTileRows) return fail(GDWS_ERR_UNSUPPORTED, "too many pixels for the bf16 pointwise kernel");
    if (p->sm_count <= 0) {
        cudaError_t e0 = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
        if (e0 != cudaSuccess) return cuda_fail(e0, "cudaDeviceGetAttribute(MultiProcessorCount)");
    }
    tensor_map_encode_fn encode = encode_fn();
    if (!encode) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    PwParams P;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)p->Gpad, (cuuint64_t)npix};
        const cuuint64_t strides[1] = {(cuuint64_t)p->Gpad * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kChunk, (cuuint32_t)kTileRows};
        const cuuint32_t estr[2] = {1, 1};
        const CUresult r = encode(&P.tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(z), dims, strides, box,
                                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    }
    P.pw_img = p->d_pw_img; P.bias = p->d_bias; P.y = (uint16_t *)y->ptr; P.status = p->d_status;
    P.npix = npix; P.ntiles = (int)tiles; P.nchunks = p->nchunks; P.D = p->D; P.Dpad = p->Dpad; P.relu = (p->opt_relu ? kOutRelu : 0) | (y->dtype == GDWS_F32 ? kOutF32 : 0);
    P.stage_bytes = 16384 + p->Dpad * kChunk * 2;
    P.ns = (kMaxSmem - 1024) / P.stage_bytes;
    if (P.ns > kPwMaxStages) P.ns = kPwMaxStages;
    if (P.ns < 2) return fail(GDWS_ERR_UNSUPPORTED, "no room for two stages");
    P.acc_cols = tmem_cols_for(p->Dpad);
    P.nacc = P.acc_cols <= 256 ? 2 : 1;
    // one block per SM: ask for more than half of the shared memory even when fewer stages would do
    size_t smem = 1024 + (size_t)P.ns * P.stage_bytes;
    if (smem < (size_t)kMaxSmem / 2 + 2048) smem = (size_t)kMaxSmem / 2 + 2048;
    cudaError_t e = cudaSuccess;
    static bool attr_set[64] = {};
    if (!attr_set[p->device & 63]) {   // once per device: allow the full dynamic shared memory
        e = cudaFuncSetAttribute(pw_bf16_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(pw_bf16_tc_kernel)");
        attr_set[p->device & 63] = true;
    }
    const int grid = (int)(tiles < p->sm_count ? tiles : p->sm_count);
    e = launch_overlapped(pw_bf16_tc_kernel, (unsigned)grid, kPwThreads, smem, st, P);
    p->launches++;
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "pw_bf16_tc_kernel launch");
}

}  // namespace gdws
