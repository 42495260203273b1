// bf16 NHWC kernels for sm_100a: weight packing, the unfused GDW kernel, the pointwise
// 1x1 convolution as a tcgen05/TMEM GEMM, and the fused GDW -> PW kernel in which the
// intermediate channels go from the depthwise ALU stage to the tensor cores through
// shared memory only.
//
// Tensor-core operand conventions used here (sm_100 "UMMA" shared-memory descriptors):
//   * 128-byte swizzle: within every 1024-byte group of eight 128-byte rows, the 16-byte
//     column index is XORed with the row index (address bits [4,7) ^= bits [7,10)).
//   * K-major operand (rows = M or N index, 64 bf16 of K per 128-byte row): row groups
//     of 8 are 1024 bytes apart (stride byte offset); one MMA of K=16 reads 32 bytes of
//     each row, so successive K steps advance the start address by 32 bytes.
//   * MN-major operand (rows = K index, 64 consecutive M per 128-byte row): blocks of
//     64 M are `leading byte offset` apart, groups of 8 K rows `stride byte offset` apart.
#include <cuda_bf16.h>

#include "gdws_internal.h"

namespace gdws {

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait.  When the limit runs out (about a second) the thread records `code` in the
// status word and raises the block's abort flag; from then on every wait in the block returns
// at once, so that all threads still walk the same control flow, reach the common teardown
// (barriers stay matched, TMEM is freed) and the kernel ends.
constexpr uint32_t kSpinLimit = 1u << 22;
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (*abort_flag) return;
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if (it > 32) __nanosleep(64);
        if ((it & 1023) == 1023 && *abort_flag) return;
    }
    *abort_flag = 1;
    atomicOr(status, code);
}
// Same, but ignores the abort flag (used in teardown to drain copies that are in flight).
__device__ __forceinline__ bool mbar_wait_drain(uint32_t bar, uint32_t parity)
{
    for (uint32_t it = 0; it < (1u << 18); ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t addr, uint16_t v)
{
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}

// Instruction descriptor of tcgen05.mma kind::f16: fp32 accumulator, bf16 A and B, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool a_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(kTileRows >> 4) << 24);
}
// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
__device__ __forceinline__ uint64_t make_sdesc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f)
{
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    return (uint32_t)float_to_bf16_bits(lo) | ((uint32_t)float_to_bf16_bits(hi) << 16);
}

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

__global__ void pack_dw_kernel(const void *__restrict__ dw, int is_bf16, int G, int Gpad, int k2,
                               float *__restrict__ out, uint32_t *__restrict__ out2)
{
    const int total = Gpad * k2;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < total; t += gridDim.x * blockDim.x) {
        const int i = t / k2;
        float v = 0.f;
        if (i < G) v = load_weight(dw, t, is_bf16);
        const uint32_t b = float_to_bf16_bits(v);
        out[t] = bf16_bits_to_float((uint16_t)b);
        out2[t] = b | (b << 16);
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
    int blocks2 = (p->Gpad * k2 + 255) / 256;
    pack_dw_kernel<<<blocks2, 256, 0, st>>>(dw_w, is_bf16, p->G, p->Gpad, k2, p->d_dw, p->d_dw2);
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
// Epilogue shared by both tensor-core kernels: 16 accumulator columns of one pixel row.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void store_row16(const uint32_t (&acc)[16], const float *__restrict__ bias, int d0, int D,
                                            int relu, uint16_t *__restrict__ yrow)
{
    float v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        v[j] = __uint_as_float(acc[j]) + __ldg(bias + d0 + j);
        if (relu) v[j] = fmaxf(v[j], 0.f);
    }
    if (d0 + 8 <= D) {
        uint4 a;
        a.x = pack_bf16x2(v[0], v[1]); a.y = pack_bf16x2(v[2], v[3]);
        a.z = pack_bf16x2(v[4], v[5]); a.w = pack_bf16x2(v[6], v[7]);
        *reinterpret_cast<uint4 *>(yrow + d0) = a;
    }
    if (d0 + 16 <= D) {
        uint4 b;
        b.x = pack_bf16x2(v[8], v[9]); b.y = pack_bf16x2(v[10], v[11]);
        b.z = pack_bf16x2(v[12], v[13]); b.w = pack_bf16x2(v[14], v[15]);
        *reinterpret_cast<uint4 *>(yrow + d0 + 8) = b;
    }
}

// Issue the MMAs of one 64-wide K chunk (4 steps of K=16; output channels beyond 256 take a
// second instruction on the next 256 accumulator columns).
__device__ __forceinline__ void issue_chunk(uint32_t tmem, uint32_t a_addr, uint32_t b_addr, int Dpad, bool a_mn_major,
                                            bool first_chunk)
{
    const int n0 = Dpad > 256 ? 256 : Dpad;
    const int n1 = Dpad - n0;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
        const uint64_t adesc = a_mn_major ? make_sdesc(a_addr + ks * 4096, 1024, 2048)
                                          : make_sdesc(a_addr + ks * 32, 16, 1024);
        const uint32_t acc = (first_chunk && ks == 0) ? 0u : 1u;
        umma_bf16(tmem, adesc, make_sdesc(b_addr + ks * 32, 16, 1024), make_idesc(n0, a_mn_major), acc);
        if (n1 > 0)
            umma_bf16(tmem + 256, adesc, make_sdesc(b_addr + 256 * 128 + ks * 32, 16, 1024),
                      make_idesc(n1, a_mn_major), acc);
    }
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

static int tmem_cols_for(int Dpad)
{
    int c = 32;
    while (c < Dpad) c <<= 1;
    return c;
}

// Shared memory to request so that the blocks resident on one SM never ask for more than the
// 512 TMEM columns together (an allocation that cannot be served would wait).
static size_t smem_for_tmem(size_t need, int cols)
{
    const int max_ctas = 512 / cols;
    const size_t floor_bytes = (size_t)kMaxSmem / (max_ctas + 1) + 1024;
    return need > floor_bytes ? need : floor_bytes;
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

// ------------------------------------------------------------------------------------------
// Fused kernel
// ------------------------------------------------------------------------------------------
struct FusedParams {
    const uint16_t *x;
    uint16_t *y;
    const float *dw;
    const uint32_t *dw2;
    const uint16_t *pw_img;
    const float *bias;
    const int32_t *off;
    const int32_t *chan;
    int *status;
    int N, H, W, C, Ho, Wo, D, Dpad, G, Gpad, nchunks, k, stride, pad, relu;
    int TN, PH, PW, tiles_h, tiles_w;
    int IH, IW, IWp, plane, CB, nblocks, nsb;
    int tmem_cols, a_kmajor, dw_math;
};

constexpr int kDwThreads = 256;
constexpr int kFusedThreads = kDwThreads + 32;
constexpr int kMaxPrefetch = 12;

// Where the 8 bf16 results of pixel group `o` (rows 8o..8o+7 of the tile) and intermediate
// channel column kk go in a pixel-contiguous (MN-major) stage: K group kk/8 and 64-row block
// o/8 select a 1024-byte atom, kk%8 the 128-byte row, and the 16-byte piece is swizzled.
__device__ __forceinline__ uint32_t a_off_mn(int o, int kk)
{
    return (uint32_t)(((kk >> 3) * 2 + (o >> 3)) * 1024 + (kk & 7) * 128 + (((o & 7) ^ (kk & 7)) << 4));
}
// Channel-contiguous (K-major) stage: byte offset of element (row r, column kk).
__device__ __forceinline__ uint32_t a_off_k(int r, int kk)
{
    return (uint32_t)(r * 128 + (((kk >> 3) ^ (r & 7)) << 4) + (kk & 7) * 2);
}

// Depthwise work of intermediate channels [i_lo, i_hi) (all inside K chunk i_lo/64) for the
// 16 pixel groups of the tile.  Generic in filter size and stride; fp32 FMAs.
template <int K>
__device__ __forceinline__ void dw_items_generic(const FusedParams &P, const uint16_t *__restrict__ xs, int c0, int i_lo,
                                                 int i_hi, uint32_t a_stage, int tid)
{
    const int ni = i_hi - i_lo;
    const int hw = P.PH * P.PW;
    for (int it = tid; it < ni * 16; it += kDwThreads) {
        const int o = it / ni;
        const int i = i_lo + (it - o * ni);
        const int kk = i & (kChunk - 1);
        float out[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = 0.f;
        if (i < P.G) {
            float w[K * K];
            const float *wp = P.dw + (size_t)i * (K * K);
#pragma unroll
            for (int t = 0; t < K * K; ++t) w[t] = __ldg(wp + t);
            const int cl = __ldg(P.chan + i) - c0;
            const int r0 = o * 8;
            const int tn = r0 / hw;
            const int rem = r0 - tn * hw;
            const int ph = rem / P.PW;
            const int pw0 = rem - ph * P.PW;
            if (tn < P.TN) {
                const uint16_t *xc = xs + (size_t)cl * P.plane + (size_t)tn * P.IH * P.IWp;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int phe = (P.PW >= 8) ? ph : ph + (e >> 2);
                    const int pwe = (P.PW >= 8) ? pw0 + e : (e & 3);
                    const uint16_t *xp = xc + phe * P.stride * P.IWp + pwe * P.stride;
                    float acc = 0.f;
#pragma unroll
                    for (int u = 0; u < K; ++u)
#pragma unroll
                        for (int v = 0; v < K; ++v)
                            acc = fmaf(w[u * K + v], bf16_bits_to_float(xp[u * P.IWp + v]), acc);
                    out[e] = acc;
                }
            }
        }
        if (!P.a_kmajor) {
            uint4 v4;
            v4.x = pack_bf16x2(out[0], out[1]); v4.y = pack_bf16x2(out[2], out[3]);
            v4.z = pack_bf16x2(out[4], out[5]); v4.w = pack_bf16x2(out[6], out[7]);
            sts128(a_stage + a_off_mn(o, kk), v4);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) sts16(a_stage + a_off_k(o * 8 + e, kk), float_to_bf16_bits(out[e]));
        }
    }
}

template <int K>
__global__ void __launch_bounds__(kFusedThreads, 1) fused_bf16_kernel(const __grid_constant__ FusedParams P)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[12];   // a_full[2] | mma_done[2] | b_full[4] | b_free[4]
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_s = smem_u32(base);
    const uint32_t b_bytes = (uint32_t)P.Dpad * kChunk * 2;
    const uint32_t b_s = a_s + 2 * 16384;
    const uint32_t x_bytes = (uint32_t)P.CB * P.plane * 2;
    uint16_t *xs_base = (uint16_t *)(base + 2 * 16384 + (size_t)P.nsb * b_bytes);
    const uint32_t bar_afull = smem_u32(&bars[0]), bar_done = smem_u32(&bars[2]);
    const uint32_t bar_bfull = smem_u32(&bars[4]), bar_bfree = smem_u32(&bars[8]);

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < 2; ++i) { mbar_init(bar_afull + 8 * i, kDwThreads); mbar_init(bar_done + 8 * i, 1); }
        for (int i = 0; i < 4; ++i) { mbar_init(bar_bfull + 8 * i, 1); mbar_init(bar_bfree + 8 * i, 1); }
        fence_mbar_init();
    }
    if (warp == kDwThreads / 32) tmem_alloc(smem_u32(&tmem_slot), (uint32_t)P.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    // tile -> first image / output row / output column
    int tile = blockIdx.x;
    const int bw = tile % P.tiles_w;
    tile /= P.tiles_w;
    const int bh = tile % P.tiles_h;
    const int bn = tile / P.tiles_h;
    const int n0 = bn * P.TN, ho0 = bh * P.PH, wo0 = bw * P.PW;

    if (warp == kDwThreads / 32) {
        // ---------------- control warp: weight copies and MMA issue (one lane) ----------------
        if (lane == 0) {
            const int pre = P.nchunks < P.nsb ? P.nchunks : P.nsb;
            for (int q = 0; q < pre; ++q) {
                mbar_expect_tx(bar_bfull + 8 * q, b_bytes);
                bulk_g2s(b_s + q * b_bytes, P.pw_img + (size_t)q * P.Dpad * kChunk, b_bytes, bar_bfull + 8 * q);
            }
            for (int q = 0; q < P.nchunks; ++q) {
                const int sa = q & 1, sb = q % P.nsb;
                mbar_wait(bar_bfull + 8 * sb, (q / P.nsb) & 1, &abort_flag, P.status, kStatusWaitOperand);
                mbar_wait(bar_afull + 8 * sa, (q >> 1) & 1, &abort_flag, P.status, kStatusWaitOperand);
                tc_fence_after();
                issue_chunk(tmem, a_s + sa * 16384, b_s + sb * b_bytes, P.Dpad, !P.a_kmajor, q == 0);
                umma_commit(bar_done + 8 * sa);
                umma_commit(bar_bfree + 8 * sb);
                // refill the stage of the previous chunk once its MMAs have finished
                const int qn = q - 1 + P.nsb;
                if (q >= 1 && qn < P.nchunks) {
                    const int sp = (q - 1) % P.nsb;
                    mbar_wait(bar_bfree + 8 * sp, ((q - 1) / P.nsb) & 1, &abort_flag, P.status, kStatusWaitStage);
                    mbar_expect_tx(bar_bfull + 8 * sp, b_bytes);
                    bulk_g2s(b_s + sp * b_bytes, P.pw_img + (size_t)qn * P.Dpad * kChunk, b_bytes, bar_bfull + 8 * sp);
                }
            }
            // drain: every copy issued has been waited for above (each chunk's b_full), and the
            // last commits are awaited so that no arrival is pending when the block exits
            for (int q = (P.nchunks > P.nsb ? P.nchunks - P.nsb : 0); q < P.nchunks; ++q)
                mbar_wait_drain(bar_bfree + 8 * (q % P.nsb), (q / P.nsb) & 1);
        }
    } else {
        // ---------------- depthwise warps ----------------
        const int items = P.TN * P.IH * P.IWp * (P.CB / 8);
        const int hi0 = ho0 * P.stride - P.pad, wi0 = wo0 * P.stride - P.pad;
        uint4 pf[kMaxPrefetch];
        auto load_block = [&](int b) {
            const int c0 = b * P.CB;
#pragma unroll
            for (int m = 0; m < kMaxPrefetch; ++m) {
                const int t = tid + m * kDwThreads;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (t < items) {
                    const int iw = t % P.IWp;
                    int r = t / P.IWp;
                    const int c8 = r % (P.CB / 8);
                    r /= (P.CB / 8);
                    const int ih = r % P.IH;
                    const int tn = r / P.IH;
                    const int n = n0 + tn, hi = hi0 + ih, wi = wi0 + iw, c = c0 + c8 * 8;
                    if (n < P.N && hi >= 0 && hi < P.H && wi >= 0 && wi < P.W && iw < P.IW && c < P.C)
                        v = __ldg(reinterpret_cast<const uint4 *>(P.x + (((size_t)n * P.H + hi) * P.W + wi) * P.C + c));
                }
                pf[m] = v;
            }
        };
        auto store_block = [&](int slot) {
            const uint32_t xs = smem_u32(xs_base) + slot * x_bytes;
#pragma unroll
            for (int m = 0; m < kMaxPrefetch; ++m) {
                const int t = tid + m * kDwThreads;
                if (t < items) {
                    const int iw = t % P.IWp;
                    int r = t / P.IWp;
                    const int c8 = r % (P.CB / 8);
                    r /= (P.CB / 8);
                    const int ih = r % P.IH;
                    const int tn = r / P.IH;
                    const uint32_t a = xs + (uint32_t)(((c8 * 8) * P.plane + (tn * P.IH + ih) * P.IWp + iw) * 2);
                    const uint32_t w[4] = {pf[m].x, pf[m].y, pf[m].z, pf[m].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        sts16(a + (uint32_t)((2 * e) * P.plane * 2), (uint16_t)(w[e] & 0xffffu));
                        sts16(a + (uint32_t)((2 * e + 1) * P.plane * 2), (uint16_t)(w[e] >> 16));
                    }
                }
            }
        };

        load_block(0);
        store_block(0);
        named_bar_sync(1, kDwThreads);
        for (int b = 0; b < P.nblocks; ++b) {
            if (b + 1 < P.nblocks) load_block(b + 1);
            const int c0 = b * P.CB;
            const int c1 = min(P.C, c0 + P.CB);
            int i = __ldg(P.off + c0);
            const int i1 = (b + 1 == P.nblocks) ? P.Gpad : __ldg(P.off + c1);
            const uint16_t *xs = xs_base + (size_t)(b & 1) * (x_bytes / 2);
            while (i < i1) {
                const int q = i >> 6;
                const int i_end = min(i1, (q + 1) << 6);
                const int sa = q & 1;
                if ((i & (kChunk - 1)) == 0 && q >= 2)
                    mbar_wait(bar_done + 8 * sa, ((q >> 1) - 1) & 1, &abort_flag, P.status, kStatusWaitStage);
                dw_items_generic<K>(P, xs, c0, i, i_end, a_s + sa * 16384, tid);
                if ((i_end & (kChunk - 1)) == 0) {   // chunk complete: hand it to the tensor cores
                    fence_proxy_async();
                    mbar_arrive(bar_afull + 8 * sa);
                }
                i = i_end;
            }
            if (b + 1 < P.nblocks) store_block((b + 1) & 1);
            named_bar_sync(1, kDwThreads);
        }

        // ---------------- epilogue: TMEM -> registers -> bias / ReLU -> bf16 -> global ----------------
        {
            const int ql = P.nchunks - 1;
            mbar_wait(bar_done + 8 * (ql & 1), (ql >> 1) & 1, &abort_flag, P.status, kStatusWaitMma);
            if (P.nchunks >= 2) {
                const int qo = P.nchunks - 2;
                mbar_wait(bar_done + 8 * (qo & 1), (qo >> 1) & 1, &abort_flag, P.status, kStatusWaitMma);
            }
        }
        tc_fence_after();
        const int lg = warp & 3, half = warp >> 2;
        const int r = lg * 32 + lane;
        const int hw = P.PH * P.PW;
        const int tn = r / hw;
        const int rem = r - tn * hw;
        const int ph = rem / P.PW, pw_ = rem - (rem / P.PW) * P.PW;
        const int n = n0 + tn, ho = ho0 + ph, wo = wo0 + pw_;
        const bool live = tn < P.TN && n < P.N && ho < P.Ho && wo < P.Wo;
        uint16_t *yrow = P.y + (((size_t)n * P.Ho + ho) * P.Wo + wo) * P.D;
        for (int d0 = half * 16; d0 < P.Dpad; d0 += 32) {
            uint32_t acc[16];
            tmem_ld16(tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)d0, acc);
            tmem_ld_wait();
            if (live) store_row16(acc, P.bias, d0, P.D, P.relu, yrow);
        }
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (warp == kDwThreads / 32) tmem_dealloc(tmem, (uint32_t)P.tmem_cols);
}

template <int K>
static gdws_status_t launch_fused(const FusedParams &P, int device, int64_t tiles, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaSuccess;
    static bool attr_set[64] = {};
    if (!attr_set[device & 63]) {   // once per device: allow the full dynamic shared memory
        e = cudaFuncSetAttribute(fused_bf16_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(fused_bf16_kernel)");
        attr_set[device & 63] = true;
    }
    fused_bf16_kernel<K><<<(int)tiles, kFusedThreads, smem, st>>>(P);
    e = cudaGetLastError();
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "fused_bf16_kernel launch");
}

gdws_status_t bf16_fused(gdws_plan_s *p, const gdws_tensor_t *x, gdws_tensor_t *y, cudaStream_t st)
{
    if (p->Dpad > 512) return fail(GDWS_ERR_UNSUPPORTED, "bf16 fused kernel supports D <= 512 (got %d)", p->D);
    if (p->D % 8 || p->C % 8)
        return fail(GDWS_ERR_UNSUPPORTED, "bf16 kernels need C %% 8 == 0 and D %% 8 == 0 (got C=%d, D=%d)", p->C, p->D);
    Tile t;
    if (!choose_tile(p, x->n, x->h, x->w, &t))
        return fail(GDWS_ERR_UNSUPPORTED, "no fused tile fits this shape in shared memory");
    if (t.tiles() > 0x7fffffffLL) return fail(GDWS_ERR_UNSUPPORTED, "too many tiles");
    FusedParams P;
    P.x = (const uint16_t *)x->ptr; P.y = (uint16_t *)y->ptr;
    P.dw = p->d_dw; P.dw2 = p->d_dw2; P.pw_img = p->d_pw_img; P.bias = p->d_bias;
    P.off = p->d_off; P.chan = p->d_chan; P.status = p->d_status;
    P.N = x->n; P.H = x->h; P.W = x->w; P.C = p->C; P.Ho = y->h; P.Wo = y->w; P.D = p->D; P.Dpad = p->Dpad;
    P.G = p->G; P.Gpad = p->Gpad; P.nchunks = p->nchunks; P.k = p->k; P.stride = p->stride; P.pad = p->pad;
    P.relu = p->opt_relu;
    P.TN = t.TN; P.PH = t.PH; P.PW = t.PW; P.tiles_h = t.tiles_h; P.tiles_w = t.tiles_w;
    P.IH = t.IH; P.IW = t.IW; P.IWp = t.IWp; P.plane = t.plane; P.CB = t.CB; P.nsb = t.nsb;
    P.nblocks = (p->C + t.CB - 1) / t.CB;
    P.tmem_cols = tmem_cols_for(p->Dpad);
    P.a_kmajor = p->opt_a_layout;
    P.dw_math = p->opt_dw_math;
    const size_t smem = smem_for_tmem(t.smem, P.tmem_cols);
    gdws_status_t rc;
    switch (p->k) {
    case 1: rc = launch_fused<1>(P, p->device, t.tiles(), smem, st); break;
    case 2: rc = launch_fused<2>(P, p->device, t.tiles(), smem, st); break;
    case 3: rc = launch_fused<3>(P, p->device, t.tiles(), smem, st); break;
    case 4: rc = launch_fused<4>(P, p->device, t.tiles(), smem, st); break;
    case 5: rc = launch_fused<5>(P, p->device, t.tiles(), smem, st); break;
    case 6: rc = launch_fused<6>(P, p->device, t.tiles(), smem, st); break;
    case 7: rc = launch_fused<7>(P, p->device, t.tiles(), smem, st); break;
    default: return fail(GDWS_ERR_UNSUPPORTED, "k=%d", p->k);
    }
    if (rc == GDWS_OK) p->launches++;
    return rc;
}

}  // namespace gdws
