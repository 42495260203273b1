// Diagnostics of libgdws: a measurement of the multiply-add rate of the plain ALUs (the bound of a GDW stage
// that runs there) and a self-test of the bounded-wait error path.
#include "sm100.cuh"

using namespace gdws;

namespace {

constexpr int kRateAcc = 16;       // independent accumulators per thread
constexpr int kRateBody = 8;       // passes over them per loop iteration: 128 multiply-adds, a loop body of 2 KB

// KIND 0: fma.rn.f32, 1: fma.rn.f32x2 (two multiply-adds per instruction), 2: fma.rn.bf16x2 (two, bf16 sums),
// 3: fma.rn.f32.bf16 (bf16 factors taken from register halves, fp32 sum).
template <int KIND>
__global__ void __launch_bounds__(1024, 1) fma_rate_kernel(float *sink, long long *cycles, int iters, float seed)
{
    float a[kRateAcc];
    uint32_t h[kRateAcc];
    unsigned long long p[kRateAcc];
#pragma unroll
    for (int i = 0; i < kRateAcc; ++i) {
        a[i] = seed * (float)(i + 1) + (float)threadIdx.x;
        h[i] = 0x3c003c00u + (uint32_t)i;
        p[i] = ((unsigned long long)__float_as_uint(a[i] + 1.f) << 32) | __float_as_uint(a[i]);
    }
    const float w0 = seed, w1 = seed * 0.5f;
    const unsigned long long wp = ((unsigned long long)__float_as_uint(w1) << 32) | __float_as_uint(w0);
    const unsigned long long xp = ((unsigned long long)__float_as_uint(w0 + 1.f) << 32) | __float_as_uint(w1 + 1.f);
    const uint32_t hw = 0x3f803f80u, hx = 0x3f003f00u;
    const uint32_t word = 0x3f803f00u + threadIdx.x;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int rep = 0; rep < kRateBody; ++rep) {
#pragma unroll
            for (int i = 0; i < kRateAcc; ++i) {
                if (KIND == 0) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(a[i]) : "f"(w0), "f"(w1));
                else if (KIND == 1) asm volatile("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(p[i]) : "l"(wp), "l"(xp));
                else if (KIND == 2) asm volatile("fma.rn.bf16x2 %0, %1, %2, %0;" : "+r"(h[i]) : "r"(hw), "r"(hx));
                else
                    asm volatile("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tfma.rn.f32.bf16 %0, lo, hi, %0;\n\t}"
                                 : "+f"(a[i]) : "r"(word + (uint32_t)i));
            }
        }
    }
    const long long t1 = clock64();
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kRateAcc; ++i)
        s += a[i] + __uint_as_float(h[i]) + __uint_as_float((uint32_t)p[i]) + __uint_as_float((uint32_t)(p[i] >> 32));
    if (s == 123.456f) sink[threadIdx.x] = s;     // never true: keeps the sums alive
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// The same independent fp32 multiply-adds with a loop body of BODY instructions (16 bytes each; the loop itself is kept
// from being unrolled, so BODY * 16 bytes is what the warps walk through): shows where straight-line code stops
// fitting the SM's instruction caches and runs at the speed of instruction fetch instead.
template <int BODY>
__global__ void __launch_bounds__(512, 1) code_size_kernel(float *sink, long long *cycles, int total_fma, float seed)
{
    float a[32], w[9], x[10];
#pragma unroll
    for (int i = 0; i < 32; ++i) a[i] = seed * (float)i;
#pragma unroll
    for (int i = 0; i < 9; ++i) w[i] = seed + (float)i + (float)threadIdx.x;
#pragma unroll
    for (int i = 0; i < 10; ++i) x[i] = seed * 3.f + (float)i + (float)threadIdx.x;
    __syncthreads();
    const int iters = total_fma / BODY;
    const long long t0 = clock64();
#pragma unroll 1
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int b = 0; b < BODY / 32; ++b)
#pragma unroll
            for (int i = 0; i < 32; ++i)
                asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(a[i]) : "f"(w[b % 9]), "f"(x[(i + b) % 10]));
    }
    const long long t1 = clock64();
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) s += a[i];
    if (s == 123.456f) sink[threadIdx.x] = s;
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// One block; nothing ever arrives at its mbarrier.  Lane 0 of warp 0 waits with the given poll limit, runs out,
// records the code and raises the abort flag; lane 0 of warp 1 waits with the library's normal limit and is
// released by that flag.  No copies, no tensor memory: the kernel returns by itself.
__global__ void wait_selftest_kernel(int *status, uint32_t polls)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        if (warp == 0) mbar_wait_limited(smem_u32(&bar), 0, polls, &abort_flag, status, kStatusWaitOperand);
        else mbar_wait(smem_u32(&bar), 0, &abort_flag, status, kStatusWaitStage);
    }
    __syncthreads();
}

}  // namespace

extern "C" {

gdws_status_t gdws_measure_fma_rate(int kind, double *macs_per_clk_per_sm, double *tmacs_per_s)
{
    if (kind < 0 || kind > 3) return fail(GDWS_ERR_INVALID_ARG, "gdws_measure_fma_rate: kind must be 0..3");
    gdws_status_t st = check_arch();
    if (st != GDWS_OK) return st;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e, "device query");
    float *sink = nullptr;
    long long *cyc = nullptr;
    e = cudaMalloc((void **)&sink, 4096);
    if (e == cudaSuccess) e = cudaMalloc((void **)&cyc, sizeof(long long) * (size_t)sms);
    if (e != cudaSuccess) { cudaFree(sink); return cuda_fail(e, "cudaMalloc"); }
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const int iters = 4000, threads = 1024;
    auto launch = [&](int n) {
        switch (kind) {
        case 0: fma_rate_kernel<0><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 1: fma_rate_kernel<1><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 2: fma_rate_kernel<2><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        default: fma_rate_kernel<3><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        }
    };
    launch(50);
    cudaEventRecord(e0);
    launch(iters);
    cudaEventRecord(e1);
    e = cudaDeviceSynchronize();
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    long long worst = 0;
    if (e == cudaSuccess) {
        std::vector<long long> h((size_t)sms);
        e = cudaMemcpy(h.data(), cyc, sizeof(long long) * (size_t)sms, cudaMemcpyDeviceToHost);
        for (long long c : h) worst = c > worst ? c : worst;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(sink);
    cudaFree(cyc);
    if (e != cudaSuccess) return cuda_fail(e, "gdws_measure_fma_rate");
    const double per_instr = (kind == 1 || kind == 2) ? 2.0 : 1.0;
    const double macs_sm = (double)iters * kRateBody * kRateAcc * threads * per_instr;
    if (macs_per_clk_per_sm) *macs_per_clk_per_sm = worst > 0 ? macs_sm / (double)worst : 0.0;
    if (tmacs_per_s) *tmacs_per_s = ms > 0.f ? macs_sm * sms / (ms * 1e-3) / 1e12 : 0.0;
    return GDWS_OK;
}

gdws_status_t gdws_measure_code_size(int body_instructions, int threads, double *instructions_per_clk_per_scheduler)
{
    if (threads != 128 && threads != 256 && threads != 512)
        return fail(GDWS_ERR_INVALID_ARG, "gdws_measure_code_size: threads must be 128, 256 or 512");
    gdws_status_t st = check_arch();
    if (st != GDWS_OK) return st;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e, "device query");
    float *sink = nullptr;
    long long *cyc = nullptr;
    e = cudaMalloc((void **)&sink, 4096);
    if (e == cudaSuccess) e = cudaMalloc((void **)&cyc, sizeof(long long) * (size_t)sms);
    if (e != cudaSuccess) { cudaFree(sink); return cuda_fail(e, "cudaMalloc"); }
    const int total = 3 << 18;      // a multiple of every body size
    bool known = true;
    for (int pass = 0; pass < 2 && known; ++pass) {
        const int n = pass == 0 ? 3 << 13 : total;
        switch (body_instructions) {
        case 128: code_size_kernel<128><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 512: code_size_kernel<512><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 1024: code_size_kernel<1024><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 2048: code_size_kernel<2048><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 3072: code_size_kernel<3072><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 4096: code_size_kernel<4096><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 6144: code_size_kernel<6144><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        case 8192: code_size_kernel<8192><<<sms, threads>>>(sink, cyc, n, 1.f); break;
        default: known = false; break;
        }
    }
    long long worst = 0;
    if (known) {
        e = cudaDeviceSynchronize();
        if (e == cudaSuccess) {
            std::vector<long long> h((size_t)sms);
            e = cudaMemcpy(h.data(), cyc, sizeof(long long) * (size_t)sms, cudaMemcpyDeviceToHost);
            for (long long c : h) worst = c > worst ? c : worst;
        }
    }
    cudaFree(sink);
    cudaFree(cyc);
    if (!known) return fail(GDWS_ERR_INVALID_ARG, "gdws_measure_code_size: body must be 128, 512, 1024, 2048, 3072, 4096, 6144 or 8192 instructions");
    if (e != cudaSuccess) return cuda_fail(e, "gdws_measure_code_size");
    if (instructions_per_clk_per_scheduler)
        *instructions_per_clk_per_scheduler = worst > 0 ? (double)total * (threads / 32) / 4.0 / (double)worst : 0.0;
    return GDWS_OK;
}

gdws_status_t gdws_selftest_wait(gdws_plan_t *p, unsigned int polls, void *stream)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_selftest_wait: plan is NULL");
    if (polls > (1u << 16)) return fail(GDWS_ERR_INVALID_ARG, "gdws_selftest_wait: at most 65536 polls");
    if (p->device < 0) return fail(GDWS_ERR_INVALID_ARG, "gdws_selftest_wait: the plan has no device tables");
    gdws_status_t st = check_arch();
    if (st != GDWS_OK) return st;
    int dev = -1;
    cudaGetDevice(&dev);
    if (dev != p->device) return fail(GDWS_ERR_INVALID_ARG, "plan lives on device %d but device %d is current", p->device, dev);
    wait_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(p->d_status, polls);
    p->launches++;
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "wait_selftest_kernel launch");
}

}  // extern "C"
