// Fused GDWS forward for bf16 NHWC tensors on sm_100a: the G intermediate channels of the GDW
// stage go from the ALUs to the tensor cores through shared memory and never reach HBM.
//
// The kernel is persistent: one block per SM walks over tiles of 128 output pixels (TN images x
// PH x PW patch, all D output channels).  Within a tile the intermediate channels are processed
// in K chunks of 64 (i = 64q .. 64q+63, canonical order i = off_c + j).  Five kinds of warps run
// as one pipeline over the sequence of (tile, chunk) pairs, coupled only by mbarriers:
//   * 8 staging warps: chunk q reads the contiguous channel range [c0(q), c0(q)+span); the warps
//     load those channels of the tile's input patch (with halo, zero filled outside the image)
//     with 16-byte loads and write them channel-major into one of `nslots` slots, so that the
//     depthwise stage reads runs of consecutive pixels of one channel with 16-byte loads;
//   * 8 depthwise warps: thread t owns intermediate channel 64q + (t & 63) and a quarter of the
//     tile's pixels; it keeps its k x k filter in registers, slides down the patch reusing each
//     input row for up to k output rows, and writes bf16 results as 16-byte pieces into a
//     pixel-contiguous (MN-major), 128-byte-swizzled tensor-core operand stage;
//   * 2 control threads: one streams the pre-swizzled pointwise weights (bulk copies with mbarrier
//     completion, a ring of units of at most 256 output channels x 64), the other issues
//     tcgen05.mma into a TMEM accumulator (128 lanes x D fp32 columns; two accumulators when
//     D <= 256, so that a tile's epilogue overlaps the next tile's main loop);
//   * 4 epilogue warps: read the finished accumulator (tcgen05.ld), add the bias, apply the
//     optional ReLU, round to bf16 and store y.
// Every wait is bounded; a wait that runs out raises a block-wide abort flag that turns all later
// waits into no-ops, so the block still reaches its teardown, frees TMEM and ends.
#include "sm100.cuh"

namespace gdws {

struct FusedParams {
    const uint16_t *x;
    uint16_t *y;
    const uint32_t *dwpack;
    const uint16_t *pw_img;
    const float *bias;
    const int32_t *chan;
    const int32_t *chunk_c0;
    int *status;
    int N, H, W, C, Ho, Wo, D, Dpad, G, nchunks, stride, pad, relu;
    int TN, PH, PW, tiles_h, tiles_w, ntiles;
    int IH, IW, IWp, plane, span, nslots, nsb, wstride;
    int nhalf, unit_bytes, nacc, acc_cols;
    int a_kmajor, dw_math;
};

// Warp roles, in warpgroups of 4 so that registers can be moved between the roles (setmaxnreg):
// warps 0-7 depthwise, 8-15 staging, 16 MMA issue, 17 weight loader (18-19 idle), 20-23 epilogue.
constexpr int kDwWarps = 8, kStageWarps = 8, kEpiWarps = 4;
constexpr int kDwThreads = kDwWarps * 32;
constexpr int kCtrlWarp = kDwWarps + kStageWarps;
constexpr int kEpiWarp0 = kCtrlWarp + 4;
constexpr int kFusedThreads = (kEpiWarp0 + kEpiWarps) * 32;
// Registers per thread after the split.  setmaxnreg.inc can only claim what other warpgroups of the
// same block released, so the sum must stay within the block's allocation at launch
// (768 threads x 80 registers, the most that one block of this size can get).
constexpr int kRegsLaunch = 80, kRegsDw = 112, kRegsStage = 80, kRegsCtrl = 40, kRegsEpi = 56;
static_assert(kDwThreads * kRegsDw + kStageWarps * 32 * kRegsStage + 128 * kRegsCtrl + kEpiWarps * 32 * kRegsEpi <=
                  kFusedThreads * kRegsLaunch,
              "register split exceeds the block's allocation: setmaxnreg.inc would wait forever");

// Barrier traffic is per warp, not per thread: one lane waits or arrives for its warp.
__device__ __forceinline__ void warp_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if ((threadIdx.x & 31) == 0) mbar_wait(bar, parity, abort_flag, status, code);
    __syncwarp();
}
__device__ __forceinline__ void warp_arrive(uint32_t bar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

template <int N> __device__ __forceinline__ void regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
constexpr int kMaxSlots = 8, kMaxBUnits = 8;

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint16_t lds16(uint32_t addr)
{
    uint16_t v;
    asm volatile("ld.shared.b16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

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
__device__ __forceinline__ void store_group(const FusedParams &P, uint32_t a_stage, int o, int kk, const float (&v)[8])
{
    if (!P.a_kmajor) {
        uint4 q;
        q.x = pack_bf16x2(v[0], v[1]); q.y = pack_bf16x2(v[2], v[3]);
        q.z = pack_bf16x2(v[4], v[5]); q.w = pack_bf16x2(v[6], v[7]);
        sts128(a_stage + a_off_mn(o, kk), q);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) sts16(a_stage + a_off_k(o * 8 + e, kk), float_to_bf16_bits(v[e]));
    }
}

// ---- depthwise, k = 3, patches at least 8 wide: a thread computes 4 consecutive output rows of one
// 8-pixel column group, reading each input row once (16-byte loads) and using it for up to 3 rows.
template <int S>
__device__ __forceinline__ void dw_rows_k3(const FusedParams &P, uint32_t xs, int cl, const float (&w)[9], int kk,
                                           int run, bool live_i, uint32_t a_stage)
{
    const int nseg = P.PW >> 3;
    const int seg = run % nseg;
    const int R0 = (run / nseg) * 4;               // first of the 4 rows (row index = tn*PH + ph)
    const int o0 = R0 * nseg + seg;
    float acc[4][8];
#pragma unroll
    for (int ro = 0; ro < 4; ++ro)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[ro][e] = 0.f;
    if (live_i && R0 < P.TN * P.PH) {
        const int tn = R0 / P.PH, ph0 = R0 - tn * P.PH;
        const uint32_t rowb = (uint32_t)P.IWp * 2;
        const uint32_t base = xs + (uint32_t)(cl * P.plane + (tn * P.IH + ph0 * S) * P.IWp + seg * 8 * S) * 2;
        constexpr int NR = 3 * S + 3;              // input rows feeding 4 output rows
        constexpr int NX = 7 * S + 3;              // input columns feeding 8 output columns
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            float xr[NX + 1];
            const uint4 a = lds128(base + r * rowb);
            xr[0] = bf_lo(a.x); xr[1] = bf_hi(a.x); xr[2] = bf_lo(a.y); xr[3] = bf_hi(a.y);
            xr[4] = bf_lo(a.z); xr[5] = bf_hi(a.z); xr[6] = bf_lo(a.w); xr[7] = bf_hi(a.w);
            if (S == 1) {
                const uint32_t b = lds32(base + r * rowb + 16);
                xr[8] = bf_lo(b); xr[9] = bf_hi(b);
            } else {
                const uint4 b = lds128(base + r * rowb + 16);
                const uint32_t c = lds32(base + r * rowb + 32);
                xr[8] = bf_lo(b.x); xr[9] = bf_hi(b.x); xr[10] = bf_lo(b.y); xr[11] = bf_hi(b.y);
                xr[12] = bf_lo(b.z); xr[13] = bf_hi(b.z); xr[14] = bf_lo(b.w); xr[15] = bf_hi(b.w);
                xr[16] = bf_lo(c);
            }
#pragma unroll
            for (int ro = 0; ro < 4; ++ro) {
                const int u = r - ro * S;
                if (u >= 0 && u < 3) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
#pragma unroll
                        for (int v = 0; v < 3; ++v) acc[ro][e] = fmaf(w[u * 3 + v], xr[e * S + v], acc[ro][e]);
                }
            }
        }
    }
#pragma unroll
    for (int ro = 0; ro < 4; ++ro) store_group(P, a_stage, o0 + ro * nseg, kk, acc[ro]);
}

// ---- depthwise, k = 3, 4-wide patches: a pixel group is 2 output rows x 4 columns of one image.
template <int S>
__device__ __forceinline__ void dw_quads_k3(const FusedParams &P, uint32_t xs, int cl, const float (&w)[9], int kk,
                                            int run, bool live_i, uint32_t a_stage)
{
    const int gpi = P.PH >> 1;                      // pixel groups per image
#pragma unroll 1
    for (int m = 0; m < 4; ++m) {
        const int o = run * 4 + m;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        const int tn = o / gpi, ph0 = (o - tn * gpi) * 2;
        if (live_i && tn < P.TN) {
            const uint32_t rowb = (uint32_t)P.IWp * 2;
            const uint32_t base = xs + (uint32_t)(cl * P.plane + (tn * P.IH + ph0 * S) * P.IWp) * 2;
            constexpr int NR = S + 3;               // input rows feeding 2 output rows
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                float xr[10];
                const uint4 a = lds128(base + r * rowb);
                xr[0] = bf_lo(a.x); xr[1] = bf_hi(a.x); xr[2] = bf_lo(a.y); xr[3] = bf_hi(a.y);
                xr[4] = bf_lo(a.z); xr[5] = bf_hi(a.z); xr[6] = bf_lo(a.w); xr[7] = bf_hi(a.w);
                if (S == 2) {
                    const uint32_t b = lds32(base + r * rowb + 16);
                    xr[8] = bf_lo(b); xr[9] = bf_hi(b);
                }
#pragma unroll
                for (int ro = 0; ro < 2; ++ro) {
                    const int u = r - ro * S;
                    if (u >= 0 && u < 3) {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
#pragma unroll
                            for (int v = 0; v < 3; ++v)
                                acc[ro * 4 + e] = fmaf(w[u * 3 + v], xr[e * S + v], acc[ro * 4 + e]);
                    }
                }
            }
        }
        store_group(P, a_stage, o, kk, acc);
    }
}

// ---- depthwise, any k and stride: one pixel group at a time, 2-byte loads.
template <int K>
__device__ __forceinline__ void dw_generic(const FusedParams &P, uint32_t xs, int cl, uint32_t wsm, int kk,
                                           int run, bool live_i, uint32_t a_stage)
{
    const int hw = P.PH * P.PW;
#pragma unroll 1
    for (int m = 0; m < 4; ++m) {
        const int o = run * 4 + m;
        float out[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = 0.f;
        const int r0 = o * 8;
        const int tn = r0 / hw;
        if (live_i && tn < P.TN) {
            const int rem = r0 - tn * hw;
            const int ph = rem / P.PW, pw0 = rem - ph * P.PW;
            const uint32_t xc = xs + (uint32_t)(cl * P.plane + tn * P.IH * P.IWp) * 2;
#pragma unroll 1
            for (int e = 0; e < 8; ++e) {
                const int phe = (P.PW >= 8) ? ph : ph + (e >> 2);
                const int pwe = (P.PW >= 8) ? pw0 + e : (e & 3);
                const uint32_t xp = xc + (uint32_t)(phe * P.stride * P.IWp + pwe * P.stride) * 2;
                float acc = 0.f;
#pragma unroll
                for (int u = 0; u < K; ++u)
#pragma unroll
                    for (int v = 0; v < K; ++v)
                        acc = fmaf(__uint_as_float(lds32(wsm + (uint32_t)(u * K + v) * 4)),
                                   bf16_bits_to_float(lds16(xp + (uint32_t)(u * P.IWp + v) * 2)), acc);
                out[e] = acc;
            }
        }
        store_group(P, a_stage, o, kk, out);
    }
}

// MODE: 0 generic, 1 row runs (k=3), 2 4-wide patches (k=3); S = stride for modes 1/2.
template <int K, int MODE, int S>
__global__ void __launch_bounds__(kFusedThreads, 1) fused_bf16_kernel(const __grid_constant__ FusedParams P)
{
    extern __shared__ uint8_t smem_raw[];
    // a_full[2] a_free[2] | b_full[8] b_free[8] | x_full[8] x_free[8] | acc_full[2] acc_free[2]
    __shared__ __align__(8) uint64_t bars[4 + 2 * kMaxBUnits + 2 * kMaxSlots + 4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_s = smem_u32(base);
    const uint32_t b_s = a_s + 2 * 16384;
    const uint32_t x_s = b_s + (uint32_t)P.nsb * P.unit_bytes;
    const uint32_t xplanes_bytes = (uint32_t)P.span * P.plane * 2;       // a slot: channel planes, then the chunk's filters
    const uint32_t slot_bytes = xplanes_bytes + (uint32_t)kChunk * P.wstride * 4;
    const uint32_t bar_afull = smem_u32(&bars[0]), bar_afree = smem_u32(&bars[2]);
    const uint32_t bar_bfull = smem_u32(&bars[4]), bar_bfree = smem_u32(&bars[4 + kMaxBUnits]);
    const uint32_t bar_xfull = smem_u32(&bars[4 + 2 * kMaxBUnits]);
    const uint32_t bar_xfree = smem_u32(&bars[4 + 2 * kMaxBUnits + kMaxSlots]);
    const uint32_t bar_accfull = smem_u32(&bars[4 + 2 * kMaxBUnits + 2 * kMaxSlots]);
    const uint32_t bar_accfree = bar_accfull + 16;
    const int npair = (P.TN * P.IH * P.IWp) >> 1;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_afull + 8 * i, kDwWarps);
            mbar_init(bar_afree + 8 * i, 1);
            mbar_init(bar_accfull + 8 * i, 1);
            mbar_init(bar_accfree + 8 * i, kEpiWarps);
        }
        for (int i = 0; i < kMaxBUnits; ++i) { mbar_init(bar_bfull + 8 * i, 1); mbar_init(bar_bfree + 8 * i, 1); }
        for (int i = 0; i < kMaxSlots; ++i) { mbar_init(bar_xfull + 8 * i, kStageWarps); mbar_init(bar_xfree + 8 * i, kDwWarps); }
        fence_mbar_init();
    }
    if (warp == kCtrlWarp) tmem_alloc(smem_u32(&tmem_slot), (uint32_t)(P.nacc * P.acc_cols));

    // Patch table (the same for every tile): for each pair of horizontally adjacent patch positions
    // the pixel offset (tn*H + ih)*W + iw relative to the tile's first input pixel, and tn, ih, iw.
    int2 *pix_tab = reinterpret_cast<int2 *>(base + (x_s - a_s) + (size_t)P.nslots * slot_bytes);
    for (int pp = tid; pp < npair; pp += kFusedThreads) {
        const int t = 2 * pp;
        const int iw = t % P.IWp;
        const int r = t / P.IWp;
        const int ih = r % P.IH, tn = r / P.IH;
        pix_tab[pp] = make_int2((tn * P.H + ih) * P.W + iw, tn | (ih << 8) | (iw << 16));
    }
    // Channel range [c0, c1] read by every K chunk.
    int2 *chunk_rng = pix_tab + npair;
    for (int q = tid; q < P.nchunks; q += kFusedThreads) {
        const int c0 = __ldg(P.chunk_c0 + q);
        const int ilast = min(P.G, (q + 1) * kChunk) - 1;
        chunk_rng[q] = make_int2(c0, q * kChunk < P.G ? __ldg(P.chan + ilast) : c0);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    const int my_tiles = (P.ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int total_chunks = my_tiles * P.nchunks;
    const int tiles_hw = P.tiles_h * P.tiles_w;

    if (warp >= kCtrlWarp && warp < kEpiWarp0) {
        regs_dec<kRegsCtrl>();
        const int units_per_tile = P.nchunks * P.nhalf;
        const int total_units = my_tiles * units_per_tile;
        const int rows0 = P.Dpad > 256 ? 256 : P.Dpad, rows1 = P.Dpad - rows0;
        if (warp == kCtrlWarp && lane == 0) {
            // ---------------- MMA issue (one thread) ----------------
            const bool a_mn = !P.a_kmajor;
            const uint64_t adesc0 = a_mn ? make_sdesc(a_s, 1024, 2048) : make_sdesc(a_s, 16, 1024);
            const uint64_t bdesc0 = make_sdesc(b_s, 16, 1024);
            const uint32_t a_step = a_mn ? (4096u >> 4) : (32u >> 4);     // descriptor advance per K step of 16
            const uint32_t idesc0 = make_idesc(rows0, a_mn), idesc1 = make_idesc(rows1 > 0 ? rows1 : 16, a_mn);
            uint32_t sa = 0, pa = 0;          // intermediate-tile stage and its phase parity
            uint32_t sb = 0, pb = 0;          // weight-ring slot and its phase parity
            for (int tl = 0; tl < my_tiles; ++tl) {
                const int buf = tl % P.nacc;
                if (tl >= P.nacc)
                    mbar_wait(bar_accfree + 8 * buf, ((tl / P.nacc) - 1) & 1, &abort_flag, P.status, kStatusWaitStage);
                tc_fence_after();
                for (int q = 0; q < P.nchunks; ++q) {
                    mbar_wait(bar_afull + 8 * sa, pa, &abort_flag, P.status, kStatusWaitOperand);
                    const uint64_t adesc = adesc0 + (uint64_t)(sa * (16384u >> 4));
                    for (int h = 0; h < P.nhalf; ++h) {
                        mbar_wait(bar_bfull + 8 * sb, pb, &abort_flag, P.status, kStatusWaitOperand);
                        tc_fence_after();
                        const uint32_t d_tmem = tmem + (uint32_t)(buf * P.acc_cols + h * 256);
                        const uint64_t bdesc = bdesc0 + (uint64_t)(sb * ((uint32_t)P.unit_bytes >> 4));
                        const uint32_t idesc = h ? idesc1 : idesc0;
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_bf16(d_tmem, adesc + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * 2), idesc,
                                      (q == 0 && ks == 0) ? 0u : 1u);
                        umma_commit(bar_bfree + 8 * sb);
                        if (++sb == (uint32_t)P.nsb) { sb = 0; pb ^= 1; }
                    }
                    umma_commit(bar_afree + 8 * sa);
                    sa ^= 1;
                    if (sa == 0) pa ^= 1;
                }
                umma_commit(bar_accfull + 8 * buf);
            }
        } else if (warp == kCtrlWarp + 1 && lane == 0) {
            // ---------------- pointwise-weight loader (one thread): ring of nsb units ----------------
            uint32_t sb = 0, pb = 1;          // parity of the "slot free" phase awaited (first round: nothing to wait for)
            int q = 0, h = 0;
            for (int u = 0; u < total_units; ++u) {
                if (u >= P.nsb) mbar_wait(bar_bfree + 8 * sb, pb, &abort_flag, P.status, kStatusWaitStage);
                const uint32_t bytes = (uint32_t)(h ? rows1 : rows0) * 128u;
                mbar_expect_tx(bar_bfull + 8 * sb, bytes);
                bulk_g2s(b_s + sb * P.unit_bytes, P.pw_img + ((size_t)q * P.Dpad + h * 256) * kChunk, bytes,
                         bar_bfull + 8 * sb);
                if (++sb == (uint32_t)P.nsb) { sb = 0; pb ^= 1; }
                if (++h == P.nhalf) { h = 0; if (++q == P.nchunks) q = 0; }
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ---------------- epilogue warps: TMEM -> registers -> bias / ReLU -> bf16 -> global ----------------
        regs_dec<kRegsEpi>();
        const int lg = warp & 3;                          // TMEM lanes 32*lg .. 32*lg+31 belong to this warp
        const int r = lg * 32 + lane;
        const int hw = P.PH * P.PW;
        const int tn = r / hw;
        const int rem = r - tn * hw;
        const int ph = rem / P.PW, pw_ = rem - (rem / P.PW) * P.PW;
        for (int tl = 0; tl < my_tiles; ++tl) {
            int tile = (int)blockIdx.x + tl * (int)gridDim.x;
            const int bn = tile / tiles_hw;
            tile -= bn * tiles_hw;
            const int bh = tile / P.tiles_w, bw = tile - bh * P.tiles_w;
            const int n = bn * P.TN + tn, ho = bh * P.PH + ph, wo = bw * P.PW + pw_;
            const bool live = tn < P.TN && n < P.N && ho < P.Ho && wo < P.Wo;
            uint16_t *yrow = P.y + (((size_t)n * P.Ho + ho) * P.Wo + wo) * P.D;
            const int buf = tl % P.nacc;
            warp_wait(bar_accfull + 8 * buf, (tl / P.nacc) & 1, &abort_flag, P.status, kStatusWaitMma);
            tc_fence_after();
            const uint32_t t_base = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * P.acc_cols);
            for (int d0 = 0; d0 < P.Dpad; d0 += 16) {
                uint32_t acc[16];
                tmem_ld16(t_base + (uint32_t)d0, acc);
                tmem_ld_wait();
                if (live) store_row16(acc, P.bias, d0, P.D, P.relu, yrow);
            }
            tc_fence_before();
            warp_arrive(bar_accfree + 8 * buf);
        }
    } else if (warp >= kDwWarps) {
        // ---------------- staging warps: all 8 work on every chunk, software-pipelined ----------------
        // A chunk is staged in rounds of 256 x kSet pixel pairs (one channel group of 8 each).  The loads of
        // round e+1 are issued before the stores of round e, also across chunk and tile boundaries, so the
        // global-memory latency is overlapped with the shared-memory scatter of the previous round.
        if (kRegsStage < kRegsLaunch) regs_dec<kRegsStage>();
        const int st = tid - kDwThreads;                       // 0..255
        constexpr int kSet = 3;                                // pixel pairs per thread and round (6 loads)
        struct ChunkInfo {
            int gq, q, n0, hi0, wi0, c0, gr0, items, rounds;
            long long pbase;
        };
        auto chunk_info = [&](int gq, ChunkInfo &ci) {
            ci.gq = gq;
            const int tl = gq / P.nchunks;
            ci.q = gq - tl * P.nchunks;
            int tile = (int)blockIdx.x + tl * (int)gridDim.x;
            const int bn = tile / tiles_hw;
            tile -= bn * tiles_hw;
            const int bh = tile / P.tiles_w, bw = tile - bh * P.tiles_w;
            ci.n0 = bn * P.TN;
            ci.hi0 = bh * P.PH * P.stride - P.pad;
            ci.wi0 = bw * P.PW * P.stride - P.pad;
            ci.pbase = ((long long)ci.n0 * P.H + ci.hi0) * P.W + ci.wi0;
            const int2 rng = chunk_rng[ci.q];
            ci.c0 = rng.x;
            ci.gr0 = rng.x >> 3;
            ci.items = ((rng.y >> 3) - ci.gr0 + 1) * npair;    // (channel group, pixel pair), pixel pair fastest
            ci.rounds = (ci.items + kStageWarps * 32 * kSet - 1) / (kStageWarps * 32 * kSet);
        };
        uint4 va[2][kSet], vb[2][kSet];
        auto load_round = [&](const ChunkInfo &ci, int r, int set) {
#pragma unroll
            for (int m = 0; m < kSet; ++m) {
                const int t = (r * kSet + m) * (kStageWarps * 32) + st;
                va[set][m] = make_uint4(0, 0, 0, 0);
                vb[set][m] = make_uint4(0, 0, 0, 0);
                if (t < ci.items) {
                    const int gr = t / npair, pp = t - gr * npair;
                    const int2 e = pix_tab[pp];
                    const int tn = e.y & 0xff, ih = (e.y >> 8) & 0xff, iw = e.y >> 16;
                    const int hi = ci.hi0 + ih, wi = ci.wi0 + iw;
                    const bool rowok = ci.n0 + tn < P.N && hi >= 0 && hi < P.H;
                    const uint16_t *xp = P.x + (ci.pbase + e.x) * P.C + (ci.gr0 + gr) * 8;
                    if (rowok && wi >= 0 && wi < P.W && iw < P.IW) va[set][m] = __ldg(reinterpret_cast<const uint4 *>(xp));
                    if (rowok && wi + 1 >= 0 && wi + 1 < P.W && iw + 1 < P.IW)
                        vb[set][m] = __ldg(reinterpret_cast<const uint4 *>(xp + P.C));
                }
            }
        };
        auto store_round = [&](const ChunkInfo &ci, int r, int set, uint32_t xs) {
#pragma unroll
            for (int m = 0; m < kSet; ++m) {
                const int t = (r * kSet + m) * (kStageWarps * 32) + st;
                if (t < ci.items) {
                    const int gr = t / npair, pp = t - gr * npair;
                    const int cb = (ci.gr0 + gr) * 8 - ci.c0;   // slot channel of the group's first channel
                    const bool whole = cb >= 0 && cb + 8 <= P.span;
                    const uint32_t a4[4] = {va[set][m].x, va[set][m].y, va[set][m].z, va[set][m].w};
                    const uint32_t b4[4] = {vb[set][m].x, vb[set][m].y, vb[set][m].z, vb[set][m].w};
                    const uint32_t dst = xs + (uint32_t)(cb * P.plane + 2 * pp) * 2;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        // channel cb+e of the two pixels -> one 32-bit store
                        const uint32_t word = (e & 1) ? __byte_perm(a4[e >> 1], b4[e >> 1], 0x7632)
                                                      : __byte_perm(a4[e >> 1], b4[e >> 1], 0x5410);
                        if (whole || (cb + e >= 0 && cb + e < P.span)) sts32(dst + (uint32_t)(e * P.plane * 2), word);
                    }
                }
            }
        };
        if (total_chunks > 0) {
            ChunkInfo LC, SC;
            chunk_info(0, LC);
            SC = LC;
            int lr = 0, sr = 0, set = 0;
            load_round(LC, 0, 0);
            while (true) {
                // advance the load cursor and issue its loads into the other register set
                bool more = true;
                if (++lr == LC.rounds) {
                    lr = 0;
                    if (LC.gq + 1 < total_chunks) chunk_info(LC.gq + 1, LC);
                    else more = false;
                }
                if (more) {
                    if (set == 0) load_round(LC, lr, 1);
                    else load_round(LC, lr, 0);
                    if (lr == 0 && LC.q == 0 && warp == kDwWarps + 1) {
                        // first chunk of a tile: pull the rest of that tile's input patch towards L2
                        for (int pp = lane; pp < npair; pp += 32) {
                            const int2 e = pix_tab[pp];
                            const int tn = e.y & 0xff, ih = (e.y >> 8) & 0xff, iw = e.y >> 16;
                            const int hi = LC.hi0 + ih, wi = LC.wi0 + iw;
                            if (LC.n0 + tn < P.N && hi >= 0 && hi < P.H && wi >= 0 && wi + 1 < P.W && iw + 1 < P.IW) {
                                const char *px = reinterpret_cast<const char *>(P.x + (LC.pbase + e.x) * P.C);
                                for (int bb = 0; bb < P.C * 4; bb += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(px + bb));
                            }
                        }
                    }
                }
                // store the round loaded one step earlier
                const int slot = SC.gq % P.nslots;
                const uint32_t xs = x_s + slot * slot_bytes;
                if (sr == 0) {
                    const int use = SC.gq / P.nslots;
                    if (use >= 1) warp_wait(bar_xfree + 8 * slot, (use - 1) & 1, &abort_flag, P.status, kStatusWaitStage);
                    if (st == 0) {   // the chunk's filters and slot-channel indices: one bulk copy, counted by the slot's barrier
                        const uint32_t wbytes = (uint32_t)kChunk * P.wstride * 4;
                        mbar_expect_tx_only(bar_xfull + 8 * slot, wbytes);
                        bulk_g2s(xs + xplanes_bytes, P.dwpack + (size_t)SC.q * kChunk * P.wstride, wbytes, bar_xfull + 8 * slot);
                    }
                }
                if (set == 0) store_round(SC, sr, 0, xs);
                else store_round(SC, sr, 1, xs);
                if (++sr == SC.rounds) {
                    sr = 0;
                    warp_arrive(bar_xfull + 8 * slot);
                    if (SC.gq + 1 >= total_chunks) break;
                    chunk_info(SC.gq + 1, SC);
                }
                set ^= 1;
            }
        }
    } else {
        // ---------------- depthwise warps ----------------
        regs_inc<kRegsDw>();
        const int il = tid & 63, run = tid >> 6;
        int q = 0;
        for (int gq = 0; gq < total_chunks; ++gq) {
            const int sa = gq & 1, slot = gq % P.nslots;
            const bool live_i = q * kChunk + il < P.G;
            warp_wait(bar_xfull + 8 * slot, (gq / P.nslots) & 1, &abort_flag, P.status, kStatusWaitOperand);
            const uint32_t xs = x_s + slot * slot_bytes;
            const uint32_t wsm = xs + xplanes_bytes + (uint32_t)(il * P.wstride) * 4;   // this thread's filter
            float w[9];
            int cl;
            if (MODE != 0) {
                const uint4 w0 = lds128(wsm), w1 = lds128(wsm + 16), w2 = lds128(wsm + 32);
                w[0] = __uint_as_float(w0.x); w[1] = __uint_as_float(w0.y); w[2] = __uint_as_float(w0.z);
                w[3] = __uint_as_float(w0.w); w[4] = __uint_as_float(w1.x); w[5] = __uint_as_float(w1.y);
                w[6] = __uint_as_float(w1.z); w[7] = __uint_as_float(w1.w); w[8] = __uint_as_float(w2.x);
                cl = (int)w2.y;
            } else {
                cl = (int)lds32(wsm + (uint32_t)(K * K) * 4);
            }
            if (gq >= 2) warp_wait(bar_afree + 8 * sa, ((gq >> 1) - 1) & 1, &abort_flag, P.status, kStatusWaitStage);
            const uint32_t a_stage = a_s + sa * 16384;
            if (MODE == 1) dw_rows_k3<S>(P, xs, cl, w, il, run, live_i, a_stage);
            else if (MODE == 2) dw_quads_k3<S>(P, xs, cl, w, il, run, live_i, a_stage);
            else dw_generic<K>(P, xs, cl, wsm, il, run, live_i, a_stage);
            fence_proxy_async();      // every thread: its own writes become visible to the tensor-core proxy
            warp_arrive(bar_afull + 8 * sa);
            warp_arrive(bar_xfree + 8 * slot);
            q = (q + 1 == P.nchunks) ? 0 : q + 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (warp == kCtrlWarp) tmem_dealloc(tmem, (uint32_t)(P.nacc * P.acc_cols));
}

template <int K, int MODE, int S>
static gdws_status_t launch_fused(const FusedParams &P, int device, int grid, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaSuccess;
    static bool attr_set[64] = {};
    if (!attr_set[device & 63]) {   // once per device: allow the full dynamic shared memory
        e = cudaFuncSetAttribute(fused_bf16_kernel<K, MODE, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(fused_bf16_kernel)");
        attr_set[device & 63] = true;
    }
    fused_bf16_kernel<K, MODE, S><<<grid, kFusedThreads, smem, st>>>(P);
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
    if ((long long)x->n * x->h * x->w > 0x7fffffffLL) return fail(GDWS_ERR_UNSUPPORTED, "more than 2^31 input pixels");
    if (p->sm_count <= 0) {
        cudaError_t e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute(MultiProcessorCount)");
    }
    FusedParams P;
    P.x = (const uint16_t *)x->ptr; P.y = (uint16_t *)y->ptr;
    P.dwpack = p->d_dwpack; P.pw_img = p->d_pw_img; P.bias = p->d_bias;
    P.chan = p->d_chan; P.chunk_c0 = p->d_chunk_c0; P.status = p->d_status;
    P.N = x->n; P.H = x->h; P.W = x->w; P.C = p->C; P.Ho = y->h; P.Wo = y->w; P.D = p->D; P.Dpad = p->Dpad;
    P.G = p->G; P.nchunks = p->nchunks; P.stride = p->stride; P.pad = p->pad;
    P.relu = p->opt_relu;
    P.TN = t.TN; P.PH = t.PH; P.PW = t.PW; P.tiles_h = t.tiles_h; P.tiles_w = t.tiles_w; P.ntiles = (int)t.tiles();
    P.IH = t.IH; P.IW = t.IW; P.IWp = t.IWp; P.plane = t.plane; P.span = t.span; P.nslots = t.nslots; P.nsb = t.nsb; P.wstride = p->wstride;
    P.nhalf = p->Dpad > 256 ? 2 : 1;
    P.unit_bytes = (p->Dpad > 256 ? 256 : p->Dpad) * kChunk * 2;
    P.acc_cols = tmem_cols_for(p->Dpad);
    P.nacc = P.acc_cols <= 256 ? 2 : 1;
    P.a_kmajor = p->opt_a_layout;
    P.dw_math = p->opt_dw_math;
    const size_t smem = t.smem;     // one block per SM (register file), so the TMEM columns are never oversubscribed
    const int grid = P.ntiles < p->sm_count ? P.ntiles : p->sm_count;
    gdws_status_t rc;
    if (t.fast == 1 && p->stride == 1) rc = launch_fused<3, 1, 1>(P, p->device, grid, smem, st);
    else if (t.fast == 1 && p->stride == 2) rc = launch_fused<3, 1, 2>(P, p->device, grid, smem, st);
    else if (t.fast == 2 && p->stride == 1) rc = launch_fused<3, 2, 1>(P, p->device, grid, smem, st);
    else if (t.fast == 2 && p->stride == 2) rc = launch_fused<3, 2, 2>(P, p->device, grid, smem, st);
    else {
        switch (p->k) {
        case 1: rc = launch_fused<1, 0, 1>(P, p->device, grid, smem, st); break;
        case 2: rc = launch_fused<2, 0, 1>(P, p->device, grid, smem, st); break;
        case 3: rc = launch_fused<3, 0, 1>(P, p->device, grid, smem, st); break;
        case 4: rc = launch_fused<4, 0, 1>(P, p->device, grid, smem, st); break;
        case 5: rc = launch_fused<5, 0, 1>(P, p->device, grid, smem, st); break;
        case 6: rc = launch_fused<6, 0, 1>(P, p->device, grid, smem, st); break;
        case 7: rc = launch_fused<7, 0, 1>(P, p->device, grid, smem, st); break;
        default: return fail(GDWS_ERR_UNSUPPORTED, "k=%d", p->k);
        }
    }
    if (rc == GDWS_OK) p->launches++;
    return rc;
}

}  // namespace gdws
