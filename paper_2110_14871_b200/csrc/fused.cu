// Fused GDWS forward for bf16 NHWC tensors on sm_100a: the G intermediate channels of the GDW
// stage go from the ALUs to the tensor cores through shared memory and never reach HBM.
//
// The kernel is persistent: one block per SM walks over tiles of 128 output pixels (TN images x
// PH x PW patch, all D output channels).  Within a tile the intermediate channels are processed
// in K chunks of 64 (i = 64q .. 64q+63, canonical order i = off_c + j).  The warps form one
// pipeline over the sequence of (tile, chunk) pairs, coupled only by mbarriers:
//   * input loader (one thread): chunk q reads a contiguous range of input channels, and
//     consecutive chunks whose ranges fit into one box of `cbox` channels share it; one TMA
//     tiled load per box (x seen as a rank-4 tensor C x W x H x N, box = channels x patch with
//     halo, out-of-image positions filled with zeros) brings those channels of the tile's input
//     patch into one of `nslots` shared-memory slots; one bulk copy per chunk adds its 64 filters;
//   * 16 depthwise warps in two groups that take alternate chunks: thread t of a group owns
//     intermediate channel 64q + (t & 63) and a quarter of the tile's pixels; it keeps its k x k
//     filter in registers, slides down the patch reusing each input row for up to k output rows,
//     and writes bf16 results as 16-byte pieces into one of the group's (one or two) pixel-contiguous
//     (MN-major), 128-byte-swizzled tensor-core operand stages; a finished chunk is handed over through
//     a hardware named barrier on which the depthwise threads only arrive, so that they go on to their
//     next chunk at once;
//   * weight loader (one thread): streams the pre-swizzled pointwise weights (bulk copies with
//     mbarrier completion, a ring of units of at most 256 output channels x 64);
//   * gate warp: waits for a chunk's filters, input box and free operand stage and opens the group's
//     gate barrier, so that no depthwise thread ever polls a shared-memory barrier;
//   * MMA warp: waits on the hand-over barrier chunk by chunk, and one lane issues tcgen05.mma into a
//     TMEM accumulator (128 lanes x D fp32 columns; two accumulators when D <= 256, so that a tile's
//     epilogue overlaps the next tile's main loop);
//   * 4 epilogue warps: read the finished accumulator (tcgen05.ld), add the bias, apply the
//     optional ReLU, round to bf16 and store y.
// Every wait is bounded; a wait that runs out raises a block-wide abort flag that turns all later
// waits into no-ops, so the block still reaches its teardown, frees TMEM and ends.
#include "sm100.cuh"

namespace gdws {

struct alignas(64) FusedParams {
    CUtensorMap tmap;            // x as (C, W, H, N) bf16, box (cbox, IW, IH, TN)
    CUtensorMap tmap_y;          // y as (D, Wo, Ho, N) bf16, box (64, PW, PH, TN), 128-byte swizzle (when ostage != 0)
    uint16_t *y;
    const uint32_t *dwpack;
    const uint16_t *pw_img;
    const float *bias;
    const int4 *chunk_meta;      // per chunk: {box index, flags, first channel of the box, 0}
    int *status;
    int N, H, W, C, Ho, Wo, D, Dpad, G, nchunks, stride, pad, relu;
    int TN, PH, PW, tiles_h, tiles_w, ntiles;
    uint32_t dv_thw[2], dv_tw[2];   // multiplier and shift for the divisions by tiles_h * tiles_w and by tiles_w
    int IH, IW, ps, nslots, nwslots, nboxes, nsb, wstride;
    int spg_shift;                 // log2 of the operand stages per depthwise group (0 or 1)
    int ostage;                    // bytes of output staging (0: the epilogue stores rows directly)
    int nsplit;                    // blocks per tile: each takes Dpad of the Dtot output channels (D, Dpad: one block's share)
    int Dtot, Dpad_tot;            // output channels of the layer (row pitch of y), rows per chunk of the packed pointwise matrix
    int box_bytes, slot_bytes;
    int nhalf, unit_bytes, nacc, acc_cols;
    int a_kmajor, zout;
};

// Warp roles, in warpgroups of 4 so that registers can be moved between the roles (setmaxnreg):
// warp 0 MMA issue, 1 weight loader, 2 input loader, 3 gate, 4-19 depthwise (two groups of 8),
// 20-23 epilogue.  The control warps come first: the schedulers favour a block's oldest warps, and a
// control lane that has to queue behind the depthwise warps' instruction streams stalls the pipeline.
constexpr int kDwWarps = 16, kDwGroupWarps = 8, kEpiWarps = 4;
constexpr int kDwThreads = kDwWarps * 32;
constexpr int kCtrlWarp = 0;
constexpr int kDwWarp0 = kCtrlWarp + 4;
constexpr int kEpiWarp0 = kDwWarp0 + kDwWarps;
constexpr int kFusedThreads = (kEpiWarp0 + kEpiWarps) * 32;
// Registers per thread after the split.  setmaxnreg.inc can only claim what other warpgroups of the
// same block released, so the sum must stay within the block's allocation at launch
// (768 threads x 80 registers, the most that one block of this size can get).
constexpr int kRegsLaunch = 80, kRegsDw = 96, kRegsCtrl = 40, kRegsEpi = 56;
static_assert(kDwThreads * kRegsDw + 128 * kRegsCtrl + kEpiWarps * 32 * kRegsEpi <= kFusedThreads * kRegsLaunch,
              "register split exceeds the block's allocation: setmaxnreg.inc would wait forever");
constexpr int kMaxSlots = 8, kMaxBUnits = 8;
constexpr int kTailShare = 1 + kDwWarps / 4;   // warps per TMEM lane quarter that share the last tile's epilogue
constexpr int kPollNs = 1000;        // longest suspension of one poll by a waiter that runs ahead of the pipeline
constexpr int kBarChunk0 = 5;       // named barriers 5..8: hand-over of a finished chunk
constexpr int kBarEpi = 9;          // named barrier 9: the epilogue warps around the output staging buffer

// Barrier traffic is per warp, not per thread: one lane waits or arrives for its warp.
__device__ __forceinline__ void warp_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if ((threadIdx.x & 31) == 0) mbar_wait_relaxed<kPollNs>(bar, parity, abort_flag, status, code);
    __syncwarp();
}
__device__ __forceinline__ void warp_arrive(uint32_t bar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

// n / d for n < 2^31 as a multiplication: md = (ceil(2^(31+s) / d), 31 + s) with s = ceil(log2 d) is exact in that range
// (a division by a run-time value is some fifty instructions; a tile's coordinates need two of them).
__device__ __forceinline__ int fdiv31(int n, const uint32_t (&md)[2]) { return (int)(((uint64_t)(uint32_t)n * md[0]) >> md[1]); }

template <int N> __device__ __forceinline__ void regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

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
// One bf16 element of the staged input, as loaded: the 16 bits sit in the low half of the register.
__device__ __forceinline__ uint32_t lds_bf16(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
// The depthwise multiply-add.  Filter taps are kept as fp32 words whose value is a bf16 (low half zero) and
// inputs as loaded (bf16 in the low half): the mixed-precision FMA of sm_100 takes the two bf16 halves as they
// are and accumulates in fp32 with one rounding, which is the fp32 FMA of the widened values without the
// widening instruction (a shift per input on the 16-lane integer pipe, which holds the issue port for two
// cycles: measured, a third of the depthwise warps' time).
__device__ __forceinline__ float fma_bf(uint32_t w, uint32_t x, float acc)
{
    asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %1;\n\t"
        "mov.b32 {xl, xh}, %2;\n\t"
        "fma.rn.f32.bf16 %0, wh, xl, %0;\n\t}"
        : "+f"(acc) : "r"(w), "r"(x));
    return acc;
}
// The first tap starts the sum: w * x + 0.
__device__ __forceinline__ float mul_bf(uint32_t w, uint32_t x)
{
    float r;
    asm("{\n\t.reg .b16 wl, wh, xl, xh;\n\t"
        "mov.b32 {wl, wh}, %1;\n\t"
        "mov.b32 {xl, xh}, %2;\n\t"
        "fma.rn.f32.bf16 %0, wh, xl, 0f00000000;\n\t}"
        : "=f"(r) : "r"(w), "r"(x));
    return r;
}

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

// The staged input of a slot is the TMA box as it lies in x: [tn][ih][iw][channel], PS bytes per
// pixel.  Lanes of a warp read different channels of the same pixel, i.e. one or two 32-byte
// sectors: a single shared-memory wavefront per load.

// What a depthwise thread needs to know about its share of a tile; none of it changes from chunk to
// chunk, so it is worked out once per kernel.  The thread owns up to four pixel groups (8 pixels each):
// `in_off[m]` is where group m's input window starts inside a staged box (bytes, channel 0), `st_off[m]`
// where its results go inside an operand stage, and bit m of `live` says whether the group has pixels.
// In a pixel-contiguous stage a group's 8 results are one 16-byte piece at st_off[m]; in a channel-contiguous
// stage (KMAJOR, the unfused GDW kernel) they are 8 two-byte elements in 8 consecutive 128-byte rows, each
// in the 16-byte piece (kk/8) ^ (row & 7), and st_off[m] is the address of the first row's unswizzled piece 0.
struct DwShare {
    uint32_t in_off[4];
    uint32_t st_off[4];
    uint32_t rowb;              // bytes per input row of the staged box
    uint32_t live;
    uint32_t kg4;               // KMAJOR: 16 * (kk / 8)
};
template <bool KMAJOR>
__device__ __forceinline__ uint32_t dw_st_off(int o, int kk)
{
    return KMAJOR ? (uint32_t)(o * 1024 + (kk & 7) * 2) : a_off_mn(o, kk);
}
template <bool KMAJOR>
__device__ __forceinline__ void store_group_at(uint32_t addr, uint32_t kg4, const float (&v)[8])
{
    if (!KMAJOR) {
        uint4 q;
        q.x = pack_bf16x2(v[0], v[1]); q.y = pack_bf16x2(v[2], v[3]);
        q.z = pack_bf16x2(v[4], v[5]); q.w = pack_bf16x2(v[6], v[7]);
        sts128(addr, q);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) sts16(addr + (uint32_t)(e * 128) + (kg4 ^ (uint32_t)(e << 4)), float_to_bf16_bits(v[e]));
    }
}

// ---- depthwise, k = 3 or 5, patches at least 8 wide: a thread computes 4 consecutive output rows of one
// 8-pixel column group (its four pixel groups), reading each input row once and using it for up to K
// output rows.
template <int S, int PS, bool KMAJOR>
__device__ __forceinline__ DwShare dw_rows_share(const FusedParams &P, int kk, int run)
{
    DwShare sh;
    const int nseg = P.PW >> 3;
    const int seg = run % nseg;
    const int R0 = (run / nseg) * 4;               // first of the 4 rows (row index = tn*PH + ph)
    const int o0 = R0 * nseg + seg;
    const int tn = R0 / P.PH, ph0 = R0 - tn * P.PH;
    sh.rowb = (uint32_t)P.IW * PS;
    sh.live = R0 < P.TN * P.PH ? 1u : 0u;
    sh.in_off[0] = (uint32_t)((tn * P.IH + ph0 * S) * P.IW + seg * 8 * S) * PS;
#pragma unroll
    for (int ro = 0; ro < 4; ++ro) sh.st_off[ro] = dw_st_off<KMAJOR>(o0 + ro * nseg, kk);
    sh.kg4 = (uint32_t)(kk >> 3) << 4;
    return sh;
}
template <int K, int S, int PS, bool KMAJOR>
__device__ __forceinline__ void dw_rows(const DwShare &sh, uint32_t xs, int clb, const uint32_t (&w)[K * K], bool live_i,
                                        uint32_t a_stage)
{
    float acc[4][8];
    if (live_i && sh.live) {
        const uint32_t base = xs + sh.in_off[0] + (uint32_t)clb * 2;
        constexpr int NR = 3 * S + K;
        constexpr int NX = 7 * S + K;
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            uint32_t xr[NX];
#pragma unroll
            for (int j = 0; j < NX; ++j) xr[j] = lds_bf16(base + r * sh.rowb + j * PS);
#pragma unroll
            for (int ro = 0; ro < 4; ++ro) {
                const int u = r - ro * S;
                if (u >= 0 && u < K) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        // the first tap starts the sum
                        float a = u == 0 ? mul_bf(w[0], xr[e * S]) : fma_bf(w[u * K], xr[e * S], acc[ro][e]);
#pragma unroll
                        for (int v = 1; v < K; ++v) a = fma_bf(w[u * K + v], xr[e * S + v], a);
                        acc[ro][e] = a;
                    }
                }
            }
        }
    } else {
#pragma unroll
        for (int ro = 0; ro < 4; ++ro)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[ro][e] = 0.f;
    }
#pragma unroll
    for (int ro = 0; ro < 4; ++ro) store_group_at<KMAJOR>(a_stage + sh.st_off[ro], sh.kg4, acc[ro]);
}

// ---- depthwise, k = 3, 4-wide patches: a pixel group is 2 output rows x 4 columns of one image.
template <int S, int PS, bool KMAJOR>
__device__ __forceinline__ DwShare dw_quads_share(const FusedParams &P, int kk, int run)
{
    DwShare sh;
    const int gpi = P.PH >> 1;                      // pixel groups per image
    sh.rowb = (uint32_t)P.IW * PS;
    sh.live = 0;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        const int o = run * 4 + m;
        const int tn = o / gpi, ph0 = (o - tn * gpi) * 2;
        if (tn < P.TN) sh.live |= 1u << m;
        sh.in_off[m] = (uint32_t)((tn * P.IH + ph0 * S) * P.IW) * PS;
        sh.st_off[m] = dw_st_off<KMAJOR>(o, kk);
    }
    sh.kg4 = (uint32_t)(kk >> 3) << 4;
    return sh;
}
template <int S, int PS, bool KMAJOR>
__device__ __forceinline__ void dw_quads_k3(const DwShare &sh, uint32_t xs, int clb, const uint32_t (&w)[9], bool live_i,
                                            uint32_t a_stage)
{
#pragma unroll
    for (int m = 0; m < 4; ++m) {
        float acc[8];
        if (live_i && ((sh.live >> m) & 1u)) {
            const uint32_t base = xs + sh.in_off[m] + (uint32_t)clb * 2;
            constexpr int NR = S + 3;               // input rows feeding 2 output rows
            constexpr int NX = 3 * S + 3;           // input columns feeding 4 output columns
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                uint32_t xr[NX];
#pragma unroll
                for (int j = 0; j < NX; ++j) xr[j] = lds_bf16(base + r * sh.rowb + j * PS);
#pragma unroll
                for (int ro = 0; ro < 2; ++ro) {
                    const int u = r - ro * S;
                    if (u >= 0 && u < 3) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float a = u == 0 ? mul_bf(w[0], xr[e * S]) : fma_bf(w[u * 3], xr[e * S], acc[ro * 4 + e]);
                            a = fma_bf(w[u * 3 + 1], xr[e * S + 1], a);
                            acc[ro * 4 + e] = fma_bf(w[u * 3 + 2], xr[e * S + 2], a);
                        }
                    }
                }
            }
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        }
        store_group_at<KMAJOR>(a_stage + sh.st_off[m], sh.kg4, acc);
    }
}

// ---- depthwise, any k and stride: one pixel group at a time.
template <int K>
__device__ __forceinline__ void dw_generic(const FusedParams &P, uint32_t xs, int clb, uint32_t wsm, int kk,
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
            const uint32_t xc = xs + (uint32_t)(tn * P.IH * P.IW) * P.ps + (uint32_t)clb * 2;
#pragma unroll 1
            for (int e = 0; e < 8; ++e) {
                const int phe = (P.PW >= 8) ? ph : ph + (e >> 2);
                const int pwe = (P.PW >= 8) ? pw0 + e : (e & 3);
                const uint32_t xp = xc + (uint32_t)(phe * P.stride * P.IW + pwe * P.stride) * P.ps;
                float acc = 0.f;
#pragma unroll
                for (int u = 0; u < K; ++u)
#pragma unroll
                    for (int v = 0; v < K; ++v)
                        acc = fma_bf(lds32(wsm + (uint32_t)(u * K + v) * 4), lds_bf16(xp + (uint32_t)(u * P.IW + v) * P.ps), acc);
                out[e] = acc;
            }
        }
        store_group(P, a_stage, o, kk, out);
    }
}

// Epilogue of one thread's accumulator row with direct stores: the 16-column granules first, first + step, ...
// go from TMEM through bias / ReLU / bf16 rounding to y.
__device__ __forceinline__ void epilogue_row(const FusedParams &P, uint32_t t_base, uint32_t bias_s, size_t yrow, bool live,
                                             int first, int step)
{
    const int ngran = P.Dpad >> 4;
    for (int j = first; j < ngran; j += step) {
        uint32_t acc[16];
        tmem_ld16(t_base + (uint32_t)(j * 16), acc);
        tmem_ld_wait();
        if (live) {
            float bv[16];
            bias16_shared(bias_s + (uint32_t)j * 64, bv);
            if (P.relu & kOutF32) {          // fp32 output asked for: the sums are not rounded to bf16
                finish_store_row16_f32(acc, bv, P.relu & kOutRelu, j * 16, P.D, reinterpret_cast<float *>(P.y) + yrow);
            } else {
                uint32_t o[8];
                finish_row16(acc, bv, P.relu & kOutRelu, o);
                store_packed16(o, j * 16, P.D, P.y + yrow);
            }
        }
    }
}

// MODE: 0 generic, 1 row runs (k=3), 2 4-wide patches (k=3); S = stride and PS = bytes per staged
// pixel for modes 1/2 (mode 0 reads both from the parameters).
// ZOUT = true turns the kernel into the unfused GDW stage: the depthwise warps write channel-contiguous
// stages and the four "epilogue" warps copy each finished stage to z[pixel][Gpad] in global memory
// (16-byte stores, 128 contiguous bytes per pixel and chunk); no weights are streamed, no MMA is issued
// and no TMEM is used.  P.y then points to z and P.D holds Gpad.
// VAR: 0 the fused kernel, 1 ZOUT, 2 the fused kernel with several blocks per tile (P.nsplit > 1).
template <int K, int MODE, int S, int PS, int VAR>
__global__ void __launch_bounds__(kFusedThreads, 1) fused_bf16_kernel(const __grid_constant__ FusedParams P)
{
    constexpr bool ZOUT = VAR == 1, SPLIT = VAR == 2;
    extern __shared__ uint8_t smem_raw[];
    // a_free[4] | b_full[8] b_free[8] | x_full[8] x_free[8] | acc_full[2] acc_free[2] | w_full[8] w_free[8] | open[4] | drain
    __shared__ __align__(8) uint64_t bars[4 + 2 * kMaxBUnits + 2 * kMaxSlots + 4 + 2 * kMaxSlots + 4 + 1];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ uint32_t xinfo[kMaxSlots];      // per filter-ring slot: input slot (bits 0-7) and phase parity (bit 8) of the chunk's box
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int *const vabort = &abort_flag;
    // With few tiles, nsplit blocks share a tile: each does the whole depthwise stage and its share of the output channels.
    // (worked out where it is needed, not kept in registers through the depthwise loop)
#define GDWS_BLOCK_SHARE                                                                                     \
    const int part = SPLIT ? (int)blockIdx.x % P.nsplit : 0, bid = SPLIT ? (int)blockIdx.x / P.nsplit : (int)blockIdx.x, \
              nblocks = SPLIT ? (int)gridDim.x / P.nsplit : (int)gridDim.x;                                 \
    (void)part; (void)bid; (void)nblocks
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_s = smem_u32(base);
    const uint32_t o_s = a_s + (32768u << P.spg_shift);   // after the one or two operand stages per depthwise group: output staging
    const uint32_t b_s = o_s + (uint32_t)P.ostage;
    const uint32_t x_s = b_s + (uint32_t)P.nsb * P.unit_bytes;
    const uint32_t bar_afree = smem_u32(&bars[0]);
    const uint32_t bar_bfull = smem_u32(&bars[4]), bar_bfree = smem_u32(&bars[4 + kMaxBUnits]);
    const uint32_t bar_xfull = smem_u32(&bars[4 + 2 * kMaxBUnits]);
    const uint32_t bar_xfree = smem_u32(&bars[4 + 2 * kMaxBUnits + kMaxSlots]);
    const uint32_t bar_accfull = smem_u32(&bars[4 + 2 * kMaxBUnits + 2 * kMaxSlots]);
    const uint32_t bar_accfree = bar_accfull + 16;
    const uint32_t bar_wfull = bar_accfull + 32, bar_wfree = bar_wfull + 8 * kMaxSlots;
    const uint32_t bar_open = bar_wfree + 8 * kMaxSlots;       // a group's next chunk may start (two per group, alternating)
    const uint32_t bar_drain = bar_open + 32;                  // the MMA warp's last commit, awaited before TMEM is freed
    const uint32_t wblock = (uint32_t)kChunk * P.wstride * 4;             // one chunk's filters
    const uint32_t w_s = x_s + (uint32_t)P.nslots * P.slot_bytes;         // ring of nwslots filter blocks
    int4 *meta_tab = reinterpret_cast<int4 *>(base + (w_s - a_s) + (size_t)P.nwslots * wblock);

    grid_launch_dependents();      // the next kernel in the stream may start its prologue as SMs become free
    if (tid == 0) abort_flag = 0;
    {
        // Eight threads of warp 1 initialise the barriers, one ring slot each (warp 0 allocates tensor memory meanwhile).
        static_assert(kMaxBUnits == 8 && kMaxSlots == 8, "one ring slot per initialising thread");
        const int i = tid - 32;
        if (i >= 0 && i < 8) {
            if (i < 4) {
                mbar_init(bar_afree + 8 * i, ZOUT ? kEpiWarps : 1);
                mbar_init(bar_open + 8 * i, 1);
            }
            if (i < 2) {
                mbar_init(bar_accfull + 8 * i, 1);
                mbar_init(bar_accfree + 8 * i, kEpiWarps);
            }
            if (i == 0) mbar_init(bar_drain, 1);
            mbar_init(bar_bfull + 8 * i, 1); mbar_init(bar_bfree + 8 * i, 1);
            mbar_init(bar_xfull + 8 * i, 1);
            mbar_init(bar_xfree + 8 * i, 2 * kDwGroupWarps);   // the last two chunks that use a box release it, warp by warp
            mbar_init(bar_wfull + 8 * i, 1);
            mbar_init(bar_wfree + 8 * i, kDwGroupWarps);
            fence_mbar_init();
        }
    }
    if (!ZOUT && warp == kCtrlWarp) tmem_alloc(smem_u32(&tmem_slot), (uint32_t)(P.nacc * P.acc_cols));
    // up to here only this block's shared and tensor memory were touched; the kernel before this one in the stream has
    // to be complete before global memory is read or written
    grid_dependency_wait();
    for (int q = tid; q < P.nchunks; q += kFusedThreads) meta_tab[q] = __ldg(P.chunk_meta + q);
    // a copy of the bias next to the chunk table: the epilogue reads it per 16 columns, with the accumulator in hand
    float *bias_sm = reinterpret_cast<float *>(meta_tab + P.nchunks);
    const uint32_t bias_s = smem_u32(bias_sm);
    if (!ZOUT) {
        GDWS_BLOCK_SHARE;
        for (int d = tid; d < P.Dpad; d += kFusedThreads) bias_sm[d] = __ldg(P.bias + part * P.Dpad + d);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ZOUT ? 0u : tmem_slot;

    int my_tiles;
    {
        GDWS_BLOCK_SHARE;
        my_tiles = (P.ntiles - bid + nblocks - 1) / nblocks;
    }
    const int total_chunks = my_tiles * P.nchunks;
    const int tiles_hw = P.tiles_h * P.tiles_w;

    if (warp < kDwWarp0) {
        regs_dec<kRegsCtrl>();
        const int units_per_tile = P.nchunks * P.nhalf;
        const int total_units = my_tiles * units_per_tile;
        const int rows0 = P.Dpad > 256 ? 256 : P.Dpad, rows1 = P.Dpad - rows0;
        if (!ZOUT && warp == kCtrlWarp) {
            // ---------------- MMA warp ----------------
            // All 32 lanes wait for the weights and at the chunk's hand-over barrier; one elected lane then issues the
            // chunk's MMAs and commits.  Its per-chunk instruction stream is kept as short as possible (32-bit
            // descriptor words, no table lookups): the pipeline cannot run faster than this one lane.
            const bool a_mn = !P.a_kmajor;
            const uint64_t adesc0 = a_mn ? make_sdesc(a_s, 1024, 2048) : make_sdesc(a_s, 16, 1024);
            const uint64_t bdesc0 = make_sdesc(b_s, 16, 1024);
            const uint32_t a_lo0 = (uint32_t)adesc0, a_hi = (uint32_t)(adesc0 >> 32);
            const uint32_t b_lo0 = (uint32_t)bdesc0, b_hi = (uint32_t)(bdesc0 >> 32);
            const uint32_t a_step = a_mn ? (4096u >> 4) : (32u >> 4);     // descriptor advance per K step of 16
            const uint32_t b_unit = (uint32_t)P.unit_bytes >> 4;
            const uint32_t idesc0 = make_idesc(rows0, a_mn), idesc1 = make_idesc(rows1 > 0 ? rows1 : 16, a_mn);
            const uint32_t spg_mask = (1u << P.spg_shift) - 1u;
            uint32_t sb = 0, pb = 0;          // weight-ring slot and its phase parity
            uint32_t gq = 0;
            int buf = 0;
            uint32_t accuse = 0;              // accumulator of the tile in turn, and how often it has been used
            for (int tl = 0; tl < my_tiles; ++tl, buf = (buf + 1 == P.nacc ? 0 : buf + 1), accuse += (buf == 0)) {
                const uint32_t d_tmem = tmem + (uint32_t)(buf * P.acc_cols);
                if (accuse)
                    mbar_wait_call(bar_accfree + 8 * buf, (accuse - 1u) & 1u, &abort_flag, P.status, kStatusWaitStage);
                for (int q = 0; q < P.nchunks; ++q, ++gq) {
                    // chunk gq is the (gq >> 1)-th chunk of group gq & 1, which cycles through its own stages
                    const uint32_t sa = ((gq & 1u) << P.spg_shift) + ((gq >> 1) & spg_mask);
                    const uint32_t a_lo = a_lo0 + sa * (16384u >> 4);
                    mbar_wait_call(bar_bfull + 8 * sb, pb, &abort_flag, P.status, kStatusWaitOperand);   // long there
                    named_bar_sync(kBarChunk0 + (int)(gq & 3u), kDwGroupWarps * 32 + 32);   // the group has written chunk gq
                    tc_fence_after();
                    if (elect_one()) {
                        const uint32_t b_lo = b_lo0 + sb * b_unit;
                        umma_bf16_words(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc0, q != 0);
                        umma_bf16_words(d_tmem, a_lo + a_step, a_hi, b_lo + 2, b_hi, idesc0, 1u);
                        umma_bf16_words(d_tmem, a_lo + 2 * a_step, a_hi, b_lo + 4, b_hi, idesc0, 1u);
                        umma_bf16_words(d_tmem, a_lo + 3 * a_step, a_hi, b_lo + 6, b_hi, idesc0, 1u);
                        umma_commit(bar_bfree + 8 * sb);
                    }
                    if (++sb == (uint32_t)P.nsb) { sb = 0; pb ^= 1; }
                    if (P.nhalf == 2) {       // output channels 256 and up: a second weight unit, a second set of columns
                        mbar_wait_call(bar_bfull + 8 * sb, pb, &abort_flag, P.status, kStatusWaitOperand);
                        tc_fence_after();
                        if (elect_one()) {
                            const uint32_t b_lo = b_lo0 + sb * b_unit;
                            umma_bf16_words(d_tmem + 256, a_lo, a_hi, b_lo, b_hi, idesc1, q != 0);
                            umma_bf16_words(d_tmem + 256, a_lo + a_step, a_hi, b_lo + 2, b_hi, idesc1, 1u);
                            umma_bf16_words(d_tmem + 256, a_lo + 2 * a_step, a_hi, b_lo + 4, b_hi, idesc1, 1u);
                            umma_bf16_words(d_tmem + 256, a_lo + 3 * a_step, a_hi, b_lo + 6, b_hi, idesc1, 1u);
                            umma_commit(bar_bfree + 8 * sb);
                        }
                        if (++sb == (uint32_t)P.nsb) { sb = 0; pb ^= 1; }
                    }
                    if (elect_one()) {
                        umma_commit(bar_afree + 8 * sa);
                        if (q == P.nchunks - 1) umma_commit(bar_accfull + 8 * buf);
                    }
                    __syncwarp();
                }
            }
            // Teardown: everything this warp issued has to be complete before the block frees its tensor memory
            // and gives back its shared memory (after an abort the waits above return at once, and products may have
            // been issued on operands that were not there: their results are undefined, but they too must have ended).
            // One more commit covers all earlier products; its wait is bounded and does not look at the abort flag.
            if (lane == 0) {
                umma_commit(bar_drain);
                mbar_wait_drain(bar_drain, 0);
            }
            __syncwarp();
        } else if (!ZOUT && warp == kCtrlWarp + 1 && lane == 0) {
            // ---------------- pointwise-weight loader (one thread): ring of nsb units ----------------
            GDWS_BLOCK_SHARE;
            uint32_t sb = 0, pb = 1;          // parity of the "slot free" phase awaited (first round: nothing to wait for)
            int q = 0, h = 0, issued = 0;
            for (int u = 0; u < total_units; ++u) {
                if (u >= P.nsb) mbar_wait_relaxed_call<kPollNs>(bar_bfree + 8 * sb, pb, &abort_flag, P.status, kStatusWaitStage);
                if (*vabort) break;                    // a wait ran out somewhere: no new copies
                ++issued;
                const uint32_t bytes = (uint32_t)(h ? rows1 : rows0) * 128u;
                mbar_expect_tx(bar_bfull + 8 * sb, bytes);
                bulk_g2s(b_s + sb * P.unit_bytes, P.pw_img + ((size_t)q * P.Dpad_tot + part * P.Dpad + h * 256) * kChunk, bytes,
                         bar_bfull + 8 * sb);
                if (++sb == (uint32_t)P.nsb) { sb = 0; pb ^= 1; }
                if (++h == P.nhalf) { h = 0; if (++q == P.nchunks) q = 0; }
            }
            // Teardown: the block's shared memory must not be given back while a copy into it is in flight.  The last
            // phase armed on each ring slot completes when its copy has landed (earlier phases completed before it).
            for (int j = 0; j < P.nsb && j < issued; ++j)
                mbar_wait_drain(bar_bfull + 8 * j, (uint32_t)((issued - 1 - j) / P.nsb) & 1u);
        } else if (warp == kCtrlWarp + 2 && lane == 0) {
            // ---------------- input loader (one thread): ring of boxes, ring of filter blocks ----------------
            GDWS_BLOCK_SHARE;
            uint32_t xslot = 0, xpar = 1;     // next box slot; parity of the "slot free" phase awaited
            uint32_t wslot = 0, wpar = 1;
            uint32_t cur_x = 0;               // slot and "full" phase parity of the box the current chunks read
            int gq = 0, gb = 0;
            bool stop = false;
            for (int tl = 0; tl < my_tiles && !stop; ++tl) {
                int tile = bid + tl * nblocks;
                const int bn = fdiv31(tile, P.dv_thw);
                tile -= bn * tiles_hw;
                const int bh = fdiv31(tile, P.dv_tw), bw = tile - bh * P.tiles_w;
                const int n0 = bn * P.TN, hi0 = bh * P.PH * P.stride - P.pad, wi0 = bw * P.PW * P.stride - P.pad;
                for (int q = 0; q < P.nchunks; ++q, ++gq) {
                    const int4 meta = meta_tab[q];
                    if (*vabort) { stop = true; break; }        // a wait ran out somewhere: no new copies
                    if (meta.y & 4) {         // first chunk of a box: fetch the box
                        if (gb >= P.nslots) mbar_wait_relaxed_call<kPollNs>(bar_xfree + 8 * xslot, xpar, &abort_flag, P.status, kStatusWaitStage);
                        mbar_expect_tx(bar_xfull + 8 * xslot, (uint32_t)P.box_bytes);
                        tma_load_4d(x_s + xslot * (uint32_t)P.slot_bytes, &P.tmap, meta.z, wi0, hi0, n0, bar_xfull + 8 * xslot);
                        cur_x = xslot | ((xpar ^ 1u) << 8);   // "full" phase parity = the opposite of the "free" parity awaited
                        ++gb;
                        if (++xslot == (uint32_t)P.nslots) { xslot = 0; xpar ^= 1; }
                    }
                    if (gq >= P.nwslots) mbar_wait_relaxed_call<kPollNs>(bar_wfree + 8 * wslot, wpar, &abort_flag, P.status, kStatusWaitStage);
                    xinfo[wslot] = cur_x;                     // published by the arrive below
                    mbar_expect_tx(bar_wfull + 8 * wslot, wblock);
                    bulk_g2s(w_s + wslot * wblock, P.dwpack + (size_t)q * kChunk * P.wstride, wblock, bar_wfull + 8 * wslot);
                    if (++wslot == (uint32_t)P.nwslots) { wslot = 0; wpar ^= 1; }
                }
            }
            // Teardown, as for the weight ring: gb boxes and gq filter blocks were requested.
            for (int j = 0; j < P.nslots && j < gb; ++j)
                mbar_wait_drain(bar_xfull + 8 * j, (uint32_t)((gb - 1 - j) / P.nslots) & 1u);
            for (int j = 0; j < P.nwslots && j < gq; ++j)
                mbar_wait_drain(bar_wfull + 8 * j, (uint32_t)((gq - 1 - j) / P.nwslots) & 1u);
        } else if (warp == kCtrlWarp + 3) {
            // ---------------- gate warp ----------------
            // Waits, chunk by chunk, until the chunk's filters and input box have landed and its operand stage
            // is free again, then completes a phase of the group's "open" barrier (two per group, alternating).
            // Each depthwise warp checks that one barrier before a chunk, on its own: the warps of a group do
            // not wait for one another.  An "open" barrier is used again two chunks of the group later; by then
            // the stage wait has shown that every warp of the group is past its earlier use.
            uint32_t wslot = 0, wpar = 0;
            uint32_t xs_cur = 0, xp_cur = 0, xs_next = 0, xp_next = 0;   // box slot and the parity of its "full" phase
            int gq = 0;
            for (int tl = 0; tl < my_tiles; ++tl) {
                for (int q = 0; q < P.nchunks; ++q, ++gq) {
                    const int flags = meta_tab[q].y;
                    const int g = gq & 1, k = gq >> 1;
                    mbar_wait_relaxed_call<kPollNs>(bar_wfull + 8 * wslot, wpar, &abort_flag, P.status, kStatusWaitOperand);
                    if (flags & 4) {
                        xs_cur = xs_next; xp_cur = xp_next;
                        if (++xs_next == (uint32_t)P.nslots) { xs_next = 0; xp_next ^= 1; }
                        mbar_wait_relaxed_call<kPollNs>(bar_xfull + 8 * xs_cur, xp_cur, &abort_flag, P.status, kStatusWaitOperand);
                    }
                    if ((k >> P.spg_shift) >= 1) {
                        const uint32_t sa = ((uint32_t)g << P.spg_shift) + ((uint32_t)k & ((1u << P.spg_shift) - 1u));
                        mbar_wait_relaxed_call<kPollNs>(bar_afree + 8 * sa, ((k >> P.spg_shift) - 1) & 1, &abort_flag, P.status, kStatusWaitStage);
                    }
                    if (lane == 0) mbar_arrive(bar_open + 8 * (2 * g + (k & 1)));
                    __syncwarp();
                    if (++wslot == (uint32_t)P.nwslots) { wslot = 0; wpar ^= 1; }
                }
            }
        }
    } else if (warp >= kEpiWarp0) {
        // ---------------- epilogue warps: TMEM -> registers -> bias / ReLU -> bf16 -> global ----------------
        GDWS_BLOCK_SHARE;
        regs_dec<kRegsEpi>();
        const int lg = warp & 3;                          // TMEM lanes 32*lg .. 32*lg+31 belong to this warp
        const int r = lg * 32 + lane;
        const int hw = P.PH * P.PW;
        const int tn = r / hw;
        const int rem = r - tn * hw;
        const int ph = rem / P.PW, pw_ = rem - (rem / P.PW) * P.PW;
        int wq = 0;                                       // ZOUT: running index of the next finished chunk
        for (int tl = 0; tl < my_tiles; ++tl) {
            int tile = bid + tl * nblocks;
            const int bn = fdiv31(tile, P.dv_thw);
            tile -= bn * tiles_hw;
            const int bh = fdiv31(tile, P.dv_tw), bw = tile - bh * P.tiles_w;
            const int n = bn * P.TN + tn, ho = bh * P.PH + ph, wo = bw * P.PW + pw_;
            const bool live = tn < P.TN && n < P.N && ho < P.Ho && wo < P.Wo;
            const size_t yrow = (((size_t)n * P.Ho + ho) * P.Wo + wo) * P.Dtot + part * P.Dpad;   // element index of the row's first channel
            if (ZOUT) {
                // this thread's pixel row of every finished stage goes to z (row r of the stage: 128 bytes, swizzled)
                for (int q = 0; q < P.nchunks; ++q, ++wq) {
                    named_bar_sync(kBarChunk0 + (wq & 3), kDwGroupWarps * 32 + kEpiWarps * 32);   // chunk wq is written
                    const uint32_t sa = ((uint32_t)(wq & 1) << P.spg_shift) + ((uint32_t)(wq >> 1) & ((1u << P.spg_shift) - 1u));
                    const uint32_t row_s = a_s + sa * 16384 + (uint32_t)r * 128;
                    uint4 v[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) v[c] = lds128(row_s + (uint32_t)((c ^ (r & 7)) << 4));
                    warp_arrive(bar_afree + 8 * sa);
                    if (live) {
                        uint4 *dst = reinterpret_cast<uint4 *>(P.y + yrow + (size_t)q * kChunk);
#pragma unroll
                        for (int c = 0; c < 8; ++c) dst[c] = v[c];
                    }
                }
                continue;
            }
            const int buf = tl & (P.nacc - 1);            // one or two accumulators
            warp_wait(bar_accfull + 8 * buf, (tl >> (P.nacc - 1)) & 1, &abort_flag, P.status, kStatusWaitMma);
            tc_fence_after();
            const uint32_t t_base = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * P.acc_cols);
            if (P.ostage) {
                // 64 output channels at a time: every thread puts its row's 128 bytes into the staging buffer
                // (rows in tile order = the order of a (64, PW, PH, TN) box of y; 16-byte pieces swizzled by
                // row), then one thread stores the box by TMA, which also clips it to the tensor.  Row-wise
                // stores from registers would touch 32 different lines per instruction.
                const bool issuer = warp == kEpiWarp0 && lane == 0;
                const uint32_t row_s = o_s + (uint32_t)r * 128;
                const int nblk = P.Dpad >> 6;
                for (int cb = 0; cb < nblk; ++cb) {
                    if (issuer) bulk_wait_read_all();          // the last box has left the staging buffer
                    named_bar_sync(kBarEpi, kEpiWarps * 32);
#pragma unroll 1
                    for (int h4 = 0; h4 < 4; ++h4) {
                        uint32_t acc[16], o[8];
                        tmem_ld16(t_base + (uint32_t)(cb * 64 + h4 * 16), acc);
                        tmem_ld_wait();
                        float bv[16];
                        bias16_shared(bias_s + (uint32_t)(cb * 64 + h4 * 16) * 4, bv);
                        finish_row16(acc, bv, P.relu & kOutRelu, o);
                        sts128(row_s + (uint32_t)(((2 * h4) ^ (r & 7)) << 4), make_uint4(o[0], o[1], o[2], o[3]));
                        sts128(row_s + (uint32_t)(((2 * h4 + 1) ^ (r & 7)) << 4), make_uint4(o[4], o[5], o[6], o[7]));
                    }
                    fence_proxy_async();
                    if (cb == nblk - 1) {                      // the accumulator has been read: the next tile may use it
                        tc_fence_before();
                        warp_arrive(bar_accfree + 8 * buf);
                    }
                    named_bar_sync(kBarEpi, kEpiWarps * 32);
                    if (issuer) {
                        tma_store_4d(o_s, &P.tmap_y, part * P.Dpad + cb * 64, bw * P.PW, bh * P.PH, bn * P.TN);
                        bulk_commit();
                    }
                }
                continue;
            }
            // the block's last tile: the depthwise warps, idle by then, take four fifths of the columns
            epilogue_row(P, t_base, bias_s, yrow, live, 0, tl == my_tiles - 1 ? kTailShare : 1);
            tc_fence_before();
            warp_arrive(bar_accfree + 8 * buf);
        }
        if (!ZOUT && P.ostage && warp == kEpiWarp0 && lane == 0) bulk_wait_all();   // the staging buffer must outlive its stores
    } else {
        // ---------------- depthwise warps: group g takes the chunks gq = g, g+2, ... ----------------
        regs_inc<kRegsDw>();
        const int dt = tid - kDwWarp0 * 32;               // index among the depthwise threads
        const int g = dt >> 8;
        const int il = dt & 63, run = (dt >> 6) & 3;
        int q = g;
        while (q >= P.nchunks) q -= P.nchunks;
        int wslot = g;
        while (wslot >= P.nwslots) wslot -= P.nwslots;
        DwShare share = {};
        if (MODE == 1) share = dw_rows_share<S, PS, ZOUT>(P, il, run);
        else if (MODE == 2) share = dw_quads_share<S, PS, ZOUT>(P, il, run);
        // A depthwise warp checks one shared-memory barrier per chunk (the group's "open" barrier, kept by the
        // gate warp), and after the chunk's arithmetic its threads arrive, without waiting, at the chunk's
        // hand-over barrier, where the consumer waits.  A hand-over barrier is used again four chunks later, by the same group
        // and for the same stage (two chunks later with one stage per group); by then the gate warp has seen
        // that stage released, hence the consumer past the barrier.
        for (int gq = g, k = 0; gq < total_chunks; gq += 2, ++k) {
            const bool live_i = q * kChunk + il < P.G;
            const uint32_t sa = ((uint32_t)g << P.spg_shift) + ((uint32_t)k & ((1u << P.spg_shift) - 1u));   // this chunk's stage
            const uint32_t a_stage = a_s + sa * 16384;
            if (lane == 0) mbar_wait(bar_open + 8 * (2 * g + (k & 1)), (k >> 1) & 1, &abort_flag, P.status, kStatusWaitOperand);
            __syncwarp();
            const uint32_t xslot = xinfo[wslot] & 0xffu;
            const uint32_t xs = x_s + xslot * (uint32_t)P.slot_bytes;
            const uint32_t wsm = w_s + wslot * wblock + (uint32_t)(il * P.wstride) * 4;   // this thread's filter
            uint32_t w[K * K];                            // taps: fp32 words holding bf16 values
            int clb;                                      // channel index inside the staged box
            if (MODE != 0) {
                constexpr int NV = (K * K + 4) / 4;       // 16-byte pieces holding the taps and the channel index
                uint32_t wv[NV * 4];
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const uint4 t = lds128(wsm + 16 * j);
                    wv[4 * j] = t.x; wv[4 * j + 1] = t.y; wv[4 * j + 2] = t.z; wv[4 * j + 3] = t.w;
                }
#pragma unroll
                for (int j = 0; j < K * K; ++j) w[j] = wv[j];
                clb = (int)wv[K * K];
            } else {
                clb = (int)lds32(wsm + (uint32_t)(K * K) * 4);
            }
            if (MODE == 1) dw_rows<K, S, PS, ZOUT>(share, xs, clb, w, live_i, a_stage);
            else if (MODE == 2) dw_quads_k3<S, PS, ZOUT>(share, xs, clb, reinterpret_cast<const uint32_t (&)[9]>(w), live_i, a_stage);
            else dw_generic<K>(P, xs, clb, wsm, il, run, live_i, a_stage);
            fence_proxy_async();      // every thread: its own writes become visible to the tensor-core proxy
            __syncwarp();
            if (lane == 0) {          // this warp is done with the chunk's filters and input box
                const int flags = meta_tab[q].y;
                mbar_arrive(bar_wfree + 8 * wslot);
                if (flags & 1) mbar_arrive(bar_xfree + 8 * xslot);
                if (flags & 2) mbar_arrive(bar_xfree + 8 * xslot);
            }
            __syncwarp();
            named_bar_arrive(kBarChunk0 + (gq & 3), kDwGroupWarps * 32 + (ZOUT ? kEpiWarps * 32 : 32));
            q += 2;
            while (q >= P.nchunks) q -= P.nchunks;
            wslot += 2;
            while (wslot >= P.nwslots) wslot -= P.nwslots;
        }
    }
    if (!ZOUT && !P.ostage && warp >= kDwWarp0 && warp < kEpiWarp0) {
        // ---------------- depthwise warps, done with their chunks: help with the last tile's epilogue ----------------
        GDWS_BLOCK_SHARE;
        // A warp reads the TMEM lanes 32 * (warp % 4) ...; the four depthwise warps and the epilogue warp of a
        // lane quarter share its columns in granules of 16.
        const int tl = my_tiles - 1;
        const int lg = warp & 3;
        const int r = lg * 32 + lane;
        const int hw = P.PH * P.PW;
        const int tn = r / hw;
        const int rem = r - tn * hw;
        const int ph = rem / P.PW, pw_ = rem - (rem / P.PW) * P.PW;
        int tile = bid + tl * nblocks;
        const int bn = fdiv31(tile, P.dv_thw);
        tile -= bn * tiles_hw;
        const int bh = fdiv31(tile, P.dv_tw), bw = tile - bh * P.tiles_w;
        const int n = bn * P.TN + tn, ho = bh * P.PH + ph, wo = bw * P.PW + pw_;
        const bool live = tn < P.TN && n < P.N && ho < P.Ho && wo < P.Wo;
        const size_t yrow = (((size_t)n * P.Ho + ho) * P.Wo + wo) * P.Dtot + part * P.Dpad;
        const int buf = tl & (P.nacc - 1);            // one or two accumulators
        warp_wait(bar_accfull + 8 * buf, (tl >> (P.nacc - 1)) & 1, &abort_flag, P.status, kStatusWaitMma);
        tc_fence_after();
        const uint32_t t_base = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * P.acc_cols);
        epilogue_row(P, t_base, bias_s, yrow, live, 1 + ((warp - kDwWarp0) >> 2), kTailShare);
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (!ZOUT && warp == kCtrlWarp) tmem_dealloc(tmem, (uint32_t)(P.nacc * P.acc_cols));
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
template <int K, int MODE, int S, int PS, int VAR>
static gdws_status_t launch_one(const FusedParams &P, int device, int grid, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaSuccess;
    static bool attr_set[64] = {};
    if (!attr_set[device & 63]) {   // once per device: allow the full dynamic shared memory
        e = cudaFuncSetAttribute(fused_bf16_kernel<K, MODE, S, PS, VAR>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(fused_bf16_kernel)");
        attr_set[device & 63] = true;
    }
    e = launch_overlapped(fused_bf16_kernel<K, MODE, S, PS, VAR>, (unsigned)grid, kFusedThreads, smem, st, P);
    return e == cudaSuccess ? GDWS_OK : cuda_fail(e, "fused_bf16_kernel launch");
}

template <int K, int MODE, int S, int PS>
static gdws_status_t launch_fused(const FusedParams &P, int device, int grid, size_t smem, cudaStream_t st)
{
    if (P.zout) return launch_one<K, MODE, S, PS, 1>(P, device, grid, smem, st);
    if (P.nsplit > 1) {
        if constexpr (K == 3 && MODE != 0) return launch_one<K, MODE, S, PS, 2>(P, device, grid, smem, st);
        else return fail(GDWS_ERR_UNSUPPORTED, "several blocks per tile: no such kernel for k=%d", K);
    }
    return launch_one<K, MODE, S, PS, 0>(P, device, grid, smem, st);
}

template <int K, int MODE, int S>
static gdws_status_t launch_fast(const FusedParams &P, int device, int grid, size_t smem, cudaStream_t st)
{
    switch (P.ps) {
    case 64: return launch_fused<K, MODE, S, 64>(P, device, grid, smem, st);
    case 128: return launch_fused<K, MODE, S, 128>(P, device, grid, smem, st);
    case 256: return launch_fused<K, MODE, S, 256>(P, device, grid, smem, st);
    default: return fail(GDWS_ERR_UNSUPPORTED, "staged pixel size %d", P.ps);
    }
}

static gdws_status_t run_tiled(gdws_plan_s *p, const gdws_tensor_t *x, void *out, int Ho, int Wo, bool zout, bool out_f32, cudaStream_t st)
{
    if (!zout && p->Dpad > 512) return fail(GDWS_ERR_UNSUPPORTED, "bf16 fused kernel supports D <= 512 (got %d)", p->D);
    if (p->D % 8 || p->C % 8)
        return fail(GDWS_ERR_UNSUPPORTED, "bf16 kernels need C %% 8 == 0 and D %% 8 == 0 (got C=%d, D=%d)", p->C, p->D);
    if (p->sm_count <= 0) {
        cudaError_t e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute(MultiProcessorCount)");
    }
    Tile t;
    if (!choose_tile(p, x->n, x->h, x->w, &t))
        return fail(GDWS_ERR_UNSUPPORTED, "no fused tile fits this shape in shared memory");
    if (t.tiles() > 0x7fffffffLL) return fail(GDWS_ERR_UNSUPPORTED, "too many tiles");
    tensor_map_encode_fn encode = encode_fn();
    if (!encode) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    FusedParams P;
    {
        // x as a rank-4 tensor, innermost first: channels, width, height, batch
        const cuuint64_t dims[4] = {(cuuint64_t)p->C, (cuuint64_t)x->w, (cuuint64_t)x->h, (cuuint64_t)x->n};
        const cuuint64_t strides[3] = {(cuuint64_t)p->C * 2, (cuuint64_t)x->w * p->C * 2,
                                       (cuuint64_t)x->h * x->w * p->C * 2};
        const cuuint32_t box[4] = {(cuuint32_t)t.cbox, (cuuint32_t)t.IW, (cuuint32_t)t.IH, (cuuint32_t)t.TN};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        const CUresult r = encode(&P.tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, x->ptr, dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    }
    // The staged epilogue pays when it overlaps the next tile's main loop; a block with a single tile would
    // only wait for its one staging buffer between the column blocks.
    const bool tma_out = !zout && !out_f32 && t.ostage && (reinterpret_cast<uintptr_t>(out) & 15) == 0 && t.tiles() > p->sm_count;
    if (tma_out) {
        // y as a rank-4 tensor, innermost first: channels, width, height, batch
        const cuuint64_t dims[4] = {(cuuint64_t)p->D, (cuuint64_t)Wo, (cuuint64_t)Ho, (cuuint64_t)x->n};
        const cuuint64_t strides[3] = {(cuuint64_t)p->D * 2, (cuuint64_t)Wo * p->D * 2, (cuuint64_t)Ho * Wo * p->D * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)t.PW, (cuuint32_t)t.PH, (cuuint32_t)t.TN};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        const CUresult r = encode(&P.tmap_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, out, dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled (y) failed with code %d", (int)r);
    } else {
        P.tmap_y = P.tmap;
    }
    P.y = (uint16_t *)out;
    P.dwpack = p->d_dwpack; P.pw_img = p->d_pw_img; P.bias = p->d_bias;
    P.chunk_meta = reinterpret_cast<const int4 *>(p->d_chunk_meta); P.status = p->d_status;
    // Few tiles and many output channels: two blocks per tile, each with half of the channels (and of the weight stream).
    const int nsplit = (!zout && t.fast && p->k == 3 && p->Dpad == p->D && p->D >= 256 && p->D % 32 == 0 && 2 * t.tiles() <= p->sm_count) ? 2 : 1;
    const int Dloc = p->Dpad / nsplit;
    P.nsplit = nsplit; P.Dtot = zout ? p->Gpad : p->D; P.Dpad_tot = p->Dpad;
    P.N = x->n; P.H = x->h; P.W = x->w; P.C = p->C; P.Ho = Ho; P.Wo = Wo; P.D = zout ? p->Gpad : (nsplit > 1 ? Dloc : p->D); P.Dpad = Dloc;
    P.G = p->G; P.nchunks = p->nchunks; P.stride = p->stride; P.pad = p->pad;
    P.relu = (p->opt_relu ? kOutRelu : 0) | (out_f32 ? kOutF32 : 0);
    P.TN = t.TN; P.PH = t.PH; P.PW = t.PW; P.tiles_h = t.tiles_h; P.tiles_w = t.tiles_w; P.ntiles = (int)t.tiles();
    {
        auto magic = [](int d, uint32_t (&md)[2]) {
            int sh = 0;
            while ((1 << sh) < d) ++sh;
            md[0] = (uint32_t)((((uint64_t)1 << (31 + sh)) + (uint64_t)d - 1) / (uint64_t)d);
            md[1] = (uint32_t)(31 + sh);
        };
        magic(t.tiles_h * t.tiles_w, P.dv_thw); magic(t.tiles_w, P.dv_tw);
    }
    P.IH = t.IH; P.IW = t.IW; P.ps = t.cbox * 2; P.nslots = t.nslots; P.nwslots = t.nwslots; P.nboxes = p->nboxes; P.nsb = t.nsb; P.wstride = p->wstride;
    P.spg_shift = t.spg == 2 ? 1 : 0;
    P.ostage = tma_out ? t.ostage : 0;
    P.box_bytes = t.box_bytes; P.slot_bytes = t.slot_bytes;
    P.nhalf = Dloc > 256 ? 2 : 1;
    P.unit_bytes = (Dloc > 256 ? 256 : Dloc) * kChunk * 2;
    P.acc_cols = tmem_cols_for(Dloc);
    P.nacc = P.acc_cols <= 256 ? 2 : 1;
    P.a_kmajor = zout ? 1 : p->opt_a_layout;
    P.zout = zout ? 1 : 0;
    const size_t smem = t.smem;     // one block per SM (register file), so the TMEM columns are never oversubscribed
    const int grid = nsplit > 1 ? P.ntiles * nsplit : (P.ntiles < p->sm_count ? P.ntiles : p->sm_count);
    const int dev = p->device;
    gdws_status_t rc;
    if (t.fast == 1 && p->k == 3 && p->stride == 1) rc = launch_fast<3, 1, 1>(P, dev, grid, smem, st);
    else if (t.fast == 1 && p->k == 3 && p->stride == 2) rc = launch_fast<3, 1, 2>(P, dev, grid, smem, st);
    else if (t.fast == 1 && p->k == 5 && p->stride == 1) rc = launch_fast<5, 1, 1>(P, dev, grid, smem, st);
    else if (t.fast == 1 && p->k == 5 && p->stride == 2) rc = launch_fast<5, 1, 2>(P, dev, grid, smem, st);
    else if (t.fast == 2 && p->stride == 1) rc = launch_fast<3, 2, 1>(P, dev, grid, smem, st);
    else if (t.fast == 2 && p->stride == 2) rc = launch_fast<3, 2, 2>(P, dev, grid, smem, st);
    else {
        switch (p->k) {
        case 1: rc = launch_fused<1, 0, 1, 0>(P, dev, grid, smem, st); break;
        case 2: rc = launch_fused<2, 0, 1, 0>(P, dev, grid, smem, st); break;
        case 3: rc = launch_fused<3, 0, 1, 0>(P, dev, grid, smem, st); break;
        case 4: rc = launch_fused<4, 0, 1, 0>(P, dev, grid, smem, st); break;
        case 5: rc = launch_fused<5, 0, 1, 0>(P, dev, grid, smem, st); break;
        case 6: rc = launch_fused<6, 0, 1, 0>(P, dev, grid, smem, st); break;
        case 7: rc = launch_fused<7, 0, 1, 0>(P, dev, grid, smem, st); break;
        default: return fail(GDWS_ERR_UNSUPPORTED, "k=%d", p->k);
        }
    }
    if (rc == GDWS_OK) p->launches++;
    return rc;
}

gdws_status_t bf16_fused(gdws_plan_s *p, const gdws_tensor_t *x, gdws_tensor_t *y, cudaStream_t st)
{
    // GDWS_OPT_DW_MATH: 1 = GDW stage on the ALUs, 2 = on the tensor cores, 0 = whichever measured faster for this kind of layer
    if (gdw_stage_of(p) == 2) {
        const gdws_status_t rc = bf16_fused_tc(p, x, y, st);
        if (rc != GDWS_ERR_UNSUPPORTED || p->opt_dw_math == 2) return rc;     // chosen automatically but no tile fits: the ALU kernel
    }
    return run_tiled(p, x, y->ptr, y->h, y->w, false, y->dtype == GDWS_F32, st);
}

// The unfused GDW stage with the tiled pipeline (TMA-staged input, register-blocked depthwise warps,
// coalesced 16-byte stores of z).  GDWS_ERR_UNSUPPORTED if no tile fits; the caller then takes the
// simple kernel.
gdws_status_t bf16_depthwise_tiled(gdws_plan_s *p, const gdws_tensor_t *x, void *z, cudaStream_t st)
{
    const int Ho = gdws_out_dim(x->h, p->k, p->stride, p->pad), Wo = gdws_out_dim(x->w, p->k, p->stride, p->pad);
    return run_tiled(p, x, z, Ho, Wo, true, false, st);
}

}  // namespace gdws
