// Fused GDWS forward for bf16 NHWC tensors on sm_100a with BOTH stages on the tensor cores.
//
// GDW stage as a sum of k*k small GEMMs (Section 3.1, Definition of the (C,K,g) GDW convolution).  For filter
// tap (u,v) the GDW output of a tile of 128 pixels and a window of 16 input channels is
//     z[pixel, i] += x[pixel shifted by (u,v), c] * B_uv[c, i],   B_uv[c, i] = K[i,u,v] if c = c(i), else 0,
// i.e. a [128 x 16] x [16 x n] product per tap whose B operand has one non-zero per column.  The A operand is
// not copied per tap: the staged input box lies in shared memory as [row][column][16 channels] (32 bytes per
// pixel, 32-byte swizzle, written by TMA), which for every tap is a valid K-major tensor-core operand (8
// consecutive pixels of an output row are 8 consecutive 32-byte rows) that differs from the next tap's only in
// its start address.  The fp32 result z (128 lanes x n columns of TMEM) is read back by the converter warps,
// rounded to bf16 and written as the K-major A operand of the pointwise stage (Property 1: W_P is M x G), whose
// products accumulate in a second TMEM region over all windows of the tile.  The ALUs only round z, scatter the
// filter taps into the B operands and run the epilogue; they execute no multiply of the GDW stage.
// With stride 2 the box is staged from four dense views of x (one per parity of input row and column), in each of which
// a tap is again a unit-stride shift; which copy a tap reads and where its operand starts come from tables.
//
// One persistent block of 20 warps per SM walks over work items (tile of 128 output pixels x block of up to
// 256 output channels).  Roles, coupled by mbarriers only:
//   warp 0             issues the k*k GDW products of every chunk (one elected lane) and, with commits of its own,
//                      hands back the B buffer and the input box they have read;
//   warp 3             issues the PW products of every chunk, once its z slabs and weights are in place;
//   warp 1 (one lane)  fetches the input boxes by TMA (x as a rank-4 tensor: C, W, H, N; 16 channels per box);
//   warp 2 (one lane)  streams the packed pointwise weights (one bulk copy per chunk into a ring of 16-channel slabs);
//   warps 4-11         converter: TMEM z -> bf16 -> 16-channel operand slabs; two groups of four warps (one per TMEM
//                      lane quarter) that take alternate chunks;
//   warps 12-15        epilogue: TMEM y -> bias, ReLU, bf16 -> global memory (TMA store or direct);
//   warps 16-19        builder: one thread per intermediate channel of the chunk scatters its k*k taps into B
//                      operand planes that are otherwise zero, and clears what it wrote when the buffer comes back.
// A chunk's slabs are contiguous in the two rings (a chunk that does not fit behind its predecessor starts over at
// slab 0), at places that are the same for every work item and come from a table computed at launch.
// All operands are K-major with 32-byte rows and the 32-byte swizzle (address bit 4 ^= bit 7), 8-row groups
// `stride byte offset` apart.  Every wait is bounded (see mbar_wait, tc_wait).
#include <string.h>

#include <algorithm>
#include <vector>

#include "sm100.cuh"

namespace gdws {

static_assert(sizeof(TcChunk) == 32, "chunk table entries are copied as two 16-byte words");

constexpr int kTcConvWarp0 = 4, kTcConvWarps = 8;    // converter warps 4 .. 11: two groups of four (one warp per TMEM lane quarter)
constexpr int kTcEpiWarp0 = kTcConvWarp0 + kTcConvWarps, kTcBuildWarp0 = kTcEpiWarp0 + 4, kTcBuildWarps = 4;
constexpr int kTcThreads = (kTcBuildWarp0 + kTcBuildWarps) * 32;
constexpr int kTcNU = 4;              // chunks in flight per ring (barriers per ring)
static_assert(kTcNU == 4, "unit parity is taken from bit 2 of the unit index");
constexpr int kTcMaxNB = 4;           // B operand buffers of the GDW stage (one chunk each: k*k planes), up to two per chunk parity
constexpr int kTcMaxNX = 4;           // input box slots
constexpr int kTcMaxTaps = 25;
constexpr int kTcZCol = 256;          // TMEM columns 256..511: two GDW accumulators of up to 128 columns
constexpr uint32_t kTcSw32 = 6u << 29;   // descriptor high word: layout type "32-byte swizzle"
constexpr int kTcSlab = 4096;         // bytes of one z slab: 128 pixels x 16 channels of bf16
constexpr int kTcMaxChunks = 256;

struct alignas(64) TcParams {
    CUtensorMap tmap_xp[4];      // x as (C, W, H, N) bf16, box (16, IW, rows, TN), 32-byte swizzle; with stride 2 one map per
                                 // parity of the input row and column (index 2 * row parity + column parity), each a dense
                                 // (C, W/2, H/2, N) view of every other row and column
    CUtensorMap tmap_y;          // y as (D, Wo, Ho, N) bf16, box (64, PW, PH, TN), 128-byte swizzle (when ostage != 0)
    uint16_t *y;
    const uint16_t *filt;
    const uint16_t *pw;
    const float *bias;
    const TcChunk *chunks;
    int *status;
    int N, Ho, Wo, D, Dloc, Dpad_tot, nparts, nchunks, pad, relu;
    int TN, PH, PW, tiles_h, tiles_w, nitems;
    int nloads, xbox_bytes;
    int load_dw[kTcMaxTaps], load_dh[kTcMaxTaps], load_map[kTcMaxTaps];   // per copy of the box: start relative to the tile's first output pixel, which map
    uint32_t load_off[kTcMaxTaps];
    uint32_t tap_off[kTcMaxTaps];          // the A operand of tap (u, v) starts this many bytes into the box slot
    uint32_t a_sbo;              // GDW A operand: bytes between 8-pixel groups
    int nb, nx, nz, nw, nacc;
    uint32_t dv_parts[2], dv_thw[2], dv_tw[2];   // multiplier and shift for the divisions by nparts, tiles_h * tiles_w, tiles_w
    int first_cbase;             // first input channel of the window the block takes first
    int nbw;                     // builder warps that have rows to fill (32 rows each; the layer's largest chunk decides)
    uint32_t bbuf_bytes, bplane, xslot_bytes, wslab_bytes;
    uint32_t off_b, off_z, off_w, off_x, off_tab;    // from the 1024-aligned base; the output staging comes first
    int ostage, rec_hw, nslabs_total, bias_len;
    // Per chunk of the work item, where its slabs sit in the two rings and which older chunk must have left them:
    // bits 0-7 first z slab, 8-15 first weight slab, 16-18 / 19-21 how many units back the PW products must be done
    // before the z slabs / the weight slabs are overwritten (0: no wait).  A chunk's slabs are contiguous (no wrap).
    uint32_t ring[kTcMaxChunks];
    uint8_t order[kTcMaxChunks];   // the chunk the block takes i-th within a work item (an index into `chunks`)
};

// Bounded wait of every role but the issuing warps: each poll lets the hardware suspend the thread until the phase
// completes (or 16 us pass), so that waiting warps issue next to nothing.  The polling loop is a call (one copy of it in
// the kernel; inlined and unrolled at every site it was a third of the kernel's code), the first poll is inline.
__device__ __forceinline__ void tc_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (!mbar_try_wait(bar, parity)) mbar_wait_relaxed_slow(bar, parity, 16384u, abort_flag, status, code);
}
// The same with the polling loop as a call: for the warps whose per-chunk code has to stay small.
__device__ __forceinline__ void tc_warp_wait_call(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if ((threadIdx.x & 31) == 0 && !mbar_try_wait(bar, parity)) mbar_wait_relaxed_slow(bar, parity, 16384u, abort_flag, status, code);
    __syncwarp();
}
__device__ __forceinline__ void tc_warp_arrive(uint32_t bar)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

// Producer-side bookkeeping of a ring of slabs whose consumer frees whole chunks (in order, one barrier
// per chunk, kTcNU barriers in rotation).
struct SlabRing {
    int head = 0, free_slabs = 0, oldest = 0;
};

// n / d for n < 2^31 as a multiplication: md = (ceil(2^(31+s) / d), 31 + s) with s = ceil(log2 d) is exact in that range
// (a division by a run-time value is some fifty instructions, and the work item's coordinates need three of them).
__device__ __forceinline__ int tc_fdiv(int n, const uint32_t (&md)[2]) { return (int)(((uint64_t)(uint32_t)n * md[0]) >> md[1]); }

// Filters of more than 9 taps: a B buffer holds the operands of up to 13 taps at a time (8 for k = 4), and a chunk's GDW
// products are issued group by group as the groups' operands arrive, all into the same accumulator.
__host__ __device__ constexpr int tc_taps_per_build(int k) { return k * k <= 9 ? k * k : (k == 4 ? 8 : 13); }

template <int K>
__global__ void __launch_bounds__(kTcThreads, 1) fused_tc_kernel(const __grid_constant__ TcParams P)
{
    constexpr int TPB = tc_taps_per_build(K), NBUILD = (K * K + TPB - 1) / TPB;   // taps per B buffer, buffers per chunk
    extern __shared__ uint8_t smem_raw[];
    // dwready[4] | zfull[2] (2 unused) | pwready[4] pwdone[4] | bfree[4] xfree[4] | accfull[2] accfree[2] | drain[2] | 2 unused | bready[4]
    __shared__ __align__(8) uint64_t bars[4 + 4 + 2 * kTcNU + kTcMaxNB + kTcMaxNX + 4 + 4 + kTcMaxNB];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t *base = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t base_s = smem_u32(base);
    const uint32_t o_s = base_s, b_s = base_s + P.off_b, z_s = base_s + P.off_z, w_s = base_s + P.off_w, x_s = base_s + P.off_x;
    // dwready: the B operands (the builder warps that have rows to fill) and the input box (the loader's arrive, with the
    // box's bytes when the chunk opens a window) of a chunk are in place.  zfull[h]: the GDW products of a chunk of parity h
    // are done.  pwready: the chunk's z slabs (the 4 converter warps of its parity) and its pointwise weights (the loader's
    // arrive with their bytes) are in place.  pwdone: its PW products are done.  bfree / xfree: committed by the GDW
    // issuing warp once the products that read a B buffer / the last ones that read a box are done.
    const uint32_t bar_dwready = smem_u32(&bars[0]);
    const uint32_t bar_zfull = bar_dwready + 32;
    const uint32_t bar_pwready = bar_zfull + 32, bar_pwdone = bar_pwready + 8 * kTcNU;
    const uint32_t bar_bfree = bar_pwdone + 8 * kTcNU, bar_xfree = bar_bfree + 8 * kTcMaxNB;
    const uint32_t bar_accfull = bar_xfree + 8 * kTcMaxNX, bar_accfree = bar_accfull + 16;
    const uint32_t bar_drain = bar_accfull + 32;       // the issuing warps' last commits, awaited before TMEM is freed
    const uint32_t bar_bready = bar_drain + 32;        // (filters of more than 9 taps) the operands of a group of taps are in a B buffer
    volatile int *const vabort = &abort_flag;
    TcChunk *tab = reinterpret_cast<TcChunk *>(base + P.off_tab);
    float *bias_sm = reinterpret_cast<float *>(tab + P.nchunks);
    uint16_t *bold = reinterpret_cast<uint16_t *>(bias_sm + P.Dpad_tot);     // [2 * nb][128]: what each builder thread wrote last
    const uint32_t bias_s = smem_u32(bias_sm);

    // The chunk table was written when the plan was built (by a synchronous copy), not by a kernel: its loads may start
    // at once and be in flight during the rest of the set-up (one 16-byte word per thread; at most 256 chunks).
    static_assert(2 * kTcMaxChunks <= kTcThreads, "one table word per thread");
    uint4 tabw = make_uint4(0u, 0u, 0u, 0u);
    if (tid < P.nchunks * 2) {
        tabw = __ldg(reinterpret_cast<const uint4 *>(P.chunks) + 2 * (int)P.order[tid >> 1] + (tid & 1));
        if (tid & 1) tabw.z = P.ring[tid >> 1];      // second half of the entry: slab0, flags, places in the rings, (unused)
    }
    if (tid == 0) abort_flag = 0;
    {
        // One barrier per thread of warps 1 and 2 (warp 0 allocates tensor memory meanwhile).  Layout of bars[] as above;
        // with one B buffer per chunk the builder warps count towards dwready, else they have barriers of their own.
        constexpr int kBars = 4 + 4 + 2 * kTcNU + kTcMaxNB + kTcMaxNX + 4 + 4 + kTcMaxNB;
        const int b = tid - 32;
        if (b >= 0 && b < kBars) {
            uint32_t count = 1;                                                       // zfull, pwdone, bfree, xfree, accfull, drain
            if (b < 4) count = NBUILD == 1 ? 1u + (uint32_t)P.nbw : 1u;               // dwready
            else if (b >= 8 && b < 8 + kTcNU) count = kTcConvWarps / 2 + 1;           // pwready
            else if (b >= 8 + 2 * kTcNU + kTcMaxNB + kTcMaxNX + 2 && b < 8 + 2 * kTcNU + kTcMaxNB + kTcMaxNX + 4) count = 4;   // accfree
            else if (b >= kBars - kTcMaxNB) count = (uint32_t)P.nbw;                   // bready
            mbar_init(bar_dwready + 8 * (uint32_t)b, count);
            fence_mbar_init();
        }
    }
    // The kernel that follows in the stream (launched with programmatic serialisation, as this one is) may start its
    // blocks as SMs become free; it reads nothing from global memory before its own grid_dependency_wait below.
    grid_launch_dependents();
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 512u);
    {
        for (int i = tid; i < P.nb * 128; i += kTcThreads) bold[i] = 0xFFFFu;
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        const uint32_t nb16 = (uint32_t)P.nb * P.bbuf_bytes / 16u;
        for (uint32_t i = tid; i < nb16; i += kTcThreads) sts128(b_s + i * 16u, zero);
        fence_proxy_async();
        if (tid < P.nchunks * 2) reinterpret_cast<uint4 *>(tab)[tid] = tabw;
        // Everything above touches this block's shared and tensor memory and the plan's chunk table only.  From here on
        // what other kernels write is read and written: the kernel before this one in the stream (which may have
        // produced x or the packed weights, or may still be reading what this one overwrites) has to be complete.
        grid_dependency_wait();
        // The block's first input box is asked for right here, by the thread that initialised its barrier (the loader's
        // lane, which skips this box later): it is what the first products wait for longest.
        if (tid == 32 && (int)blockIdx.x < P.nitems) {
            const int item = (int)blockIdx.x;
            int tile = tc_fdiv(item, P.dv_parts);
            const int bn = tc_fdiv(tile, P.dv_thw);
            tile -= bn * (P.tiles_h * P.tiles_w);
            const int bh = tc_fdiv(tile, P.dv_tw), bw = tile - bh * P.tiles_w;
            mbar_expect_tx(bar_dwready, (uint32_t)P.xbox_bytes);
#pragma unroll 1
            for (int l = 0; l < P.nloads; ++l)
                tma_load_4d(x_s + P.load_off[l], &P.tmap_xp[P.load_map[l]], P.first_cbase, bw * P.PW + P.load_dw[l], bh * P.PH + P.load_dh[l],
                            bn * P.TN, bar_dwready);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    const int my_items = ((int)P.nitems - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int total = my_items * P.nchunks;
    const int tiles_hw = P.tiles_h * P.tiles_w;
    const uint32_t p_hi = (256u >> 4) | (1u << 14) | kTcSw32;   // descriptor high word: 8-row groups 256 bytes apart, version 1, 32-byte swizzle

    // A warp runs a dozen cycles per instruction on this control-heavy code (every step waits for the one before), so the
    // code each role runs per chunk is kept short: slab positions come from a table instead of ring bookkeeping, the
    // issuing warps release the buffers their products have read with commits of their own, and the converters, whose
    // per-chunk work is the longest, take alternate chunks in two groups.
    if (warp == 0) {
        // ---------------- GDW issue ----------------
        // Unit u: the k*k GDW products of chunk u into accumulator u & 1, which is free again once the converters have
        // announced the slabs of chunk u - 2 (they read TMEM before that).  Three commits: the accumulator is full, the
        // B buffer may be rebuilt, and (after a window's last chunk) the input box may be overwritten.
        const uint32_t a_hi = ((P.a_sbo >> 4) & 0x3FFFu) | (1u << 14) | kTcSw32;
        const uint32_t a_lo0 = ((x_s & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t b_lo0 = ((b_s & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t xstep = P.xslot_bytes >> 4, bstep = P.bbuf_bytes >> 4, pstep = P.bplane >> 4;
        uint32_t tap_a[K * K], tap_b[K * K];
#pragma unroll
        for (int ur = 0; ur < K; ++ur)
#pragma unroll
            for (int v = 0; v < K; ++v) {
                tap_a[ur * K + v] = P.tap_off[ur * K + v] >> 4;
                tap_b[ur * K + v] = (uint32_t)((ur * K + v) % TPB) * pstep;
            }
        uint32_t xslot = 0, bslot = 0, buse = 0, a_lo = a_lo0, b_lo = b_lo0;
        (void)buse;
        int q = 0;                  // chunk index of unit u within its work item
#pragma unroll 1
        for (int u = 0; u < total; ++u) {
            const int npad = tab[q].npad, flags = tab[q].flags;
            mbar_wait_call(bar_dwready + 8 * (u & 3), (uint32_t)(u >> 2) & 1u, &abort_flag, P.status, kStatusWaitOperand);
            if (u >= 2) mbar_wait_call(bar_pwready + 8 * ((u - 2) & 3), (uint32_t)((u - 2) >> 2) & 1u, &abort_flag, P.status, kStatusWaitStage);
            tc_fence_after();
            if constexpr (NBUILD == 1) {
                if (elect_one()) {
                    const uint32_t idesc = make_idesc(npad, false);
                    const uint32_t d_z = tmem + (uint32_t)(kTcZCol + 128 * (u & 1));
#pragma unroll
                    for (int i = 0; i < K * K; ++i)
                        umma_bf16_words(d_z, a_lo + tap_a[i], a_hi, b_lo + tap_b[i], p_hi, idesc, i != 0);
                    umma_commit(bar_zfull + 8 * (u & 1));
                    umma_commit(bar_bfree + 8 * bslot);
                    if (flags & 2) umma_commit(bar_xfree + 8 * xslot);
                }
                __syncwarp();
                b_lo += bstep;
                if (++bslot == (uint32_t)P.nb) { bslot = 0; b_lo = b_lo0; }
            } else {
                const uint32_t idesc = make_idesc(npad, false);
                const uint32_t d_z = tmem + (uint32_t)(kTcZCol + 128 * (u & 1));
#pragma unroll
                for (int r = 0; r < NBUILD; ++r) {
                    // the operands of tap group r: buffer bslot, for the buse-th time
                    mbar_wait_call(bar_bready + 8 * bslot, buse & 1u, &abort_flag, P.status, kStatusWaitOperand);
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int j = 0; j < TPB; ++j)
                            if (r * TPB + j < K * K)
                                umma_bf16_words(d_z, a_lo + tap_a[r * TPB + j], a_hi, b_lo + tap_b[r * TPB + j], p_hi, idesc, (r | j) != 0);
                        umma_commit(bar_bfree + 8 * bslot);
                        if (r == NBUILD - 1) {
                            umma_commit(bar_zfull + 8 * (u & 1));
                            if (flags & 2) umma_commit(bar_xfree + 8 * xslot);
                        }
                    }
                    __syncwarp();
                    b_lo += bstep;
                    if (++bslot == (uint32_t)P.nb) { bslot = 0; b_lo = b_lo0; ++buse; }
                }
            }
            if (flags & 2) {
                a_lo += xstep;
                if (++xslot == (uint32_t)P.nx) { xslot = 0; a_lo = a_lo0; }
            }
            if (++q == P.nchunks) q = 0;
        }
        // Teardown: one more commit covers every product this thread issued (after an abort, products may have been issued
        // on operands that were not there; they must have ended all the same); its wait is bounded and ignores the abort flag.
        if (elect_one()) {
            umma_commit(bar_drain);
            mbar_wait_drain(bar_drain, 0);
        }
        __syncwarp();
    } else if (warp == 3) {
        // ---------------- PW issue, every chunk in order ----------------
        const uint32_t idesc_pw = make_idesc(P.Dloc, false);
        const uint32_t z_lo0 = ((z_s & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t w_lo0 = ((w_s & 0x3FFFFu) >> 4) | (1u << 16);
        const uint32_t wstep = P.wslab_bytes >> 4;
        uint32_t buf = 0, accpar = 1;
        int qp = 0, itp = 0;
#pragma unroll 1
        for (int v = 0; v < total; ++v) {
            const int ns = tab[qp].npad >> 4;
            const uint32_t ring = (uint32_t)tab[qp].reserved0;
            if (qp == 0 && itp >= P.nacc) mbar_wait_call(bar_accfree + 8 * buf, accpar, &abort_flag, P.status, kStatusWaitStage);
            mbar_wait_call(bar_pwready + 8 * (v & 3), (uint32_t)(v >> 2) & 1u, &abort_flag, P.status, kStatusWaitOperand);
            tc_fence_after();
            if (elect_one()) {
                const uint32_t d_y = tmem + buf * 128u;
                const uint32_t z_lo = z_lo0 + (ring & 0xFFu) * (uint32_t)(kTcSlab >> 4);
                const uint32_t w_lo = w_lo0 + ((ring >> 8) & 0xFFu) * wstep;
#pragma unroll
                for (int s = 0; s < 8; ++s)          // a chunk has at most 8 slabs
                    if (s < ns) umma_bf16_words(d_y, z_lo + (uint32_t)s * (uint32_t)(kTcSlab >> 4), p_hi, w_lo + (uint32_t)s * wstep, p_hi, idesc_pw,
                                                (uint32_t)(qp | s));
                umma_commit(bar_pwdone + 8 * (v & 3));
                if (qp == P.nchunks - 1) umma_commit(bar_accfull + 8 * buf);
            }
            __syncwarp();
            if (++qp == P.nchunks) {
                qp = 0; ++itp;
                if (++buf == (uint32_t)P.nacc) { buf = 0; accpar ^= 1; }
            }
        }
        if (elect_one()) {
            umma_commit(bar_drain + 8);
            mbar_wait_drain(bar_drain + 8, 0);
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- input loader ----------------
            int box = 0, u = 0;
            uint32_t xslot = 0, xuse = 0;      // slot of the next box, and how often that slot has been used
            bool stop = false;
#pragma unroll 1
            for (int it = 0; it < my_items && !stop; ++it) {
                const int item = (int)blockIdx.x + it * (int)gridDim.x;
                int tile = tc_fdiv(item, P.dv_parts);
                const int bn = tc_fdiv(tile, P.dv_thw);
                tile -= bn * tiles_hw;
                const int bh = tc_fdiv(tile, P.dv_tw), bw = tile - bh * P.tiles_w;
                const int n0 = bn * P.TN, hi0 = bh * P.PH, wi0 = bw * P.PW;     // the copies' offsets carry the padding
#pragma unroll 1
                for (int q = 0; q < P.nchunks; ++q, ++u) {
                    const int cbase = tab[q].cbase, flags = tab[q].flags;
                    const uint32_t bar = bar_dwready + 8 * (u & 3);
                    // This barrier's last phase (chunk u - 4) must be complete, and seen by the issuing warp, before anything
                    // counts towards chunk u.  Where the builder warps count towards it too, they keep this thread within
                    // four chunks of the issuing warp (they wait for its commits); where they do not (filters of more than
                    // 9 taps), this thread waits until chunk u - 4 has been converted, which is after its products were issued.
                    if (u >= 4) {
                        if constexpr (NBUILD == 1) tc_wait(bar, (uint32_t)((u >> 2) - 1) & 1u, &abort_flag, P.status, kStatusWaitStage);
                        else tc_wait(bar_pwready + 8 * (u & 3), (uint32_t)((u >> 2) - 1) & 1u, &abort_flag, P.status, kStatusWaitStage);
                    }
                    if (*vabort) { stop = true; break; }       // a wait ran out somewhere: no new copies
                    if (!(flags & 1)) { mbar_arrive(bar); continue; }
                    if (box >= P.nx)
                        tc_wait(bar_xfree + 8 * xslot, (xuse - 1u) & 1u, &abort_flag, P.status, kStatusWaitStage);
                    if (u > 0) {       // the block's first box was asked for in the prologue
                        mbar_expect_tx(bar, (uint32_t)P.xbox_bytes);
                        const uint32_t dst = x_s + xslot * P.xslot_bytes;
#pragma unroll 1
                        for (int l = 0; l < P.nloads; ++l)
                            tma_load_4d(dst + P.load_off[l], &P.tmap_xp[P.load_map[l]], cbase, wi0 + P.load_dw[l], hi0 + P.load_dh[l], n0, bar);
                    }
                    ++box;
                    if (++xslot == (uint32_t)P.nx) { xslot = 0; ++xuse; }
                }
            }
            // Teardown: no box copy may be in flight when the block ends.  This thread arrived for units 0 .. u-1; the
            // last phase of each of the four barriers completes once its box (if any) has landed and the builder warps
            // have arrived, and the phases before it completed earlier (bounded wait).
            for (int j = 0; j < 4 && j < u; ++j) {
                const int v = u - 1 - j;
                mbar_wait_drain(bar_dwready + 8 * (v & 3), (uint32_t)(v >> 2) & 1u);
            }
        }
    } else if (warp == 2) {
        if (lane == 0) {
            // ---------------- pointwise-weight loader ----------------
            int q = 0, it = 0, issued = 0;
#pragma unroll 1
            for (int v = 0; v < total; ++v) {
                const int ns = tab[q].npad >> 4, slab0 = tab[q].slab0;
                const uint32_t ring = (uint32_t)tab[q].reserved0;
                // the chunk's place in the ring was last used wdep units ago (1 .. 4, which also keeps the four pwready
                // barriers apart): the PW products of that chunk must be done
                const int wdep = (int)((ring >> 19) & 7u);
                if (v >= wdep) tc_wait(bar_pwdone + 8 * ((v - wdep) & 3), (uint32_t)((v - wdep) >> 2) & 1u, &abort_flag, P.status, kStatusWaitStage);
                if (*vabort) break;                            // a wait ran out somewhere: no new copies
                issued = v + 1;
                const int item = (int)blockIdx.x + it * (int)gridDim.x;
                const int part = P.nparts == 1 ? 0 : item - tc_fdiv(item, P.dv_parts) * P.nparts;
                const uint32_t bar = bar_pwready + 8 * (v & 3);
                mbar_expect_tx(bar, (uint32_t)ns * P.wslab_bytes);
                const uint16_t *src = P.pw + ((size_t)part * P.nslabs_total + slab0) * 16 * P.Dloc;
                bulk_g2s(w_s + ((ring >> 8) & 0xFFu) * P.wslab_bytes, src, (uint32_t)ns * P.wslab_bytes, bar);
                if (++q == P.nchunks) { q = 0; ++it; }
            }
            // Teardown: the last phase armed on each pwready barrier completes when its weights have landed and the
            // converter warps have arrived (bounded wait).
            for (int j = 0; j < kTcNU && j < issued; ++j) {
                const int v = issued - 1 - j;
                mbar_wait_drain(bar_pwready + 8 * (v & 3), (uint32_t)(v >> 2) & 1u);
            }
        }
    } else if (warp >= kTcConvWarp0 && warp < kTcConvWarp0 + kTcConvWarps) {
        // ---------------- converter: z (fp32, TMEM) -> bf16 operand slabs ----------------
        // Group grp (four warps, one per TMEM lane quarter) takes the chunks of parity grp: it reads the chunk's
        // accumulator granule by granule (16 columns; the next granule's load is in flight while one is rounded and
        // stored) and writes the slabs the table names.
        const int lg = warp & 3, grp = (warp - kTcConvWarp0) >> 2;
        const uint32_t r = (uint32_t)(lg * 32 + lane);
        const uint32_t sw = ((r >> 2) & 1u) << 4;           // 32-byte swizzle: address bit 4 ^= bit 7
        const uint32_t row_s = z_s + r * 32u;
        const uint32_t taddr = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(kTcZCol + 128 * grp);
        int q = 0;
        auto round_store = [&](const uint32_t (&acc)[16], uint32_t addr) {
            uint4 lo, hi;
            lo.x = pack_bf16x2(__uint_as_float(acc[0]), __uint_as_float(acc[1]));
            lo.y = pack_bf16x2(__uint_as_float(acc[2]), __uint_as_float(acc[3]));
            lo.z = pack_bf16x2(__uint_as_float(acc[4]), __uint_as_float(acc[5]));
            lo.w = pack_bf16x2(__uint_as_float(acc[6]), __uint_as_float(acc[7]));
            hi.x = pack_bf16x2(__uint_as_float(acc[8]), __uint_as_float(acc[9]));
            hi.y = pack_bf16x2(__uint_as_float(acc[10]), __uint_as_float(acc[11]));
            hi.z = pack_bf16x2(__uint_as_float(acc[12]), __uint_as_float(acc[13]));
            hi.w = pack_bf16x2(__uint_as_float(acc[14]), __uint_as_float(acc[15]));
            sts128(addr + sw, lo);                 // channels 0 .. 7 of the slab for this pixel
            sts128(addr + (sw ^ 16u), hi);         // channels 8 .. 15
        };
#pragma unroll 1
        for (int v = 0; v < total; ++v) {
            const int ns = tab[q].npad >> 4;
            if ((v & 1) == grp) {
                const uint32_t ring = (uint32_t)tab[q].reserved0;
                const int zdep = (int)((ring >> 16) & 7u);
                if (zdep && v >= zdep)
                    tc_warp_wait_call(bar_pwdone + 8 * ((v - zdep) & 3), (uint32_t)((v - zdep) >> 2) & 1u, &abort_flag, P.status, kStatusWaitStage);
                tc_warp_wait_call(bar_zfull + 8 * grp, (uint32_t)(v >> 1) & 1u, &abort_flag, P.status, kStatusWaitMma);
                tc_fence_after();
                uint32_t addr = row_s + (ring & 0xFFu) * (uint32_t)kTcSlab;
                uint32_t acc0[16], acc1[16];
                tmem_ld16(taddr, acc0);
#pragma unroll 1
                for (int g = 0; g < ns; g += 2) {
                    tmem_ld_wait();
                    if (g + 1 < ns) tmem_ld16(taddr + (uint32_t)((g + 1) * 16), acc1);
                    round_store(acc0, addr);
                    if (g + 1 < ns) {
                        tmem_ld_wait();
                        if (g + 2 < ns) tmem_ld16(taddr + (uint32_t)((g + 2) * 16), acc0);
                        round_store(acc1, addr + (uint32_t)kTcSlab);
                    }
                    addr += 2u * (uint32_t)kTcSlab;
                }
                fence_proxy_async();
                tc_fence_before();
                tc_warp_arrive(bar_pwready + 8 * (v & 3));
            }
            if (++q == P.nchunks) q = 0;
        }
    } else if (warp >= kTcEpiWarp0 && warp < kTcEpiWarp0 + 4) {
        // ---------------- epilogue: TMEM -> bias / ReLU -> bf16 -> global ----------------
        const int lg = warp & 3;
        const int r = lg * 32 + lane;
        const int hw = P.PH * P.PW;
        const int tn = r / hw;
        const int rem = r - tn * hw;
        const int ph = rem / P.PW, pw_ = rem - (rem / P.PW) * P.PW;
        const bool issuer = warp == kTcEpiWarp0 && lane == 0;
        // the bias is first needed here: these warps copy it while the first tile is being computed
        for (int d = r; d < P.Dpad_tot; d += 128) bias_sm[d] = d < P.bias_len ? __ldg(P.bias + d) : 0.f;
        named_bar_sync(1, 128);
        int buf = 0;
        uint32_t accuse = 0;          // accumulator of the tile in turn, and how often it has been used
#pragma unroll 1
        for (int it = 0; it < my_items; ++it) {
            const int item = (int)blockIdx.x + it * (int)gridDim.x;
            int tile = tc_fdiv(item, P.dv_parts);
            const int part = item - tile * P.nparts;
            const int bn = tc_fdiv(tile, P.dv_thw);
            tile -= bn * tiles_hw;
            const int bh = tc_fdiv(tile, P.dv_tw), bw = tile - bh * P.tiles_w;
            const int n = bn * P.TN + tn, ho = bh * P.PH + ph, wo = bw * P.PW + pw_;
            const bool live = n < P.N && ho < P.Ho && wo < P.Wo;
            const size_t yrow = (((size_t)n * P.Ho + ho) * P.Wo + wo) * P.D + part * P.Dloc;   // element index of the row's first channel
            const int dvalid = P.D - part * P.Dloc < P.Dloc ? P.D - part * P.Dloc : P.Dloc;
            tc_warp_wait_call(bar_accfull + 8 * buf, accuse & 1u, &abort_flag, P.status, kStatusWaitMma);
            tc_fence_after();
            const uint32_t t_base = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(buf * 128);
            const uint32_t bias_part = bias_s + (uint32_t)(part * P.Dloc) * 4u;
            if (P.ostage) {
                // 64 output channels at a time through a staging buffer (rows in tile order = the order of a
                // (64, PW, PH, TN) box of y; 16-byte pieces swizzled by row), stored by TMA, which clips the box.
                const uint32_t row_s = o_s + (uint32_t)r * 128;
                const int nblk = P.Dloc >> 6;
#pragma unroll 1
                for (int cb = 0; cb < nblk; ++cb) {
                    if (issuer) bulk_wait_read_all();
                    named_bar_sync(1, 128);
#pragma unroll 1
                    for (int h4 = 0; h4 < 4; ++h4) {
                        uint32_t acc[16], o[8];
                        tmem_ld16(t_base + (uint32_t)(cb * 64 + h4 * 16), acc);
                        tmem_ld_wait();
                        float bv[16];
                        bias16_shared(bias_part + (uint32_t)(cb * 64 + h4 * 16) * 4, bv);
                        finish_row16(acc, bv, P.relu & kOutRelu, o);
                        sts128(row_s + (uint32_t)(((2 * h4) ^ (r & 7)) << 4), make_uint4(o[0], o[1], o[2], o[3]));
                        sts128(row_s + (uint32_t)(((2 * h4 + 1) ^ (r & 7)) << 4), make_uint4(o[4], o[5], o[6], o[7]));
                    }
                    fence_proxy_async();
                    if (cb == nblk - 1) {
                        tc_fence_before();
                        tc_warp_arrive(bar_accfree + 8 * buf);
                    }
                    named_bar_sync(1, 128);
                    if (issuer) {
                        tma_store_4d(o_s, &P.tmap_y, part * P.Dloc + cb * 64, bw * P.PW, bh * P.PH, bn * P.TN);
                        bulk_commit();
                    }
                }
            } else {
                const int ngran = P.Dloc >> 4;
#pragma unroll 1
                for (int j = 0; j < ngran; ++j) {
                    uint32_t acc[16];
                    tmem_ld16(t_base + (uint32_t)(j * 16), acc);
                    tmem_ld_wait();
                    if (live && j * 16 < dvalid) {
                        float bv[16];
                        bias16_shared(bias_part + (uint32_t)j * 64, bv);
                        if (P.relu & kOutF32) {      // fp32 output asked for: the sums are not rounded to bf16
                            finish_store_row16_f32(acc, bv, P.relu & kOutRelu, j * 16, dvalid, reinterpret_cast<float *>(P.y) + yrow);
                        } else {
                            uint32_t o[8];
                            finish_row16(acc, bv, P.relu & kOutRelu, o);
                            store_packed16(o, j * 16, dvalid, P.y + yrow);
                        }
                    }
                }
                tc_fence_before();
                tc_warp_arrive(bar_accfree + 8 * buf);
            }
            if (++buf == P.nacc) { buf = 0; ++accuse; }
        }
        if (P.ostage && issuer) bulk_wait_all();
    } else if (warp >= kTcBuildWarp0 && warp < kTcBuildWarp0 + P.nbw) {
        // ---------------- builder: filter taps -> B operands of the GDW products ----------------
        // Thread t owns intermediate slot t of the current chunk.  The B operand of tap (ur, v) is a [n x 16]
        // K-major matrix whose row t has the tap's value in column `channel of slot t inside the window`.
        const int t = tid - kTcBuildWarp0 * 32;
        constexpr int RW = (1 + K * K + 7) / 8 * 4;         // 32-bit words of a filter record
        const uint32_t rowoff = (uint32_t)t * 32u, rowsw = (uint32_t)(t >> 2) & 1u;   // row of slot t; 32-byte swizzle phase
        uint32_t rec[RW], nxt[RW];
        auto load_rec = [&](const TcChunk &ch, uint32_t (&dst)[RW]) {
            if (t < ch.npad) {
                const uint4 *src = reinterpret_cast<const uint4 *>(P.filt + ((size_t)ch.slab0 * 16 + t) * (RW * 2));
#pragma unroll
                for (int j = 0; j < RW / 4; ++j) {
                    const uint4 w4 = __ldg(src + j);
                    dst[4 * j] = w4.x; dst[4 * j + 1] = w4.y; dst[4 * j + 2] = w4.z; dst[4 * j + 3] = w4.w;
                }
            } else {
#pragma unroll
                for (int j = 0; j < RW; ++j) dst[j] = 0xFFFFu;
            }
        };
        if (total > 0) load_rec(tab[0], nxt);
        uint32_t bslot = 0, bpar = 0, buse = 0;      // B buffer in turn, the parity of the "free" phase it waits for / how often it was used
        (void)bpar; (void)buse;
        int q = 0;
#pragma unroll 1
        for (int v = 0; v < total; ++v) {
#pragma unroll
            for (int j = 0; j < RW; ++j) rec[j] = nxt[j];
            if (++q == P.nchunks) q = 0;
            if (v + 1 < total) load_rec(tab[q], nxt);
            const uint32_t cw = rec[0] & 0xFFFFu;
            const bool valid = cw != 0xFFFFu;
            const uint32_t off = rowoff + ((((cw >> 3) & 1u) ^ rowsw) << 4) + (cw & 7u) * 2u;
            if constexpr (NBUILD == 1) {
                if (v >= P.nb) tc_warp_wait_call(bar_bfree + 8 * bslot, bpar, &abort_flag, P.status, kStatusWaitStage);
                const uint32_t bb = b_s + bslot * P.bbuf_bytes;
                const uint32_t old = bold[bslot * 128 + t];
                if (old != 0xFFFFu) {
                    uint32_t a = bb + old;
#pragma unroll 1
                    for (int j = 0; j < K * K; ++j, a += P.bplane) sts16(a, (uint16_t)0);
                }
                if (valid) {
#pragma unroll
                    for (int j = 0; j < K * K; ++j)     // 16-bit word 1 + j of the record holds tap j
                        sts16(bb + (uint32_t)j * P.bplane + off, (uint16_t)(rec[(1 + j) >> 1] >> (16 * ((1 + j) & 1))));
                }
                bold[bslot * 128 + t] = (uint16_t)(valid ? off : 0xFFFFu);
                fence_proxy_async();
                tc_warp_arrive(bar_dwready + 8 * (v & 3));
                if (++bslot == (uint32_t)P.nb) { bslot = 0; if (v >= P.nb) bpar ^= 1u; }
            } else {
                // up to TPB taps per buffer: NBUILD buffers per chunk, each announced on its own barrier
#pragma unroll
                for (int r = 0; r < NBUILD; ++r) {
                    if (buse) tc_warp_wait_call(bar_bfree + 8 * bslot, (buse - 1u) & 1u, &abort_flag, P.status, kStatusWaitStage);
                    const uint32_t bb = b_s + bslot * P.bbuf_bytes;
                    const uint32_t old = bold[bslot * 128 + t];
                    if (old != 0xFFFFu) {
                        uint32_t a = bb + old;
#pragma unroll 1
                        for (int j = 0; j < TPB; ++j, a += P.bplane) sts16(a, (uint16_t)0);
                    }
                    if (valid) {
#pragma unroll
                        for (int j = 0; j < TPB; ++j) {
                            const int h = 1 + r * TPB + j;          // 16-bit word h of the record holds tap h - 1
                            if (h <= K * K) sts16(bb + (uint32_t)j * P.bplane + off, (uint16_t)(rec[h >> 1] >> (16 * (h & 1))));
                        }
                    }
                    bold[bslot * 128 + t] = (uint16_t)(valid ? off : 0xFFFFu);
                    fence_proxy_async();
                    tc_warp_arrive(bar_bready + 8 * bslot);
                    if (++bslot == (uint32_t)P.nb) { bslot = 0; ++buse; }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (warp == 0) tmem_dealloc(tmem, 512u);
}

// ------------------------------------------------------------------------------------------
// Weight packing
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float tc_load_weight(const void *w, size_t idx, int is_bf16)
{
    return is_bf16 ? bf16_bits_to_float(((const uint16_t *)w)[idx]) : ((const float *)w)[idx];
}

// dw_w[G][k][k] -> one record per intermediate slot: the slot's channel inside its 16-channel window
// (0xFFFF for the padding slots of a chunk), then the k*k taps as bf16.
__global__ void tc_pack_filt_kernel(const void *__restrict__ dw, int is_bf16, int k2, int rec_hw, const TcChunk *__restrict__ chunks,
                                    const int32_t *__restrict__ chan, uint16_t *__restrict__ out)
{
    const TcChunk ch = chunks[blockIdx.x];
    for (int e = threadIdx.x; e < ch.npad * rec_hw; e += blockDim.x) {
        const int t = e / rec_hw, h = e - t * rec_hw;
        uint16_t val = 0;
        if (h == 0) val = t < ch.n ? (uint16_t)(chan[ch.i0 + t] - ch.cbase) : (uint16_t)0xFFFFu;
        else if (h <= k2 && t < ch.n) val = float_to_bf16_bits(tc_load_weight(dw, (size_t)(ch.i0 + t) * k2 + (h - 1), is_bf16));
        out[((size_t)ch.slab0 * 16 + t) * rec_hw + h] = val;
    }
}

// pw_w[D][G] -> [part][slab][output channel][16] bf16: per 16 intermediate slots one K-major operand slab of the
// pointwise product, 32 bytes per output channel, 32-byte swizzle.
__global__ void tc_pack_pw_kernel(const void *__restrict__ pw, int is_bf16, int D, int G, int Dloc, int nslabs,
                                  const TcChunk *__restrict__ chunks, uint16_t *__restrict__ out)
{
    const TcChunk ch = chunks[blockIdx.x];
    const int part = blockIdx.y;
    const int per_slab = 16 * Dloc;
    for (int e = threadIdx.x; e < (ch.npad >> 4) * per_slab; e += blockDim.x) {
        const int s = e / per_slab;
        int rem = e - s * per_slab;
        const int dl = rem >> 4, kk = rem & 15;
        const int t = s * 16 + kk, d = part * Dloc + dl;
        float val = 0.f;
        if (t < ch.n && d < D) val = tc_load_weight(pw, (size_t)d * G + ch.i0 + t, is_bf16);
        // row dl of the slab: 32 bytes, its two 16-byte halves swapped in rows 4..7 of every 8 (32-byte swizzle)
        out[((size_t)part * nslabs + ch.slab0 + s) * per_slab + dl * 16 + ((((kk >> 3) ^ ((dl >> 2) & 1))) << 3) + (kk & 7)] =
            float_to_bf16_bits(val);
    }
}

void tc_pack(gdws_plan_s *p, const void *dw_w, const void *pw_w, int is_bf16, cudaStream_t st)
{
    if (!p->tc_ok) return;
    const int nch = (int)p->tc_chunks.size();
    tc_pack_filt_kernel<<<nch, 256, 0, st>>>(dw_w, is_bf16, p->k * p->k, p->tc_rec_hw, p->d_tc_chunks, p->d_chan, p->d_tc_filt);
    tc_pack_pw_kernel<<<dim3(nch, p->tc_nparts), 256, 0, st>>>(pw_w, is_bf16, p->D, p->G, p->tc_dloc, p->tc_nslabs, p->d_tc_chunks,
                                                            p->d_tc_pw);
    p->launches += 2;
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
namespace {

// Input row h = stride * ho + u - pad of filter row u (columns alike).  With stride 2 the input is read through four
// dense views, one per parity of row and column (every other row, every other column): in the view of parity par
// filter row u reads row ho + off of the view, which turns the strided access into a unit-stride one.
struct TcTaps {
    int par[5] = {}, off[5] = {};          // per filter row (the filter is square and padded alike: same for columns)
    int omin[2] = {}, omax[2] = {};        // per parity: smallest and largest offset
    bool used[2] = {};
    int ext = 0;                           // halo of a copy: the largest omax - omin
    int npar = 0;
};

TcTaps tc_taps(int k, int stride, int pad)
{
    TcTaps t;
    for (int par = 0; par < 2; ++par) { t.omin[par] = 1 << 20; t.omax[par] = -(1 << 20); }
    for (int u = 0; u < k; ++u) {
        const int i = u - pad;
        const int par = ((i % stride) + stride) % stride;
        t.par[u] = par; t.off[u] = (i - par) / stride;
        t.used[par] = true;
        t.omin[par] = std::min(t.omin[par], t.off[u]); t.omax[par] = std::max(t.omax[par], t.off[u]);
    }
    for (int par = 0; par < 2; ++par)
        if (t.used[par]) { t.ext = std::max(t.ext, t.omax[par] - t.omin[par]); ++t.npar; }
    return t;
}

struct TcGeom {
    int layout = 0;              // 1: boxes with halo rows (one image per tile; one box per parity pair), 2: one copy per
                                 // filter row and column parity, 3: one copy per tap (maps at most 4 wide)
    int TN = 0, PH = 0, PW = 0, IW = 0, IH = 0;
    int tiles_n = 0, tiles_h = 0, tiles_w = 0;
    int nloads = 0, xbox = 0, copy = 0;     // copies per box, bytes of a box, bytes of one copy (in shared memory: a multiple of 256)
    int64_t tiles() const { return (int64_t)tiles_n * tiles_h * tiles_w; }
};

bool tc_geometry(const gdws_plan_s *p, int n, int Ho, int Wo, TcGeom *out)
{
    const int k = p->k;
    const TcTaps t = tc_taps(k, p->stride, p->pad);
    double best = 1e300;
    bool found = false;
    auto consider = [&](int layout, int TN, int PH, int PW) {
        TcGeom g;
        g.layout = layout; g.TN = TN; g.PH = PH; g.PW = PW;
        g.tiles_n = (n + TN - 1) / TN; g.tiles_h = (Ho + PH - 1) / PH; g.tiles_w = (Wo + PW - 1) / PW;
        g.IW = layout == 3 ? 4 : PW + t.ext;
        g.IH = layout == 1 ? PH + t.ext : PH;
        g.nloads = layout == 1 ? t.npar * t.npar : (layout == 2 ? k * t.npar : k * k);
        g.copy = (TN * g.IH * g.IW * 32 + 255) / 256 * 256;
        g.xbox = g.nloads * g.copy;
        if (g.nloads > kTcMaxTaps) return;
        const double cost = (double)g.tiles() * (1.0 + 0.02 * (g.nloads - 1));
        if (cost < best) { best = cost; *out = g; found = true; }
    };
    if (Wo > 4) {
        consider(1, 1, 16, 8);
        for (int PH = 8; PH >= 1; PH >>= 1) consider(2, 16 / PH, PH, 8);
    } else {
        for (int PH = 32; PH >= 2; PH >>= 1) consider(3, 32 / PH, PH, 4);
    }
    return found;
}

// Places of the chunks' slabs in a ring of `cap` slabs, the same for every work item: a chunk's slabs are contiguous,
// and a chunk that does not fit behind its predecessor starts over at slab 0.  dep[q] = how many units before chunk q
// the last chunk that used any of its slabs ran (in steady state, work item after work item), at most 4: the four
// barriers of a ring are reused every four units, so a producer never runs further ahead than that anyway.
bool tc_ring_places(const std::vector<int> &slabs, int cap, std::vector<int> *pos, std::vector<int> *dep)
{
    const int n = (int)slabs.size();
    pos->assign(n, 0);
    dep->assign(n, 4);
    int head = 0;
    for (int q = 0; q < n; ++q) {
        const int ns = slabs[q];
        if (ns > cap) return false;
        if (head + ns > cap) head = 0;
        (*pos)[q] = head;
        head += ns;
    }
    std::vector<int> last(cap, -1000000);
    for (int v = 0; v < 3 * n; ++v) {
        const int q = v % n, ns = slabs[q];
        int newest = -1000000;
        for (int s2 = (*pos)[q]; s2 < (*pos)[q] + ns; ++s2) { newest = std::max(newest, last[s2]); last[s2] = v; }
        if (v >= 2 * n) (*dep)[q] = std::max(1, std::min(4, v - newest));
    }
    return true;
}

// The windows of a work item may be taken in any order (their contributions to y add up), and the order decides how
// well consecutive chunks share the two slab rings: a chunk whose slabs are still held by the chunk right before it
// waits for that one's PW products, and with them the weight copy or the conversion loses its head start.  A few
// orders (as planned, large and small windows alternating, sorted, some shuffles) are laid out; the one with the
// fewest such waits wins, the planned order on a tie.  Chunks of one window stay together.
void tc_choose_order(const std::vector<TcChunk> &chunks, int nz, int nw, std::vector<int> *order)
{
    std::vector<std::vector<int>> windows;
    for (int i = 0; i < (int)chunks.size(); ++i) {
        if (chunks[i].flags & 1) windows.emplace_back();
        windows.back().push_back(i);
    }
    const int nwin = (int)windows.size();
    auto slabs_of = [&](int w) { int t = 0; for (int i : windows[w]) t += chunks[i].npad / 16; return t; };
    std::vector<int> base(nwin), sorted(nwin);
    for (int w = 0; w < nwin; ++w) base[w] = sorted[w] = w;
    std::stable_sort(sorted.begin(), sorted.end(), [&](int a, int b) { return slabs_of(a) > slabs_of(b); });
    std::vector<std::vector<int>> cands;
    cands.push_back(base);
    {
        std::vector<int> alt;
        for (int lo = 0, hi = nwin, turn = 0; lo < hi; ++turn) alt.push_back((turn & 1) ? sorted[--hi] : sorted[lo++]);
        cands.push_back(alt);
    }
    cands.push_back(sorted);
    cands.push_back(std::vector<int>(sorted.rbegin(), sorted.rend()));
    uint32_t rng = 0x9E3779B9u ^ (uint32_t)chunks.size() * 2654435761u;
    for (int t = 0; t < 24; ++t) {
        std::vector<int> sh = base;
        for (int i = nwin - 1; i > 0; --i) {
            rng = rng * 1664525u + 1013904223u;
            std::swap(sh[i], sh[(rng >> 8) % (uint32_t)(i + 1)]);
        }
        cands.push_back(sh);
    }
    double best = 1e300;
    for (const std::vector<int> &cand : cands) {
        std::vector<int> seq, slabs;
        for (int w : cand) for (int i : windows[w]) { seq.push_back(i); slabs.push_back(chunks[i].npad / 16); }
        std::vector<int> zp, zd, wp, wd;
        if (!tc_ring_places(slabs, nz, &zp, &zd) || !tc_ring_places(slabs, nw, &wp, &wd)) continue;
        double cost = 0;
        for (size_t u = 0; u < seq.size(); ++u)
            cost += (zd[u] == 1 ? 1.0 : 0.0) + (wd[u] == 1 ? 1.0 : 0.0);
        if (cost < best - 1e-9) { best = cost; *order = seq; }
    }
    if (order->empty()) for (int i = 0; i < (int)chunks.size(); ++i) order->push_back(i);
}

}  // namespace

gdws_status_t bf16_fused_tc(gdws_plan_s *p, const gdws_tensor_t *x, gdws_tensor_t *y, cudaStream_t st)
{
    if (!p->tc_ok) return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: layer not covered (stride 1 or 2, k <= 5, C and D multiples of 8)");
    const int nchunks = (int)p->tc_chunks.size();
    if (nchunks > kTcMaxChunks) return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: %d chunks (at most %d)", nchunks, kTcMaxChunks);
    if (p->sm_count <= 0) {
        cudaError_t e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute(MultiProcessorCount)");
    }
    const int Ho = y->h, Wo = y->w, k = p->k;
    TcGeom g;
    if (!tc_geometry(p, x->n, Ho, Wo, &g)) return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: no tile");
    const int64_t nitems = g.tiles() * p->tc_nparts;
    if (nitems > 0x7fffffffLL) return fail(GDWS_ERR_UNSUPPORTED, "too many tiles");
    tensor_map_encode_fn encode = encode_fn();
    if (!encode) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");

    TcParams P;
    memset(&P, 0, sizeof(P));
    const int Dloc = p->tc_dloc, m = p->tc_maxslabs;
    // a B operand plane holds one 32-byte row per intermediate channel of the layer's largest chunk
    P.bplane = (uint32_t)m * 16u * 32u; P.bbuf_bytes = (uint32_t)tc_taps_per_build(k) * P.bplane;
    P.wslab_bytes = (uint32_t)Dloc * 32u;
    P.xslot_bytes = (uint32_t)((g.xbox + 255) / 256 * 256);
    // Shared memory: output staging (optional) | B operand buffers | z slabs | weight slabs | input boxes | tables
    const bool can_stage = y->dtype != GDWS_F32 && p->D % 64 == 0 && Dloc % 64 == 0 && ((uintptr_t)y->ptr & 15) == 0 && nitems > p->sm_count;
    const size_t tables = (size_t)nchunks * sizeof(TcChunk) + (size_t)p->tc_nparts * Dloc * 4 + kTcMaxNB * 256 + 256;
    double best_score = -1;
    int b_ost = 0, b_nx = 0, b_nb = 0, b_nz = 0, b_nw = 0;
    for (int ost = can_stage ? 1 : 0; ost >= 0; --ost)
        for (int nx = 3; nx >= 2; --nx)
            for (int nb = 3; nb >= 2; --nb)
                for (int nz = 3 * m; nz >= m; --nz) {
                    const size_t fixed = 1024 + (ost ? 16384 : 0) + (size_t)nb * P.bbuf_bytes + (size_t)nz * kTcSlab +
                                         (size_t)nx * P.xslot_bytes + tables;
                    if (fixed + (size_t)m * P.wslab_bytes > (size_t)kMaxSmem) continue;
                    int nw = (int)(((size_t)kMaxSmem - fixed) / P.wslab_bytes);
                    if (nw > 3 * m) nw = 3 * m;
                    // First two chunks of z slabs (one is converted while the PW products of the one before are pending)
                    // and of weights, then a second B buffer per parity (a chunk's operands are built while the products
                    // of the chunk before it run), then the rest.
                    const double score = 10.0 * std::min(nz, 2 * m) / m + 6.0 * std::min(nw, 2 * m) / m + 1.0 * std::min(nw, 3 * m) / m +
                                         0.5 * nz / m + 0.8 * ost + 0.6 * nb + 0.3 * nx;
                    if (score > best_score) { best_score = score; b_ost = ost; b_nx = nx; b_nb = nb; b_nz = nz; b_nw = nw; }
                }
    if (best_score < 0) return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: shared memory does not fit this layer");
    P.ostage = b_ost ? 16384 : 0; P.nx = b_nx; P.nb = b_nb; P.nz = b_nz; P.nw = b_nw;
    {
        if (p->tc_lay_nz != P.nz || p->tc_lay_nw != P.nw || (int)p->tc_lay_order.size() != nchunks) {
            std::vector<int> order, slabs, zpos, zdep, wpos, wdep;
            tc_choose_order(p->tc_chunks, P.nz, P.nw, &order);
            for (int i : order) slabs.push_back(p->tc_chunks[i].npad / 16);
            if (!tc_ring_places(slabs, P.nz, &zpos, &zdep) || !tc_ring_places(slabs, P.nw, &wpos, &wdep))
                return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: a chunk does not fit the slab rings");
            p->tc_lay_order.resize(nchunks); p->tc_lay_ring.resize(nchunks);
            for (int q = 0; q < nchunks; ++q) {
                p->tc_lay_order[q] = (uint8_t)order[q];
                p->tc_lay_ring[q] = (uint32_t)zpos[q] | ((uint32_t)wpos[q] << 8) | ((uint32_t)zdep[q] << 16) | ((uint32_t)wdep[q] << 19);
            }
            p->tc_lay_nz = P.nz; p->tc_lay_nw = P.nw;
        }
        memcpy(P.order, p->tc_lay_order.data(), (size_t)nchunks);
        memcpy(P.ring, p->tc_lay_ring.data(), (size_t)nchunks * 4);
    }
    P.off_b = (uint32_t)P.ostage;
    P.off_z = P.off_b + (uint32_t)P.nb * P.bbuf_bytes;
    P.off_w = P.off_z + (uint32_t)P.nz * kTcSlab;
    P.off_x = P.off_w + (uint32_t)P.nw * P.wslab_bytes;
    P.off_tab = P.off_x + (uint32_t)P.nx * P.xslot_bytes;
    size_t smem = 1024 + (size_t)P.off_tab + tables;
    if (smem < (size_t)kMaxSmem / 2 + 4096) smem = (size_t)kMaxSmem / 2 + 4096;   // one block per SM: it owns all of TMEM
    if (smem > (size_t)kMaxSmem) return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: shared memory plan exceeds the limit");

    const int sd = p->stride;
    const TcTaps taps = tc_taps(k, sd, p->pad);
    for (int hp = 0; hp < sd; ++hp)
        for (int wp = 0; wp < sd; ++wp) {
            if (!taps.used[hp] || !taps.used[wp]) continue;
            // x as a rank-4 tensor, innermost first: channels, width, height, batch; a box holds 16 channels (32 bytes) per
            // pixel.  With stride 2: the rows of parity hp and the columns of parity wp only.
            const int Wp = (x->w - wp + sd - 1) / sd, Hp = (x->h - hp + sd - 1) / sd;
            if (Wp <= 0 || Hp <= 0) return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: input too small for stride %d", sd);
            const cuuint64_t dims[4] = {(cuuint64_t)p->C, (cuuint64_t)Wp, (cuuint64_t)Hp, (cuuint64_t)x->n};
            const cuuint64_t strides[3] = {(cuuint64_t)sd * p->C * 2, (cuuint64_t)sd * x->w * p->C * 2, (cuuint64_t)x->h * x->w * p->C * 2};
            const cuuint32_t box[4] = {16, (cuuint32_t)g.IW, (cuuint32_t)g.IH, (cuuint32_t)g.TN};
            const cuuint32_t estr[4] = {1, 1, 1, 1};
            void *base = (uint8_t *)x->ptr + ((size_t)hp * x->w + wp) * p->C * 2;
            const CUresult r = encode(&P.tmap_xp[hp * 2 + wp], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B,
                                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled (x) failed with code %d", (int)r);
        }
    if (P.ostage) {
        const cuuint64_t dims[4] = {(cuuint64_t)p->D, (cuuint64_t)Wo, (cuuint64_t)Ho, (cuuint64_t)x->n};
        const cuuint64_t strides[3] = {(cuuint64_t)p->D * 2, (cuuint64_t)Wo * p->D * 2, (cuuint64_t)Ho * Wo * p->D * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)g.PW, (cuuint32_t)g.PH, (cuuint32_t)g.TN};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        const CUresult r = encode(&P.tmap_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, y->ptr, dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(GDWS_ERR_CUDA, "cuTensorMapEncodeTiled (y) failed with code %d", (int)r);
    } else {
        P.tmap_y = P.tmap_xp[taps.used[0] ? 0 : 3];
    }
    // Where each copy of the box goes, and where the A operand of tap (u, v) starts.
    const uint32_t px = 32;      // bytes of one staged pixel (16 channels)
    int nl = 0;
    if (g.layout == 1) {
        int idx[2][2] = {{-1, -1}, {-1, -1}};
        for (int hp = 0; hp < sd; ++hp)
            for (int wp = 0; wp < sd; ++wp) {
                if (!taps.used[hp] || !taps.used[wp]) continue;
                idx[hp][wp] = nl;
                P.load_map[nl] = hp * 2 + wp; P.load_dh[nl] = taps.omin[hp]; P.load_dw[nl] = taps.omin[wp];
                P.load_off[nl] = (uint32_t)nl * (uint32_t)g.copy;
                ++nl;
            }
        for (int u = 0; u < k; ++u)
            for (int v = 0; v < k; ++v) {
                const int hp = taps.par[u], wp = taps.par[v];
                P.tap_off[u * k + v] = P.load_off[idx[hp][wp]] +
                                       (uint32_t)((taps.off[u] - taps.omin[hp]) * g.IW + (taps.off[v] - taps.omin[wp])) * px;
            }
        P.a_sbo = (uint32_t)g.IW * px;
    } else if (g.layout == 2) {
        int idx[5][2];
        for (int u = 0; u < k; ++u)
            for (int wp = 0; wp < sd; ++wp) {
                if (!taps.used[wp]) continue;
                idx[u][wp] = nl;
                P.load_map[nl] = taps.par[u] * 2 + wp; P.load_dh[nl] = taps.off[u]; P.load_dw[nl] = taps.omin[wp];
                P.load_off[nl] = (uint32_t)nl * (uint32_t)g.copy;
                ++nl;
            }
        for (int u = 0; u < k; ++u)
            for (int v = 0; v < k; ++v) {
                const int wp = taps.par[v];
                P.tap_off[u * k + v] = P.load_off[idx[u][wp]] + (uint32_t)(taps.off[v] - taps.omin[wp]) * px;
            }
        P.a_sbo = (uint32_t)g.IW * px;
    } else {
        for (int u = 0; u < k; ++u)
            for (int v = 0; v < k; ++v) {
                P.load_map[nl] = taps.par[u] * 2 + taps.par[v]; P.load_dh[nl] = taps.off[u]; P.load_dw[nl] = taps.off[v];
                P.load_off[nl] = (uint32_t)nl * (uint32_t)g.copy;
                P.tap_off[u * k + v] = P.load_off[nl];
                ++nl;
            }
        P.a_sbo = 256u;
    }
    if (nl != g.nloads) return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: internal error in the box plan");
    P.nloads = nl;
    // bytes that arrive per box: every copy delivers its full box (positions outside the image are zero-filled)
    P.xbox_bytes = nl * g.TN * g.IH * g.IW * 32;
    P.y = (uint16_t *)y->ptr; P.filt = p->d_tc_filt; P.pw = p->d_tc_pw; P.bias = p->d_bias; P.chunks = p->d_tc_chunks;
    P.status = p->d_status;
    P.N = x->n; P.Ho = Ho; P.Wo = Wo; P.D = p->D; P.Dloc = Dloc; P.Dpad_tot = p->tc_nparts * Dloc; P.nparts = p->tc_nparts;
    P.nchunks = nchunks; P.pad = p->pad; P.relu = (p->opt_relu ? kOutRelu : 0) | (y->dtype == GDWS_F32 ? kOutF32 : 0);
    P.TN = g.TN; P.PH = g.PH; P.PW = g.PW; P.tiles_h = g.tiles_h; P.tiles_w = g.tiles_w; P.nitems = (int)nitems;
    P.nacc = Dloc <= 128 ? 2 : 1;
    P.rec_hw = p->tc_rec_hw; P.nslabs_total = p->tc_nslabs;
    P.bias_len = p->Dpad;
    P.nbw = std::min(kTcBuildWarps, (m * 16 + 31) / 32);
    P.first_cbase = p->tc_chunks[P.order[0]].cbase;
    auto magic = [](int d, uint32_t (&md)[2]) {
        int sh = 0;
        while ((1 << sh) < d) ++sh;
        md[0] = (uint32_t)((((uint64_t)1 << (31 + sh)) + (uint64_t)d - 1) / (uint64_t)d);
        md[1] = (uint32_t)(31 + sh);
    };
    magic(p->tc_nparts, P.dv_parts); magic(g.tiles_h * g.tiles_w, P.dv_thw); magic(g.tiles_w, P.dv_tw);

    const int grid = (int)(nitems < p->sm_count ? nitems : p->sm_count);
    cudaError_t e = cudaSuccess;
#define GDWS_TC_LAUNCH(KK)                                                                                              \
    do {                                                                                                                \
        static bool attr_set[64] = {};                                                                                  \
        if (!attr_set[p->device & 63]) {                                                                                \
            e = cudaFuncSetAttribute(fused_tc_kernel<KK>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);       \
            if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(fused_tc_kernel)");                         \
            attr_set[p->device & 63] = true;                                                                            \
        }                                                                                                               \
        e = launch_overlapped(fused_tc_kernel<KK>, (unsigned)grid, kTcThreads, smem, st, P);                              \
        if (e != cudaSuccess) return cuda_fail(e, "fused_tc_kernel launch");                                            \
    } while (0)
    switch (k) {
    case 1: GDWS_TC_LAUNCH(1); break;
    case 2: GDWS_TC_LAUNCH(2); break;
    case 3: GDWS_TC_LAUNCH(3); break;
    case 4: GDWS_TC_LAUNCH(4); break;
    case 5: GDWS_TC_LAUNCH(5); break;
    default: return fail(GDWS_ERR_UNSUPPORTED, "tensor-core GDW path: k=%d", k);
    }
#undef GDWS_TC_LAUNCH
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "fused_tc_kernel launch");
    p->launches++;
    return GDWS_OK;
}

}  // namespace gdws
