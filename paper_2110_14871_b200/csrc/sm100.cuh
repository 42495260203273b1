// Device-side building blocks for sm_100a shared by the tensor-core kernels: mbarrier, bulk-copy,
// tcgen05 (TMEM allocation, MMA, commit, loads) wrappers, operand descriptors, the epilogue.
//
// Tensor-core operand conventions used here (sm_100 "UMMA" shared-memory descriptors):
//   * 128-byte swizzle: within every 1024-byte group of eight 128-byte rows, the 16-byte
//     column index is XORed with the row index (address bits [4,7) ^= bits [7,10)).
//   * K-major operand (rows = M or N index, 64 bf16 of K per 128-byte row): row groups
//     of 8 are 1024 bytes apart (stride byte offset); one MMA of K=16 reads 32 bytes of
//     each row, so successive K steps advance the start address by 32 bytes.
//   * MN-major operand (rows = K index, 64 consecutive M per 128-byte row): blocks of
//     64 M are `leading byte offset` apart, groups of 8 K rows `stride byte offset` apart.
#pragma once

#include <cuda.h>
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
// Adds `bytes` to the barrier's pending transaction count without arriving.
__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Programmatic dependent launch.  grid_launch_dependents: the next kernel in the stream, if it was launched with
// programmatic stream serialisation, may be scheduled once every block of this grid has executed this (or exited).
// grid_dependency_wait: returns once the kernel before this one in the stream has completed and its writes are visible
// (at once when this kernel was not launched with the attribute).  A kernel must execute it, in every thread that
// touches global memory afterwards, before its first global access.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Bounded wait.  When the limit runs out (about a second) the thread records `code` in the
// status word and raises the block's abort flag; from then on every wait in the block returns
// at once, so that all threads still walk the same control flow, reach the common teardown
// (barriers stay matched, TMEM is freed) and the kernel ends.  The first few thousand polls
// are back to back (waits in the pipeline are short and a sleeping waiter wakes up late).
constexpr uint32_t kSpinLimit = 1u << 22;
// The waiting loops are kept out of line on purpose: inlined (and unrolled by the compiler) at every site they were a
// third of a kernel's code, and code that the warps of an SM walk through runs at the speed of instruction fetch once it
// exceeds some 32 KB (measured: gdws_measure_code_size).  Inline is only the first poll, which succeeds in the common case.
static __device__ __noinline__ void mbar_wait_slow(uint32_t bar, uint32_t parity, uint32_t limit, volatile int *abort_flag, int *status, int code)
{
    if (*abort_flag) return;
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if (it > 4096) __nanosleep(64);
        if ((it & 1023) == 1023 && *abort_flag) return;
    }
    *abort_flag = 1;
    atomicOr(status, code);
}
__device__ __forceinline__ void mbar_wait_limited(uint32_t bar, uint32_t parity, uint32_t limit, volatile int *abort_flag,
                                                  int *status, int code)
{
    if (mbar_try_wait(bar, parity)) return;           // the common case costs one shared-memory round trip
    if (*abort_flag) return;
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return;
        if (it > 4096) __nanosleep(64);
        if ((it & 1023) == 1023 && *abort_flag) return;
    }
    *abort_flag = 1;
    atomicOr(status, code);
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    mbar_wait_limited(bar, parity, kSpinLimit, abort_flag, status, code);
}
// For the control warps (few live registers, code size matters most): the loop is a call.
__device__ __forceinline__ void mbar_wait_call(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (mbar_try_wait(bar, parity)) return;
    mbar_wait_slow(bar, parity, kSpinLimit, abort_flag, status, code);
}
// The same for waiters that run ahead of the pipeline (loaders, the gate warp, epilogue warps): each poll
// lets the hardware suspend the thread for up to `ns` or until the phase completes, so that polling
// does not take issue slots from the arithmetic warps.
__device__ __forceinline__ uint32_t mbar_try_wait_suspend(uint32_t bar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok;
}
static __device__ __noinline__ void mbar_wait_relaxed_slow(uint32_t bar, uint32_t parity, uint32_t ns, volatile int *abort_flag, int *status, int code)
{
    if (*abort_flag) return;
    for (uint32_t it = 0; it < (1u << 20); ++it) {     // bounded: about a second at a microsecond per poll
        if (mbar_try_wait_suspend(bar, parity, ns)) return;
        if ((it & 63) == 63 && *abort_flag) return;
    }
    *abort_flag = 1;
    atomicOr(status, code);
}
template <int SUSPEND_NS>
__device__ __forceinline__ void mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (mbar_try_wait(bar, parity)) return;
    if (*abort_flag) return;
    for (uint32_t it = 0; it < (1u << 20); ++it) {     // bounded: about a second at a microsecond per poll
        if (mbar_try_wait_suspend(bar, parity, SUSPEND_NS)) return;
        if ((it & 63) == 63 && *abort_flag) return;
    }
    *abort_flag = 1;
    atomicOr(status, code);
}
template <int SUSPEND_NS>
__device__ __forceinline__ void mbar_wait_relaxed_call(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status, int code)
{
    if (mbar_try_wait(bar, parity)) return;
    mbar_wait_relaxed_slow(bar, parity, (uint32_t)SUSPEND_NS, abort_flag, status, code);
}
// Same, but ignores the abort flag (used in teardown to drain copies that are in flight).
static __device__ __noinline__ bool mbar_wait_drain(uint32_t bar, uint32_t parity)
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
// The same with each descriptor given as its two 32-bit words: stepping through a tile only changes the
// address field in the low word, so the caller advances 32-bit values.
__device__ __forceinline__ void umma_bf16_words(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                                uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\t"
        "mov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// True in exactly one lane of a converged warp.  (The compiler knows that a region guarded by this
// predicate runs in a single thread and keeps its operands in uniform registers.)
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
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
// Producer side of a named barrier: counts this thread in without waiting.
__device__ __forceinline__ void named_bar_arrive(int id, int count)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
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
    uint32_t r;   // one packed conversion: low half <- lo, high half <- hi (round to nearest even)
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// ------------------------------------------------------------------------------------------
// Epilogue shared by both tensor-core kernels: 16 accumulator columns of one pixel row.
// ------------------------------------------------------------------------------------------
// 16 bias values from global memory as two 32-byte loads (every lane reads the same address: one sector each).
__device__ __forceinline__ void bias16_global(const float *__restrict__ bias, float (&bv)[16])
{
    asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(bv[0]), "=f"(bv[1]), "=f"(bv[2]), "=f"(bv[3]), "=f"(bv[4]), "=f"(bv[5]), "=f"(bv[6]), "=f"(bv[7])
                 : "l"(bias));
    asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(bv[8]), "=f"(bv[9]), "=f"(bv[10]), "=f"(bv[11]), "=f"(bv[12]), "=f"(bv[13]), "=f"(bv[14]), "=f"(bv[15])
                 : "l"(bias + 8));
}
// The same from a copy in shared memory (address of the first of the 16; 16-byte aligned).
__device__ __forceinline__ void bias16_shared(uint32_t addr, float (&bv)[16])
{
#pragma unroll
    for (int j = 0; j < 4; ++j)
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(bv[4 * j]), "=f"(bv[4 * j + 1]), "=f"(bv[4 * j + 2]), "=f"(bv[4 * j + 3]) : "r"(addr + 16 * j));
}
// 16 accumulator columns of one row -> bias, optional ReLU, bf16: eight packed words.
__device__ __forceinline__ void finish_row16(const uint32_t (&acc)[16], const float (&bv)[16], int relu, uint32_t (&o)[8])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float lo = __uint_as_float(acc[2 * j]) + bv[2 * j], hi = __uint_as_float(acc[2 * j + 1]) + bv[2 * j + 1];
        if (relu) { lo = fmaxf(lo, 0.f); hi = fmaxf(hi, 0.f); }
        o[j] = pack_bf16x2(lo, hi);
    }
}
// The same 16 columns kept as fp32 (bias, optional ReLU) and stored to an fp32 row: channels d0 .. d0+15 below D,
// in 16-byte pieces (D is a multiple of 8 for these kernels, the row 16-byte aligned).
__device__ __forceinline__ void finish_store_row16_f32(const uint32_t (&acc)[16], const float (&bv)[16], int relu, int d0, int D,
                                                       float *__restrict__ yrow)
{
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float4 v;
        v.x = __uint_as_float(acc[4 * q]) + bv[4 * q];
        v.y = __uint_as_float(acc[4 * q + 1]) + bv[4 * q + 1];
        v.z = __uint_as_float(acc[4 * q + 2]) + bv[4 * q + 2];
        v.w = __uint_as_float(acc[4 * q + 3]) + bv[4 * q + 3];
        if (relu) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
        if (d0 + 4 * q + 4 <= D) *reinterpret_cast<float4 *>(yrow + d0 + 4 * q) = v;
    }
}
// Flags carried in the kernels' `relu` parameter.
enum : int { kOutRelu = 1, kOutF32 = 2 };
// Stores a row's 16 finished channels d0 .. d0+15 (those below D) to yrow.
__device__ __forceinline__ void store_packed16(const uint32_t (&o)[8], int d0, int D, uint16_t *__restrict__ yrow)
{
    uint16_t *dst = yrow + d0;
    if (d0 + 16 <= D && (reinterpret_cast<uintptr_t>(dst) & 31) == 0) {
        // a lane's 16 outputs are one 32-byte sector: one store instead of two half-sector stores
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"l"(dst), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
    } else {
        if (d0 + 8 <= D) *reinterpret_cast<uint4 *>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
        if (d0 + 16 <= D) *reinterpret_cast<uint4 *>(dst + 8) = make_uint4(o[4], o[5], o[6], o[7]);
    }
}
// `y` is the output tensor's base, `row` the element index of the row's first channel; flags: kOutRelu, kOutF32.
__device__ __forceinline__ void store_row16(const uint32_t (&acc)[16], const float *__restrict__ bias, int d0, int D,
                                            int flags, void *__restrict__ y, size_t row)
{
    float bv[16];
    bias16_global(bias + d0, bv);
    if (flags & kOutF32) {
        finish_store_row16_f32(acc, bv, flags & kOutRelu, d0, D, reinterpret_cast<float *>(y) + row);
    } else {
        uint32_t o[8];
        finish_row16(acc, bv, flags & kOutRelu, o);
        store_packed16(o, d0, D, reinterpret_cast<uint16_t *>(y) + row);
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

inline int tmem_cols_for(int Dpad)
{
    int c = 32;
    while (c < Dpad) c <<= 1;
    return c;
}

// Shared memory to request so that the blocks resident on one SM never ask for more than the
// 512 TMEM columns together (an allocation that cannot be served would wait).
inline size_t smem_for_tmem(size_t need, int cols)
{
    const int max_ctas = 512 / cols;
    const size_t floor_bytes = (size_t)kMaxSmem / (max_ctas + 1) + 1024;
    return need > floor_bytes ? need : floor_bytes;
}


// TMA tiled load of a rank-4 box; coordinates innermost first.  The innermost coordinate times the
// element size must be a multiple of 16 bytes (here: a multiple of 8 channels).
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *tmap, int c0, int c1, int c2, int c3,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}

// TMA tiled store of a rank-4 box from shared memory (bulk async-group completion).  Coordinates
// innermost first and non-negative; elements outside the tensor are not written.
__device__ __forceinline__ void tma_store_4d(uint32_t src, const CUtensorMap *tmap, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
        ::"l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Until the bulk stores this thread committed have read their shared-memory source.
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// Until they are complete.
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// TMA tiled load of a rank-2 box (innermost coordinate first; it must start on a 16-byte boundary).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tmap, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

// cuTensorMapEncodeTiled, looked up through the runtime (no link against the driver library).
typedef CUresult (*tensor_map_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                         const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                         CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                         CUtensorMapFloatOOBfill);

inline tensor_map_encode_fn encode_fn()
{
    static tensor_map_encode_fn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (tensor_map_encode_fn)p;
    }
    return fn;
}


}  // namespace gdws
