// Internal declarations shared by the translation units of libgdws.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <utility>
#include <vector>

#include "gdws.h"

namespace gdws {

constexpr int kChunk = 64;          // intermediate channels per tensor-core K chunk (one 128-byte swizzle row of bf16)
constexpr int kTileRows = 128;      // output pixels per tensor-core tile (UMMA M)
constexpr int kMaxK = 7;
constexpr int kMaxSmem = 225 * 1024;      // dynamic shared memory a block may ask for (227 KB minus static use)

// Bits of the device status word.
enum : int {
    kStatusWaitStage = 1,   // wait for a free shared-memory stage ran out
    kStatusWaitOperand = 2, // wait for an operand (bulk copy / producer warps) ran out
    kStatusWaitMma = 4,     // wait for the tensor-core commit ran out
};

// One unit of work of the tensor-core GDW path: the intermediate channels i0 .. i0+n-1, all fed by the
// 16 input channels cbase .. cbase+15 (a "window"; cbase is a multiple of 16).  Windows whose channels
// produce more than the path's limit of intermediate channels are cut into several chunks.
struct TcChunk {
    int32_t cbase;       // first input channel of the window
    int32_t i0;          // first intermediate channel (canonical order, Property 2)
    int32_t n;           // intermediate channels of the chunk
    int32_t npad;        // n rounded up to a multiple of 16 (columns of the GDW product, K of the PW product)
    int32_t slab0;       // index of the chunk's first 16-channel slab in the packed arrays
    int32_t flags;       // 1: first chunk of its window (its input box is fetched), 2: last chunk of its window
    int32_t reserved0, reserved1;
};

// Most intermediate channels one chunk of the tensor-core GDW path holds: its B operands (32 bytes per channel and
// tap; up to 9 taps per buffer) must fit shared memory twice, and two GDW
// accumulators must fit beside the PW accumulator in TMEM.
inline int tc_nmax(int k, int dloc) { (void)k; return dloc > 128 ? 96 : 128; }

struct Tile {
    int TN = 0, PH = 0, PW = 0;      // images x rows x columns of output pixels per 128-row tile
    int tiles_n = 0, tiles_h = 0, tiles_w = 0;
    int IH = 0, IW = 0;              // input patch rows / columns per image (with halo)
    int cbox = 0;                    // channels per staged box (32, 64 or 128)
    int box_bytes = 0;               // TN*IH*IW*cbox*2: one TMA box
    int slot_bytes = 0;              // box rounded up to 128
    int nslots = 0;                  // staged-input slots (boxes in flight)
    int nwslots = 0;                 // filter blocks in flight (one per chunk)
    int nsb = 0;                     // pointwise-weight units in the ring
    int spg = 2;                     // operand stages per depthwise group (1 or 2)
    int ostage = 0;                  // bytes of output staging for the TMA-store epilogue (0: direct stores)
    int fast = 0;                    // 1: row-run depthwise path, 2: 4-wide-patch path, 0: generic
    size_t smem = 0;                 // dynamic shared memory of the fused kernel
    int64_t tiles() const { return (int64_t)tiles_n * tiles_h * tiles_w; }
};

}  // namespace gdws

struct gdws_plan_s {
    int C = 0, D = 0, k = 0, stride = 0, pad = 0;
    int G = 0, Gpad = 0, Dpad = 0, nchunks = 0;
    int wstride = 0;                 // 32-bit words per intermediate channel in d_dwpack (multiple of 4)
    std::vector<int32_t> g, off, chan;
    std::vector<int32_t> chunk_c0;   // first input channel read by K chunk q (intermediate channels 64q..64q+63)
    std::vector<int32_t> chunk_c1;   // last input channel read by K chunk q
    int span_max = 0;                // widest channel range of one K chunk, counted from the chunk's first
                                     // channel rounded down to a multiple of 8 (a staged box starts there)
    // Input boxes of the fused kernel: consecutive chunks whose channels fit into one box of `cbox`
    // channels share it.  chunk_meta[q] = {box index within the tile, flags, first channel of the box, 0};
    // flags: 1 = this chunk releases the box when done (last or second-to-last chunk using it),
    // 2 = it is the only chunk of its box (releases twice), 4 = first chunk of its box (the loader fetches it),
    // 8 = first or second chunk of its box (must wait for the box to land).
    int cbox = 0, nboxes = 0;
    std::vector<int32_t> chunk_meta; // 4 ints per chunk

    // Tensor-core GDW path (fused_tc.cu): chunk list, output-channel split, packed sizes.
    bool tc_ok = false;              // the layer is one the path covers (stride 1, k <= 5, ...)
    std::vector<gdws::TcChunk> tc_chunks;
    // last layout of the tensor-core path's slab rings (chunk order within a work item, places and waits), kept per
    // ring sizes: working it out tries a few dozen orders
    int tc_lay_nz = 0, tc_lay_nw = 0;
    std::vector<uint8_t> tc_lay_order;
    std::vector<uint32_t> tc_lay_ring;
    int tc_nslabs = 0;               // sum of npad / 16 over the chunks
    int tc_maxslabs = 0;             // largest npad / 16 of one chunk
    int tc_nparts = 1, tc_dloc = 0;  // blocks per tile along D, output channels per block (multiple of 16, <= 256)
    int tc_rec_hw = 0;               // 16-bit words per filter record (channel slot, then k*k taps; multiple of 8)

    int opt_path = GDWS_PATH_AUTO;
    int opt_relu = 0;
    int opt_tile = 0;
    int opt_a_layout = 0;
    int opt_dw_math = 0;
    int opt_out_f32 = 0;           // bf16 plans: y is fp32

    // device side (allocated by ensure_device)
    int device = -1;
    int sm_count = 0;              // SMs of the plan's device (grid size of the persistent kernel)
    bool arch_ok = false;          // the plan's device was checked to be compute capability 10.x
    int32_t *d_off = nullptr;      // [C+1]
    int32_t *d_chan = nullptr;     // [Gpad], -1 for padding
    int32_t *d_chunk_meta = nullptr; // [nchunks][4]
    float *d_dw = nullptr;         // [Gpad][k*k] fp32 depthwise filters, zero rows for padding
    uint32_t *d_dwpack = nullptr;  // [Gpad][wstride]: k*k fp32 filter taps, then the channel's index within its K chunk's slot
    uint16_t *d_pw_img = nullptr;  // [nchunks][Dpad*64] bf16, 128-byte-swizzled K-major operand images
    float *d_bias = nullptr;       // [Dpad]
    gdws::TcChunk *d_tc_chunks = nullptr;
    uint16_t *d_tc_filt = nullptr; // [tc_nslabs * 16][tc_rec_hw]: per intermediate slot, channel index inside the window and the taps (bf16)
    uint16_t *d_tc_pw = nullptr;   // [tc_nparts][tc_nslabs][2][tc_dloc][8] bf16: pointwise weights, one K = 16 operand slab per 16 slots
    int *d_status = nullptr;       // device status word
    bool packed = false;

    void *ws = nullptr;
    size_t ws_bytes = 0;

    void *stage_x = nullptr, *stage_y = nullptr;  // gdws_forward_host staging
    size_t stage_x_bytes = 0, stage_y_bytes = 0;

    int64_t launches = 0;
};

namespace gdws {

void set_error(const char *fmt, ...);
gdws_status_t fail(gdws_status_t st, const char *fmt, ...);
gdws_status_t cuda_fail(cudaError_t e, const char *what);
gdws_status_t ensure_device(gdws_plan_s *p);   // allocate device tables on the current device
gdws_status_t check_arch();

// Launch with programmatic stream serialisation: the kernel may be scheduled while the kernel before it in the stream
// is still running (once all blocks of that one have executed griddepcontrol.launch_dependents, which the library's
// kernels do first thing).  Such a kernel touches global memory only after its own griddepcontrol.wait.
template <class... KArgs, class... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
// x and y of a forward call against the plan: pointers, alignment, extents, dtype/layout pair, no overlap
gdws_status_t check_pair(const gdws_plan_s *p, const gdws_tensor_t *x, const gdws_tensor_t *y);
// static_ws.cu: looks up (once per device, the device being current) the address of the built-in scratch array
gdws_status_t static_scratch_prepare(int device);
bool choose_tile(const gdws_plan_s *p, int n, int h, int w, Tile *t);

inline size_t dtype_size(gdws_dtype_t d) { return d == GDWS_F32 ? 4 : 2; }

// Where the fused bf16 kernel runs the GDW stage: 1 = ALUs, 2 = tensor cores.  With the option left at 0 the
// tensor cores are taken where they measured faster on B200: their cost is k*k products per 16-channel window
// whatever the multipliers, the ALU kernel's is proportional to G (and its stride-2 code reuses less of each input
// row), and beyond 256 output channels the tensor-core kernel computes the GDW stage once per 256 of them.
inline int gdw_stage_of(const gdws_plan_s *p)
{
    if (p->opt_dw_math == 1 || p->opt_dw_math == 2) return p->opt_dw_math;
    if (!(p->tc_ok && (p->k == 3 || p->k == 5) && p->stride <= 2)) return 1;
    if (p->stride == 1 && p->Dpad > 256) return 1;     // measured equal or slower there; with stride 2 faster at D = 512 too
    // average multiplier of at least 4, or of at least 2.7 when the PW products are small (at most 128 output channels)
    return (p->G >= 4 * p->C || (p->Dpad <= 128 && 10 * (long long)p->G >= 27 * (long long)p->C)) ? 2 : 1;
}

// SMs of the plan's device; a plan built without a device (host-side queries only) assumes a B200's 148.
constexpr int kB200Sms = 148;
inline int sm_count_of(const gdws_plan_s *p) { return p->sm_count > 0 ? p->sm_count : kB200Sms; }

// f32.cu
gdws_status_t f32_depthwise(gdws_plan_s *p, const gdws_tensor_t *x, const float *dw_w, float *z, cudaStream_t s);
gdws_status_t f32_pointwise(gdws_plan_s *p, const float *z, const float *pw_w, const float *bias,
                            gdws_tensor_t *y, cudaStream_t s);
gdws_status_t f32_fused(gdws_plan_s *p, const gdws_tensor_t *x, const float *dw_w, const float *pw_w,
                        const float *bias, gdws_tensor_t *y, cudaStream_t s);

// bf16.cu
gdws_status_t bf16_pack(gdws_plan_s *p, const void *dw_w, const void *pw_w, const float *bias,
                        gdws_dtype_t dtype, cudaStream_t s);
gdws_status_t bf16_depthwise(gdws_plan_s *p, const gdws_tensor_t *x, void *z, cudaStream_t s);
gdws_status_t bf16_pointwise(gdws_plan_s *p, const void *z, gdws_tensor_t *y, cudaStream_t s);
gdws_status_t bf16_fused(gdws_plan_s *p, const gdws_tensor_t *x, gdws_tensor_t *y, cudaStream_t s);
gdws_status_t bf16_depthwise_tiled(gdws_plan_s *p, const gdws_tensor_t *x, void *z, cudaStream_t s);

// fused_tc.cu
void tc_pack(gdws_plan_s *p, const void *dw_w, const void *pw_w, int is_bf16, cudaStream_t s);
gdws_status_t bf16_fused_tc(gdws_plan_s *p, const gdws_tensor_t *x, gdws_tensor_t *y, cudaStream_t s);

}  // namespace gdws
