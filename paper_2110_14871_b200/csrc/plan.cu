// Host side of libgdws: plan construction, options, queries, tile choice, errors.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "gdws_internal.h"

namespace gdws {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

gdws_status_t fail(gdws_status_t st, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return st;
}

gdws_status_t cuda_fail(cudaError_t e, const char *what)
{
    snprintf(g_err, sizeof(g_err), "%s: %s", what, cudaGetErrorString(e));
    return GDWS_ERR_CUDA;
}

gdws_status_t check_arch()
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
    if (major != 10)
        return fail(GDWS_ERR_ARCH, "device %d has compute capability %d.x; this library needs 10.x (sm_100a)", dev, major);
    return GDWS_OK;
}

static void free_device(gdws_plan_s *p)
{
    if (p->device < 0) return;
    int cur = 0;
    cudaGetDevice(&cur);
    cudaSetDevice(p->device);
    cudaDeviceSynchronize();
    // every pointer is cleared as it is freed: a plan that outlives a failed set-up is set up again from scratch
    auto release = [](auto *&ptr) { cudaFree(ptr); ptr = nullptr; };
    release(p->d_off);
    release(p->d_chan);
    release(p->d_chunk_meta);
    release(p->d_dw);
    release(p->d_dwpack);
    release(p->d_pw_img);
    release(p->d_bias);
    release(p->d_status);
    release(p->d_tc_chunks);
    release(p->d_tc_filt);
    release(p->d_tc_pw);
    release(p->stage_x);
    release(p->stage_y);
    p->stage_x_bytes = 0;
    p->stage_y_bytes = 0;
    p->packed = false;
    cudaSetDevice(cur);
    p->device = -1;
}

gdws_status_t ensure_device(gdws_plan_s *p)
{
    if (p->device >= 0) return GDWS_OK;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    const size_t k2 = (size_t)p->k * p->k;
    const size_t img = (size_t)p->nchunks * p->Dpad * kChunk * sizeof(uint16_t);
#define GDWS_TRY_ALLOC(ptr, bytes)                                                   \
    do {                                                                             \
        e = cudaMalloc((void **)&(ptr), (bytes));                                    \
        if (e != cudaSuccess) {                                                      \
            p->device = dev;                                                         \
            free_device(p);                                                          \
            cudaGetLastError();                                                      \
            return fail(GDWS_ERR_ALLOC, "cudaMalloc(%zu) failed: %s", (size_t)(bytes), cudaGetErrorString(e)); \
        }                                                                            \
    } while (0)
    GDWS_TRY_ALLOC(p->d_off, sizeof(int32_t) * (p->C + 1));
    GDWS_TRY_ALLOC(p->d_chan, sizeof(int32_t) * p->Gpad);
    GDWS_TRY_ALLOC(p->d_chunk_meta, sizeof(int32_t) * 4 * p->nchunks);
    GDWS_TRY_ALLOC(p->d_dw, sizeof(float) * p->Gpad * k2);
    GDWS_TRY_ALLOC(p->d_dwpack, sizeof(uint32_t) * p->Gpad * p->wstride);
    GDWS_TRY_ALLOC(p->d_pw_img, img);
    GDWS_TRY_ALLOC(p->d_bias, sizeof(float) * p->Dpad);
    GDWS_TRY_ALLOC(p->d_status, sizeof(int));
    if (p->tc_ok) {
        GDWS_TRY_ALLOC(p->d_tc_chunks, sizeof(TcChunk) * p->tc_chunks.size());
        GDWS_TRY_ALLOC(p->d_tc_filt, sizeof(uint16_t) * (size_t)p->tc_nslabs * 16 * p->tc_rec_hw);
        GDWS_TRY_ALLOC(p->d_tc_pw, sizeof(uint16_t) * (size_t)p->tc_nparts * p->tc_nslabs * 16 * p->tc_dloc);
    }
#undef GDWS_TRY_ALLOC
    p->device = dev;
    if (cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) p->sm_count = 0;
    e = cudaMemcpy(p->d_off, p->off.data(), sizeof(int32_t) * (p->C + 1), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(p->d_chan, p->chan.data(), sizeof(int32_t) * p->Gpad, cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(p->d_chunk_meta, p->chunk_meta.data(), sizeof(int32_t) * 4 * p->nchunks, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && p->tc_ok)
        e = cudaMemcpy(p->d_tc_chunks, p->tc_chunks.data(), sizeof(TcChunk) * p->tc_chunks.size(), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(p->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(p->d_bias, 0, sizeof(float) * p->Dpad);
    if (e != cudaSuccess) {
        free_device(p);
        return cuda_fail(e, "plan table upload");
    }
    // The built-in scratch array of gdws_forward_static is part of a module that the first look-up of its
    // address may load (committing its 16 MiB on this device): do that here, where allocation is expected.
    static_scratch_prepare(dev);
    return GDWS_OK;
}

static int round_up(int a, int b) { return (a + b - 1) / b * b; }

// Chunk list of the tensor-core GDW path.  The input channels are taken in windows of 16 (what one tensor-core
// instruction contracts over); a window's intermediate channels (Property 2: contiguous, in channel order) form
// one chunk, or several of equal size when there are more than the path handles at once.
static void build_tc_chunks(gdws_plan_s *p)
{
    p->tc_ok = false;
    if (p->stride > 2 || p->k > 5 || p->C % 8 || p->D % 8 || p->Dpad > 1024) return;
    p->tc_nparts = (p->Dpad + 255) / 256;
    p->tc_dloc = round_up((p->Dpad + p->tc_nparts - 1) / p->tc_nparts, 16);
    const int nmax = tc_nmax(p->k, p->tc_dloc);
    p->tc_rec_hw = round_up(1 + p->k * p->k, 8);
    int slab = 0;
    for (int c0 = 0; c0 < p->C; c0 += 16) {
        const int c1 = std::min(p->C, c0 + 16);
        const int i0 = p->off[c0], n = p->off[c1] - i0;
        if (n == 0) continue;
        const int pieces = (n + nmax - 1) / nmax;
        const int size = round_up((n + pieces - 1) / pieces, 16);
        for (int done = 0, piece = 0; done < n; done += size, ++piece) {
            TcChunk ch = {};
            ch.cbase = c0;
            ch.i0 = i0 + done;
            ch.n = std::min(size, n - done);
            ch.npad = round_up(ch.n, 16);
            ch.slab0 = slab;
            ch.flags = (done == 0 ? 1 : 0) | (done + size >= n ? 2 : 0);
            slab += ch.npad / 16;
            p->tc_maxslabs = std::max(p->tc_maxslabs, ch.npad / 16);
            p->tc_chunks.push_back(ch);
        }
    }
    p->tc_nslabs = slab;
    p->tc_ok = !p->tc_chunks.empty();
}

// Shared-memory layout of the fused bf16 kernel: 2 * t.spg intermediate-tile stages, a ring of `nsb`
// pointwise-weight units (a unit = one K chunk x up to 256 output channels, at most 32 KB) and
// `nslots` staged-input slots (one TMA box), a ring of filter blocks and, where the epilogue stores by TMA,
// one output staging buffer.  Fills t.nsb / t.nslots / t.nwslots / t.ostage / t.smem; false if it cannot fit.  Prefers at least 3 chunks of weights and 4 input slots in flight.
static bool fit_smem(const gdws_plan_s *p, Tile &t, bool stage_out, bool several_tiles)
{
    const size_t a = 2 * (size_t)t.spg * kTileRows * kChunk * 2;
    const int nhalf = p->Dpad > 256 ? 2 : 1;
    const size_t unit = (size_t)(p->Dpad > 256 ? 256 : p->Dpad) * kChunk * 2;
    const size_t slot = (size_t)t.slot_bytes;
    const size_t wblock = (size_t)kChunk * p->wstride * 4;                 // one chunk's filters
    t.nwslots = 3;                   // at least: two groups at work and one block in flight
    // Output channels in whole 64-column blocks: the epilogue stages 128 rows x 64 columns and stores them by TMA.
    // (Not beyond 256 channels: there the weight ring needs the shared memory more.)
    t.ostage = stage_out && p->D % 64 == 0 && p->Dpad <= 256 ? kTileRows * 128 : 0;
    const size_t fixed = a + t.ostage + 1024 /*alignment slack*/ + t.nwslots * wblock + (size_t)p->nchunks * 16 /*chunk table*/ + (size_t)p->Dpad * 4 /*bias*/;
    int best_score = -1;
    for (int ns = 2; ns <= 8; ++ns) {
        if (fixed + ns * slot + (size_t)(nhalf + 1) * unit > (size_t)kMaxSmem) break;
        int nsb = (int)(((size_t)kMaxSmem - fixed - ns * slot) / unit);
        if (nsb > 8) nsb = 8;
        const int depth_b = nsb / nhalf;
        const int score = 100 * std::min(std::min(depth_b, ns), 4) + 10 * std::min(depth_b, 6) + ns;
        if (score > best_score) {
            best_score = score;
            t.nsb = nsb;
            t.nslots = ns;
            t.smem = fixed + nsb * unit + ns * slot;
        }
    }
    if (best_score < 0) return false;
    // With several tiles per block, what is left goes to a deeper filter ring: a block released by the depthwise
    // warps comes back through the loader, the copy and the gate warp only thousands of cycles later.  (Measured:
    // 4 % faster on the 64-channel layers; a block with a single tile is 4 % slower with the deeper ring.)
    while (several_tiles && t.nwslots < 6 && t.smem + wblock <= (size_t)kMaxSmem) { ++t.nwslots; t.smem += wblock; }
    return true;
}

bool choose_tile(const gdws_plan_s *p, int n, int h, int w, Tile *out)
{
    const int Ho = gdws_out_dim(h, p->k, p->stride, p->pad);
    const int Wo = gdws_out_dim(w, p->k, p->stride, p->pad);
    if (n < 1 || Ho < 1 || Wo < 1) return false;
    const int cbox = p->cbox;
    if (cbox <= 0) return false;            // some chunk reads more than 128 channels: no fused kernel
    const int sms = sm_count_of(p);
    double best = 1e300;
    bool found = false;
    const int forced = p->opt_tile;
    const bool fast_shape = (p->k == 3 || p->k == 5) && (p->stride == 1 || p->stride == 2) && p->opt_a_layout == 0;
    static const int pws[4] = {32, 16, 8, 4};
    for (int pi = 0; pi < 4; ++pi) {
        const int PW = pws[pi];
        for (int PH = 1; PH * PW <= kTileRows; ++PH) {
            if (PW == 4 && (PH & 1)) continue;   // 4-wide patches pair two rows into one 8-pixel group
            const int maxTN = kTileRows / (PH * PW);
            for (int TN = 1; TN <= maxTN; ++TN) {
                if (TN > 1 && (PH * PW) % 8) continue;
                Tile t;
                t.TN = TN; t.PH = PH; t.PW = PW;
                if (fast_shape && PW >= 8 && PH % 4 == 0) t.fast = 1;
                else if (fast_shape && p->k == 3 && PW == 4) t.fast = 2;
                if (forced) {
                    if (TN != ((forced >> 16) & 0xff) || PH != ((forced >> 8) & 0xff) || PW != (forced & 0xff)) continue;
                } else if (fast_shape && p->k == 3 && !t.fast) {
                    continue;                    // k = 3: every shape has a tile that a specialised depthwise path covers
                }
                t.tiles_w = (Wo + PW - 1) / PW;
                t.tiles_h = (Ho + PH - 1) / PH;
                t.tiles_n = (n + TN - 1) / TN;
                t.IH = (PH - 1) * p->stride + p->k;
                t.IW = (PW - 1) * p->stride + p->k;
                if (t.IH > 256 || t.IW > 256 || TN > 256) continue;      // TMA box extents
                t.cbox = cbox;
                t.box_bytes = TN * t.IH * t.IW * cbox * 2;
                t.slot_bytes = round_up(t.box_bytes, 128);
                for (int variant = 0; variant < 4; ++variant) {
                    // one operand stage per group costs some overlap, an epilogue without staging costs store bandwidth
                    t.spg = 2 - (variant & 1);
                    const bool stage_out = variant < 2;
                    if (stage_out && t.tiles() <= sms) continue;     // staging pays only when a block has several tiles
                    if (!fit_smem(p, t, stage_out, t.tiles() > sms)) continue;
                    const double tiles = (double)t.tiles();
                    const double cost = tiles * (128.0 + 0.3 * TN * t.IH * t.IW) * (t.fast ? 1.0 : 4.0) * (t.spg == 1 ? 1.08 : 1.0) *
                                            (stage_out ? 1.0 : 1.07) - 1e-3 * PW;
                    if (cost < best) { best = cost; *out = t; found = true; }
                }
            }
        }
    }
    return found;
}

}  // namespace gdws

using namespace gdws;

extern "C" {

int gdws_out_dim(int in, int k, int stride, int pad)
{
    if (k < 1 || stride < 1) return 0;
    const int span = in + 2 * pad - k;
    return span < 0 ? 0 : span / stride + 1;
}

gdws_status_t gdws_plan(int C, int D, int k, int stride, int pad, const int32_t *g, gdws_plan_t **out)
{
    if (!out) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: out is NULL");
    *out = nullptr;
    if (!g) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: g is NULL");
    if (C < 1 || D < 1) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: C=%d, D=%d must be >= 1", C, D);
    if (C > (1 << 20) || D > (1 << 20)) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: C or D too large");
    if (k < 1 || k > kMaxK) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: k=%d outside 1..%d", k, kMaxK);
    if (stride < 1 || stride > 4) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: stride=%d outside 1..4", stride);
    if (pad < 0 || pad > k) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: pad=%d outside 0..k", pad);
    int64_t G = 0;
    for (int c = 0; c < C; ++c) {
        if (g[c] < 0) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: g[%d]=%d is negative", c, g[c]);
        if (g[c] > (1 << 16)) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: g[%d]=%d too large", c, g[c]);
        G += g[c];
    }
    if (G < 1) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: sum of g is 0");
    if (G > (1 << 24)) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan: sum of g too large");
    gdws_plan_s *p = new (std::nothrow) gdws_plan_s;
    if (!p) return fail(GDWS_ERR_ALLOC, "gdws_plan: out of host memory");
    p->C = C; p->D = D; p->k = k; p->stride = stride; p->pad = pad;
    p->G = (int)G;
    p->Gpad = round_up((int)G, kChunk);
    p->Dpad = round_up(D, 16);
    p->nchunks = p->Gpad / kChunk;
    p->wstride = round_up(k * k + 1, 4);
    try {
        p->g.assign(g, g + C);
        p->off.resize(C + 1);
        p->chan.assign(p->Gpad, -1);
    } catch (...) {
        delete p;
        return fail(GDWS_ERR_ALLOC, "gdws_plan: out of host memory");
    }
    int32_t acc = 0;
    for (int c = 0; c < C; ++c) {          // Property 2: rows of channel c start at off_c
        p->off[c] = acc;
        for (int j = 0; j < g[c]; ++j) p->chan[acc + j] = c;
        acc += g[c];
    }
    p->off[C] = acc;
    try {
        p->chunk_c0.assign(p->nchunks, 0);
    } catch (...) {
        delete p;
        return fail(GDWS_ERR_ALLOC, "gdws_plan: out of host memory");
    }
    try {
        p->chunk_c1.assign(p->nchunks, 0);
        p->chunk_meta.assign((size_t)p->nchunks * 4, 0);
    } catch (...) {
        delete p;
        return fail(GDWS_ERR_ALLOC, "gdws_plan: out of host memory");
    }
    for (int q = 0; q < p->nchunks; ++q) {   // channel range read by K chunk q
        const int lo = p->chan[q * kChunk];
        const int last = std::min(p->G, (q + 1) * kChunk) - 1;
        p->chunk_c0[q] = lo;
        p->chunk_c1[q] = p->chan[last];
        p->span_max = std::max(p->span_max, p->chan[last] - (lo & ~7) + 1);
    }
    // Group consecutive chunks into input boxes of cbox channels (32, 64 or 128): take the size that
    // moves the fewest channels per tile, but no more than 64 unless a single chunk needs it.
    {
        long best_cost = -1;
        for (int cb = 32; cb <= 128; cb *= 2) {
            if (cb < p->span_max) continue;
            if (cb > 64 && best_cost >= 0) break;
            if (cb > 32 && best_cost >= 0 && p->Dpad >= 256) break;   // wide layers: shared memory goes to the weight ring
            int nb = 0;
            for (int q = 0; q < p->nchunks;) {
                const int cbase = p->chunk_c0[q] & ~7;
                int e = q;
                while (e + 1 < p->nchunks && p->chunk_c1[e + 1] < cbase + cb) ++e;
                q = e + 1;
                ++nb;
            }
            const long cost = (long)nb * cb;
            if (best_cost < 0 || cost < best_cost) { best_cost = cost; p->cbox = cb; p->nboxes = nb; }
        }
        if (p->cbox > 0) {
            int b = 0;
            for (int q = 0; q < p->nchunks; ++b) {
                const int cbase = p->chunk_c0[q] & ~7;
                int e = q;
                while (e + 1 < p->nchunks && p->chunk_c1[e + 1] < cbase + p->cbox) ++e;
                for (int c = q; c <= e; ++c) {
                    int flags = 0;
                    if (c == e || c == e - 1) flags |= 1;
                    if (q == e) flags |= 2;
                    if (c == q) flags |= 4;
                    if (c == q || c == q + 1) flags |= 8;
                    p->chunk_meta[4 * c + 0] = b;
                    p->chunk_meta[4 * c + 1] = flags;
                    p->chunk_meta[4 * c + 2] = cbase;
                }
                q = e + 1;
            }
        }
    }
    try {
        build_tc_chunks(p);
    } catch (...) {
        delete p;
        return fail(GDWS_ERR_ALLOC, "gdws_plan: out of host memory");
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) == cudaSuccess && ndev > 0) {
        gdws_status_t st = ensure_device(p);
        if (st != GDWS_OK) { delete p; return st; }
    } else {
        cudaGetLastError();
    }
    *out = p;
    return GDWS_OK;
}

gdws_status_t gdws_plan_set_option(gdws_plan_t *p, int key, int value)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan_set_option: plan is NULL");
    switch (key) {
    case GDWS_OPT_PATH:
        if (value < GDWS_PATH_AUTO || value > GDWS_PATH_UNFUSED) return fail(GDWS_ERR_INVALID_ARG, "bad path %d", value);
        p->opt_path = value; return GDWS_OK;
    case GDWS_OPT_RELU:
        if (value != 0 && value != 1) return fail(GDWS_ERR_INVALID_ARG, "relu must be 0 or 1");
        p->opt_relu = value; return GDWS_OK;
    case GDWS_OPT_TILE: {
        if (value != 0) {
            const int TN = (value >> 16) & 0xff, PH = (value >> 8) & 0xff, PW = value & 0xff;
            if (!(PW == 4 || PW == 8 || PW == 16 || PW == 32) || TN < 1 || PH < 1 || TN * PH * PW > kTileRows ||
                (PW == 4 && (PH & 1)) || (TN > 1 && (PH * PW) % 8))
                return fail(GDWS_ERR_INVALID_ARG, "bad tile TN=%d PH=%d PW=%d", TN, PH, PW);
        }
        p->opt_tile = value; return GDWS_OK;
    }
    case GDWS_OPT_A_LAYOUT:
        if (value != 0 && value != 1) return fail(GDWS_ERR_INVALID_ARG, "a_layout must be 0 or 1");
        p->opt_a_layout = value; return GDWS_OK;
    case GDWS_OPT_DW_MATH:
        if (value < 0 || value > 2) return fail(GDWS_ERR_INVALID_ARG, "dw_math must be 0, 1 or 2");
        p->opt_dw_math = value; return GDWS_OK;
    case GDWS_OPT_OUT_DTYPE:
        if (value != 0 && value != 1) return fail(GDWS_ERR_INVALID_ARG, "out_dtype must be 0 (as x) or 1 (fp32)");
        p->opt_out_f32 = value; return GDWS_OK;
    default:
        return fail(GDWS_ERR_INVALID_ARG, "unknown option %d", key);
    }
}

gdws_status_t gdws_plan_info(const gdws_plan_t *p, int *G, int *G_pad, int64_t *macs_per_pixel, int64_t *params)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan_info: plan is NULL");
    if (G) *G = p->G;
    if (G_pad) *G_pad = p->Gpad;
    const int64_t v = (int64_t)p->G * ((int64_t)p->k * p->k + p->D);   // Eq. 3 per output pixel
    if (macs_per_pixel) *macs_per_pixel = v;
    if (params) *params = v;
    return GDWS_OK;
}

gdws_status_t gdws_plan_tables(const gdws_plan_t *p, int32_t *off, int32_t *chan)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan_tables: plan is NULL");
    if (off) memcpy(off, p->off.data(), sizeof(int32_t) * (p->C + 1));
    if (chan) memcpy(chan, p->chan.data(), sizeof(int32_t) * p->Gpad);
    return GDWS_OK;
}

gdws_status_t gdws_plan_tile(const gdws_plan_t *p, int n, int h, int w, int *TN, int *PH, int *PW, int64_t *tiles)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan_tile: plan is NULL");
    Tile t;
    if (!choose_tile(p, n, h, w, &t))
        return fail(GDWS_ERR_UNSUPPORTED, "no fused tile fits n=%d h=%d w=%d", n, h, w);
    if (TN) *TN = t.TN;
    if (PH) *PH = t.PH;
    if (PW) *PW = t.PW;
    if (tiles) *tiles = t.tiles();
    return GDWS_OK;
}

size_t gdws_workspace_bytes(const gdws_plan_t *p, gdws_dtype_t dtype, int n, int h, int w)
{
    if (!p || n < 1) return 0;
    const int Ho = gdws_out_dim(h, p->k, p->stride, p->pad);
    const int Wo = gdws_out_dim(w, p->k, p->stride, p->pad);
    if (Ho < 1 || Wo < 1) return 0;
    const size_t px = (size_t)n * Ho * Wo;
    if (dtype == GDWS_F32) return px * p->G * sizeof(float);
    if (dtype == GDWS_BF16) return px * p->Gpad * sizeof(uint16_t);
    return 0;
}

gdws_status_t gdws_set_workspace(gdws_plan_t *p, void *ws, size_t bytes)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_set_workspace: plan is NULL");
    if (ws && ((uintptr_t)ws & 255)) return fail(GDWS_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    p->ws = ws;
    p->ws_bytes = ws ? bytes : 0;
    return GDWS_OK;
}

gdws_status_t gdws_plan_gdw_stage(const gdws_plan_t *p, int *stage)
{
    if (!p || !stage) return fail(GDWS_ERR_INVALID_ARG, "gdws_plan_gdw_stage: NULL argument");
    *stage = gdw_stage_of(p);
    return GDWS_OK;
}

int64_t gdws_launch_count(const gdws_plan_t *p) { return p ? p->launches : 0; }

const char *gdws_last_error(void) { return gdws::g_err; }

const char *gdws_version(void) { return "gdws-b200 0.1.0 (sm_100a)"; }

void gdws_destroy(gdws_plan_t *p)
{
    if (!p) return;
    free_device(p);
    delete p;
}

}  // extern "C"
