/*
 * gdws.h -- C interface of the GDWS convolution forward library for NVIDIA B200 (sm_100a).
 *
 * A (C,K,g,M) generalized depthwise-separable (GDWS) convolution (arXiv 2110.14871,
 * Section 3.1, Definition) is a (C,K,g) generalized depthwise (GDW) convolution --
 * input channel c is convolved with g_c depthwise KxK filters, giving G = sum_c g_c
 * intermediate channels of size H'xW' -- followed by a (G,1,M) pointwise (PW)
 * convolution.  In this interface M is called D, K is called k.
 *
 *   z[n,i,h',w'] = sum_{u,v<k} dw_w[i,u,v] * xpad[n, c(i), h'*stride+u-pad, w'*stride+v-pad]
 *   y[n,d,h',w'] = bias[d] + sum_{i<G} pw_w[d,i] * z[n,i,h',w']          (optionally ReLU)
 *
 * with i = off_c + j, j < g_c, off_c = sum_{c'<c} g_c' (the row order of W_D in
 * Property 2 / Fig. 3, 0-based), xpad = x extended by zeros, no filter flip,
 * H' = floor((H + 2 pad - k)/stride) + 1 and W' likewise.  pw_w is W_P (M x G,
 * Property 1), dw_w holds the non-zero rows of W_D, taps row-major.  The bias is
 * not part of the paper's operator; it is the bias of the layer being replaced.
 *
 * General rules
 *   - Every function returns a gdws_status_t (GDWS_OK = 0) unless stated; nothing
 *     throws or aborts.  gdws_last_error() gives a thread-local message for the
 *     last failing call of the calling thread.
 *   - Pointers are marked HOST or DEVICE.  Device buffers are owned by the caller,
 *     must be 16-byte aligned, must stay valid until the stream work that uses them
 *     has finished, and outputs must not overlap inputs.
 *   - Calls that take a stream only enqueue work on it (cudaStream_t passed as
 *     void*; NULL is the default stream) and never synchronise, except where noted.
 *   - A plan may be used by one host thread at a time; different plans are independent.
 *   - The library runs only on compute capability 10.x devices.  There is no
 *     fallback path: on any other device gdws_forward returns GDWS_ERR_ARCH.
 */
#ifndef GDWS_H_
#define GDWS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define GDWS_API
#else
#define GDWS_API __attribute__((visibility("default")))
#endif

typedef struct gdws_plan_s gdws_plan_t; /* opaque, owned by the library */

typedef enum {
    GDWS_OK = 0,
    GDWS_ERR_INVALID_ARG = 1,    /* bad pointer, size, alignment or enum value            */
    GDWS_ERR_UNSUPPORTED = 2,    /* valid request that this build has no kernel for       */
    GDWS_ERR_ALLOC = 3,          /* host or device allocation failed                      */
    GDWS_ERR_CUDA = 4,           /* a CUDA runtime call or a kernel launch failed         */
    GDWS_ERR_DEVICE_TIMEOUT = 5, /* a bounded wait inside a kernel ran out (status word)  */
    GDWS_ERR_ARCH = 6,           /* current device is not compute capability 10.x         */
    GDWS_ERR_WORKSPACE = 7       /* the chosen path needs a workspace that was not set    */
} gdws_status_t;

typedef enum { GDWS_F32 = 0, GDWS_BF16 = 1 } gdws_dtype_t;
typedef enum { GDWS_NCHW = 0, GDWS_NHWC = 1 } gdws_layout_t;

/* A dense 4-D activation tensor.  n,c,h,w are logical extents; `layout` says how
 * they are ordered in memory (NCHW: w fastest; NHWC: c fastest).  ptr: DEVICE. */
typedef struct {
    void *ptr;
    gdws_dtype_t dtype;
    gdws_layout_t layout;
    int n, c, h, w;
} gdws_tensor_t;

/* Options (gdws_plan_set_option).  Set them before the first forward call. */
typedef enum {
    GDWS_OPT_PATH = 0,     /* gdws_path_t, default GDWS_PATH_AUTO                           */
    GDWS_OPT_RELU = 1,     /* 0/1: y = max(y, 0) after the bias (between chained layers)   */
    GDWS_OPT_TILE = 2,     /* bf16 fused path: force the output patch; value =
                              (TN << 16) | (PH << 8) | PW with PW in {4,8,16,32} and
                              TN*PH*PW <= 128; 0 = choose automatically                    */
    GDWS_OPT_A_LAYOUT = 3, /* bf16 fused path, shared-memory layout of the intermediate
                              tile handed to the tensor cores: 0 = pixel-contiguous
                              (default), 1 = channel-contiguous                            */
    GDWS_OPT_DW_MATH = 4,  /* bf16 fused path, where the GDW stage runs: 1 = on the ALUs (fp32
                              multiply-adds); 2 = on the tensor cores as k*k block-sparse
                              products per 16-channel window (fp32 accumulation), for stride 1
                              or 2 and k <= 5, else GDWS_ERR_UNSUPPORTED; 0 (default) = the library
                              chooses (see gdws_plan_gdw_stage).  Both give the same result
                              up to summation order                                         */
    GDWS_OPT_OUT_DTYPE = 5 /* bf16 plans: 0 (default) = y has the dtype of x; 1 = y is fp32
                              (GDWS_F32, NHWC): bias and ReLU are applied to the fp32 sums of
                              the PW stage and stored without the rounding to bf16.  Every
                              forward call of the plan then expects such a y               */
} gdws_option_t;

typedef enum {
    GDWS_PATH_AUTO = 0,    /* fused where a fused kernel exists for the tensors, else unfused */
    GDWS_PATH_FUSED = 1,   /* one kernel; the G intermediate channels never reach HBM       */
    GDWS_PATH_UNFUSED = 2  /* GDW kernel -> z in the workspace -> PW kernel                 */
} gdws_path_t;

/*
 * gdws_plan -- build the plan of a (C,k,g,D) GDWS layer (Section 3.1, Definition;
 * Property 2 for the intermediate-channel order).
 *   C, D    input / output channels, >= 1
 *   k       filter size, 1..7;  stride 1..4;  pad 0..k
 *   g       HOST, C entries, copied.  g_c >= 0 (g_c = 0: channel c is unused),
 *           sum_c g_c >= 1.  g_c > k*k is accepted (rank of W_c is capped at k*k,
 *           Lemma 1) and simply runs g_c filters.
 *   out     receives the plan.
 * Host work: offsets off_c, the intermediate-channel -> input-channel table, the
 * padding of G to the tensor-core chunk, output-patch choice.  If a CUDA device is
 * current, the plan also allocates its device tables and packed-weight buffers
 * (O(G*(k*k+D)) bytes) on it; with no device the plan is still valid for the
 * host-side queries below and allocates at the first device call.
 * Errors: GDWS_ERR_INVALID_ARG, GDWS_ERR_ALLOC, GDWS_ERR_CUDA.
 */
GDWS_API gdws_status_t gdws_plan(int C, int D, int k, int stride, int pad, const int32_t *g,
                                 gdws_plan_t **out);

/* Change one option; see gdws_option_t.  Errors: GDWS_ERR_INVALID_ARG. */
GDWS_API gdws_status_t gdws_plan_set_option(gdws_plan_t *plan, int key, int value);

/*
 * gdws_plan_info -- sizes and complexity of the planned layer (any pointer may be NULL).
 *   G               sum of g_c
 *   G_pad           G rounded up to the tensor-core K chunk (64)
 *   macs_per_pixel  G*(k*k + D): Eq. 3 of the paper divided by H'W'
 *   params          G*(k*k + D) weights (bias not counted)
 */
GDWS_API gdws_status_t gdws_plan_info(const gdws_plan_t *plan, int *G, int *G_pad,
                                      int64_t *macs_per_pixel, int64_t *params);

/*
 * gdws_plan_tables -- host copies of the plan's integer tables, for inspection.
 *   off    HOST, C+1 entries or NULL: off[c] = sum_{c'<c} g_c', off[C] = G (Property 2)
 *   chan   HOST, G_pad entries or NULL: input channel read by intermediate channel i,
 *          -1 for the padding entries i >= G
 */
GDWS_API gdws_status_t gdws_plan_tables(const gdws_plan_t *plan, int32_t *off, int32_t *chan);

/*
 * gdws_plan_tile -- the output patch the fused bf16 kernel would use for an input of
 * h x w and batch n: each 128-row tensor-core tile covers TN images x PH x PW output
 * pixels.  Pure host computation.
 */
GDWS_API gdws_status_t gdws_plan_tile(const gdws_plan_t *plan, int n, int h, int w, int *TN,
                                      int *PH, int *PW, int64_t *tiles);

/* Output extent H' (or W') for input extent `in`: floor((in + 2 pad - k)/stride) + 1, 0 if negative. */
GDWS_API int gdws_out_dim(int in, int k, int stride, int pad);

/*
 * gdws_plan_gdw_stage -- where the fused bf16 kernel of this plan runs the GDW stage (Section 3.1,
 * Definition) with the current GDWS_OPT_DW_MATH: *stage = 1 (ALUs) or 2 (tensor cores).  With the option
 * at 0 the choice follows the measured cost of the two kernels: the tensor-core form costs k*k products
 * per window of 16 input channels whatever their g_c, the ALU form costs in proportion to sum g_c; the
 * tensor cores are taken for k = 3 or 5, stride 1 (with at most 256 output channels) or 2, and an average
 * g_c of at least 4 (at least 2.7 with at most 128 output channels).  Host only; errors: GDWS_ERR_INVALID_ARG.
 */
GDWS_API gdws_status_t gdws_plan_gdw_stage(const gdws_plan_t *plan, int *stage);

/*
 * gdws_pack_weights -- convert one weight set to the kernels' internal form
 * (bf16 paths; Property 1 / 2 give the shapes).  Enqueues small kernels on `stream`.
 *   dw_w   DEVICE, [G][k][k], dtype `dtype`, canonical order i = off_c + j
 *   pw_w   DEVICE, [D][G] row-major, dtype `dtype`
 *   bias   DEVICE float[D] or NULL (zero)
 * The packed copy lives in the plan.  After it, gdws_forward may be called with
 * dw_w = pw_w = NULL to reuse it (bias too).  Call again whenever the weights change.
 * Errors: GDWS_ERR_INVALID_ARG, GDWS_ERR_ARCH, GDWS_ERR_ALLOC, GDWS_ERR_CUDA.
 */
GDWS_API gdws_status_t gdws_pack_weights(gdws_plan_t *plan, const void *dw_w, const void *pw_w,
                                         const float *bias, gdws_dtype_t dtype, void *stream);

/*
 * gdws_workspace_bytes -- bytes of DEVICE scratch the unfused path needs for an input of
 * n x C x h x w with element type `dtype` (the G intermediate channels z); 0 for sizes it
 * cannot run.  The fused path needs none.
 * gdws_set_workspace -- hand the plan a DEVICE buffer (256-byte aligned) to use as that
 * scratch; the caller keeps ownership and may pass NULL/0 to withdraw it.
 */
GDWS_API size_t gdws_workspace_bytes(const gdws_plan_t *plan, gdws_dtype_t dtype, int n, int h, int w);
GDWS_API gdws_status_t gdws_set_workspace(gdws_plan_t *plan, void *workspace, size_t bytes);

/*
 * gdws_forward -- y = PW(GDW(x)) + bias  (Section 3.1, Definition; formulas at the top).
 *   x      DEVICE tensor, x->c == C.  Supported: F32 (NCHW or NHWC), BF16 NHWC.
 *   dw_w, pw_w, bias   DEVICE, as in gdws_pack_weights, same dtype as x; or all NULL to
 *          use the weights packed earlier.  With non-NULL weights a bf16 plan re-packs
 *          them on `stream` first (F32 plans read them in place).
 *   y      DEVICE tensor, same dtype and layout as x, y->n == x->n, y->c == D,
 *          y->h/w == H'/W'.
 * Accumulation is fp32 on both paths; the bf16 path rounds the intermediate z to bf16
 * before the tensor-core contraction and y to bf16 on store.
 * Device memory is never allocated here.  Errors: GDWS_ERR_INVALID_ARG (shape, dtype,
 * alignment, NULL), GDWS_ERR_UNSUPPORTED, GDWS_ERR_WORKSPACE (unfused path without a large
 * enough workspace), GDWS_ERR_ARCH, GDWS_ERR_CUDA (launch failure, reported synchronously).
 */
GDWS_API gdws_status_t gdws_forward(gdws_plan_t *plan, const gdws_tensor_t *x, const void *dw_w,
                                    const void *pw_w, const float *bias, gdws_tensor_t *y,
                                    void *stream);

/*
 * The two stages on their own (Section 3.1: the GDW convolution and the PW convolution).
 * gdws_depthwise:  z = GDW(x).  z: DEVICE; F32: [n][G][H'][W'] (NCHW) or [n][H'][W'][G] (NHWC)
 *                  following x's layout; BF16 NHWC: [n*H'*W'][G_pad] with zero padding columns.
 * gdws_pointwise:  y = PW(z) + bias (optionally ReLU), z in the layout gdws_depthwise writes.
 *                  `pixels`-style shapes are taken from y.
 * Weight arguments follow gdws_forward (NULL = packed weights; F32 plans need them non-NULL).
 */
GDWS_API gdws_status_t gdws_depthwise(gdws_plan_t *plan, const gdws_tensor_t *x, const void *dw_w,
                                      void *z, void *stream);
GDWS_API gdws_status_t gdws_pointwise(gdws_plan_t *plan, const void *z, const void *pw_w,
                                      const float *bias, gdws_tensor_t *y, void *stream);

/*
 * gdws_forward_host -- the same forward with HOST activations: copies x_host to the
 * device, runs gdws_forward with the packed weights, copies y back, all on `stream`,
 * then waits for the stream.  x_host / y_host: HOST, same dtype/layout rules as
 * gdws_forward (pinned memory makes the copies asynchronous with respect to the host).
 * The plan keeps device staging buffers that grow (cudaMalloc) when a call needs more
 * than any earlier one; weights must have been packed (bf16) or be passed (f32).
 */
GDWS_API gdws_status_t gdws_forward_host(gdws_plan_t *plan, const gdws_tensor_t *x_host,
                                         const void *dw_w, const void *pw_w, const float *bias,
                                         gdws_tensor_t *y_host, void *stream);

/*
 * gdws_forward_static -- gdws_forward on the unfused path, for callers that cannot allocate device
 * memory.  (The paper has no counterpart; this is an addition of the library.)
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region whose memory plan
 * was fixed up front (a real-time or safety-checked inference loop that forbids allocation after
 * start-up, a process whose device memory is handed out entirely by another framework's pool, a
 * callback that may not block on the allocator) -- and that therefore can neither size a workspace
 * with gdws_workspace_bytes / gdws_set_workspace nor let the library grow one.
 * What it does: the GDW kernel writes the G intermediate channels z into a fixed scratch array that
 * is part of the library image (GDWS_STATIC_SCRATCH_BYTES, 16 MiB; every GPU that loads the library
 * holds it until the process ends), and the PW kernel reads them from there.  Arguments, supported
 * tensors, weight rules and results are those of gdws_forward with GDWS_PATH_UNFUSED; the plan's
 * workspace and path options are ignored.  The call itself, and the kernels it launches, allocate
 * nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 * Limits and rules:
 *   - z must fit: gdws_workspace_bytes(plan, dtype, n, h, w) <= gdws_static_scratch_bytes(), else
 *     GDWS_ERR_UNSUPPORTED (nothing is launched).
 *   - The plan must have been built with its device current (that is where the plan's own tables
 *     were allocated); otherwise GDWS_ERR_INVALID_ARG.
 *   - The scratch array's device address is looked up once per device (cudaGetSymbolAddress): when
 *     a plan sets up its tables on that device (gdws_plan with the device current), which is also
 *     the moment the CUDA runtime may load the array's module and commit its 16 MiB there -- a
 *     set-up cost of the allocating phase, not of this call.  Build the plan, and make the first
 *     call on a device, outside any stream capture.
 *   - All calls on one GPU share the one array, whatever the plan or stream, and it keeps what the
 *     last call left there.  Nothing has to be cleared: each call overwrites every element of z that
 *     it reads.  Two calls whose kernels may overlap on the GPU (different streams) race on it:
 *     order them on one stream or with events.
 */
#define GDWS_STATIC_SCRATCH_BYTES (16u << 20)
GDWS_API gdws_status_t gdws_forward_static(gdws_plan_t *plan, const gdws_tensor_t *x, const void *dw_w,
                                           const void *pw_w, const float *bias, gdws_tensor_t *y,
                                           void *stream);
/* Size in bytes of the built-in scratch array used by gdws_forward_static. */
GDWS_API size_t gdws_static_scratch_bytes(void);

/*
 * gdws_status -- read (and clear) the plan's device status word; synchronises with the
 * device.  GDWS_OK, or GDWS_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel expired
 * (the kernel then skipped its remaining work; outputs of that launch are undefined).
 */
GDWS_API gdws_status_t gdws_status(gdws_plan_t *plan);

/*
 * gdws_measure_fma_rate -- diagnostic: multiply-adds per clock and SM (and per second on the whole
 * current device, in 1e12) that the plain ALUs sustain, measured with a kernel of independent
 * register-to-register multiply-adds.  This is the bound of a GDW stage (Section 3.1, Definition:
 * K*K multiply-adds per intermediate channel and output pixel) that runs on the ALUs.
 *   kind  0: fma.rn.f32, 1: fma.rn.f32x2, 2: fma.rn.bf16x2, 3: fma.rn.f32.bf16 (bf16 factors, fp32 sum)
 * Allocates a few KB on the current device, runs for a few milliseconds, synchronises.  Either output
 * pointer may be NULL (HOST).  Errors: GDWS_ERR_INVALID_ARG, GDWS_ERR_ARCH, GDWS_ERR_CUDA.
 */
GDWS_API gdws_status_t gdws_measure_fma_rate(int kind, double *macs_per_clk_per_sm, double *tmacs_per_s);

/*
 * gdws_measure_code_size -- diagnostic: instructions per clock and warp scheduler that `threads` threads per SM
 * (128, 256 or 512) sustain on independent fp32 multiply-adds in a loop whose body is `body_instructions` long
 * (128, 512, 1024, 2048, 3072, 4096, 6144 or 8192; 16 bytes each, the loop is not unrolled).  Measured on B200: up to
 * 2048 instructions (32 KB) 0.7 to 0.9 per clock and scheduler; from 3072 (48 KB) on 0.31 with one warp per scheduler,
 * 0.70 with two, 0.45 to 0.50 with four: code that all warps walk through has to stay below some 32 KB per SM, else it
 * runs at the speed of instruction fetch.  (No counterpart in the paper.)  Allocates a few KB, runs for about a
 * millisecond, synchronises.
 */
GDWS_API gdws_status_t gdws_measure_code_size(int body_instructions, int threads, double *instructions_per_clk_per_scheduler);

/*
 * gdws_selftest_wait -- diagnostic of the error path behind GDWS_ERR_DEVICE_TIMEOUT: enqueues a
 * one-block kernel in which one thread waits, with a limit of `polls` polls (at most 65536), on a
 * shared-memory barrier that nothing ever completes.  The wait runs out, the thread records the
 * condition in the plan's status word and raises the block's abort flag, which releases a second
 * waiter; the kernel then returns by itself (it uses no copies and no tensor memory).  The next
 * gdws_status(plan) reports GDWS_ERR_DEVICE_TIMEOUT once and clears the word.  (No counterpart in
 * the paper.)  Errors: GDWS_ERR_INVALID_ARG, GDWS_ERR_ARCH, GDWS_ERR_CUDA.
 */
GDWS_API gdws_status_t gdws_selftest_wait(gdws_plan_t *plan, unsigned int polls, void *stream);

/* Number of kernels this plan has launched so far (all entry points). */
GDWS_API int64_t gdws_launch_count(const gdws_plan_t *plan);

/* Message for the calling thread's last failing call ("" if none).  Never NULL. */
GDWS_API const char *gdws_last_error(void);

/* Library version string. */
GDWS_API const char *gdws_version(void);

/* Free the plan and everything it allocated (not the caller's buffers).  NULL is a no-op.
 * Synchronises with the device if the plan holds device memory. */
GDWS_API void gdws_destroy(gdws_plan_t *plan);

#ifdef __cplusplus
}
#endif
#endif /* GDWS_H_ */
