// gdws_forward_static: the unfused forward (GDW kernel -> z -> PW kernel) for callers that must not
// allocate device memory.  The intermediate z lives in a fixed array that is part of the library
// image, so nothing is asked of the CUDA allocator, neither here nor by the caller.
#include <mutex>

#include "gdws_internal.h"

using namespace gdws;

// Scratch for z.  Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[GDWS_STATIC_SCRATCH_BYTES];

namespace {

// In host code `g_static_scratch` is only a handle of the symbol, not a device address; the address
// a kernel can use has to be looked up, once per device, with that device current.  The table is
// shared by all host threads, hence the lock.
void *g_scratch_addr[64] = {};
std::mutex g_scratch_lock;

gdws_status_t scratch_address(int device, void **out)
{
    if (device < 0 || device >= 64) return fail(GDWS_ERR_UNSUPPORTED, "device index %d is outside 0..63", device);
    std::lock_guard<std::mutex> hold(g_scratch_lock);
    if (!g_scratch_addr[device]) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        g_scratch_addr[device] = ptr;
    }
    if (out) *out = g_scratch_addr[device];
    return GDWS_OK;
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

}  // namespace

// Called while a plan sets up its device tables, i.e. in the phase that allocates anyway: this translation
// unit holds no kernel, so its module (and with it the array) may only be loaded by this first look-up.
gdws_status_t gdws::static_scratch_prepare(int device) { return scratch_address(device, nullptr); }

extern "C" {

size_t gdws_static_scratch_bytes(void) { return (size_t)GDWS_STATIC_SCRATCH_BYTES; }

gdws_status_t gdws_forward_static(gdws_plan_t *p, const gdws_tensor_t *x, const void *dw_w, const void *pw_w,
                                  const float *bias, gdws_tensor_t *y, void *stream)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_forward_static: plan is NULL");
    gdws_status_t st = check_pair(p, x, y);      // the checks of gdws_forward, overlap of x and y included
    if (st != GDWS_OK) return st;
    if (bias && ((uintptr_t)bias & 3)) return fail(GDWS_ERR_INVALID_ARG, "gdws_forward_static: bias must be 4-byte aligned");
    if (x->dtype == GDWS_BF16 && (p->C % 8 || p->D % 8)) return fail(GDWS_ERR_UNSUPPORTED, "bf16 kernels need C %% 8 == 0 and D %% 8 == 0");
    // The plan's own tables were allocated when it was built on a device; this call never allocates.
    if (p->device < 0)
        return fail(GDWS_ERR_INVALID_ARG, "gdws_forward_static: build the plan with its CUDA device current (it allocates the plan's tables)");
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev != p->device) return fail(GDWS_ERR_INVALID_ARG, "plan lives on device %d but device %d is current", p->device, dev);
    if (!p->arch_ok) {
        st = check_arch();
        if (st != GDWS_OK) return st;
        p->arch_ok = true;
    }
    const size_t need = gdws_workspace_bytes(p, x->dtype, x->n, x->h, x->w);
    if (need == 0 || need > (size_t)GDWS_STATIC_SCRATCH_BYTES)
        return fail(GDWS_ERR_UNSUPPORTED,
                    "gdws_forward_static: the intermediate needs %zu bytes, the built-in scratch holds %zu; use gdws_forward",
                    need, (size_t)GDWS_STATIC_SCRATCH_BYTES);
    void *z = nullptr;
    st = scratch_address(dev, &z);
    if (st != GDWS_OK) return st;
    cudaStream_t cs = (cudaStream_t)stream;
    if (x->dtype == GDWS_F32) {
        if (!dw_w || !pw_w || !aligned16(dw_w) || !aligned16(pw_w))
            return fail(GDWS_ERR_INVALID_ARG, "fp32 plans read the weights in place: dw_w/pw_w must be 16-byte aligned device pointers");
        st = f32_depthwise(p, x, (const float *)dw_w, (float *)z, cs);
        if (st != GDWS_OK) return st;
        return f32_pointwise(p, (const float *)z, (const float *)pw_w, bias, y, cs);
    }
    if ((dw_w == nullptr) != (pw_w == nullptr))
        return fail(GDWS_ERR_INVALID_ARG, "dw_w and pw_w must both be given or both be NULL");
    if (dw_w) {   // re-pack into the plan's buffers (kernels only)
        if (!aligned16(dw_w) || !aligned16(pw_w)) return fail(GDWS_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
        st = bf16_pack(p, dw_w, pw_w, bias, GDWS_BF16, cs);
        if (st != GDWS_OK) return st;
    } else if (!p->packed) {
        return fail(GDWS_ERR_INVALID_ARG, "no weights: pass dw_w/pw_w or call gdws_pack_weights first");
    }
    st = bf16_depthwise(p, x, z, cs);     // writes every element of z it later reads, padding columns included
    if (st != GDWS_OK) return st;
    return bf16_pointwise(p, z, y, cs);
}

}  // extern "C"
