// Entry points that touch the device: argument checks, path choice, launches.
#include "gdws_internal.h"

using namespace gdws;

namespace {

bool aligned16(const void *p) { return ((uintptr_t)p & 15) == 0; }

gdws_status_t check_tensor(const char *name, const gdws_tensor_t *t)
{
    if (!t) return fail(GDWS_ERR_INVALID_ARG, "%s is NULL", name);
    if (!t->ptr) return fail(GDWS_ERR_INVALID_ARG, "%s->ptr is NULL", name);
    if (!aligned16(t->ptr)) return fail(GDWS_ERR_INVALID_ARG, "%s->ptr is not 16-byte aligned", name);
    if (t->dtype != GDWS_F32 && t->dtype != GDWS_BF16) return fail(GDWS_ERR_INVALID_ARG, "%s: bad dtype", name);
    if (t->layout != GDWS_NCHW && t->layout != GDWS_NHWC) return fail(GDWS_ERR_INVALID_ARG, "%s: bad layout", name);
    if (t->n < 1 || t->c < 1 || t->h < 1 || t->w < 1)
        return fail(GDWS_ERR_INVALID_ARG, "%s: extents must be >= 1 (n=%d c=%d h=%d w=%d)", name, t->n, t->c, t->h, t->w);
    return GDWS_OK;
}

size_t tensor_bytes(const gdws_tensor_t *t) { return (size_t)t->n * t->c * t->h * t->w * dtype_size(t->dtype); }

}  // namespace

namespace gdws {

gdws_status_t check_pair(const gdws_plan_s *p, const gdws_tensor_t *x, const gdws_tensor_t *y)
{
    gdws_status_t st = check_tensor("x", x);
    if (st != GDWS_OK) return st;
    st = check_tensor("y", y);
    if (st != GDWS_OK) return st;
    if (x->c != p->C) return fail(GDWS_ERR_INVALID_ARG, "x->c=%d but the plan has C=%d", x->c, p->C);
    if (y->c != p->D) return fail(GDWS_ERR_INVALID_ARG, "y->c=%d but the plan has D=%d", y->c, p->D);
    if (x->n != y->n) return fail(GDWS_ERR_INVALID_ARG, "batch mismatch: x->n=%d y->n=%d", x->n, y->n);
    const gdws_dtype_t want = (x->dtype == GDWS_BF16 && p->opt_out_f32) ? GDWS_F32 : x->dtype;
    if (y->dtype != want)
        return fail(GDWS_ERR_INVALID_ARG, "y must be %s for this plan and x", want == GDWS_F32 ? "fp32" : "bf16 (GDWS_OPT_OUT_DTYPE is 0)");
    if (x->layout != y->layout) return fail(GDWS_ERR_INVALID_ARG, "x and y must share the layout");
    const int Ho = gdws_out_dim(x->h, p->k, p->stride, p->pad), Wo = gdws_out_dim(x->w, p->k, p->stride, p->pad);
    if (Ho < 1 || Wo < 1) return fail(GDWS_ERR_INVALID_ARG, "input %dx%d is smaller than the filter", x->h, x->w);
    if (y->h != Ho || y->w != Wo)
        return fail(GDWS_ERR_INVALID_ARG, "y is %dx%d but the output of this layer is %dx%d", y->h, y->w, Ho, Wo);
    if (x->dtype == GDWS_BF16 && x->layout != GDWS_NHWC)
        return fail(GDWS_ERR_UNSUPPORTED, "bf16 tensors must be NHWC");
    const char *xb = (const char *)x->ptr, *yb = (const char *)y->ptr;
    if (xb < yb + tensor_bytes(y) && yb < xb + tensor_bytes(x))
        return fail(GDWS_ERR_INVALID_ARG, "x and y overlap");
    return GDWS_OK;
}

}  // namespace gdws

namespace {

gdws_status_t prepare(gdws_plan_s *p)
{
    gdws_status_t st = GDWS_OK;
    if (!p->arch_ok) {
        st = check_arch();
        if (st != GDWS_OK) return st;
        p->arch_ok = true;
    }
    st = ensure_device(p);
    if (st != GDWS_OK) return st;
    int dev = -1;
    cudaGetDevice(&dev);
    if (dev != p->device)
        return fail(GDWS_ERR_INVALID_ARG, "plan lives on device %d but device %d is current", p->device, dev);
    return GDWS_OK;
}

gdws_status_t weights_ready(gdws_plan_s *p, const void *dw_w, const void *pw_w, const float *bias,
                            gdws_dtype_t dtype, cudaStream_t st)
{
    if ((dw_w == nullptr) != (pw_w == nullptr))
        return fail(GDWS_ERR_INVALID_ARG, "dw_w and pw_w must both be given or both be NULL");
    if (dw_w) {
        if (!aligned16(dw_w) || !aligned16(pw_w) || (bias && ((uintptr_t)bias & 3)))
            return fail(GDWS_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
        return bf16_pack(p, dw_w, pw_w, bias, dtype, st);
    }
    if (!p->packed) return fail(GDWS_ERR_INVALID_ARG, "no weights: pass dw_w/pw_w or call gdws_pack_weights first");
    return GDWS_OK;
}

}  // namespace

extern "C" {

gdws_status_t gdws_pack_weights(gdws_plan_t *p, const void *dw_w, const void *pw_w, const float *bias,
                                gdws_dtype_t dtype, void *stream)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_pack_weights: plan is NULL");
    if (!dw_w || !pw_w) return fail(GDWS_ERR_INVALID_ARG, "gdws_pack_weights: dw_w and pw_w must not be NULL");
    if (dtype != GDWS_F32 && dtype != GDWS_BF16) return fail(GDWS_ERR_INVALID_ARG, "gdws_pack_weights: bad dtype");
    gdws_status_t st = prepare(p);
    if (st != GDWS_OK) return st;
    return weights_ready(p, dw_w, pw_w, bias, dtype, (cudaStream_t)stream);
}

gdws_status_t gdws_forward(gdws_plan_t *p, const gdws_tensor_t *x, const void *dw_w, const void *pw_w,
                           const float *bias, gdws_tensor_t *y, void *stream)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_forward: plan is NULL");
    gdws_status_t st = check_pair(p, x, y);
    if (st != GDWS_OK) return st;
    st = prepare(p);
    if (st != GDWS_OK) return st;
    cudaStream_t cs = (cudaStream_t)stream;
    const bool fused = p->opt_path != GDWS_PATH_UNFUSED;
    if (x->dtype == GDWS_F32) {
        if (!dw_w || !pw_w) return fail(GDWS_ERR_INVALID_ARG, "fp32 plans read the weights in place: dw_w/pw_w must not be NULL");
        if (!aligned16(dw_w) || !aligned16(pw_w)) return fail(GDWS_ERR_INVALID_ARG, "weight pointers must be 16-byte aligned");
        if (fused) return f32_fused(p, x, (const float *)dw_w, (const float *)pw_w, bias, y, cs);
        const size_t need = gdws_workspace_bytes(p, GDWS_F32, x->n, x->h, x->w);
        if (!p->ws || p->ws_bytes < need)
            return fail(GDWS_ERR_WORKSPACE, "unfused path needs a %zu-byte workspace (have %zu)", need, p->ws_bytes);
        st = f32_depthwise(p, x, (const float *)dw_w, (float *)p->ws, cs);
        if (st != GDWS_OK) return st;
        return f32_pointwise(p, (const float *)p->ws, (const float *)pw_w, bias, y, cs);
    }
    st = weights_ready(p, dw_w, pw_w, bias, GDWS_BF16, cs);
    if (st != GDWS_OK) return st;
    if (fused) {
        st = bf16_fused(p, x, y, cs);
        if (st != GDWS_ERR_UNSUPPORTED || p->opt_path == GDWS_PATH_FUSED) return st;
        // GDWS_PATH_AUTO and no fused kernel for this shape: take the unfused pair
    }
    const size_t need = gdws_workspace_bytes(p, GDWS_BF16, x->n, x->h, x->w);
    if (!p->ws || p->ws_bytes < need)
        return fail(GDWS_ERR_WORKSPACE, "unfused path needs a %zu-byte workspace (have %zu)", need, p->ws_bytes);
    st = bf16_depthwise(p, x, p->ws, cs);
    if (st != GDWS_OK) return st;
    return bf16_pointwise(p, p->ws, y, cs);
}

gdws_status_t gdws_depthwise(gdws_plan_t *p, const gdws_tensor_t *x, const void *dw_w, void *z, void *stream)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_depthwise: plan is NULL");
    gdws_status_t st = check_tensor("x", x);
    if (st != GDWS_OK) return st;
    if (x->c != p->C) return fail(GDWS_ERR_INVALID_ARG, "x->c=%d but the plan has C=%d", x->c, p->C);
    if (!z || !aligned16(z)) return fail(GDWS_ERR_INVALID_ARG, "z must be a 16-byte aligned device pointer");
    if (gdws_out_dim(x->h, p->k, p->stride, p->pad) < 1 || gdws_out_dim(x->w, p->k, p->stride, p->pad) < 1)
        return fail(GDWS_ERR_INVALID_ARG, "input %dx%d is smaller than the filter", x->h, x->w);
    st = prepare(p);
    if (st != GDWS_OK) return st;
    cudaStream_t cs = (cudaStream_t)stream;
    if (x->dtype == GDWS_F32) {
        if (!dw_w || !aligned16(dw_w)) return fail(GDWS_ERR_INVALID_ARG, "fp32 plans need dw_w (16-byte aligned)");
        return f32_depthwise(p, x, (const float *)dw_w, (float *)z, cs);
    }
    if (x->layout != GDWS_NHWC) return fail(GDWS_ERR_UNSUPPORTED, "bf16 tensors must be NHWC");
    if (p->C % 8) return fail(GDWS_ERR_UNSUPPORTED, "bf16 kernels need C %% 8 == 0");
    if (dw_w) return fail(GDWS_ERR_INVALID_ARG, "bf16 stage calls use packed weights: call gdws_pack_weights, pass NULL");
    if (!p->packed) return fail(GDWS_ERR_INVALID_ARG, "no packed weights: call gdws_pack_weights first");
    return bf16_depthwise(p, x, z, cs);
}

gdws_status_t gdws_pointwise(gdws_plan_t *p, const void *z, const void *pw_w, const float *bias, gdws_tensor_t *y,
                             void *stream)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_pointwise: plan is NULL");
    gdws_status_t st = check_tensor("y", y);
    if (st != GDWS_OK) return st;
    if (y->c != p->D) return fail(GDWS_ERR_INVALID_ARG, "y->c=%d but the plan has D=%d", y->c, p->D);
    if (!z || !aligned16(z)) return fail(GDWS_ERR_INVALID_ARG, "z must be a 16-byte aligned device pointer");
    st = prepare(p);
    if (st != GDWS_OK) return st;
    cudaStream_t cs = (cudaStream_t)stream;
    if (y->dtype == GDWS_F32 && !p->opt_out_f32) {
        if (!pw_w || !aligned16(pw_w)) return fail(GDWS_ERR_INVALID_ARG, "fp32 plans need pw_w (16-byte aligned)");
        return f32_pointwise(p, (const float *)z, (const float *)pw_w, bias, y, cs);
    }
    if (y->layout != GDWS_NHWC) return fail(GDWS_ERR_UNSUPPORTED, "bf16 tensors must be NHWC");
    if (pw_w) return fail(GDWS_ERR_INVALID_ARG, "bf16 stage calls use packed weights: call gdws_pack_weights, pass NULL");
    if (!p->packed) return fail(GDWS_ERR_INVALID_ARG, "no packed weights: call gdws_pack_weights first");
    return bf16_pointwise(p, z, y, cs);
}

gdws_status_t gdws_forward_host(gdws_plan_t *p, const gdws_tensor_t *xh, const void *dw_w, const void *pw_w,
                                const float *bias, gdws_tensor_t *yh, void *stream)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_forward_host: plan is NULL");
    if (!xh || !yh || !xh->ptr || !yh->ptr) return fail(GDWS_ERR_INVALID_ARG, "gdws_forward_host: NULL tensor");
    gdws_status_t st = prepare(p);
    if (st != GDWS_OK) return st;
    if (xh->n < 1 || xh->c < 1 || xh->h < 1 || xh->w < 1 || yh->n < 1 || yh->c < 1 || yh->h < 1 || yh->w < 1)
        return fail(GDWS_ERR_INVALID_ARG, "gdws_forward_host: extents must be >= 1");
    const size_t xb = tensor_bytes(xh), yb = tensor_bytes(yh);
    cudaError_t e;
    if (p->stage_x_bytes < xb) {
        cudaFree(p->stage_x); p->stage_x = nullptr; p->stage_x_bytes = 0;
        e = cudaMalloc(&p->stage_x, xb);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(GDWS_ERR_ALLOC, "cudaMalloc(%zu) failed", xb); }
        p->stage_x_bytes = xb;
    }
    if (p->stage_y_bytes < yb) {
        cudaFree(p->stage_y); p->stage_y = nullptr; p->stage_y_bytes = 0;
        e = cudaMalloc(&p->stage_y, yb);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(GDWS_ERR_ALLOC, "cudaMalloc(%zu) failed", yb); }
        p->stage_y_bytes = yb;
    }
    cudaStream_t cs = (cudaStream_t)stream;
    gdws_tensor_t xd = *xh, yd = *yh;
    xd.ptr = p->stage_x;
    yd.ptr = p->stage_y;
    e = cudaMemcpyAsync(xd.ptr, xh->ptr, xb, cudaMemcpyHostToDevice, cs);
    if (e != cudaSuccess) return cuda_fail(e, "host to device copy");
    st = gdws_forward(p, &xd, dw_w, pw_w, bias, &yd, stream);
    if (st != GDWS_OK) return st;
    e = cudaMemcpyAsync(yh->ptr, yd.ptr, yb, cudaMemcpyDeviceToHost, cs);
    if (e != cudaSuccess) return cuda_fail(e, "device to host copy");
    e = cudaStreamSynchronize(cs);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    return GDWS_OK;
}

gdws_status_t gdws_status(gdws_plan_t *p)
{
    if (!p) return fail(GDWS_ERR_INVALID_ARG, "gdws_status: plan is NULL");
    if (p->device < 0) return GDWS_OK;
    // the status word lives on the plan's device: wait for that device, whichever is current
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (cur != p->device) {
        e = cudaSetDevice(p->device);
        if (e != cudaSuccess) return cuda_fail(e, "cudaSetDevice");
    }
    int word = 0;
    e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&word, p->d_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && word) e = cudaMemset(p->d_status, 0, sizeof(int));
    if (cur != p->device) cudaSetDevice(cur);
    if (e != cudaSuccess) return cuda_fail(e, "status read");
    if (word) return fail(GDWS_ERR_DEVICE_TIMEOUT, "a bounded wait inside a kernel expired (status word 0x%x)", word);
    return GDWS_OK;
}

}  // extern "C"
