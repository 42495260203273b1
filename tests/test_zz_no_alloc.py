"""gdws_forward_static: the forward for callers that may not allocate device memory (an inference
loop whose memory plan is frozen after start-up, a process whose GPU memory belongs to another
framework's pool).  Its intermediate lives in a fixed array inside the library, so the call needs no
workspace.  This file is collected last on purpose: a run that stops at the first failure has then
already gone through every other test.

Checked here, through the C ABI: two calls in a row give what gdws_forward gives on the unfused path
with a caller-provided workspace (same kernels, so the same tolerance as the other parity tests is
ample), for a bf16 and an fp32 layer.  Before them another, wider layer fed with NaN inputs goes through
the same entry point, so the shared array holds NaNs wherever the target layer does not overwrite it: a
stale element read by the second layer would show.  Across the calls the device's free memory and
torch's allocation count must not move.  A layer whose intermediate exceeds the built-in array is
refused without a launch; overlapping x and y are refused as gdws_forward refuses them."""
import gc

import numpy as np
import pytest
import torch

from paper_2110_14871_b200 import build as gbuild
from paper_2110_14871_b200 import gdws
from paper_2110_14871_b200 import inputs as gi

from util import TOL, make_plan, rel_err, run_gpu, run_oracle, small_spec, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    gbuild.build_library()


@pytest.mark.parametrize("dtype,layout", [("bf16", "NHWC"), ("f32", "NCHW")])
def test_forward_static_matches_forward_twice(dtype, layout):
    spec = small_spec("t", 5, 16, 24, 11, 9, 3, 1, 1, ("uniform", 1, 9), dtype, layout, seed=77)
    data = gi.make_layer(spec)
    want = run_gpu(data, path=gdws.PATH_UNFUSED)            # existing entry point, caller's workspace
    ref, _ = run_oracle(data)
    code = gdws.F32 if dtype == "f32" else gdws.BF16
    # a wider layer with NaN activations first: it leaves NaNs all over the shared scratch array
    wide = small_spec("w", 6, 32, 16, 13, 12, 3, 1, 1, ("uniform", 4, 9), dtype, layout, seed=79)
    wdata = gi.make_layer(wide)
    wplan = make_plan(wdata)
    wx = torch.full(tuple(wdata.x.shape), float("nan"), dtype=torch.float32 if dtype == "f32" else torch.bfloat16, device="cuda")
    wdw, wpw = (to_device(a, dtype) for a in (wdata.dw_w, wdata.pw_w))
    wshape = (wide.N, wide.D, wide.Ho, wide.Wo) if layout == "NCHW" else (wide.N, wide.Ho, wide.Wo, wide.D)
    wy = torch.zeros(wshape, dtype=wx.dtype, device="cuda")
    plan = make_plan(data)
    assert wplan.workspace_bytes(code, wide.N, wide.H, wide.W) > plan.workspace_bytes(code, spec.N, spec.H, spec.W)
    wplan.forward_static(wx, wy, layout, wdw, wpw)
    torch.cuda.synchronize()
    assert torch.isnan(wy.float()).any()
    x, dw, pw = (to_device(a, dtype) for a in (data.x, data.dw_w, data.pw_w))
    b = torch.from_numpy(data.bias).cuda()
    shape = (spec.N, spec.D, spec.Ho, spec.Wo) if layout == "NCHW" else (spec.N, spec.Ho, spec.Wo, spec.D)
    assert plan.workspace_bytes(code, spec.N, spec.H, spec.W) <= gdws.static_scratch_bytes()
    ys = [torch.full(shape, float("nan"), dtype=x.dtype, device="cuda") for _ in range(2)]
    if dtype == "bf16":
        plan.pack_weights(dw, pw, b)          # the allocation-free call then takes no weight arguments
    torch.cuda.synchronize()
    gc.collect()                  # tensors of earlier tests that only the cycle collector frees must not go in between
    gc.disable()
    free_before, _ = torch.cuda.mem_get_info()
    count_before = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
    held_before = torch.cuda.memory_allocated()
    for call in range(2):
        if dtype == "bf16":
            plan.forward_static(x, ys[call], layout)
        else:
            plan.forward_static(x, ys[call], layout, dw, pw, b)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "device memory in use changed across gdws_forward_static"
    assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == count_before
    held_after = torch.cuda.memory_allocated()
    gc.enable()
    assert held_after == held_before
    for call in range(2):
        got = ys[call].float().cpu().numpy().astype(np.float64)
        assert rel_err(got, want) <= TOL[dtype], call
        assert rel_err(got, ref) <= TOL[dtype], call
    plan.destroy()
    wplan.destroy()


def test_forward_static_refuses_overlap():
    spec = small_spec("t", 2, 16, 16, 8, 8, 3, 1, 1, ("uniform", 1, 3), "bf16", "NHWC", seed=80)
    data = gi.make_layer(spec)
    plan = make_plan(data)
    buf = torch.zeros((spec.N, spec.H, spec.W, spec.C), dtype=torch.bfloat16, device="cuda")
    dw, pw = (to_device(a, "bf16") for a in (data.dw_w, data.pw_w))
    before = plan.launch_count()
    with pytest.raises(gdws.GdwsError) as e:
        plan.forward_static(buf, buf, "NHWC", dw, pw)
    assert e.value.status == gdws.ERR_INVALID_ARG and plan.launch_count() == before
    plan.destroy()


def test_forward_static_refuses_what_does_not_fit():
    spec = small_spec("t", 64, 64, 64, 56, 56, 3, 1, 1, ("uniform", 1, 9), "bf16", "NHWC", seed=78)
    rng = np.random.Generator(np.random.PCG64(1))
    g = gi.make_g(rng, spec.C, spec.g_dist)
    plan = gdws.Plan(spec.C, spec.D, spec.k, spec.stride, spec.pad, g)
    assert plan.workspace_bytes(gdws.BF16, spec.N, spec.H, spec.W) > gdws.static_scratch_bytes() == 16 << 20
    G = int(g.sum())
    x = torch.zeros((spec.N, spec.H, spec.W, spec.C), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((spec.N, spec.Ho, spec.Wo, spec.D), dtype=torch.bfloat16, device="cuda")
    dw = torch.zeros((G, 3, 3), dtype=torch.bfloat16, device="cuda")
    pw = torch.zeros((spec.D, G), dtype=torch.bfloat16, device="cuda")
    before = plan.launch_count()
    with pytest.raises(gdws.GdwsError) as e:
        plan.forward_static(x, y, "NHWC", dw, pw)
    assert e.value.status == gdws.ERR_UNSUPPORTED and plan.launch_count() == before
    plan.destroy()
