"""gdws_forward_static: the forward for callers that may not allocate device memory (an inference
loop whose memory plan is frozen after start-up, a process whose GPU memory belongs to another
framework's pool).  Its intermediate lives in a fixed array inside the library, so the call needs no
workspace.  This file is collected last on purpose: a run that stops at the first failure has then
already gone through every other test.

Checked here, through the C ABI: two calls in a row give what gdws_forward gives on the unfused path
with a caller-provided workspace (same kernels, so the same tolerance as the other parity tests is
ample), for a bf16 and an fp32 layer; a layer whose intermediate exceeds the built-in array is
refused without a launch."""
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
    plan = make_plan(data)
    x, dw, pw = (to_device(a, dtype) for a in (data.x, data.dw_w, data.pw_w))
    b = torch.from_numpy(data.bias).cuda()
    shape = (spec.N, spec.D, spec.Ho, spec.Wo) if layout == "NCHW" else (spec.N, spec.Ho, spec.Wo, spec.D)
    assert plan.workspace_bytes(gdws.F32 if dtype == "f32" else gdws.BF16, spec.N, spec.H, spec.W) <= gdws.static_scratch_bytes()
    for call in range(2):
        y = torch.full(shape, float("nan"), dtype=x.dtype, device="cuda")
        plan.forward_static(x, y, layout, dw, pw, b)
        torch.cuda.synchronize()
        got = y.float().cpu().numpy().astype(np.float64)
        assert rel_err(got, want) <= TOL[dtype], call
        assert rel_err(got, ref) <= TOL[dtype], call
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
