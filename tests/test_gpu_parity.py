"""Parity of the CUDA library (through the C ABI) with the CPU reference, element by
element on the same seeded inputs.  Bars: max|y - y_ref| / max|y_ref| <= 1e-4 on the
fp32 path and <= 2e-2 on the bf16-in / fp32-accumulate path."""
import numpy as np
import pytest
import torch

from oracle import gdws_oracle as orc
from paper_2110_14871_b200 import build as gbuild
from paper_2110_14871_b200 import gdws
from paper_2110_14871_b200 import inputs as gi

from util import TOL, make_plan, rel_err, run_gpu, run_oracle, small_spec, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    gbuild.build_library()
    assert torch.cuda.get_device_capability(0)[0] == 10, "these tests need an sm_100 device"


# ------------------------------------------------------------------ fp32 path
F32_SHAPES = [
    # N, C, D, H, W, k, stride, pad, g_dist
    (1, 16, 16, 32, 32, 3, 1, 1, ("uniform", 1, 3)),
    (2, 5, 7, 9, 11, 3, 2, 1, ("uniform", 0, 9)),
    (3, 4, 130, 7, 6, 5, 1, 2, ("uniform", 1, 25)),
    (1, 3, 4, 6, 5, 2, 1, 0, ("uniform", 1, 4)),
    (2, 6, 3, 5, 5, 1, 1, 0, ("const", 1)),
    (1, 40, 20, 13, 13, 3, 1, 1, ("uniform", 1, 9)),
]


@pytest.mark.parametrize("layout", ["NCHW", "NHWC"])
@pytest.mark.parametrize("path", [gdws.PATH_FUSED, gdws.PATH_UNFUSED])
@pytest.mark.parametrize("shape", F32_SHAPES)
def test_f32_forward_matches_reference(shape, path, layout):
    N, C, D, H, W, k, s, p, gd = shape
    spec = small_spec("t", N, C, D, H, W, k, s, p, gd, "f32", layout, relu=(C == 5), seed=sum(shape[:8]))
    data = gi.make_layer(spec)
    if data.G == 0:
        pytest.skip("empty g")
    y = run_gpu(data, path=path)
    ref, _ = run_oracle(data)
    assert rel_err(y, ref) <= TOL["f32"]


def test_config0_exact_recipe():
    data = gi.make_layer(gi.config_layers(0)[0])
    ref, _ = run_oracle(data)
    for path in (gdws.PATH_FUSED, gdws.PATH_UNFUSED):
        assert rel_err(run_gpu(data, path=path), ref) <= TOL["f32"]


def test_f32_stages_match_reference():
    spec = small_spec("t", 2, 6, 10, 9, 8, 3, 2, 1, ("uniform", 1, 9), "f32", "NCHW", seed=5)
    data = gi.make_layer(spec)
    plan = make_plan(data)
    x, dw, pw = to_device(data.x, "f32"), to_device(data.dw_w, "f32"), to_device(data.pw_w, "f32")
    b = torch.from_numpy(data.bias).cuda()
    z = torch.full((spec.N, data.G, spec.Ho, spec.Wo), float("nan"), device="cuda")
    y = torch.full((spec.N, spec.D, spec.Ho, spec.Wo), float("nan"), device="cuda")
    plan.depthwise(x, z, "NCHW", dw)
    plan.pointwise(z, y, "NCHW", pw, b)
    torch.cuda.synchronize()
    yr, zr, _ = run_oracle(data, return_z=True)
    assert rel_err(z.cpu().numpy(), zr) <= 1e-5
    assert rel_err(y.cpu().numpy(), yr) <= TOL["f32"]
    assert plan.launch_count() == 2
    plan.destroy()


# ------------------------------------------------------------------ bf16 path
BF16_SHAPES = [
    # N, C, D, H, W, k, stride, pad, g_dist   (several tiles + ragged tails in n, h and w)
    (3, 16, 16, 8, 8, 3, 1, 1, ("uniform", 1, 9)),
    (5, 32, 24, 9, 11, 3, 1, 1, ("uniform", 0, 9)),
    (2, 24, 40, 20, 17, 3, 2, 1, ("uniform", 1, 9)),
    (9, 16, 64, 4, 4, 3, 1, 1, ("uniform", 1, 9)),
    (2, 8, 16, 14, 14, 5, 1, 2, ("uniform", 1, 25)),
    (1, 16, 8, 12, 10, 2, 1, 0, ("uniform", 1, 4)),
    (2, 40, 272, 7, 7, 1, 1, 0, ("uniform", 1, 1)),
    (1, 64, 512, 9, 9, 3, 2, 1, ("heavy",)),
    (2, 16, 32, 33, 35, 3, 1, 1, ("heavy",)),
    (9, 16, 64, 8, 8, 3, 2, 1, ("uniform", 1, 9)),       # stride 2 onto 4x4 outputs
    (3, 72, 48, 16, 16, 3, 1, 1, ("const", 1)),            # depthwise-separable special case (g = 1)
    (1, 8, 16, 40, 70, 3, 1, 1, ("uniform", 5, 9)),
    (2, 16, 24, 19, 17, 5, 2, 2, ("uniform", 1, 25)),      # k = 5, stride 2: the row-run depthwise code for 5 x 5 filters
    (1, 8, 32, 16, 24, 5, 1, 2, ("heavy",)),
]


# dw_math: 0 = the library chooses where the GDW stage runs, 1 = on the ALUs, 2 = on the tensor cores (own tests below)
@pytest.mark.parametrize("path,a_layout,dw_math", [(gdws.PATH_UNFUSED, 0, 0), (gdws.PATH_FUSED, 0, 0), (gdws.PATH_FUSED, 1, 1)])
@pytest.mark.parametrize("shape", BF16_SHAPES)
def test_bf16_forward_matches_reference(shape, path, a_layout, dw_math):
    N, C, D, H, W, k, s, p, gd = shape
    spec = small_spec("t", N, C, D, H, W, k, s, p, gd, "bf16", "NHWC", relu=(C == 24), seed=sum(shape[:8]))
    data = gi.make_layer(spec)
    y = run_gpu(data, path=path, a_layout=a_layout, dw_math=dw_math)
    ref, _ = run_oracle(data)
    err = rel_err(y, ref)
    assert err <= TOL["bf16"], err
    # two bf16 roundings (z and y) should sit far inside the bar
    assert err <= 1e-2, err


@pytest.mark.parametrize("tile", [(1 << 16) | (3 << 8) | 32, (2 << 16) | (6 << 8) | 8, (1 << 16) | (1 << 8) | 16])
def test_bf16_fused_generic_depthwise_path_with_forced_tiles(tile):
    """Patches the specialised k=3 depthwise code does not cover run the generic code."""
    spec = small_spec("t", 3, 16, 24, 13, 19, 3, 1, 1, ("uniform", 1, 9), seed=33)
    data = gi.make_layer(spec)
    ref, _ = run_oracle(data)
    assert rel_err(run_gpu(data, path=gdws.PATH_FUSED, tile=tile, dw_math=1), ref) <= 1e-2


# Shapes for the kernel that runs the GDW stage on the tensor cores: every tile family (one image with halo rows,
# several images per tile, maps at most 4 wide), ragged tails, windows of 8 and 16 input channels, chunks that a
# window is cut into (many intermediate channels), D beyond 256 (two blocks per tile), k = 1, 2, 3, 5.
TC_SHAPES = [
    (2, 16, 16, 16, 8, 3, 1, 1, ("uniform", 1, 9)),
    (3, 32, 64, 8, 8, 3, 1, 1, ("uniform", 1, 9)),
    (5, 24, 40, 9, 11, 3, 1, 1, ("uniform", 0, 9)),
    (9, 16, 64, 4, 4, 3, 1, 1, ("uniform", 1, 9)),
    (3, 48, 272, 14, 14, 3, 1, 1, ("heavy",)),
    (1, 32, 512, 28, 28, 3, 1, 1, ("uniform", 7, 9)),
    (2, 8, 16, 14, 14, 5, 1, 2, ("uniform", 1, 25)),
    (1, 16, 8, 12, 10, 2, 1, 0, ("uniform", 1, 4)),
    (2, 40, 24, 7, 7, 1, 1, 0, ("uniform", 1, 1)),
    (1, 64, 64, 40, 33, 3, 1, 1, ("heavy",)),
    (4, 16, 128, 3, 3, 3, 1, 1, ("uniform", 1, 9)),
    (2, 16, 32, 6, 20, 3, 1, 0, ("uniform", 1, 9)),
    (1, 16, 16, 9, 9, 3, 1, 1, ("const", 12)),              # g_c > k*k is legal (Lemma 1 caps the rank, not the count)
    # stride 2: the input is read through one dense view per parity of row and column
    (2, 16, 16, 8, 8, 3, 2, 1, ("uniform", 1, 9)),          # 4 x 4 output maps: one copy per tap
    (3, 32, 64, 17, 15, 3, 2, 1, ("uniform", 1, 9)),        # odd input sizes: the views differ in size
    (1, 16, 32, 32, 32, 3, 2, 1, ("uniform", 1, 9)),        # one image per tile, four boxes with halo
    (5, 16, 24, 16, 16, 3, 2, 1, ("uniform", 0, 9)),        # 8 x 8 output maps: two images per tile
    (2, 24, 40, 19, 23, 5, 2, 2, ("uniform", 1, 25)),
    (2, 16, 16, 12, 12, 1, 2, 0, ("uniform", 1, 1)),        # k = 1: only the even rows and columns are read
    (1, 64, 272, 28, 28, 3, 2, 1, ("heavy",)),
    # more than 9 taps: the B operands go through the buffers in groups of taps
    (2, 16, 32, 12, 12, 4, 1, 1, ("uniform", 1, 16)),
    (3, 32, 48, 13, 13, 4, 2, 1, ("uniform", 1, 16)),
    (80, 32, 32, 16, 16, 5, 1, 2, ("uniform", 1, 25)),      # more tiles than SMs, windows of three chunks
]


@pytest.mark.parametrize("shape", TC_SHAPES)
def test_bf16_tensor_core_gdw_matches_reference(shape):
    N, C, D, H, W, k, s, p, gd = shape
    spec = small_spec("t", N, C, D, H, W, k, s, p, gd, "bf16", "NHWC", relu=(C == 24), seed=7 + sum(shape[:8]))
    data = gi.make_layer(spec)
    y = run_gpu(data, path=gdws.PATH_FUSED, dw_math=2)
    ref, _ = run_oracle(data)
    err = rel_err(y, ref)
    assert err <= 1e-2, err


def test_tensor_core_gdw_agrees_with_alu_gdw_and_refuses_stride_3():
    spec = small_spec("t", 6, 32, 48, 16, 16, seed=77)
    data = gi.make_layer(spec)
    a = run_gpu(data, path=gdws.PATH_FUSED, dw_math=2)
    b = run_gpu(data, path=gdws.PATH_FUSED, dw_math=1)
    # both round z to bf16 once and accumulate in fp32; only the summation order differs
    assert rel_err(a, b) <= 4e-3
    data2 = gi.make_layer(small_spec("t", 2, 16, 16, 9, 9, 3, 3, 1, seed=78))
    with pytest.raises(gdws.GdwsError) as e:
        run_gpu(data2, path=gdws.PATH_FUSED, dw_math=2)
    assert e.value.status == gdws.ERR_UNSUPPORTED


def test_bf16_depthwise_and_pointwise_stages():
    spec = small_spec("t", 3, 16, 24, 10, 9, 3, 1, 1, ("uniform", 1, 9), seed=9)
    data = gi.make_layer(spec)
    plan = make_plan(data)
    x, dw, pw = (to_device(a, "bf16") for a in (data.x, data.dw_w, data.pw_w))
    b = torch.from_numpy(data.bias).cuda()
    plan.pack_weights(dw, pw, b)
    G, Gp, _, _ = plan.info()
    npix = spec.N * spec.Ho * spec.Wo
    z = torch.full((npix, Gp), float("nan"), dtype=torch.bfloat16, device="cuda")
    y = torch.full((spec.N, spec.Ho, spec.Wo, spec.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.depthwise(x, z, "NHWC")
    plan.pointwise(z, y, "NHWC")
    torch.cuda.synchronize()
    plan.status()
    yr, zr, _ = run_oracle(data, return_z=True)
    zg = z.float().cpu().numpy()
    assert (zg[:, G:] == 0).all()                      # padding columns are zeros
    assert rel_err(zg[:, :G].reshape(spec.N, spec.Ho, spec.Wo, G), zr) <= 2 ** -8
    # the PW stage alone, against the reference PW applied to the GPU's own (rounded) z
    yr2, _ = orc.pw(zg[:, :G].reshape(spec.N, spec.Ho, spec.Wo, G).astype(np.float64), data.pw_w, data.bias, layout="NHWC")
    assert rel_err(y.float().cpu().numpy(), yr2) <= 2 ** -7
    assert rel_err(y.float().cpu().numpy(), yr) <= TOL["bf16"]
    plan.destroy()


def test_bf16_prepacked_weights_and_rerun_is_bitwise_stable():
    spec = small_spec("t", 4, 32, 32, 8, 8, seed=13)
    data = gi.make_layer(spec)
    a = run_gpu(data, path=gdws.PATH_FUSED, prepack=True)
    b = run_gpu(data, path=gdws.PATH_FUSED, prepack=False)
    c = run_gpu(data, path=gdws.PATH_FUSED, prepack=True)
    assert np.array_equal(a, b) and np.array_equal(a, c)
    ref, _ = run_oracle(data)
    assert rel_err(a, ref) <= TOL["bf16"]


def test_config1_shape_reduced_batch():
    """Config-1 layer (C=D=256, 8x8, g~U[1,9]) at a batch the reference finishes in seconds."""
    spec = gi.config_layers(1)[0]
    data = gi.make_layer(spec, N=20)
    ref, _ = run_oracle(data)
    for path in (gdws.PATH_FUSED, gdws.PATH_UNFUSED):
        err = rel_err(run_gpu(data, path=path), ref)
        assert err <= TOL["bf16"], (path, err)


def test_forward_rejects_bad_tensors():
    data = gi.make_layer(small_spec("t", 2, 16, 16, 8, 8, seed=3))
    plan = make_plan(data)
    x = to_device(data.x, "bf16")
    y = torch.empty((2, 8, 8, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdws.GdwsError) as e:
        plan.forward(x, y, "NHWC")                                  # no weights yet
    assert e.value.status == gdws.ERR_INVALID_ARG
    dw, pw = to_device(data.dw_w, "bf16"), to_device(data.pw_w, "bf16")
    ybad = torch.empty((2, 7, 8, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdws.GdwsError) as e:
        plan.forward(x, ybad, "NHWC", dw, pw)
    assert e.value.status == gdws.ERR_INVALID_ARG
    with pytest.raises(gdws.GdwsError) as e:
        plan.forward(x, x, "NHWC", dw, pw)                          # aliasing
    assert e.value.status == gdws.ERR_INVALID_ARG
    plan.set_option(gdws.OPT_PATH, gdws.PATH_UNFUSED)
    with pytest.raises(gdws.GdwsError) as e:
        plan.forward(x, y, "NHWC", dw, pw)                          # no workspace
    assert e.value.status == gdws.ERR_WORKSPACE
    before = plan.launch_count()
    xn = torch.empty((2, 16, 8, 8), dtype=torch.bfloat16, device="cuda")
    yn = torch.empty((2, 16, 8, 8), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdws.GdwsError) as e:
        plan.forward(xn, yn, "NCHW", dw, pw)
    assert e.value.status == gdws.ERR_UNSUPPORTED and plan.launch_count() == before
    plan.destroy()


def test_forward_host_matches_device_forward():
    spec = small_spec("t", 4, 16, 16, 8, 8, seed=21)
    data = gi.make_layer(spec)
    plan = make_plan(data)
    dw, pw = to_device(data.dw_w, "bf16"), to_device(data.pw_w, "bf16")
    b = torch.from_numpy(data.bias).cuda()
    plan.pack_weights(dw, pw, b)
    xh = torch.from_numpy(data.x).to(torch.bfloat16).pin_memory()
    yh = torch.empty((spec.N, spec.Ho, spec.Wo, spec.D), dtype=torch.bfloat16).pin_memory()
    plan.forward_host(xh, yh, "NHWC")
    ref, _ = run_oracle(data)
    assert rel_err(yh.float().numpy(), ref) <= TOL["bf16"]
    plan.destroy()


# ------------------------------------------------------------------ diagnostics
def test_bounded_wait_reports_once_and_plan_stays_usable():
    """A wait that nothing satisfies runs out after its poll limit: the kernel returns by itself, the
    status word reports the time-out once, and the same plan then runs a normal forward."""
    spec = small_spec("t", 2, 16, 16, 8, 8, 3, 1, 1, ("uniform", 1, 9), "bf16", "NHWC", seed=81)
    data = gi.make_layer(spec)
    plan = make_plan(data, path=gdws.PATH_FUSED)
    plan.status()
    plan.selftest_wait(polls=32)
    torch.cuda.synchronize()
    with pytest.raises(gdws.GdwsError) as e:
        plan.status()
    assert e.value.status == gdws.ERR_DEVICE_TIMEOUT
    plan.status()                                   # cleared by the report
    x, dw, pw = (to_device(a, "bf16") for a in (data.x, data.dw_w, data.pw_w))
    b = torch.from_numpy(data.bias).cuda()
    y = torch.full((spec.N, spec.Ho, spec.Wo, spec.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.forward(x, y, "NHWC", dw, pw, b)
    torch.cuda.synchronize()
    plan.status()
    ref, _ = run_oracle(data)
    assert rel_err(y.float().cpu().numpy().astype(np.float64), ref) <= TOL["bf16"]
    plan.destroy()


def test_fma_rate_measurement_is_plausible():
    """The ALU multiply-add rate that bench.py reports as the bound of a GDW stage on the ALUs: between
    half and all of the 128 fp32 lanes of an SM, and the packed forms no faster in multiply-adds."""
    per_clk, tmacs = gdws.measure_fma_rate(gdws.FMA_F32)
    assert 64.0 <= per_clk <= 130.0 and tmacs > 5.0
    per_clk2, _ = gdws.measure_fma_rate(gdws.FMA_F32X2)
    assert 64.0 <= per_clk2 <= 135.0


def test_code_size_cliff_is_where_the_kernels_assume_it():
    """A loop of 16 KB runs from the SM's instruction caches, a loop of 64 KB at the speed of instruction fetch: why
    the kernels keep what their warps execute per chunk small and their polling loops out of line."""
    small = gdws.measure_code_size(1024, 512)
    large = gdws.measure_code_size(4096, 512)
    assert small > 0.7 and large < 0.75 * small, (small, large)


@pytest.mark.parametrize("variant", ["alu", "tensor_cores", "unfused"])
def test_fp32_output_of_a_bf16_plan(variant):
    """GDWS_OPT_OUT_DTYPE = 1: y keeps the fp32 sums of the PW stage (bias, ReLU applied, no rounding to bf16), so it
    is at least as close to the reference as the bf16 output, and equal to it after rounding."""
    spec = small_spec("t", 3, 32, 40, 12, 9, 3, 1, 1, ("uniform", 1, 9), "bf16", "NHWC", relu=True, seed=91)
    data = gi.make_layer(spec)
    ref, _ = run_oracle(data)
    path = gdws.PATH_UNFUSED if variant == "unfused" else gdws.PATH_FUSED
    dw_math = 2 if variant == "tensor_cores" else 1
    want16 = run_gpu(data, path=path, dw_math=dw_math)
    plan = make_plan(data, path=path, dw_math=dw_math)
    plan.set_option(gdws.OPT_OUT_DTYPE, 1)
    x, dw, pw = (to_device(a, "bf16") for a in (data.x, data.dw_w, data.pw_w))
    b = torch.from_numpy(data.bias).cuda()
    if path == gdws.PATH_UNFUSED:
        ws = torch.empty(plan.workspace_bytes(gdws.BF16, spec.N, spec.H, spec.W), dtype=torch.uint8, device="cuda")
        plan.set_workspace(ws)
    y = torch.full((spec.N, spec.Ho, spec.Wo, spec.D), float("nan"), dtype=torch.float32, device="cuda")
    plan.forward(x, y, "NHWC", dw, pw, b)
    torch.cuda.synchronize()
    plan.status()
    got = y.cpu().numpy().astype(np.float64)
    assert rel_err(got, ref) <= TOL["bf16"]
    assert rel_err(got, ref) <= rel_err(want16, ref) + 1e-6
    assert np.array_equal(y.to(torch.bfloat16).float().cpu().numpy().astype(np.float64), want16)
    y16 = torch.empty((spec.N, spec.Ho, spec.Wo, spec.D), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdws.GdwsError):
        plan.forward(x, y16, "NHWC", dw, pw, b)        # the plan now expects an fp32 y
    plan.destroy()
