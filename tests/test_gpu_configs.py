"""Parity at the benchmark's full layer sizes (configs 1-4), in the launch configuration that
bench.py times (fused path, packed weights), on sampled images the CPU reference can compute one
by one; and the 16-layer chain of config 3 checked layer by layer (teacher forced).

Layers whose input fits host memory comfortably take exactly the seeded instance that bench.py times
(`inputs.make_layer(spec)`); for the largest ones the activations are drawn on the device with a seeded
generator and the weights with the recipe's generator.  Every full-size launch writes into a buffer with
guard bands, and runs twice with bitwise-equal results."""
import numpy as np
import pytest
import torch

from oracle import gdws_oracle as orc
from paper_2110_14871_b200 import build as gbuild
from paper_2110_14871_b200 import gdws
from paper_2110_14871_b200 import inputs as gi

from util import TOL, Guarded, rel_err

pytestmark = pytest.mark.gpu

HOST_DRAW_LIMIT = 60_000_000      # activations up to this many elements are drawn on the host by the recipe


@pytest.fixture(scope="module", autouse=True)
def built():
    gbuild.build_library()


def _layer_on_gpu(spec, g, x, dw_w, pw_w, bias, path=gdws.PATH_FUSED, dw_math=0, twice=False):
    """x: torch bf16 NHWC on the device.  Returns y (torch bf16 NHWC)."""
    plan = gdws.Plan(spec.C, spec.D, spec.k, spec.stride, spec.pad, g)
    plan.set_option(gdws.OPT_PATH, path)
    plan.set_option(gdws.OPT_RELU, int(spec.relu))
    plan.set_option(gdws.OPT_DW_MATH, dw_math)
    dw = torch.from_numpy(dw_w).to(torch.bfloat16).cuda()
    pw = torch.from_numpy(pw_w).to(torch.bfloat16).cuda()
    b = torch.from_numpy(bias).cuda()
    plan.pack_weights(dw, pw, b)
    wsg = None
    if path == gdws.PATH_UNFUSED:
        wsg = Guarded((plan.workspace_bytes(gdws.BF16, x.shape[0], spec.H, spec.W),), torch.uint8, fill=0xFF)
        plan.set_workspace(wsg.t)
    yg = Guarded((x.shape[0], spec.Ho, spec.Wo, spec.D), torch.bfloat16, fill=float("nan"))
    plan.forward(x, yg.t, "NHWC")
    torch.cuda.synchronize()
    plan.status()
    yg.check("y")
    if wsg is not None:
        wsg.check("the workspace")
    if twice:
        first = yg.t.clone()
        yg.t.fill_(float("nan"))
        plan.forward(x, yg.t, "NHWC")
        torch.cuda.synchronize()
        plan.status()
        yg.check("y (second launch)")
        assert torch.equal(first.view(torch.int16), yg.t.view(torch.int16)), "two launches on the same input differ"
    plan.destroy()
    return yg.t


def _weights(spec):
    """Seeded g and weights of a layer, drawn as the recipe draws them when the activations are skipped."""
    rng = np.random.Generator(np.random.PCG64(spec.seed))
    g = gi.make_g(rng, spec.C, spec.g_dist)
    G = int(g.sum())
    dw_w = gi.round_to_bf16((rng.standard_normal((G, spec.k, spec.k)) / spec.k).astype(np.float32))
    pw_w = gi.round_to_bf16((rng.standard_normal((spec.D, G)) / np.sqrt(G)).astype(np.float32))
    bias = (rng.standard_normal(spec.D) * 0.1).astype(np.float32)
    return g, dw_w, pw_w, bias


def _instance(spec):
    """(g, x on the device, dw_w, pw_w, bias, what) of a full-size layer."""
    if spec.N * spec.H * spec.W * spec.C <= HOST_DRAW_LIMIT:
        d = gi.make_layer(spec)                 # the instance bench.py times
        x = torch.from_numpy(d.x).to(torch.bfloat16).cuda()
        return d.g, x, d.dw_w, d.pw_w, d.bias, "recipe"
    g, dw_w, pw_w, bias = _weights(spec)
    gen = torch.Generator(device="cuda").manual_seed(spec.seed)
    x = torch.randn((spec.N, spec.H, spec.W, spec.C), generator=gen, device="cuda").to(torch.bfloat16)
    return g, x, dw_w, pw_w, bias, "device draw"


def _check_sampled(spec, g, x, dw_w, pw_w, bias, y):
    assert torch.isfinite(y.float()).all()
    sel = sorted({0, spec.N // 2, spec.N - 1}) if spec.H <= 56 else [spec.N - 1]
    xs = x[sel].float().cpu().numpy()
    ref, _ = orc.forward(xs, g, dw_w, pw_w, bias, stride=spec.stride, pad=spec.pad, relu=spec.relu, layout="NHWC")
    got = y[sel].float().cpu().numpy()
    assert rel_err(got, ref) <= TOL["bf16"]


SINGLE = [(c, l) for c in (1, 2, 4) for l in range(len(gi.config_layers(c)))]


@pytest.mark.parametrize("cfg,layer", SINGLE)
def test_full_size_layer_sampled_images(cfg, layer):
    spec = gi.config_layers(cfg)[layer]
    g, x, dw_w, pw_w, bias, _ = _instance(spec)
    y = _layer_on_gpu(spec, g, x, dw_w, pw_w, bias, twice=True)
    _check_sampled(spec, g, x, dw_w, pw_w, bias, y)


# the other launch configurations at full size: GDW stage forced onto the ALUs / the tensor cores (the default
# lets the library choose), and the unfused pair
OTHER = [(1, 0), (2, 0), (4, 4)]


@pytest.mark.parametrize("cfg,layer", OTHER)
@pytest.mark.parametrize("variant", ["alu_gdw", "tensor_core_gdw", "unfused"])
def test_full_size_other_paths(cfg, layer, variant):
    spec = gi.config_layers(cfg)[layer]
    g, x, dw_w, pw_w, bias, _ = _instance(spec)
    if variant == "alu_gdw":
        y = _layer_on_gpu(spec, g, x, dw_w, pw_w, bias, path=gdws.PATH_FUSED, dw_math=1, twice=True)
    elif variant == "tensor_core_gdw":
        y = _layer_on_gpu(spec, g, x, dw_w, pw_w, bias, path=gdws.PATH_FUSED, dw_math=2, twice=True)
    else:
        y = _layer_on_gpu(spec, g, x, dw_w, pw_w, bias, path=gdws.PATH_UNFUSED, twice=True)
    _check_sampled(spec, g, x, dw_w, pw_w, bias, y)


def test_config3_chain_teacher_forced():
    """The 16 chained layers (ReLU between them) at N=512: layer l's GPU output is compared with the
    reference applied to the GPU's own layer l-1 output, on sampled images; the free-running error of
    the last layer against a reference chain is reported as well."""
    layers = gi.config_layers(3)
    N = layers[0].N
    gen = torch.Generator(device="cuda").manual_seed(3000)
    x = torch.randn((N, layers[0].H, layers[0].W, layers[0].C), generator=gen, device="cuda").to(torch.bfloat16)
    sel = [0, N // 2, N - 1]
    free = x[sel].float().cpu().numpy().astype(np.float64)
    for spec in layers:
        g, dw_w, pw_w, bias = _weights(spec)
        y = _layer_on_gpu(spec, g, x, dw_w, pw_w, bias)
        ref, _ = orc.forward(x[sel].float().cpu().numpy(), g, dw_w, pw_w, bias, stride=spec.stride, pad=spec.pad,
                             relu=spec.relu, layout="NHWC")
        err = rel_err(y[sel].float().cpu().numpy(), ref)
        assert err <= TOL["bf16"], (spec.name, err)
        free, _ = orc.forward(free, g, dw_w, pw_w, bias, stride=spec.stride, pad=spec.pad, relu=spec.relu, layout="NHWC")
        x = y
    end_to_end = rel_err(x[sel].float().cpu().numpy(), free)
    assert end_to_end <= 0.1, end_to_end      # 16 layers of bf16 rounding; informational bound
