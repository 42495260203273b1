"""Parity at the benchmark's full layer sizes (configs 1-4), in the launch configuration that
bench.py times (fused path, packed weights), on sampled images the CPU reference can compute one
by one; and the 16-layer chain of config 3 checked layer by layer (teacher forced)."""
import numpy as np
import pytest
import torch

from oracle import gdws_oracle as orc
from paper_2110_14871_b200 import build as gbuild
from paper_2110_14871_b200 import gdws
from paper_2110_14871_b200 import inputs as gi

from util import TOL, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    gbuild.build_library()


def _layer_on_gpu(spec, g, x, dw_w, pw_w, bias, path=gdws.PATH_FUSED):
    """x: torch bf16 NHWC on the device.  Returns y (torch bf16 NHWC)."""
    plan = gdws.Plan(spec.C, spec.D, spec.k, spec.stride, spec.pad, g)
    plan.set_option(gdws.OPT_PATH, path)
    plan.set_option(gdws.OPT_RELU, int(spec.relu))
    dw = torch.from_numpy(dw_w).to(torch.bfloat16).cuda()
    pw = torch.from_numpy(pw_w).to(torch.bfloat16).cuda()
    b = torch.from_numpy(bias).cuda()
    plan.pack_weights(dw, pw, b)
    y = torch.full((x.shape[0], spec.Ho, spec.Wo, spec.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.forward(x, y, "NHWC")
    torch.cuda.synchronize()
    plan.status()
    plan.destroy()
    return y


def _weights(spec):
    """Seeded g and weights of a layer (activations drawn separately, on the device)."""
    rng = np.random.Generator(np.random.PCG64(spec.seed))
    g = gi.make_g(rng, spec.C, spec.g_dist)
    G = int(g.sum())
    dw_w = gi.round_to_bf16((rng.standard_normal((G, spec.k, spec.k)) / spec.k).astype(np.float32))
    pw_w = gi.round_to_bf16((rng.standard_normal((spec.D, G)) / np.sqrt(G)).astype(np.float32))
    bias = (rng.standard_normal(spec.D) * 0.1).astype(np.float32)
    return g, dw_w, pw_w, bias


SINGLE = [(c, l) for c in (1, 2, 4) for l in range(len(gi.config_layers(c)))]


@pytest.mark.parametrize("cfg,layer", SINGLE)
def test_full_size_layer_sampled_images(cfg, layer):
    spec = gi.config_layers(cfg)[layer]
    g, dw_w, pw_w, bias = _weights(spec)
    gen = torch.Generator(device="cuda").manual_seed(spec.seed)
    x = torch.randn((spec.N, spec.H, spec.W, spec.C), generator=gen, device="cuda").to(torch.bfloat16)
    y = _layer_on_gpu(spec, g, x, dw_w, pw_w, bias)
    assert torch.isfinite(y.float()).all()
    sel = sorted({0, spec.N // 2, spec.N - 1}) if spec.H <= 56 else [spec.N - 1]
    xs = x[sel].float().cpu().numpy()
    ref, _ = orc.forward(xs, g, dw_w, pw_w, bias, stride=spec.stride, pad=spec.pad, relu=spec.relu, layout="NHWC")
    got = y[sel].float().cpu().numpy()
    assert rel_err(got, ref) <= TOL["bf16"]


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
