"""Helpers shared by the GPU parity tests: run one synthetic layer through the C-ABI
library and through the CPU reference, return both results as float64 arrays."""
import numpy as np
import torch

from oracle import gdws_oracle as orc
from paper_2110_14871_b200 import gdws
from paper_2110_14871_b200 import inputs as gi

TOL = {"f32": 1e-4, "bf16": 2e-2}   # max|y - y_ref| / max|y_ref|


def to_device(a: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)          # exact: the values are bf16-representable
    return t.cuda()


def rel_err(y: np.ndarray, ref: np.ndarray) -> float:
    assert y.shape == ref.shape, (y.shape, ref.shape)
    assert np.isfinite(y).all(), "non-finite values in the GPU output"
    return float(np.max(np.abs(y.astype(np.float64) - ref)) / max(np.max(np.abs(ref)), 1e-30))


GUARD_BYTES = 4096
_SENTINEL = 0x5A


class Guarded:
    """A device tensor of `shape` carved out of a larger byte buffer, with GUARD_BYTES of a sentinel
    before and after it.  check() fails if a kernel wrote outside the tensor (the role a memory checker
    would play)."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape))
        esz = torch.empty((), dtype=dtype).element_size()
        body = (n * esz + 255) // 256 * 256
        self.raw = torch.full((GUARD_BYTES + body + GUARD_BYTES,), _SENTINEL, dtype=torch.uint8, device="cuda")
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + n * esz].view(dtype).view(shape)
        self._tail = GUARD_BYTES + n * esz
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what="buffer"):
        before = self.raw[:GUARD_BYTES]
        after = self.raw[self._tail:]
        assert bool((before == _SENTINEL).all()), f"bytes before {what} were overwritten"
        assert bool((after == _SENTINEL).all()), f"bytes after {what} were overwritten"


def make_plan(data: gi.LayerData, path=gdws.PATH_AUTO, a_layout=0, dw_math=0, tile=0) -> gdws.Plan:
    s = data.spec
    plan = gdws.Plan(s.C, s.D, s.k, s.stride, s.pad, data.g)
    plan.set_option(gdws.OPT_PATH, path)
    plan.set_option(gdws.OPT_RELU, int(s.relu))
    plan.set_option(gdws.OPT_A_LAYOUT, a_layout)
    plan.set_option(gdws.OPT_DW_MATH, dw_math)
    if tile:
        plan.set_option(gdws.OPT_TILE, tile)
    return plan


def run_gpu(data: gi.LayerData, path=gdws.PATH_AUTO, a_layout=0, dw_math=0, tile=0, prepack=False, poison=True):
    """y of the library for `data` as float64, in the layer's layout order."""
    s = data.spec
    plan = make_plan(data, path, a_layout, dw_math, tile)
    x = to_device(data.x, s.dtype)
    dw = to_device(data.dw_w, s.dtype)
    pw = to_device(data.pw_w, s.dtype)
    b = torch.from_numpy(data.bias).cuda()
    tdt = torch.float32 if s.dtype == "f32" else torch.bfloat16
    shape = (s.N, s.D, s.Ho, s.Wo) if s.layout == "NCHW" else (s.N, s.Ho, s.Wo, s.D)
    yg = Guarded(shape, tdt, fill=float("nan") if poison else 0.0)
    y = yg.t
    code = gdws.F32 if s.dtype == "f32" else gdws.BF16
    wsg = None
    if path == gdws.PATH_UNFUSED:
        nbytes = plan.workspace_bytes(code, s.N, s.H, s.W)
        wsg = Guarded((nbytes,), torch.uint8, fill=0xFF)
        plan.set_workspace(wsg.t)
    if prepack and s.dtype == "bf16":
        plan.pack_weights(dw, pw, b)
        plan.forward(x, y, s.layout)
    else:
        plan.forward(x, y, s.layout, dw, pw, b)
    torch.cuda.synchronize()
    plan.status()
    yg.check("y")
    if wsg is not None:
        wsg.check("the workspace")
    out = y.float().cpu().numpy().astype(np.float64)
    plan.destroy()
    return out


def run_oracle(data: gi.LayerData, return_z=False):
    s = data.spec
    return orc.forward(data.x, data.g, data.dw_w, data.pw_w, data.bias, stride=s.stride, pad=s.pad,
                       relu=s.relu, layout=s.layout, return_z=return_z)


def small_spec(name, N, C, D, H, W, k=3, stride=1, pad=1, g_dist=("uniform", 1, 9), dtype="bf16",
               layout="NHWC", relu=False, seed=1):
    return gi.LayerSpec(name, N, C, D, H, W, k, stride, pad, g_dist, dtype, layout, relu, seed)
