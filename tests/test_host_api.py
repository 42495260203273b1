"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, validates arguments, and its plan tables follow
Property 2 (intermediate channel i = off_c + j) and Eq. 3 (complexity)."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import gdws_oracle as orc
from paper_2110_14871_b200 import build as gbuild
from paper_2110_14871_b200 import gdws
from paper_2110_14871_b200 import inputs as gi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    gbuild.build_library()


def declared_symbols():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"GDWS_API\s+[\w\s\*]+?\b(gdws_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 18 and set(gdws.EXPORTS) <= set(names)
    L = ctypes.CDLL(gdws.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n
    assert "sm_100a" in gdws.version()


def test_plan_rejects_bad_arguments():
    g = [1, 2, 3]
    bad = [
        dict(C=0, D=4, k=3, stride=1, pad=1, g=[]),
        dict(C=3, D=0, k=3, stride=1, pad=1, g=g),
        dict(C=3, D=4, k=0, stride=1, pad=1, g=g),
        dict(C=3, D=4, k=9, stride=1, pad=1, g=g),
        dict(C=3, D=4, k=3, stride=0, pad=1, g=g),
        dict(C=3, D=4, k=3, stride=1, pad=-1, g=g),
        dict(C=3, D=4, k=3, stride=1, pad=1, g=[1, -1, 2]),
        dict(C=3, D=4, k=3, stride=1, pad=1, g=[0, 0, 0]),
    ]
    for kw in bad:
        with pytest.raises((gdws.GdwsError, ValueError)) as ei:
            gdws.Plan(**kw)
        if isinstance(ei.value, gdws.GdwsError):
            assert ei.value.status == gdws.ERR_INVALID_ARG and gdws.last_error()
    L = gdws.lib()
    assert L.gdws_plan(3, 4, 3, 1, 1, None, ctypes.byref(ctypes.c_void_p())) == gdws.ERR_INVALID_ARG
    garr = (ctypes.c_int32 * 3)(1, 2, 3)
    assert L.gdws_plan(3, 4, 3, 1, 1, garr, None) == gdws.ERR_INVALID_ARG
    L.gdws_destroy(None)          # no-op


def test_plan_tables_follow_property_2_and_eq_3():
    rng = np.random.default_rng(0)
    for C, D, k in [(5, 7, 3), (64, 64, 3), (33, 16, 5), (8, 8, 1)]:
        g = rng.integers(0, k * k + 1, size=C).astype(np.int32)
        g[0] = max(g[0], 1)
        plan = gdws.Plan(C, D, k, 1, k // 2, g)
        G, Gp, macs, params = plan.info()
        assert G == g.sum() and Gp % 64 == 0 and 0 <= Gp - G < 64
        assert macs == orc.gdws_macs(1, 1, G, k, D) and params == orc.gdws_params(G, k, D)
        off, chan = plan.tables()
        assert np.array_equal(off, orc.offsets(g).astype(np.int32))
        assert np.array_equal(chan[:G], np.repeat(np.arange(C), g)) and (chan[G:] == -1).all()
        plan.destroy()


def test_options_and_workspace_queries():
    plan = gdws.Plan(8, 8, 3, 1, 1, [1] * 8)
    for key, val in [(gdws.OPT_PATH, 7), (gdws.OPT_RELU, 2), (99, 0), (gdws.OPT_TILE, (1 << 16) | (8 << 8) | 5),
                     (gdws.OPT_TILE, (2 << 16) | (16 << 8) | 8), (gdws.OPT_A_LAYOUT, 3)]:
        with pytest.raises(gdws.GdwsError):
            plan.set_option(key, val)
    plan.set_option(gdws.OPT_TILE, (2 << 16) | (8 << 8) | 8)
    assert plan.tile(4, 8, 8)[:3] == (2, 8, 8)
    assert plan.workspace_bytes(gdws.F32, 2, 6, 6) == 2 * 36 * 8 * 4
    assert plan.workspace_bytes(gdws.BF16, 2, 6, 6) == 2 * 36 * 64 * 2
    assert plan.workspace_bytes(gdws.F32, 2, 1, 1) == 2 * 8 * 4      # pad 1: 1x1 output
    assert gdws.out_dim(56, 3, 2, 1) == 28 and gdws.out_dim(2, 5, 1, 0) == 0
    assert plan.launch_count() == 0
    plan.destroy()
    plan.destroy()


@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_fused_tiles_cover_the_benchmark_layers(cfg):
    """Every bf16 benchmark layer gets a fused tile: TN*PH*PW <= 128 rows, and the
    tile grid covers the whole output."""
    for spec in gi.config_layers(cfg):
        rng = np.random.Generator(np.random.PCG64(spec.seed))
        g = gi.make_g(rng, spec.C, spec.g_dist)
        plan = gdws.Plan(spec.C, spec.D, spec.k, spec.stride, spec.pad, g)
        TN, PH, PW, tiles = plan.tile(spec.N, spec.H, spec.W)
        assert TN * PH * PW <= 128 and PW in (4, 8, 16, 32)
        need = -(-spec.N // TN) * -(-spec.Ho // PH) * -(-spec.Wo // PW)
        assert tiles == need
        waste = tiles * 128 / (spec.N * spec.Ho * spec.Wo)
        assert waste < 1.35, (spec.name, TN, PH, PW, waste)
        plan.destroy()


def test_gdw_stage_choice_follows_the_documented_rule():
    """Tensor cores for k = 3 or 5, stride 1 or 2, at most 256 output channels and an average multiplier of at least 4
    (2.7 with at most 128 output channels); the option overrides the choice."""
    def stage(C, D, k, stride, g, opt=0):
        plan = gdws.Plan(C, D, k, stride, k // 2, np.full(C, g, dtype=np.int32))
        plan.set_option(gdws.OPT_DW_MATH, opt)
        s = plan.gdw_stage()
        plan.destroy()
        return s
    assert stage(64, 64, 3, 1, 5) == 2
    assert stage(64, 64, 3, 1, 2) == 1          # few filters per channel: the ALU kernel's cost follows G
    assert stage(64, 128, 3, 1, 3) == 2 and stage(64, 256, 3, 1, 3) == 1     # small PW products move the boundary
    assert stage(64, 512, 3, 1, 5) == 1         # no room for two GDW accumulators beside 512 output columns
    assert stage(64, 64, 3, 2, 5) == 2 and stage(64, 64, 3, 3, 5) == 1     # strides 1 and 2 are covered by the tensor-core form
    assert stage(64, 512, 3, 2, 5) == 2         # with stride 2 also beyond 256 output channels
    assert stage(64, 64, 5, 1, 12) == 2 and stage(64, 64, 4, 1, 12) == 1
    assert stage(64, 64, 3, 1, 2, opt=2) == 2 and stage(64, 64, 3, 1, 5, opt=1) == 1
