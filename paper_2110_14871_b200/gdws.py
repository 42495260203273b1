"""Thin ctypes binding of ``libgdws.so`` (interface: ``include/gdws.h``).

Argument marshalling only: every step of the GDWS forward (Section 3.1 of
arXiv 2110.14871: GDW convolution, PW convolution, bias) runs in the CUDA
library.  PyTorch tensors are used as device (or pinned host) buffers; their
``data_ptr()`` and the current stream are passed through.  If the shared library
is missing this module raises: there is no other path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgdws.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_ARCH, ERR_WORKSPACE = range(8)
F32, BF16 = 0, 1
NCHW, NHWC = 0, 1
OPT_PATH, OPT_RELU, OPT_TILE, OPT_A_LAYOUT, OPT_DW_MATH, OPT_OUT_DTYPE = range(6)
PATH_AUTO, PATH_FUSED, PATH_UNFUSED = 0, 1, 2

EXPORTS = [
    "gdws_plan", "gdws_plan_set_option", "gdws_plan_info", "gdws_plan_tables", "gdws_plan_tile",
    "gdws_out_dim", "gdws_pack_weights", "gdws_workspace_bytes", "gdws_set_workspace", "gdws_forward",
    "gdws_depthwise", "gdws_pointwise", "gdws_forward_host", "gdws_status", "gdws_launch_count",
    "gdws_last_error", "gdws_version", "gdws_destroy", "gdws_forward_static", "gdws_static_scratch_bytes",
    "gdws_measure_fma_rate", "gdws_measure_code_size", "gdws_selftest_wait", "gdws_plan_gdw_stage",
]


class GdwsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"gdws status {status}: {message}")
        self.status = status


class Tensor(ctypes.Structure):
    """Mirror of gdws_tensor_t."""
    _fields_ = [("ptr", ctypes.c_void_p), ("dtype", ctypes.c_int), ("layout", ctypes.c_int),
                ("n", ctypes.c_int), ("c", ctypes.c_int), ("h", ctypes.c_int), ("w", ctypes.c_int)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libgdws.so (built in-tree by ``build.build_library``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2110_14871_b200.build` "
            "(there is no fallback implementation)")
    L = ctypes.CDLL(LIB_PATH)
    vp, ci, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    pi32 = ctypes.POINTER(ctypes.c_int32)
    pint = ctypes.POINTER(ctypes.c_int)
    pi64 = ctypes.POINTER(ctypes.c_int64)
    pt = ctypes.POINTER(Tensor)
    L.gdws_plan.argtypes = [ci, ci, ci, ci, ci, pi32, ctypes.POINTER(vp)]
    L.gdws_plan.restype = ci
    L.gdws_plan_set_option.argtypes = [vp, ci, ci]
    L.gdws_plan_set_option.restype = ci
    L.gdws_plan_info.argtypes = [vp, pint, pint, pi64, pi64]
    L.gdws_plan_info.restype = ci
    L.gdws_plan_tables.argtypes = [vp, pi32, pi32]
    L.gdws_plan_tables.restype = ci
    L.gdws_plan_tile.argtypes = [vp, ci, ci, ci, pint, pint, pint, pi64]
    L.gdws_plan_tile.restype = ci
    L.gdws_plan_gdw_stage.argtypes = [vp, pint]
    L.gdws_plan_gdw_stage.restype = ci
    L.gdws_out_dim.argtypes = [ci, ci, ci, ci]
    L.gdws_out_dim.restype = ci
    L.gdws_pack_weights.argtypes = [vp, vp, vp, vp, ci, vp]
    L.gdws_pack_weights.restype = ci
    L.gdws_workspace_bytes.argtypes = [vp, ci, ci, ci, ci]
    L.gdws_workspace_bytes.restype = ctypes.c_size_t
    L.gdws_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    L.gdws_set_workspace.restype = ci
    L.gdws_forward.argtypes = [vp, pt, vp, vp, vp, pt, vp]
    L.gdws_forward.restype = ci
    L.gdws_depthwise.argtypes = [vp, pt, vp, vp, vp]
    L.gdws_depthwise.restype = ci
    L.gdws_pointwise.argtypes = [vp, vp, vp, vp, pt, vp]
    L.gdws_pointwise.restype = ci
    L.gdws_forward_host.argtypes = [vp, pt, vp, vp, vp, pt, vp]
    L.gdws_forward_host.restype = ci
    L.gdws_forward_static.argtypes = [vp, pt, vp, vp, vp, pt, vp]
    L.gdws_forward_static.restype = ci
    L.gdws_static_scratch_bytes.argtypes = []
    L.gdws_static_scratch_bytes.restype = ctypes.c_size_t
    L.gdws_status.argtypes = [vp]
    L.gdws_status.restype = ci
    L.gdws_measure_fma_rate.argtypes = [ci, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    L.gdws_measure_fma_rate.restype = ci
    L.gdws_measure_code_size.argtypes = [ci, ci, ctypes.POINTER(ctypes.c_double)]
    L.gdws_measure_code_size.restype = ci
    L.gdws_selftest_wait.argtypes = [vp, ctypes.c_uint, vp]
    L.gdws_selftest_wait.restype = ci
    L.gdws_launch_count.argtypes = [vp]
    L.gdws_launch_count.restype = i64
    L.gdws_last_error.argtypes = []
    L.gdws_last_error.restype = ctypes.c_char_p
    L.gdws_version.argtypes = []
    L.gdws_version.restype = ctypes.c_char_p
    L.gdws_destroy.argtypes = [vp]
    L.gdws_destroy.restype = None
    _lib = L
    return L


def last_error() -> str:
    return lib().gdws_last_error().decode()


def version() -> str:
    return lib().gdws_version().decode()


def static_scratch_bytes() -> int:
    return int(lib().gdws_static_scratch_bytes())


FMA_F32, FMA_F32X2, FMA_BF16X2, FMA_F32_BF16 = range(4)


def measure_fma_rate(kind: int = FMA_F32) -> Tuple[float, float]:
    """gdws_measure_fma_rate: (multiply-adds per clock and SM, 1e12 multiply-adds per second on the device)."""
    per_clk, tmacs = ctypes.c_double(), ctypes.c_double()
    _check(lib().gdws_measure_fma_rate(kind, ctypes.byref(per_clk), ctypes.byref(tmacs)))
    return per_clk.value, tmacs.value


def measure_code_size(body_instructions: int, threads: int = 512) -> float:
    """gdws_measure_code_size: instructions per clock and scheduler for a loop body of that many instructions."""
    ipc = ctypes.c_double()
    _check(lib().gdws_measure_code_size(body_instructions, threads, ctypes.byref(ipc)))
    return ipc.value


def out_dim(size: int, k: int, stride: int, pad: int) -> int:
    return int(lib().gdws_out_dim(size, k, stride, pad))


def _check(status: int) -> None:
    if status != OK:
        raise GdwsError(status, last_error())


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def tensor_desc(t, layout: str) -> Tensor:
    """gdws_tensor_t for a contiguous 4-D torch tensor stored in ``layout`` order."""
    if t.dim() != 4 or not t.is_contiguous():
        raise ValueError("expected a contiguous 4-D tensor")
    if layout == "NCHW":
        n, c, h, w = t.shape
        code = NCHW
    elif layout == "NHWC":
        n, h, w, c = t.shape
        code = NHWC
    else:
        raise ValueError(layout)
    return Tensor(t.data_ptr(), _dtype_code(t), code, int(n), int(c), int(h), int(w))


class Plan:
    """Owner of one gdws_plan_t.  Method names follow the C entry points."""

    def __init__(self, C: int, D: int, k: int, stride: int, pad: int, g: Sequence[int]):
        garr = np.ascontiguousarray(np.asarray(g), dtype=np.int32)
        if garr.ndim != 1 or garr.size != C:
            raise ValueError("g must have C entries")
        handle = ctypes.c_void_p()
        st = lib().gdws_plan(C, D, k, stride, pad, garr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                             ctypes.byref(handle))
        _check(st)
        self._h = handle
        self.C, self.D, self.k, self.stride, self.pad = C, D, k, stride, pad
        self._keep = []

    # -- lifetime
    def destroy(self) -> None:
        if getattr(self, "_h", None):
            lib().gdws_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- host-side queries
    def set_option(self, key: int, value: int) -> None:
        _check(lib().gdws_plan_set_option(self._h, key, value))

    def info(self) -> Tuple[int, int, int, int]:
        G, Gp = ctypes.c_int(), ctypes.c_int()
        macs, params = ctypes.c_int64(), ctypes.c_int64()
        _check(lib().gdws_plan_info(self._h, ctypes.byref(G), ctypes.byref(Gp), ctypes.byref(macs), ctypes.byref(params)))
        return G.value, Gp.value, macs.value, params.value

    def tables(self) -> Tuple[np.ndarray, np.ndarray]:
        _, Gp, _, _ = self.info()
        off = np.zeros(self.C + 1, dtype=np.int32)
        chan = np.zeros(Gp, dtype=np.int32)
        p32 = ctypes.POINTER(ctypes.c_int32)
        _check(lib().gdws_plan_tables(self._h, off.ctypes.data_as(p32), chan.ctypes.data_as(p32)))
        return off, chan

    def tile(self, n: int, h: int, w: int) -> Tuple[int, int, int, int]:
        TN, PH, PW = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        tiles = ctypes.c_int64()
        _check(lib().gdws_plan_tile(self._h, n, h, w, ctypes.byref(TN), ctypes.byref(PH), ctypes.byref(PW),
                                    ctypes.byref(tiles)))
        return TN.value, PH.value, PW.value, tiles.value

    def gdw_stage(self) -> int:
        """gdws_plan_gdw_stage: 1 = the fused kernel runs the GDW stage on the ALUs, 2 = on the tensor cores."""
        st = ctypes.c_int()
        _check(lib().gdws_plan_gdw_stage(self._h, ctypes.byref(st)))
        return st.value

    def workspace_bytes(self, dtype: int, n: int, h: int, w: int) -> int:
        return int(lib().gdws_workspace_bytes(self._h, dtype, n, h, w))

    def launch_count(self) -> int:
        return int(lib().gdws_launch_count(self._h))

    # -- device calls
    def set_workspace(self, ws) -> None:
        if ws is None:
            _check(lib().gdws_set_workspace(self._h, None, 0))
            self._ws = None
        else:
            _check(lib().gdws_set_workspace(self._h, ws.data_ptr(), ws.numel() * ws.element_size()))
            self._ws = ws

    def pack_weights(self, dw_w, pw_w, bias=None, stream=None) -> None:
        _check(lib().gdws_pack_weights(self._h, _ptr(dw_w), _ptr(pw_w), _ptr(bias), _dtype_code(dw_w), _stream(stream)))

    def forward(self, x, y, layout: str, dw_w=None, pw_w=None, bias=None, stream=None) -> None:
        xd, yd = tensor_desc(x, layout), tensor_desc(y, layout)
        _check(lib().gdws_forward(self._h, ctypes.byref(xd), _ptr(dw_w), _ptr(pw_w), _ptr(bias), ctypes.byref(yd),
                                  _stream(stream)))

    def depthwise(self, x, z, layout: str, dw_w=None, stream=None) -> None:
        xd = tensor_desc(x, layout)
        _check(lib().gdws_depthwise(self._h, ctypes.byref(xd), _ptr(dw_w), z.data_ptr(), _stream(stream)))

    def pointwise(self, z, y, layout: str, pw_w=None, bias=None, stream=None) -> None:
        yd = tensor_desc(y, layout)
        _check(lib().gdws_pointwise(self._h, z.data_ptr(), _ptr(pw_w), _ptr(bias), ctypes.byref(yd), _stream(stream)))

    def forward_host(self, x_host, y_host, layout: str, dw_w=None, pw_w=None, bias=None, stream=None) -> None:
        xd, yd = tensor_desc(x_host, layout), tensor_desc(y_host, layout)
        _check(lib().gdws_forward_host(self._h, ctypes.byref(xd), _ptr(dw_w), _ptr(pw_w), _ptr(bias), ctypes.byref(yd),
                                       _stream(stream)))

    def forward_static(self, x, y, layout: str, dw_w=None, pw_w=None, bias=None, stream=None) -> None:
        """gdws_forward_static: the unfused forward with the intermediate in the library's built-in
        scratch array; for callers that must not allocate device memory."""
        xd, yd = tensor_desc(x, layout), tensor_desc(y, layout)
        _check(lib().gdws_forward_static(self._h, ctypes.byref(xd), _ptr(dw_w), _ptr(pw_w), _ptr(bias),
                                         ctypes.byref(yd), _stream(stream)))

    def status(self) -> None:
        _check(lib().gdws_status(self._h))

    def selftest_wait(self, polls: int = 64, stream=None) -> None:
        """gdws_selftest_wait: a bounded wait that runs out; the next status() raises GDWS_ERR_DEVICE_TIMEOUT once."""
        _check(lib().gdws_selftest_wait(self._h, polls, _stream(stream)))
