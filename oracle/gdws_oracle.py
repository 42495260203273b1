"""ctypes front end of the CPU reference in ``gdws_oracle.c``.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline
leg load this; the CUDA library never does, and this module never imports it.

All arithmetic happens in the C file (double precision, direct loops, written
from the paper's Section 3.1 definitions and Properties 1-2).  This wrapper only
builds the shared object with gcc, converts dtypes exactly (float32 / bfloat16
values upcast to float64) and permutes NHWC <-> NCHW.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdws_oracle.c")
_SO = os.path.join(_HERE, "libgdws_oracle.so")
_lock = threading.Lock()
_lib = None

_c_int = ctypes.c_int
_c_i64 = ctypes.c_int64
_p_i32 = ctypes.POINTER(ctypes.c_int32)
_p_i64 = ctypes.POINTER(ctypes.c_int64)
_p_f64 = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile gdws_oracle.c into libgdws_oracle.so next to it (gcc, -O2, OpenMP
    on the outermost loops only; no fast-math, so sums keep their written order)."""
    with _lock:
        stale = force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if stale:
            tmp = _SO + f".tmp{os.getpid()}"
            subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                                   "-o", tmp, _SRC])
            os.replace(tmp, _SO)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.gdws_oracle_out_dim.argtypes = [_c_int] * 4
        L.gdws_oracle_out_dim.restype = _c_int
        L.gdws_oracle_offsets.argtypes = [_c_int, _p_i32, _p_i64]
        L.gdws_oracle_offsets.restype = _c_i64
        L.gdws_oracle_dense_macs.argtypes = [_c_int] * 5
        L.gdws_oracle_dense_macs.restype = _c_i64
        L.gdws_oracle_gdws_macs.argtypes = [_c_int, _c_int, _c_i64, _c_int, _c_int]
        L.gdws_oracle_gdws_macs.restype = _c_i64
        L.gdws_oracle_gdws_params.argtypes = [_c_i64, _c_int, _c_int]
        L.gdws_oracle_gdws_params.restype = _c_i64
        L.gdws_oracle_gdw.argtypes = [_c_int] * 7 + [_p_i32, _p_f64, _p_f64, _p_f64]
        L.gdws_oracle_gdw.restype = _c_i64
        L.gdws_oracle_pw.argtypes = [_c_int, _c_i64, _c_int, _c_int, _c_int, _p_f64, _p_f64, _p_f64,
                                     _c_int, _p_f64]
        L.gdws_oracle_pw.restype = _c_i64
        L.gdws_oracle_forward.argtypes = [_c_int] * 8 + [_p_i32, _p_f64, _p_f64, _p_f64, _p_f64,
                                                         _c_int, _p_f64, _p_f64]
        L.gdws_oracle_forward.restype = _c_i64
        L.gdws_oracle_dense_conv.argtypes = [_c_int] * 8 + [_p_f64, _p_f64, _p_f64, _p_f64]
        L.gdws_oracle_dense_conv.restype = _c_i64
        L.gdws_oracle_wd_matrix.argtypes = [_c_int, _c_int, _p_i32, _p_f64, _p_f64]
        L.gdws_oracle_wd_matrix.restype = None
        L.gdws_oracle_reconstruct_dense.argtypes = [_c_int, _c_int, _c_int, _p_i32, _p_f64, _p_f64, _p_f64]
        L.gdws_oracle_reconstruct_dense.restype = None
        _lib = L
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS, else all host cores)."""
    v = os.environ.get("OMP_NUM_THREADS")
    if v:
        try:
            return max(1, int(v.split(",")[0]))
        except ValueError:
            pass
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a: Optional[np.ndarray], typ):
    return None if a is None else a.ctypes.data_as(typ)


def _nchw(x: np.ndarray, layout: str) -> np.ndarray:
    if layout == "NCHW":
        return _f64(x)
    if layout == "NHWC":
        return _f64(np.transpose(x, (0, 3, 1, 2)))
    raise ValueError(layout)


def _to_layout(y_nchw: np.ndarray, layout: str) -> np.ndarray:
    if layout == "NCHW":
        return y_nchw
    return np.ascontiguousarray(np.transpose(y_nchw, (0, 2, 3, 1)))


def out_dim(size: int, k: int, stride: int, pad: int) -> int:
    return int(lib().gdws_oracle_out_dim(size, k, stride, pad))


def offsets(g) -> np.ndarray:
    g = _i32(g)
    off = np.zeros(g.size + 1, dtype=np.int64)
    lib().gdws_oracle_offsets(g.size, _ptr(g, _p_i32), _ptr(off, _p_i64))
    return off


def dense_macs(Ho, Wo, C, K, M) -> int:
    return int(lib().gdws_oracle_dense_macs(Ho, Wo, C, K, M))


def gdws_macs(Ho, Wo, G, K, M) -> int:
    return int(lib().gdws_oracle_gdws_macs(Ho, Wo, G, K, M))


def gdws_params(G, K, M) -> int:
    return int(lib().gdws_oracle_gdws_params(G, K, M))


def gdw(x, g, dw_w, stride=1, pad=0, layout="NCHW") -> Tuple[np.ndarray, int]:
    """GDW stage: returns (z in ``layout`` order, MAC count)."""
    xn = _nchw(np.asarray(x), layout)
    g = _i32(g)
    N, C, H, W = xn.shape
    Kd = _f64(dw_w)
    G, K = Kd.shape[0], Kd.shape[-1]
    assert g.size == C and int(g.sum()) == G and Kd.shape == (G, K, K)
    Ho, Wo = out_dim(H, K, stride, pad), out_dim(W, K, stride, pad)
    z = np.zeros((N, G, Ho, Wo), dtype=np.float64)
    macs = lib().gdws_oracle_gdw(N, C, H, W, K, stride, pad, _ptr(g, _p_i32), _ptr(xn, _p_f64),
                                 _ptr(Kd, _p_f64), _ptr(z, _p_f64))
    return _to_layout(z, layout), int(macs)


def pw(z, pw_w, bias=None, relu=False, layout="NCHW") -> Tuple[np.ndarray, int]:
    """PW stage + bias: returns (y in ``layout`` order, MAC count)."""
    zn = _nchw(np.asarray(z), layout)
    N, G, Ho, Wo = zn.shape
    P = _f64(pw_w)
    M = P.shape[0]
    assert P.shape == (M, G)
    b = None if bias is None else _f64(bias)
    y = np.zeros((N, M, Ho, Wo), dtype=np.float64)
    macs = lib().gdws_oracle_pw(N, G, Ho, Wo, M, _ptr(zn, _p_f64), _ptr(P, _p_f64), _ptr(b, _p_f64),
                                int(bool(relu)), _ptr(y, _p_f64))
    return _to_layout(y, layout), int(macs)


def forward(x, g, dw_w, pw_w, bias=None, stride=1, pad=0, relu=False, layout="NCHW",
            return_z=False):
    """GDWS forward.  Returns (y, macs) or (y, z, macs); arrays in ``layout`` order."""
    xn = _nchw(np.asarray(x), layout)
    g = _i32(g)
    N, C, H, W = xn.shape
    Kd, P = _f64(dw_w), _f64(pw_w)
    G, K = Kd.shape[0], Kd.shape[-1]
    M = P.shape[0]
    assert g.size == C and int(g.sum()) == G and Kd.shape == (G, K, K) and P.shape == (M, G)
    b = None if bias is None else _f64(bias)
    Ho, Wo = out_dim(H, K, stride, pad), out_dim(W, K, stride, pad)
    y = np.zeros((N, M, Ho, Wo), dtype=np.float64)
    z = np.zeros((N, G, Ho, Wo), dtype=np.float64) if return_z else None
    macs = lib().gdws_oracle_forward(N, C, H, W, M, K, stride, pad, _ptr(g, _p_i32), _ptr(xn, _p_f64),
                                     _ptr(Kd, _p_f64), _ptr(P, _p_f64), _ptr(b, _p_f64),
                                     int(bool(relu)), _ptr(z, _p_f64), _ptr(y, _p_f64))
    if macs < 0:
        raise MemoryError("oracle scratch allocation failed")
    if return_z:
        return _to_layout(y, layout), _to_layout(z, layout), int(macs)
    return _to_layout(y, layout), int(macs)


def dense_conv(x, w, bias=None, stride=1, pad=0, layout="NCHW") -> Tuple[np.ndarray, int]:
    """Standard convolution (Eq. 1) by direct loops; w is [M][C][K][K]."""
    xn = _nchw(np.asarray(x), layout)
    N, C, H, W = xn.shape
    Wt = _f64(w)
    M, K = Wt.shape[0], Wt.shape[-1]
    assert Wt.shape == (M, C, K, K)
    b = None if bias is None else _f64(bias)
    Ho, Wo = out_dim(H, K, stride, pad), out_dim(W, K, stride, pad)
    y = np.zeros((N, M, Ho, Wo), dtype=np.float64)
    macs = lib().gdws_oracle_dense_conv(N, C, H, W, M, K, stride, pad, _ptr(xn, _p_f64),
                                        _ptr(Wt, _p_f64), _ptr(b, _p_f64), _ptr(y, _p_f64))
    return _to_layout(y, layout), int(macs)


def wd_matrix(g, dw_w) -> np.ndarray:
    """W_D as the dense G x (C K^2) matrix of Property 2."""
    g = _i32(g)
    Kd = _f64(dw_w)
    G, K = Kd.shape[0], Kd.shape[-1]
    WD = np.zeros((G, g.size * K * K), dtype=np.float64)
    lib().gdws_oracle_wd_matrix(g.size, K, _ptr(g, _p_i32), _ptr(Kd, _p_f64), _ptr(WD, _p_f64))
    return WD


def reconstruct_dense(g, dw_w, pw_w) -> np.ndarray:
    """Weights [M][C][K][K] of the standard convolution equal to the GDWS layer."""
    g = _i32(g)
    Kd, P = _f64(dw_w), _f64(pw_w)
    G, K = Kd.shape[0], Kd.shape[-1]
    M = P.shape[0]
    Wt = np.zeros((M, g.size, K, K), dtype=np.float64)
    lib().gdws_oracle_reconstruct_dense(g.size, M, K, _ptr(g, _p_i32), _ptr(Kd, _p_f64),
                                        _ptr(P, _p_f64), _ptr(Wt, _p_f64))
    return Wt
