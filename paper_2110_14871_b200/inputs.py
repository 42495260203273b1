"""Seeded synthetic inputs for GDWS layers (shapes of the paper's CIFAR / SVHN /
ImageNet networks; Section 4.1 names VGG-16, ResNet-18 and ResNet-50).

This module holds no GDWS arithmetic: it draws the channel distribution vector g,
the activations and the weights, rounds them to the storage type, and describes
the layer shapes.  Both the CPU reference used by the tests and the CUDA library
are fed from here, so that they see bit-identical inputs.

Recipe: ``numpy.random.Generator(PCG64(seed))`` with ``seed = 1000*config + layer``;
draw order g, x, dw_w, pw_w, bias; normals are drawn in float64, cast to float32
and, for bf16 layers, rounded once to bfloat16 (round to nearest even).  The
rounded values are what every consumer receives.
    x ~ N(0, 1),  dw_w ~ N(0, 1/k^2),  pw_w ~ N(0, 1/G),  bias ~ N(0, 0.01)   (variances)
g is either uniform on [lo, hi] or heavy-tailed: P(1)=0.5, P(2)=0.2, otherwise
uniform on {3..9}.  The paper restricts g_c to at most K^2 (Section 3.2, after
Lemma 1); all recipes respect that.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Tuple

import numpy as np

__all__ = [
    "LayerSpec", "LayerData", "config_layers", "make_layer", "make_g",
    "f32_to_bf16_bits", "bf16_bits_to_f32", "round_to_bf16", "out_dim",
    "to_layout", "from_layout", "CONFIG_NAMES",
]


@dataclasses.dataclass(frozen=True)
class LayerSpec:
    """Shape of one GDWS layer.  D is the paper's M (output channels)."""
    name: str
    N: int
    C: int
    D: int
    H: int
    W: int
    k: int = 3
    stride: int = 1
    pad: int = 1
    g_dist: Tuple = ("uniform", 1, 9)      # ("uniform", lo, hi) | ("heavy",)
    dtype: str = "bf16"                    # "f32" | "bf16"
    layout: str = "NHWC"                   # "NCHW" | "NHWC"
    relu: bool = False                     # ReLU after the bias (chained layers only)
    seed: int = 0

    @property
    def Ho(self) -> int:
        return out_dim(self.H, self.k, self.stride, self.pad)

    @property
    def Wo(self) -> int:
        return out_dim(self.W, self.k, self.stride, self.pad)


@dataclasses.dataclass
class LayerData:
    """Arrays of one layer.  For bf16 layers ``x``, ``dw_w`` and ``pw_w`` are
    float32 arrays that hold bf16-representable values; ``*_bits`` give the raw
    16-bit patterns.  ``x`` is in ``spec.layout`` order; weights are canonical:
    dw_w[G][k][k] with intermediate channel i = off_c + j, pw_w[D][G]."""
    spec: LayerSpec
    g: np.ndarray            # int32 [C]
    x: np.ndarray            # float32, layout order
    dw_w: np.ndarray         # float32 [G,k,k]
    pw_w: np.ndarray         # float32 [D,G]
    bias: np.ndarray         # float32 [D]

    @property
    def G(self) -> int:
        return int(self.g.sum())


def out_dim(size: int, k: int, stride: int, pad: int) -> int:
    span = size + 2 * pad - k
    return span // stride + 1 if span >= 0 else 0


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array whose values are exactly representable in bfloat16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(a)).reshape(np.shape(a))


def to_layout(a_nchw: np.ndarray, layout: str) -> np.ndarray:
    if layout == "NCHW":
        return np.ascontiguousarray(a_nchw)
    if layout == "NHWC":
        return np.ascontiguousarray(np.transpose(a_nchw, (0, 2, 3, 1)))
    raise ValueError(layout)


def from_layout(a: np.ndarray, layout: str) -> np.ndarray:
    """Inverse of :func:`to_layout`: returns an NCHW-ordered contiguous array."""
    if layout == "NCHW":
        return np.ascontiguousarray(a)
    if layout == "NHWC":
        return np.ascontiguousarray(np.transpose(a, (0, 3, 1, 2)))
    raise ValueError(layout)


def make_g(rng: np.random.Generator, C: int, g_dist: Tuple) -> np.ndarray:
    kind = g_dist[0]
    if kind == "uniform":
        lo, hi = int(g_dist[1]), int(g_dist[2])
        return rng.integers(lo, hi + 1, size=C).astype(np.int32)
    if kind == "heavy":
        u = rng.random(C)
        tail = rng.integers(3, 10, size=C)
        g = np.where(u < 0.5, 1, np.where(u < 0.7, 2, tail))
        return g.astype(np.int32)
    if kind == "const":
        return np.full(C, int(g_dist[1]), dtype=np.int32)
    raise ValueError(g_dist)


def make_layer(spec: LayerSpec, N: Optional[int] = None, with_x: bool = True) -> LayerData:
    """Draw g, x, dw_w, pw_w, bias for ``spec``.  ``N`` overrides the batch size
    (the first N images of the full batch are NOT reproduced; a different N gives
    a different but equally distributed batch).  ``with_x=False`` skips the
    activation draw (weights then differ from the with_x=True draw)."""
    n = spec.N if N is None else int(N)
    rng = np.random.Generator(np.random.PCG64(spec.seed))
    g = make_g(rng, spec.C, spec.g_dist)
    G = int(g.sum())
    if with_x:
        x = rng.standard_normal((n, spec.C, spec.H, spec.W)).astype(np.float32)
    else:
        x = np.zeros((0, spec.C, spec.H, spec.W), dtype=np.float32)
    dw_w = (rng.standard_normal((G, spec.k, spec.k)) / spec.k).astype(np.float32)
    pw_w = (rng.standard_normal((spec.D, G)) / np.sqrt(max(G, 1))).astype(np.float32)
    bias = (rng.standard_normal(spec.D) * 0.1).astype(np.float32)
    if spec.dtype == "bf16":
        x, dw_w, pw_w = round_to_bf16(x), round_to_bf16(dw_w), round_to_bf16(pw_w)
    x = to_layout(x, spec.layout)
    return LayerData(dataclasses.replace(spec, N=n), g, x, dw_w, pw_w, bias)


CONFIG_NAMES = {
    0: "fp32 single layer (N=1, C=D=16, 32x32, NCHW)",
    1: "CIFAR VGG-16 middle layer (N=256, C=D=256, 8x8, g~U[1,9], bf16 NHWC)",
    2: "ImageNet ResNet-50 3x3 layers (N=64, bf16 NHWC, heavy-tailed g)",
    3: "CIFAR ResNet-18 3x3 stack, 16 chained layers (N=512, bf16 NHWC)",
    4: "ImageNet VGG-16 3x3 layers (N=32, bf16 NHWC, heavy-tailed g) + k=5 variant",
}


def config_layers(config: int) -> List[LayerSpec]:
    """Layer list of one benchmark configuration (shapes only)."""
    def seed(layer: int) -> int:
        return 1000 * config + layer

    if config == 0:
        return [LayerSpec("c0", 1, 16, 16, 32, 32, 3, 1, 1, ("uniform", 1, 3), "f32", "NCHW", False, seed(0))]
    if config == 1:
        return [LayerSpec("c1", 256, 256, 256, 8, 8, 3, 1, 1, ("uniform", 1, 9), "bf16", "NHWC", False, seed(0))]
    if config == 2:
        return [
            LayerSpec("c2a", 64, 64, 64, 56, 56, 3, 1, 1, ("heavy",), "bf16", "NHWC", False, seed(0)),
            LayerSpec("c2b", 64, 128, 128, 56, 56, 3, 2, 1, ("heavy",), "bf16", "NHWC", False, seed(1)),
            LayerSpec("c2c", 64, 256, 256, 14, 14, 3, 1, 1, ("heavy",), "bf16", "NHWC", False, seed(2)),
        ]
    if config == 3:
        out: List[LayerSpec] = []
        res, cin = 32, 64
        layer = 0
        for stage, width in enumerate((64, 128, 256, 512)):
            for blk in range(4):
                stride = 2 if (stage > 0 and blk == 0) else 1
                out.append(LayerSpec(f"c3L{layer}", 512, cin, width, res, res, 3, stride, 1,
                                     ("uniform", 1, 9), "bf16", "NHWC", layer < 15, seed(layer)))
                res = out_dim(res, 3, stride, 1)
                cin = width
                layer += 1
        return out
    if config == 4:
        shapes = [(64, 64, 224), (64, 128, 112), (128, 128, 112), (128, 256, 56), (256, 256, 56),
                  (256, 256, 56), (256, 512, 28), (512, 512, 28), (512, 512, 28), (512, 512, 14),
                  (512, 512, 14), (512, 512, 14)]
        out = [LayerSpec(f"c4V{i}", 32, c, d, r, r, 3, 1, 1, ("heavy",), "bf16", "NHWC", False, seed(i))
               for i, (c, d, r) in enumerate(shapes)]
        out.append(LayerSpec("c4k5", 32, 256, 256, 56, 56, 5, 1, 2, ("uniform", 1, 25), "bf16", "NHWC",
                             False, seed(len(shapes))))
        return out
    raise ValueError(f"unknown config {config}")
