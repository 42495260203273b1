"""Pins for the CPU reference (oracle/): what the paper and the mathematics fix.

Nothing here touches the CUDA library.  Each test names the passage it rests on.
The pins are chosen so that a plausible mistake in the reference (a wrong channel
offset, a flipped or transposed filter, a dropped tap, padding or stride applied
wrongly, bias or intermediate order mixed up) fails at least one of them.
"""
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import gdws_oracle as orc
from paper_2110_14871_b200 import inputs as gi

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_layer(rng, N, C, D, H, W, k, g):
    g = np.asarray(g, dtype=np.int32)
    G = int(g.sum())
    x = rng.standard_normal((N, C, H, W))
    dw = rng.standard_normal((G, k, k))
    pw = rng.standard_normal((D, G))
    b = rng.standard_normal(D)
    return g, x, dw, pw, b


SHAPES = [
    # N, C, D, H, W, k, stride, pad
    (2, 5, 7, 9, 8, 3, 1, 1),
    (1, 4, 3, 11, 13, 3, 2, 1),
    (2, 3, 6, 10, 10, 5, 1, 2),
    (1, 6, 2, 7, 9, 2, 1, 0),
    (1, 3, 5, 8, 8, 1, 1, 0),
    (2, 4, 4, 9, 9, 3, 2, 0),
    (1, 2, 3, 12, 7, 5, 2, 2),
    (1, 3, 3, 6, 6, 3, 1, 2),
]


# ---------------------------------------------------------------- (a) Property 1 + 2
@pytest.mark.parametrize("shape", SHAPES)
def test_gdws_equals_dense_conv_with_reconstructed_weights(shape):
    """Property 1 (W = W_P W_D) with the block structure of Property 2: the GDWS
    layer equals the standard convolution with W[d,c] = sum_j P[d,off_c+j] K[off_c+j]."""
    N, C, D, H, W, k, s, p = shape
    rng = np.random.default_rng(hash(shape) % (2 ** 31))
    g = rng.integers(0, k * k + 1, size=C)          # ragged, zeros allowed
    if g.sum() == 0:
        g[0] = 1
    g, x, dw, pw, b = rand_layer(rng, N, C, D, H, W, k, g)
    y, _ = orc.forward(x, g, dw, pw, b, stride=s, pad=p)
    Wt = orc.reconstruct_dense(g, dw, pw)
    yd, _ = orc.dense_conv(x, Wt, b, stride=s, pad=p)
    assert y.shape == yd.shape == (N, D, gi.out_dim(H, k, s, p), gi.out_dim(W, k, s, p))
    assert np.max(np.abs(y - yd)) <= 1e-12 * max(1.0, np.max(np.abs(yd)))


@pytest.mark.parametrize("shape", SHAPES)
def test_dense_conv_matches_library_conv2d(shape):
    """Eq. 1: the direct-loop standard convolution agrees with a library routine
    (cross-correlation, zero padding, floor output size)."""
    N, C, D, H, W, k, s, p = shape
    rng = np.random.default_rng(7 + sum(shape))
    x = rng.standard_normal((N, C, H, W))
    w = rng.standard_normal((D, C, k, k))
    b = rng.standard_normal(D)
    y, _ = orc.dense_conv(x, w, b, stride=s, pad=p)
    yl = F.conv2d(torch.from_numpy(x), torch.from_numpy(w), torch.from_numpy(b), stride=s, padding=p).numpy()
    assert y.shape == yl.shape
    assert np.max(np.abs(y - yl)) <= 1e-11 * np.max(np.abs(yl))


def test_reconstructed_weights_equal_matrix_product():
    """Property 1 as matrices: reshape(W) == W_P @ W_D with W_D from Property 2."""
    rng = np.random.default_rng(3)
    C, D, k = 5, 6, 3
    g = np.array([2, 0, 9, 1, 4], dtype=np.int32)
    _, _, dw, pw, _ = rand_layer(rng, 1, C, D, 4, 4, k, g)
    WD = orc.wd_matrix(g, dw)
    assert WD.shape == (g.sum(), C * k * k)
    Wt = orc.reconstruct_dense(g, dw, pw).reshape(D, C * k * k)
    assert np.allclose(Wt, pw @ WD, rtol=0, atol=1e-12)
    # Property 2: sub-matrix c is non-zero only in rows off_c .. off_c+g_c-1
    off = orc.offsets(g)
    for c in range(C):
        blk = WD[:, c * k * k:(c + 1) * k * k]
        rows = np.nonzero(np.abs(blk).sum(axis=1))[0]
        assert set(rows.tolist()) <= set(range(int(off[c]), int(off[c + 1])))
        assert len(rows) == g[c]


def test_offsets_are_prefix_sums():
    g = np.array([3, 1, 0, 4, 2], dtype=np.int32)
    assert orc.offsets(g).tolist() == [0, 3, 4, 4, 8, 10]


# ---------------------------------------------------------------- (b) g = 1 is DWS
@pytest.mark.parametrize("shape", SHAPES[:5])
def test_all_ones_g_is_depthwise_separable(shape):
    """Section 3.1 "Relation to DWS": g_c = 1 for all c is the ordinary
    depthwise-separable convolution (library depthwise conv + 1x1 conv)."""
    N, C, D, H, W, k, s, p = shape
    rng = np.random.default_rng(11 + sum(shape))
    g, x, dw, pw, b = rand_layer(rng, N, C, D, H, W, k, np.ones(C))
    y, z, _ = orc.forward(x, g, dw, pw, b, stride=s, pad=p, return_z=True)
    xt = torch.from_numpy(x)
    zt = F.conv2d(xt, torch.from_numpy(dw).reshape(C, 1, k, k), None, stride=s, padding=p, groups=C)
    yt = F.conv2d(zt, torch.from_numpy(pw).reshape(D, C, 1, 1), torch.from_numpy(b))
    assert np.max(np.abs(z - zt.numpy())) <= 1e-12 * max(1.0, np.abs(zt.numpy()).max())
    assert np.max(np.abs(y - yt.numpy())) <= 1e-12 * max(1.0, np.abs(yt.numpy()).max())


def test_all_ones_g_loop_nest_tiny():
    """Same reduction, against a loop nest written out here (no library)."""
    rng = np.random.default_rng(5)
    N, C, D, H, W, k, s, p = 1, 2, 3, 5, 4, 3, 1, 1
    g, x, dw, pw, b = rand_layer(rng, N, C, D, H, W, k, np.ones(C))
    y, _ = orc.forward(x, g, dw, pw, b, stride=s, pad=p)
    xp = np.zeros((C, H + 2, W + 2))
    xp[:, 1:-1, 1:-1] = x[0]
    ref = np.zeros((D, H, W))
    for d, h, w in itertools.product(range(D), range(H), range(W)):
        acc = b[d]
        for c in range(C):
            dwv = sum(dw[c, u, v] * xp[c, h + u, w + v] for u in range(k) for v in range(k))
            acc += pw[d, c] * dwv
        ref[d, h, w] = acc
    assert np.allclose(y[0], ref, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- Appendix A.1 mapping
@pytest.mark.parametrize("shape", SHAPES)
def test_channel_duplication_identity(shape):
    """Appendix A.1: a (C,K,g) GDW convolution equals a depthwise convolution on
    the tensor X' obtained by repeating channel c g_c times (library routines:
    repeat_interleave + grouped conv2d), followed by a 1x1 convolution."""
    N, C, D, H, W, k, s, p = shape
    rng = np.random.default_rng(23 + sum(shape))
    g = rng.integers(1, min(k * k, 6) + 1, size=C)
    g, x, dw, pw, b = rand_layer(rng, N, C, D, H, W, k, g)
    G = int(g.sum())
    y, z, _ = orc.forward(x, g, dw, pw, b, stride=s, pad=p, return_z=True)
    xdup = torch.repeat_interleave(torch.from_numpy(x), torch.from_numpy(g.astype(np.int64)), dim=1)
    assert xdup.shape[1] == G
    zt = F.conv2d(xdup, torch.from_numpy(dw).reshape(G, 1, k, k), None, stride=s, padding=p, groups=G)
    yt = F.conv2d(zt, torch.from_numpy(pw).reshape(D, G, 1, 1), torch.from_numpy(b))
    assert np.max(np.abs(z - zt.numpy())) <= 1e-12 * max(1.0, np.abs(zt.numpy()).max())
    assert np.max(np.abs(y - yt.numpy())) <= 1e-11 * max(1.0, np.abs(yt.numpy()).max())
    # the staged entry points agree with the composed one
    z2, _ = orc.gdw(x, g, dw, stride=s, pad=p)
    y2, _ = orc.pw(z2, pw, b)
    assert np.array_equal(z2, z) and np.array_equal(y2, y)


# ---------------------------------------------------------------- Lemma 1: g = K^2
@pytest.mark.parametrize("k,s,p", [(3, 1, 1), (2, 1, 0), (3, 2, 1), (5, 1, 2)])
def test_full_rank_g_reproduces_any_dense_conv(k, s, p):
    """Lemma 1 / Section 3.2: with g_c = K^2 any standard convolution is a GDWS
    convolution.  Use K^2 delta filters per channel and P[d, off_c+t] = W[d,c,t]."""
    rng = np.random.default_rng(31 + k)
    N, C, D, H, W = 1, 3, 4, 8, 9
    Wd = rng.standard_normal((D, C, k, k))
    x = rng.standard_normal((N, C, H, W))
    b = rng.standard_normal(D)
    k2 = k * k
    g = np.full(C, k2, dtype=np.int32)
    dw = np.zeros((C * k2, k, k))
    pw = np.zeros((D, C * k2))
    for c in range(C):
        for t in range(k2):
            dw[c * k2 + t].reshape(-1)[t] = 1.0
            pw[:, c * k2 + t] = Wd[:, c].reshape(D, k2)[:, t]
    y, _ = orc.forward(x, g, dw, pw, b, stride=s, pad=p)
    yd, _ = orc.dense_conv(x, Wd, b, stride=s, pad=p)
    assert np.max(np.abs(y - yd)) <= 1e-13 * np.max(np.abs(yd))
    assert np.array_equal(orc.reconstruct_dense(g, dw, pw), Wd)


def test_rank_bound_of_submatrices():
    """Lemma 1: rank(W_c) <= min(g_c, K^2) for the reconstructed weights."""
    rng = np.random.default_rng(41)
    C, D, k = 6, 20, 3
    g = np.array([0, 1, 2, 5, 9, 12], dtype=np.int32)      # 12 > K^2: rank capped at 9
    _, _, dw, pw, _ = rand_layer(rng, 1, C, D, 4, 4, k, g)
    Wt = orc.reconstruct_dense(g, dw, pw)
    for c in range(C):
        Wc = Wt[:, c].reshape(D, k * k)
        sv = np.linalg.svd(Wc, compute_uv=False)
        rank = int((sv > 1e-10 * max(sv[0], 1e-300)).sum()) if sv[0] > 0 else 0
        assert rank == min(int(g[c]), k * k)


# ---------------------------------------------------------------- (c) complexity
@pytest.mark.parametrize("shape", SHAPES)
def test_mac_counts_match_complexity_expressions(shape):
    """Eq. 2 (H'W' M C K^2) and Eq. 3 (H'W' G (K^2 + M)); parameters G(K^2+M)."""
    N, C, D, H, W, k, s, p = shape
    rng = np.random.default_rng(51 + sum(shape))
    g = rng.integers(1, k * k + 1, size=C)
    g, x, dw, pw, b = rand_layer(rng, N, C, D, H, W, k, g)
    G = int(g.sum())
    Ho, Wo = gi.out_dim(H, k, s, p), gi.out_dim(W, k, s, p)
    _, macs = orc.forward(x, g, dw, pw, b, stride=s, pad=p)
    assert macs == N * Ho * Wo * G * (k * k + D) == N * orc.gdws_macs(Ho, Wo, G, k, D)
    _, dmacs = orc.dense_conv(x, orc.reconstruct_dense(g, dw, pw), b, stride=s, pad=p)
    assert dmacs == N * Ho * Wo * D * C * k * k == N * orc.dense_macs(Ho, Wo, C, k, D)
    _, m1 = orc.gdw(x, g, dw, stride=s, pad=p)
    assert m1 == N * Ho * Wo * G * k * k
    assert orc.gdws_params(G, k, D) == dw.size + pw.size


# ---------------------------------------------------------------- Appendix B.2 example
def _load_toy():
    sec, out = None, {}
    for line in open(os.path.join(GOLDEN, "toy_example_appendix_b2.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        if line.startswith("["):
            sec = line.strip("[]")
            out[sec] = []
            continue
        out[sec].append(line.split())
    return out


def test_toy_example_appendix_b2():
    """Appendix B.2: the printed W_PW and W_GDW multiply to the printed W, with
    g = [2,1,1]; per-pixel MACs 48 -> 32; sub-matrix ranks 2, 1, 1."""
    toy = _load_toy()
    prm = {r[0]: [int(v) for v in r[1:]] for r in toy["params"]}
    C, K, M = prm["C"][0], prm["K"][0], prm["M"][0]
    g = np.array(prm["g"], dtype=np.int32)
    vals = {"w1": 1.5, "w2": -2.25, "w3": 0.75, "w4": 3.0, "0": 0.0, "1": 1.0}
    mat = lambda rows: np.array([[vals[t] for t in r] for r in rows], dtype=np.float64)
    W, WPW, WGDW = mat(toy["W"]), mat(toy["W_PW"]), mat(toy["W_GDW"])
    assert W.shape == (M, C * K * K) and WPW.shape == (M, g.sum()) and WGDW.shape == (g.sum(), C * K * K)
    # rows of the printed W_GDW -> depthwise filters in the canonical order off_c + j
    off = orc.offsets(g)
    dw = np.zeros((int(g.sum()), K, K))
    for c in range(C):
        for j in range(g[c]):
            i = int(off[c]) + j
            dw[i] = WGDW[i, c * K * K:(c + 1) * K * K].reshape(K, K)
            # Property 2: the rest of row i is zero
            rest = np.delete(WGDW[i], np.s_[c * K * K:(c + 1) * K * K])
            assert not rest.any()
    assert np.array_equal(orc.wd_matrix(g, dw), WGDW)
    Wt = orc.reconstruct_dense(g, dw, WPW)
    assert np.array_equal(Wt.reshape(M, C * K * K), W)
    assert np.array_equal(WPW @ WGDW, W)
    for c, key in enumerate(("rank_W1", "rank_W2", "rank_W3")):
        assert np.linalg.matrix_rank(Wt[:, c].reshape(M, K * K)) == prm[key][0]
    assert orc.dense_macs(1, 1, C, K, M) == prm["dense_macs_per_pixel"][0]
    assert orc.gdws_macs(1, 1, int(g.sum()), K, M) == prm["gdws_macs_per_pixel"][0]
    assert int((WPW != 0).sum() + (WGDW != 0).sum()) == prm["nonzero_weights"][0]
    # and the forward pass agrees with the standard convolution of the printed W (even K)
    rng = np.random.default_rng(61)
    x = rng.standard_normal((2, C, 5, 6))
    y, macs = orc.forward(x, g, dw, WPW, None, stride=1, pad=0)
    yd, dmacs = orc.dense_conv(x, W.reshape(M, C, K, K), None, stride=1, pad=0)
    assert np.max(np.abs(y - yd)) <= 1e-14
    assert (dmacs, macs) == (2 * 4 * 5 * 48, 2 * 4 * 5 * 32)


# ---------------------------------------------------------------- (d) brute force, tiny
def test_ones_kernel_counts_neighbours():
    """1x1x3x3 input of ones, 3x3 all-ones filter, pad 1: each output counts the
    in-image neighbours (corners 4, edges 6, centre 9)."""
    x = np.ones((1, 1, 3, 3))
    y, _ = orc.forward(x, [1], np.ones((1, 3, 3)), np.ones((1, 1)), None, stride=1, pad=1)
    assert y[0, 0].tolist() == [[4, 6, 4], [6, 9, 6], [4, 6, 4]]


def test_delta_filter_identity_plus_bias():
    """Centre-delta filters and P = I give y = x + b."""
    rng = np.random.default_rng(71)
    C = 4
    x = rng.standard_normal((2, C, 5, 7))
    b = rng.standard_normal(C)
    dw = np.zeros((C, 3, 3))
    dw[:, 1, 1] = 1.0
    y, _ = orc.forward(x, np.ones(C), dw, np.eye(C), b, stride=1, pad=1)
    assert np.array_equal(y, x + b[None, :, None, None])


def test_single_tap_filters_shift_the_image():
    """A filter that is 1 at tap (u,v) reads x[h+u-p, w+v-p]: pins cross-correlation
    (no flip) and the (u,v) = (row, column) order, with zero fill outside."""
    x = np.arange(1.0, 1.0 + 4 * 5).reshape(1, 1, 4, 5)
    for u, v in itertools.product(range(3), range(3)):
        dw = np.zeros((1, 3, 3))
        dw[0, u, v] = 1.0
        y, _ = orc.forward(x, [1], dw, np.ones((1, 1)), None, stride=1, pad=1)
        ref = np.zeros((4, 5))
        for h, w in itertools.product(range(4), range(5)):
            hi, wi = h + u - 1, w + v - 1
            if 0 <= hi < 4 and 0 <= wi < 5:
                ref[h, w] = x[0, 0, hi, wi]
        assert np.array_equal(y[0, 0], ref), (u, v)


def test_stride_two_is_subsampled_stride_one():
    rng = np.random.default_rng(81)
    g, x, dw, pw, b = rand_layer(rng, 1, 3, 4, 9, 11, 3, [2, 1, 3])
    y1, _ = orc.forward(x, g, dw, pw, b, stride=1, pad=1)
    y2, _ = orc.forward(x, g, dw, pw, b, stride=2, pad=1)
    assert np.array_equal(y2, y1[:, :, ::2, ::2])


def test_hand_computed_two_filters_one_channel():
    """C=1, g=[2], K=2, pad 0, 2x3 input: every number written out by hand."""
    x = np.array([[[[1.0, 2.0, 3.0], [4.0, 5.0, 6.0]]]])
    dw = np.array([[[1.0, 0.0], [0.0, 1.0]],        # z0 = x[h,w] + x[h+1,w+1]
                   [[0.0, 2.0], [-1.0, 0.0]]])      # z1 = 2 x[h,w+1] - x[h+1,w]
    pw = np.array([[1.0, 1.0], [10.0, -1.0]])
    b = np.array([0.5, -0.5])
    y, z, _ = orc.forward(x, [2], dw, pw, b, stride=1, pad=0, return_z=True)
    assert z[0, :, 0, :].tolist() == [[6.0, 8.0], [0.0, 1.0]]
    assert y[0, :, 0, :].tolist() == [[6.5, 9.5], [59.5, 78.5]]


def test_channel_order_of_intermediate_maps():
    """Intermediate channel off_c + j reads input channel c: one-hot check."""
    C, k = 3, 1
    g = np.array([2, 1, 3], dtype=np.int32)
    x = np.zeros((1, C, 2, 2))
    for c in range(C):
        x[0, c] = 10.0 ** c
    dw = np.arange(1.0, 7.0).reshape(6, 1, 1)
    _, z, _ = orc.forward(x, g, dw, np.eye(6), None, stride=1, pad=0, return_z=True)
    assert z[0, :, 0, 0].tolist() == [1.0, 2.0, 30.0, 400.0, 500.0, 600.0]


def test_zero_multiplier_channel_contributes_nothing():
    rng = np.random.default_rng(91)
    g, x, dw, pw, b = rand_layer(rng, 1, 3, 2, 5, 5, 3, [2, 0, 1])
    y, _ = orc.forward(x, g, dw, pw, b, stride=1, pad=1)
    x2 = x.copy()
    x2[:, 1] = 123.0
    y2, _ = orc.forward(x2, g, dw, pw, b, stride=1, pad=1)
    assert np.array_equal(y, y2)


def test_linearity():
    rng = np.random.default_rng(101)
    g, x1, dw, pw, b = rand_layer(rng, 1, 3, 4, 6, 6, 3, [1, 3, 2])
    x2 = rng.standard_normal(x1.shape)
    a, c = 0.7, -1.3
    f = lambda x: orc.forward(x, g, dw, pw, b, stride=1, pad=1)[0]
    lhs = f(a * x1 + c * x2)
    rhs = a * f(x1) + c * f(x2) - (a + c - 1.0) * b[None, :, None, None]
    assert np.max(np.abs(lhs - rhs)) <= 1e-12


def test_relu_and_layouts():
    rng = np.random.default_rng(111)
    g, x, dw, pw, b = rand_layer(rng, 2, 3, 4, 6, 5, 3, [1, 3, 2])
    y, _ = orc.forward(x, g, dw, pw, b, stride=1, pad=1)
    yr, _ = orc.forward(x, g, dw, pw, b, stride=1, pad=1, relu=True)
    assert np.array_equal(yr, np.maximum(y, 0.0))
    xh = np.ascontiguousarray(x.transpose(0, 2, 3, 1))
    yh, zh, _ = orc.forward(xh, g, dw, pw, b, stride=1, pad=1, layout="NHWC", return_z=True)
    assert np.array_equal(yh, y.transpose(0, 2, 3, 1))
    assert zh.shape == (2, 6, 5, int(g.sum()))


# ---------------------------------------------------------------- input recipe
def test_bf16_rounding_is_nearest_even():
    a = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9, -2.5, 3.1415927], dtype=np.float32)
    r = gi.round_to_bf16(a)
    t = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(r, t)
    assert r[1] == 1.0 and r[2] == np.float32(1.0 + 2 ** -6)     # ties go to even


def test_config_recipes():
    l0 = gi.config_layers(0)[0]
    d = gi.make_layer(l0)
    assert d.g.min() >= 1 and d.g.max() <= 3 and d.x.shape == (1, 16, 32, 32) and d.x.dtype == np.float32
    d2 = gi.make_layer(l0)
    assert np.array_equal(d.x, d2.x) and np.array_equal(d.g, d2.g)
    l1 = gi.config_layers(1)[0]
    d = gi.make_layer(l1, N=2)
    assert d.x.shape == (2, 8, 8, 256) and d.g.max() <= 9 and d.pw_w.shape == (256, d.G)
    assert np.array_equal(gi.round_to_bf16(d.x), d.x)
    chain = gi.config_layers(3)
    assert len(chain) == 16 and [l.stride for l in chain].count(2) == 3
    assert [(l.C, l.D, l.H) for l in chain][4] == (64, 128, 32) and chain[-1].Ho == 4
    for a, b in zip(chain[:-1], chain[1:]):
        assert (a.D, a.Ho) == (b.C, b.H)
    v = gi.config_layers(4)
    assert len(v) == 13 and v[-1].k == 5 and v[-1].pad == 2
    heavy = gi.make_g(np.random.default_rng(0), 20000, ("heavy",))
    assert abs((heavy == 1).mean() - 0.5) < 0.02 and abs((heavy == 2).mean() - 0.2) < 0.02
    assert heavy.max() == 9 and abs(heavy.mean() - 2.7) < 0.1
