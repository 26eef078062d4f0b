"""Pins for threshold, convolution, the chained MLP (Algorithm 4) and the affine rescale."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_1609_07061_b200 import workloads


def _read(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_threshold_brute_force():
    rng = np.random.default_rng(0)
    s = rng.integers(-100, 100, (13, 37)).astype(np.int32)
    T = rng.integers(-64, 65, 37).astype(np.int32)
    flip = rng.integers(0, 2, 37).astype(np.uint8)
    got = oracle.threshold(s, T, flip)
    for m in range(13):
        for n in range(37):
            want = (1 if s[m, n] >= T[n] else 0) ^ int(flip[n])
            assert got[m, n] == want
    np.testing.assert_array_equal(oracle.threshold(s, T), (s >= T[None, :]).astype(np.uint8))
    # equality counts as +1 (Eq. 1: x >= 0)
    assert oracle.threshold(np.array([[5]], np.int32), np.array([5], np.int32))[0, 0] == 1


def test_conv_golden(golden_dir):
    rows = _read(golden_dir, "conv_border.txt")
    x = np.array([int(v) for v in rows[0][1:]], np.int32).reshape(1, 1, 2, 2)
    w = np.array([int(v) for v in rows[1][1:]], np.int32).reshape(1, 1, 3, 3)
    y = np.array([int(v) for v in rows[2][1:]], np.int32).reshape(1, 1, 2, 2)
    np.testing.assert_array_equal(oracle.conv2d(x, w, 1, 1, 1), y)


@pytest.mark.parametrize("B,C,H,W,Co,KH,KW,stride,pad", [
    (2, 3, 5, 6, 4, 3, 3, 1, 1), (1, 33, 4, 4, 5, 3, 3, 1, 1), (2, 2, 7, 5, 3, 1, 1, 1, 0),
    (1, 4, 8, 8, 2, 3, 3, 2, 1), (1, 2, 6, 6, 2, 5, 3, 1, 2)])
def test_conv_vs_library(B, C, H, W, Co, KH, KW, stride, pad):
    """torch conv2d (cross-correlation) in float64 on +-1 tensors padded with +1."""
    rng = np.random.default_rng(B + C + H)
    x = np.where(rng.standard_normal((B, C, H, W)) >= 0, 1, -1).astype(np.int32)
    w = np.where(rng.standard_normal((Co, C, KH, KW)) >= 0, 1, -1).astype(np.int32)
    xp = F.pad(torch.from_numpy(x).double(), (pad, pad, pad, pad), value=1.0)
    want = F.conv2d(xp, torch.from_numpy(w).double(), stride=stride).numpy()
    np.testing.assert_array_equal(oracle.conv2d(x, w, stride, pad, 1), want.astype(np.int32))


def test_conv_1x1_is_matrix_product_and_ones_input():
    rng = np.random.default_rng(3)
    x = np.where(rng.standard_normal((2, 8, 3, 3)) >= 0, 1, -1).astype(np.int32)
    w = np.where(rng.standard_normal((5, 8, 1, 1)) >= 0, 1, -1).astype(np.int32)
    y = oracle.conv2d(x, w, 1, 0, 1)
    rows = x.transpose(0, 2, 3, 1).reshape(-1, 8)
    want = oracle.int_gemm(rows, w.reshape(5, 8).T).reshape(2, 3, 3, 5).transpose(0, 3, 1, 2)
    np.testing.assert_array_equal(y, want)
    # an all +1 image with a +1 border sees sum(w) at every pixel, borders included
    w3 = np.where(rng.standard_normal((4, 8, 3, 3)) >= 0, 1, -1).astype(np.int32)
    ones = np.ones((1, 8, 4, 4), np.int32)
    y1 = oracle.conv2d(ones, w3, 1, 1, 1)
    for co in range(4):
        assert np.all(y1[0, co] == w3[co].sum())


def test_mlp_forward_step_by_step():
    """Algorithm 4 re-assembled from float64 matmuls and numpy comparisons."""
    wl = workloads.mnist_mlp(M=12, dims=(50, 40, 24, 10), seed=1)
    x = wl.X.numpy().astype(np.int32)
    Ws = [oracle.sign(w.numpy()) for w in wl.Ws]
    Ts = [t.numpy() for t in wl.Ts]
    got = oracle.mlp_forward(x, Ws, Ts)
    a = x.astype(np.float64)
    for l, W in enumerate(Ws):
        s = a @ W.astype(np.float64)
        if l < len(Ws) - 1:
            a = np.where(s >= Ts[l][None, :].astype(np.float64), 1.0, -1.0)
    np.testing.assert_array_equal(got, s.astype(np.int32))
    # a single flipped input pixel bit must be able to change the scores (chain is live)
    x2 = x.copy()
    x2[:, 0] = 255 - x2[:, 0]
    assert not np.array_equal(oracle.mlp_forward(x2, Ws, Ts), got)


def test_mlp_first_layer_is_eq8():
    wl = workloads.mnist_mlp(M=5, dims=(33, 16, 4), seed=1)
    x = wl.X.numpy().astype(np.int32)
    W1 = oracle.sign(wl.Ws[0].numpy())
    np.testing.assert_array_equal(oracle.int_gemm(x, W1), oracle.planewise_gemm(x, 8, W1))


def test_mlp_flip():
    wl = workloads.mnist_mlp(M=6, dims=(20, 16, 5), seed=1)
    x = wl.X.numpy().astype(np.int32)
    Ws = [oracle.sign(w.numpy()) for w in wl.Ws]
    T = wl.Ts[0].numpy()
    flip = (np.arange(16) % 2).astype(np.uint8)
    got = oracle.mlp_forward(x, Ws, [T], [flip])
    s = oracle.int_gemm(x, Ws[0])
    bits = (s >= T[None, :]) ^ (flip[None, :] != 0)
    want = oracle.int_gemm(np.where(bits, 1, -1).astype(np.int32), Ws[1])
    np.testing.assert_array_equal(got, want)


@pytest.mark.parametrize("B,C,H,W", [(2, 3, 4, 6), (1, 5, 7, 5), (3, 1, 2, 2), (1, 2, 3, 4)])
def test_maxpool_vs_library(B, C, H, W):
    rng = np.random.default_rng(H * 10 + W)
    x = rng.integers(-500, 500, (B, C, H, W)).astype(np.int32)
    want = F.max_pool2d(torch.from_numpy(x).double(), 2).numpy().astype(np.int32)
    got = oracle.maxpool2x2(x)
    assert got.shape == (B, C, H // 2, W // 2)
    np.testing.assert_array_equal(got, want)
    assert oracle.maxpool2x2(x[:, :, :1, :]).shape == (B, C, 0, W // 2)      # a single row has no window


def test_threshold_of_pooled_sums_is_or_and_of_bits():
    """Thresholding is monotone in the sum, so the bit of a window's maximum is the OR of the four
    pixels' bits, and the AND where the channel's comparison is flipped (every window checked)."""
    rng = np.random.default_rng(11)
    B, C, H, W = 2, 6, 6, 8
    s = rng.integers(-20, 20, (B, C, H, W)).astype(np.int32)
    T = rng.integers(-10, 10, C).astype(np.int32)
    flip = np.array([0, 1, 0, 1, 1, 0], np.uint8)
    rows = lambda t: t.transpose(0, 2, 3, 1).reshape(-1, C)
    pooled_bits = oracle.threshold(rows(oracle.maxpool2x2(s)), T, flip).reshape(B, H // 2, W // 2, C)
    bits = oracle.threshold(rows(s), T, flip).reshape(B, H, W, C)
    for b in range(B):
        for y in range(H // 2):
            for x in range(W // 2):
                win = bits[b, 2 * y:2 * y + 2, 2 * x:2 * x + 2, :].reshape(4, C)
                for c in range(C):
                    want = win[:, c].min() if flip[c] else win[:, c].max()
                    assert pooled_bits[b, y, x, c] == want


def test_first_layer_conv_on_pixel_codes_vs_library():
    """8-bit codes times +-1 weights with a zero border (Table 7's first layer; Eq. 8 summed over planes)."""
    rng = np.random.default_rng(5)
    x = rng.integers(0, 256, (2, 3, 6, 5)).astype(np.int32)
    w = np.where(rng.standard_normal((4, 3, 3, 3)) >= 0, 1, -1).astype(np.int32)
    want = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), padding=1).numpy()
    got = oracle.conv2d(x, w, 1, 1, 0)
    np.testing.assert_array_equal(got, want.astype(np.int32))
    # plane by plane (Eq. 8): the same sums from the eight bit planes of the codes
    acc = np.zeros_like(got)
    for i in range(8):
        acc += (1 << i) * oracle.conv2d(oracle.bit_plane(x, i).astype(np.int32), w, 1, 1, 0)
    np.testing.assert_array_equal(acc, got)


def _convnet_layers(wl):
    layers, t = [], 0
    for i, (Wc, pool) in enumerate(zip(wl.conv_W, wl.conv_pool)):
        layers.append(dict(kind="conv", W=oracle.sign(Wc.numpy()), pad=1, pad_value=0 if i == 0 else 1, pool=pool,
                           T=wl.Ts[t].numpy(), flip=wl.flips[t].numpy()))
        t += 1
    for j, Wf in enumerate(wl.fc_W):
        last = j == len(wl.fc_W) - 1
        layers.append(dict(kind="fc", W=oracle.sign(Wf.numpy()), T=None if last else wl.Ts[t].numpy(),
                           flip=None if last else wl.flips[t].numpy()))
        t += 0 if last else 1
    return layers


def test_convnet_forward_vs_library_chain():
    """Table 7 layer by layer with float64 library calls: conv2d on a padded tensor, max_pool2d, comparisons."""
    wl = workloads.cifar_convnet(B=3, H=8, W=8, widths=(8, 8, 16, 16), fc=(24, 10), seed=5, thr=3)
    layers = _convnet_layers(wl)
    got = oracle.convnet_forward(wl.X.numpy().astype(np.int32), layers)
    a = wl.X.double()
    for ly in layers:
        if ly["kind"] == "conv":
            ap = F.pad(a, (1, 1, 1, 1), value=float(ly["pad_value"]))
            s = F.conv2d(ap, torch.from_numpy(ly["W"]).double())
            if ly["pool"]:
                s = F.max_pool2d(s, 2)
            ge = s >= torch.from_numpy(ly["T"]).double()[None, :, None, None]
            bit = ge ^ (torch.from_numpy(ly["flip"]) != 0)[None, :, None, None]
            a = torch.where(bit, 1.0, -1.0).double()
        else:
            if a.dim() == 4:
                a = a.permute(0, 2, 3, 1).reshape(a.shape[0], -1)
            s = a @ torch.from_numpy(ly["W"]).double()
            if ly["T"] is not None:
                bit = (s >= torch.from_numpy(ly["T"]).double()[None, :]) ^ (torch.from_numpy(ly["flip"]) != 0)[None, :]
                a = torch.where(bit, 1.0, -1.0).double()
    assert got.shape == (3, 10)
    np.testing.assert_array_equal(got, s.numpy().astype(np.int32))
    # the chain is live: other images give other scores
    x2 = 255 - wl.X.numpy().astype(np.int32)
    assert not np.array_equal(oracle.convnet_forward(x2, layers), got)
    # both kinds of channel occur, so both the OR and the AND side of pooling are exercised
    assert any(f.any() for f in wl.flips) and any((f == 0).any() for f in wl.flips)


def test_rescale():
    rng = np.random.default_rng(1)
    p = rng.integers(-1000, 1000, (4, 6)).astype(np.int32)
    r = rng.standard_normal(4)
    c = rng.standard_normal(6)
    y = oracle.rescale(p, 0.125, r, c, -2.0)
    np.testing.assert_allclose(y, 0.125 * p + r[:, None] + c[None, :] - 2.0, rtol=0, atol=1e-12)
