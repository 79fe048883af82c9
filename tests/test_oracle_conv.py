"""Pins for the direct-convolution, max-pool and AlexNet-chain oracles."""
import os

import numpy as np
import torch

from oracle import oracle as orc
from oracle import alexnet as onet
from paper_1709_04060_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _torch_conv(In, Wt, stride, pad):
    x = torch.from_numpy(In.astype(np.float64)).permute(0, 3, 1, 2)
    w = torch.from_numpy(Wt.astype(np.float64)).permute(0, 3, 1, 2)
    y = torch.nn.functional.conv2d(x, w, stride=stride, padding=pad)
    return y.permute(0, 2, 3, 1).numpy().round().astype(np.int64)


def test_conv_against_library_routine():
    rng = np.random.default_rng(0)
    for (B, H, Wd, C, OC, KH, KW, s, p) in [
        (1, 5, 5, 3, 2, 3, 3, 1, 1), (2, 9, 7, 5, 4, 3, 3, 2, 0),
        (1, 13, 13, 8, 6, 5, 5, 1, 2), (1, 23, 23, 3, 4, 11, 11, 4, 0),
        (2, 6, 6, 33, 3, 1, 1, 1, 0),
    ]:
        In = rng.integers(0, 4, size=(B, H, Wd, C), dtype=np.int32)
        Wt = rng.integers(-2, 2, size=(OC, KH, KW, C), dtype=np.int32)
        assert np.array_equal(orc.conv_direct(In, Wt, s, p), _torch_conv(In, Wt, s, p))


def test_conv_1x1_is_plain_gemm():
    rng = np.random.default_rng(1)
    In = rng.integers(0, 4, size=(2, 4, 3, 10), dtype=np.int32)
    Wt = rng.integers(-1, 2, size=(7, 1, 1, 10), dtype=np.int32)
    acc = orc.conv_direct(In, Wt, 1, 0)
    want = orc.gemm(Wt.reshape(7, 10), In.reshape(-1, 10)).T.reshape(2, 4, 3, 7)
    assert np.array_equal(acc, want)


def test_conv_all_ones_counts_in_image_taps():
    C = 4
    In = np.ones((1, 5, 5, C), dtype=np.int32)
    Wt = np.ones((1, 3, 3, C), dtype=np.int32)
    acc = orc.conv_direct(In, Wt, 1, 1)[0, :, :, 0]
    taps = np.array([[4, 6, 6, 6, 4], [6, 9, 9, 9, 6], [6, 9, 9, 9, 6],
                     [6, 9, 9, 9, 6], [4, 6, 6, 6, 4]])
    assert np.array_equal(acc, taps * C)
    acc2 = orc.conv_direct(In, Wt, 2, 0)
    assert acc2.shape == (1, 2, 2, 1) and np.all(acc2 == 9 * C)


def _host_im2col(In, KH, KW, stride, pad):
    """Independent host lowering used only here: column order (kh, kw, c), c fastest."""
    B, H, Wd, C = In.shape
    OH = (H + 2 * pad - KH) // stride + 1
    OW = (Wd + 2 * pad - KW) // stride + 1
    padded = np.zeros((B, H + 2 * pad, Wd + 2 * pad, C), dtype=In.dtype)
    padded[:, pad:pad + H, pad:pad + Wd, :] = In
    cols = np.empty((B, OH, OW, KH, KW, C), dtype=In.dtype)
    for oh in range(OH):
        for ow in range(OW):
            cols[:, oh, ow] = padded[:, oh * stride:oh * stride + KH, ow * stride:ow * stride + KW, :]
    return cols.reshape(B * OH * OW, KH * KW * C)


def test_lowered_gemm_equals_direct_conv():
    case = synth.conv_case(11, 2, 9, 9, 40, 6, 3, 3, 2, 1, 1, 2)
    direct = orc.conv_direct(case.In, case.Wt, case.stride, case.pad)
    low = _host_im2col(case.In, 3, 3, 2, 1)
    via_gemm = orc.gemm(case.Wt.reshape(6, -1), low).T.reshape(direct.shape)
    assert np.array_equal(direct, via_gemm)


def test_maxpool_brute_force_and_commutes_with_threshold():
    rng = np.random.default_rng(2)
    x = rng.integers(-50, 50, size=(2, 7, 7, 3), dtype=np.int32)
    out = orc.maxpool(x, 3, 2)
    assert out.shape == (2, 3, 3, 3)
    for b in range(2):
        for i in range(3):
            for j in range(3):
                for c in range(3):
                    assert out[b, i, j, c] == x[b, 2 * i:2 * i + 3, 2 * j:2 * j + 3, c].max()
    # T is monotone, so pooling codes equals thresholding pooled accumulators
    thr = np.sort(rng.integers(-40, 40, size=(3, 3)), axis=1).astype(np.int32)
    a = orc.maxpool(orc.threshold_nhwc(x.astype(np.int64), thr), 3, 2)
    b = orc.threshold_nhwc(orc.maxpool(x, 3, 2).astype(np.int64), thr)
    assert np.array_equal(a, b)
    assert orc.maxpool(np.zeros((1, 55, 55, 1), np.int32), 3, 2).shape == (1, 27, 27, 1)
    assert orc.maxpool(np.zeros((1, 13, 13, 1), np.int32), 3, 2).shape == (1, 6, 6, 1)


def test_alexnet_chain_shapes_match_table3():
    want = {}
    with open(os.path.join(GOLDEN, "alexnet_shapes.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                n, r, d, c = line.split()
                want[n] = (int(r), int(d), int(c))
    net = synth.alexnet_case(1)
    H, C, flat = 227, 3, None
    for L in net.layers:
        Wt = net.weights[L.name]
        if L.kind == "conv":
            OH = (H + 2 * L.pad - L.KH) // L.stride + 1
            assert (L.OC, L.KH * L.KW * C, OH * OH) == want[L.name]
            assert Wt.shape == (L.OC, L.KH, L.KW, C)
            H = (OH - 3) // 2 + 1 if L.pool else OH
            C = L.OC
            flat = H * H * C
        else:
            assert (L.OC, flat, 1) == want[L.name]
            assert Wt.shape == (L.OC, flat)
            flat = L.OC


def test_alexnet_chain_small_runs_and_localises():
    """Chain on one image: per-layer shapes, code ranges, and an independent
    recomputation of two layers from their inputs via the lowered form."""
    net = synth.alexnet_case(1)
    logits, inter = onet.forward(net)
    assert logits.shape == (1, 1000)
    assert inter["conv1"].shape == (1, 27, 27, 96)
    assert inter["conv2"].shape == (1, 13, 13, 256)
    assert inter["conv5"].shape == (1, 6, 6, 256)
    for name in ("conv1", "conv2", "conv3", "conv4", "conv5", "fc6", "fc7"):
        v = inter[name]
        assert v.min() >= 0 and v.max() <= 3
        assert len(np.unique(v)) >= 3, name          # thresholds keep codes populated
    # conv3 from conv2's output through host lowering + numpy matmul
    x = inter["conv2"]
    low = _host_im2col(x, 3, 3, 1, 1).astype(np.int64)
    W3 = net.weights["conv3"].reshape(384, -1).astype(np.int64)
    acc = low @ W3.T
    codes = (acc[:, :, None] >= net.thr["conv3"][None, :, :]).sum(-1)
    assert np.array_equal(codes.reshape(1, 13, 13, 384), inter["conv3"])
    # fc8 logits from fc7 codes
    want = inter["fc7"].astype(np.int64) @ net.weights["fc8"].astype(np.int64).T
    assert np.array_equal(want, logits)
