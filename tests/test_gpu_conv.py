"""GPU parity: interleaved lowering, convolution by lowering, max-pool and the
AlexNet-shaped chain through the C ABI vs the CPU oracle (bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from oracle import alexnet as onet
from paper_1709_04060_b200 import synth
from qnn_testutil import unpack_planes, unpack_int8, decode_out, round_up

pytestmark = pytest.mark.gpu

BITPLANES, INT8 = 0, 1


@pytest.fixture(scope="module")
def qb():
    from paper_1709_04060_b200 import binding
    return binding


def host_im2col(In, KH, KW, stride, pad, c_pad, run_pad=False):
    """Test-side lowering: rows (b, oh, ow), columns (kh, kw, c) with each pixel padded to c_pad;
    run_pad: every filter row's KW*c_pad values are zero padded to a multiple of 16."""
    B, H, Wd, C = In.shape
    OH = (H + 2 * pad - KH) // stride + 1
    OW = (Wd + 2 * pad - KW) // stride + 1
    padded = np.zeros((B, H + 2 * pad, Wd + 2 * pad, c_pad), dtype=In.dtype)
    padded[:, pad:pad + H, pad:pad + Wd, :C] = In
    cols = np.empty((B, OH, OW, KH, KW, c_pad), dtype=In.dtype)
    for oh in range(OH):
        for ow in range(OW):
            cols[:, oh, ow] = padded[:, oh * stride:oh * stride + KH, ow * stride:ow * stride + KW, :]
    if run_pad:
        runs = np.zeros((B * OH * OW, KH, round_up(KW * c_pad, 16)), dtype=In.dtype)
        runs[:, :, :KW * c_pad] = cols.reshape(B * OH * OW, KH, KW * c_pad)
        return runs.reshape(B * OH * OW, -1)
    return cols.reshape(B * OH * OW, KH * KW * c_pad)


def device_map(qb, case, fmt, in_pitch=None):
    """Feature map on the device in the library's layout; returns (tensor, pitch)."""
    B, H, Wd, C = case.In.shape
    if fmt == BITPLANES:
        flat = qb.to_device_logical(case.In.reshape(B * H * Wd, C), case.a_enc)
        return qb.pack(flat, case.a_bits, case.a_enc, BITPLANES), 0
    pitch = in_pitch if in_pitch is not None else round_up(C, 16)
    m = np.zeros((B, H, Wd, pitch), dtype=np.uint8)
    m[..., :C] = case.In.astype(np.uint8)
    return torch.from_numpy(m).cuda(), pitch


def device_weights(qb, case, fmt):
    OC, KH, KW, C = case.Wt.shape
    if fmt == BITPLANES:
        cp = round_up(C, 32)
        Wp = np.zeros((OC, KH * KW, cp), dtype=np.int32)
        Wp[:, :, :C] = case.Wt.reshape(OC, KH * KW, C)
        flat = Wp.reshape(OC, -1)
    elif C % 16 == 0:
        flat = case.Wt.reshape(OC, -1)
    else:                       # one zero-padded run per filter row
        runs = np.zeros((OC, KH, round_up(KW * C, 16)), dtype=np.int32)
        runs[:, :, :KW * C] = case.Wt.reshape(OC, KH, KW * C)
        flat = runs.reshape(OC, -1)
    return qb.pack(qb.to_device_logical(flat, case.w_enc), case.w_bits, case.w_enc, fmt)


def conv_desc(qb, case, fmt, out_fmt, pitch):
    return qb.qnn_conv_desc(case.B, case.H, case.Wd, case.C, pitch, case.OC, case.KH, case.KW,
                            case.stride, case.pad, case.w_bits, case.a_bits, case.out_bits,
                            case.w_enc, case.a_enc, fmt, out_fmt, 0)


CONV_CASES = [
    # B, H, W, C, OC, KH, KW, stride, pad, w_bits, a_bits
    (2, 9, 9, 96, 70, 5, 5, 1, 2, 1, 2),
    (1, 13, 11, 40, 33, 3, 3, 1, 1, 2, 2),      # C not a multiple of 32 / 16
    (3, 12, 12, 32, 64, 3, 3, 2, 0, 1, 2),
    (1, 8, 8, 256, 130, 1, 1, 1, 0, 4, 4),
    (2, 7, 7, 64, 16, 7, 7, 1, 3, 3, 1),
]


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("shape", CONV_CASES)
def test_im2col_matches_host_lowering(qb, fmt, shape):
    case = synth.conv_case(800 + shape[3], *shape)
    x, pitch = device_map(qb, case, fmt)
    d = conv_desc(qb, case, fmt, INT8, pitch)
    npix = case.B * case.OH * case.OW
    low = torch.full((qb.qnn_conv_lowered_bytes(d),), 0xAB, dtype=torch.uint8, device="cuda")
    qb.check(qb.qnn_im2col(d, x, low))
    torch.cuda.synchronize()
    K = qb.qnn_conv_lowered_k(d)
    if fmt == BITPLANES:
        got = unpack_planes(low.cpu().numpy(), case.a_bits, npix, K, case.a_enc)
        want = host_im2col(case.In, case.KH, case.KW, case.stride, case.pad, round_up(case.C, 32))
    else:
        got = unpack_int8(low.cpu().numpy(), npix, K, case.a_enc)
        want = host_im2col(case.In, case.KH, case.KW, case.stride, case.pad, case.C,
                           run_pad=case.C % 16 != 0)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("lowering", ["auto", "explicit"])
@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("out_fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("shape", CONV_CASES)
def test_qconv_matches_direct_convolution(qb, monkeypatch, lowering, fmt, out_fmt, shape):
    """auto: 8-bit maps with C a multiple of 16 and stride 1 are lowered inside the GEMM's
    loader (im2col tensor map); explicit: always through the lowered matrix."""
    if lowering == "explicit":
        if fmt == BITPLANES:
            pytest.skip("bit-plane maps are always lowered explicitly")
        monkeypatch.setenv("QNN_CONV_EXPLICIT", "1")
    else:
        monkeypatch.setenv("QNN_CONV_IMPLICIT", "1")
    case = synth.conv_case(900 + shape[4], *shape)
    x, pitch = device_map(qb, case, fmt)
    Wp = device_weights(qb, case, fmt)
    d = conv_desc(qb, case, fmt, out_fmt, pitch)
    out = qb.qconv(d, Wp, x, torch.from_numpy(case.thr).cuda())
    torch.cuda.synchronize()
    npix = case.B * case.OH * case.OW
    got = decode_out(out.cpu().numpy(), out_fmt, case.out_bits, npix, case.OC, False)
    want = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
    assert np.array_equal(got, want)
    raw = qb.qconv(d, Wp, x, None)
    torch.cuda.synchronize()
    got = decode_out(raw.cpu().numpy(), out_fmt, case.out_bits, npix, case.OC, True)
    assert np.array_equal(got, orc.conv_direct(case.In, case.Wt, case.stride, case.pad).reshape(npix, case.OC))


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("B", [1, 4])
def test_config3_conv2_alexnet_shape(qb, fmt, B):
    """AlexNet conv2-shaped W1A2 layer: lowered GEMM rows 256, depth 2400, cols 729 per image."""
    case = synth.conv2_alexnet_case(B)
    x, pitch = device_map(qb, case, fmt)
    Wp = device_weights(qb, case, fmt)
    d = conv_desc(qb, case, fmt, INT8, pitch)
    assert qb.qnn_conv_lowered_k(d) == 2400
    out = qb.qconv(d, Wp, x, torch.from_numpy(case.thr).cuda())
    torch.cuda.synchronize()
    got = decode_out(out.cpu().numpy(), INT8, 2, B * 729, 256, False)
    want = orc.qconv(case.In, case.Wt, case.thr, 1, 2).reshape(B * 729, 256)
    assert np.array_equal(got, want)
    assert len(np.unique(got)) == 4


def test_conv1_shape_byte_lowering(qb):
    """First-layer shape: 3-channel uint8 image with pixel pitch 3, 11x11 stride 4 (K=363)."""
    case = synth.conv_case(950, 2, 227, 227, 3, 96, 11, 11, 4, 0, 8, 8, synth.SIGNED, synth.UNSIGNED)
    x, pitch = device_map(qb, case, INT8, in_pitch=3)
    Wp = device_weights(qb, case, INT8)
    for out_fmt in (INT8, BITPLANES):
        d = conv_desc(qb, case, INT8, out_fmt, pitch)
        out = qb.qconv(d, Wp, x, torch.from_numpy(case.thr).cuda())
        torch.cuda.synchronize()
        got = decode_out(out.cpu().numpy(), out_fmt, 2, 2 * 3025, 96, False)
        want = orc.qconv(case.In, case.Wt, case.thr, 4, 0).reshape(2 * 3025, 96)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("B,H,C,bits", [(2, 55, 96, 2), (1, 13, 256, 2), (3, 9, 40, 4), (1, 7, 33, 3), (2, 5, 64, 1)])
def test_maxpool(qb, fmt, B, H, C, bits):
    rng = np.random.default_rng(B * 100 + H)
    codes = rng.integers(0, 1 << bits, size=(B, H, H, C), dtype=np.int32)
    OH = (H - 3) // 2 + 1
    want = orc.maxpool(codes, 3, 2)
    if fmt == BITPLANES:
        x = qb.pack(qb.to_device_logical(codes.reshape(-1, C), 0), bits, 0, BITPLANES)
        out = torch.empty(bits * B * OH * OH * ((C + 31) // 32) * 4, dtype=torch.uint8, device="cuda")
    else:
        cp = round_up(C, 16)
        m = np.zeros((B, H, H, cp), dtype=np.uint8)
        m[..., :C] = codes
        x = torch.from_numpy(m).cuda()
        out = torch.empty(B * OH * OH * cp, dtype=torch.uint8, device="cuda")
    d = qb.qnn_pool_desc(B, H, H, C, 3, 2, bits, fmt)
    qb.check(qb.qnn_maxpool(d, x, out))
    torch.cuda.synchronize()
    got = decode_out(out.cpu().numpy(), fmt, bits, B * OH * OH, C, False)
    assert np.array_equal(got, want.reshape(-1, C))


@pytest.mark.parametrize("mode", ["tensor", "bitserial", "auto"])
@pytest.mark.parametrize("B", [1, 3])
def test_alexnet_chain_per_layer(qb, mode, B):
    """Every intermediate activation tensor and the final logits vs the oracle chain."""
    from paper_1709_04060_b200.alexnet import AlexNetPlan
    net = synth.alexnet_case(B)
    logits_ref, inter_ref = onet.forward(net)
    plan = AlexNetPlan(net, B, mode)
    img = torch.from_numpy(net.image.astype(np.uint8)).cuda()
    logits = plan.forward(img)
    torch.cuda.synchronize()
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    inter = plan.intermediates()
    for L in net.layers[:-1]:
        name = L.name + "_pool" if L.pool else L.name
        buf, kind, d = inter[name]
        want = inter_ref[L.name]
        C = want.shape[-1]
        npix = want.size // C
        fmt = d.fmt if kind == "pool" else d.out_fmt
        got = decode_out(buf.cpu().numpy(), fmt, 2, npix, C, False)
        assert np.array_equal(got, want.reshape(npix, C)), f"{mode}: first mismatch after {L.name}"
    assert np.array_equal(logits.cpu().numpy().astype(np.int64), logits_ref)


def test_alexnet_chain_graph_replay(qb):
    """The chain recorded into a CUDA graph gives the oracle's logits on replay, also after
    the input buffer has been overwritten with another batch."""
    from paper_1709_04060_b200.alexnet import AlexNetPlan
    net_a, net_b = synth.alexnet_case(2, seed=4), synth.alexnet_case(2, seed=5)
    net_b.weights, net_b.thr = net_a.weights, net_a.thr          # same network, other images
    plan = AlexNetPlan(net_a, 2, "tensor")
    img = torch.from_numpy(net_a.image.astype(np.uint8)).cuda()
    graph, logits = plan.capture(img)
    for net in (net_a, net_b, net_a):
        img.copy_(torch.from_numpy(net.image.astype(np.uint8)))
        graph.replay()
        torch.cuda.synchronize()
        want, _ = onet.forward(net, keep_intermediates=False)
        assert np.array_equal(logits.cpu().numpy().astype(np.int64), want)
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0


@pytest.mark.parametrize("shape", [
    # B, H, W, C, OC, KH, KW, stride, pad, w_bits, a_bits
    (2, 9, 10, 5, 20, 3, 3, 1, 1, 8, 8),
    (1, 7, 7, 3, 17, 3, 3, 2, 1, 8, 8),
    (3, 12, 11, 6, 33, 5, 4, 1, 2, 4, 4),
])
def test_byte_lowering_with_contiguous_pixels_and_padding(qb, shape):
    """Pixel pitch == C (no per-pixel padding) with zero padding around the image: the
    run-per-filter-row byte lowering against the host lowering and the direct convolution."""
    case = synth.conv_case(970 + shape[3], *shape, w_enc=synth.SIGNED, a_enc=synth.UNSIGNED)
    x, pitch = device_map(qb, case, INT8, in_pitch=case.C)
    d = conv_desc(qb, case, INT8, INT8, pitch)
    npix = case.B * case.OH * case.OW
    low = torch.full((qb.qnn_conv_lowered_bytes(d),), 0xAB, dtype=torch.uint8, device="cuda")
    qb.check(qb.qnn_im2col(d, x, low))
    torch.cuda.synchronize()
    got = unpack_int8(low.cpu().numpy(), npix, qb.qnn_conv_lowered_k(d), case.a_enc)
    want = host_im2col(case.In, case.KH, case.KW, case.stride, case.pad, case.C, run_pad=True)
    assert np.array_equal(got, want)
    Wp = device_weights(qb, case, INT8)
    out = qb.qconv(d, Wp, x, torch.from_numpy(case.thr).cuda())
    torch.cuda.synchronize()
    got = decode_out(out.cpu().numpy(), INT8, case.out_bits, npix, case.OC, False)
    want = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
    assert np.array_equal(got, want)


def test_config3_conv2_batch64_full(qb):
    """AlexNet conv2-shaped W1A2 layer at batch 64 (lowered GEMM 256 x 2400 x 46656), the
    size the benchmark's extras workload times: every output against the direct convolution."""
    case = synth.conv2_alexnet_case(64)
    x, pitch = device_map(qb, case, INT8)
    Wp = device_weights(qb, case, INT8)
    d = conv_desc(qb, case, INT8, INT8, pitch)
    out = qb.qconv(d, Wp, x, torch.from_numpy(case.thr).cuda())
    torch.cuda.synchronize()
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    got = decode_out(out.cpu().numpy(), INT8, 2, 64 * 729, 256, False)
    want = orc.qconv(case.In, case.Wt, case.thr, 1, 2).reshape(64 * 729, 256)
    assert np.array_equal(got, want)


def test_config4_alexnet_batch256_sampled_images(qb):
    """The chain at batch 256 (the large configuration): images are independent, so the
    oracle recomputes a sample of them one by one and their logits must match exactly."""
    from paper_1709_04060_b200.alexnet import AlexNetPlan
    net = synth.alexnet_case(256)
    plan = AlexNetPlan(net, 256, "tensor")
    img = torch.from_numpy(net.image.astype(np.uint8)).cuda()
    logits = plan.forward(img).cpu().numpy().astype(np.int64)
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    for b in (0, 77, 128, 255):
        one = synth.NetCase(B=1, image=net.image[b:b + 1], weights=net.weights, thr=net.thr)
        want, _ = onet.forward(one, keep_intermediates=False)
        assert np.array_equal(logits[b:b + 1], want), f"image {b}"


@pytest.mark.parametrize("shape", [
    # B, H, W, C, OC, KH, KW, stride, pad, w_bits, a_bits
    (3, 13, 13, 384, 256, 3, 3, 1, 1, 1, 2),      # conv5 shape: three 128-byte channel chunks per tap
    (2, 27, 27, 96, 256, 5, 5, 1, 2, 1, 2),       # conv2 shape: a 96-byte chunk (three of four MMAs)
    (5, 6, 7, 48, 40, 3, 2, 1, 0, 2, 2),          # no padding, ragged everything
    (1, 5, 5, 272, 33, 5, 5, 1, 4, 3, 3),         # padding larger than half the filter, 128+128+16 bytes
    (200, 4, 4, 16, 70, 2, 2, 1, 1, 4, 4),        # many small images: tiles span several images
    (3, 12, 12, 32, 64, 3, 3, 2, 0, 1, 2),        # stride 2, no padding
    (2, 23, 17, 64, 48, 5, 3, 3, 2, 2, 2),        # stride 3 with padding, rectangular filter and image
    (4, 9, 9, 128, 130, 3, 3, 2, 1, 1, 2),        # stride 2, padding 1, a full 128-byte chunk
])
@pytest.mark.parametrize("kernel", ["single", "pair"])
def test_implicit_convolution_shapes(qb, monkeypatch, shape, kernel):
    """Convolution with the lowering done by the tensor-core kernel's loader (the one-CTA kernel
    and the CTA-pair kernel, whose two CTAs fetch 128 output pixels each through the im2col tensor
    map), against the direct convolution; the explicit-lowering path must give the same bytes."""
    monkeypatch.setenv("QNN_TC_KERNEL", kernel)
    monkeypatch.setenv("QNN_CONV_LOWER", "0")         # not the lowering warps: the tensor-map loader
    monkeypatch.setenv("QNN_CONV_IMPLICIT", "1")      # also where the library would rather lower explicitly
    case = synth.conv_case(990 + shape[3], *shape)
    x, pitch = device_map(qb, case, INT8)
    Wp = device_weights(qb, case, INT8)
    npix = case.B * case.OH * case.OW
    thr = torch.from_numpy(case.thr).cuda()
    for out_fmt in (INT8, BITPLANES):
        d = conv_desc(qb, case, INT8, out_fmt, pitch)
        out = qb.qconv(d, Wp, x, thr)
        torch.cuda.synchronize()
        st, dev = qb.qnn_device_status()
        assert st == 0 and dev == 0
        got = decode_out(out.cpu().numpy(), out_fmt, case.out_bits, npix, case.OC, False)
        want = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
        assert np.array_equal(got, want)
    d = conv_desc(qb, case, INT8, INT8, pitch)
    n0 = qb.qnn_launch_count()
    raw = qb.qconv(d, Wp, x, None).clone()
    assert qb.qnn_launch_count() - n0 == 1            # one fused kernel, no lowering kernel
    monkeypatch.setenv("QNN_CONV_EXPLICIT", "1")
    n0 = qb.qnn_launch_count()
    raw_explicit = qb.qconv(d, Wp, x, None)
    assert qb.qnn_launch_count() - n0 == 2            # lowering + GEMM
    torch.cuda.synchronize()
    assert torch.equal(raw, raw_explicit)


@pytest.mark.parametrize("shape", [
    # B, H, W, C, OC, KH, KW, stride, pad, w_bits, a_bits
    (2, 39, 43, 3, 40, 11, 11, 4, 0, 8, 8),       # first-layer filter; map size not a multiple of 16 bytes
    (3, 227, 227, 3, 96, 11, 11, 4, 0, 8, 8),     # first-layer shape: 71 tiles, tiles across image boundaries
    (40, 12, 12, 3, 20, 5, 5, 1, 0, 8, 8),        # small images: a tile holds pixels of three images
    (2, 30, 29, 5, 130, 7, 3, 2, 0, 4, 4),        # more than 128 channels: explicit lowering
    (2, 30, 29, 5, 128, 7, 3, 2, 0, 4, 4),        # rectangular filter, stride 2, a full channel tile
    (1, 21, 22, 6, 33, 3, 4, 3, 0, 2, 2),         # stride 3
    (5, 9, 9, 20, 17, 3, 3, 1, 0, 2, 2),          # 20 channels: runs of 60 bytes in four 16-byte pieces
    (1, 8, 9, 1, 16, 2, 2, 1, 0, 8, 8),           # one channel, one 16-byte piece per run
    (1, 40, 41, 5, 64, 11, 11, 2, 0, 4, 4),       # depth 704: six k-blocks, two of them beyond the weight ring
    (1, 20, 2000, 3, 16, 11, 11, 4, 0, 8, 8),     # image rows too long for the staging buffers: explicit lowering
])
def test_convolution_lowered_inside_the_kernel(qb, monkeypatch, shape):
    """8-bit maps with contiguous pixels whose channel count is not a multiple of 16, no padding:
    lowering warps inside the tensor-core kernel build the activation tiles (one launch); against
    the direct convolution, and the explicit lowering must give the same accumulators."""
    case = synth.conv_case(1300 + shape[3] + shape[7], *shape, w_enc=synth.SIGNED, a_enc=synth.UNSIGNED)
    x, pitch = device_map(qb, case, INT8, in_pitch=case.C)
    Wp = device_weights(qb, case, INT8)
    npix = case.B * case.OH * case.OW
    thr = torch.from_numpy(case.thr).cuda()
    want = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
    for out_fmt in (INT8, BITPLANES):
        d = conv_desc(qb, case, INT8, out_fmt, pitch)
        n0 = qb.qnn_launch_count()
        out = qb.qconv(d, Wp, x, thr)
        # no lowering kernel while the weights fit shared memory (one tile of 128 channels)
        assert qb.qnn_launch_count() - n0 == (1 if case.OC <= 128 and case.Wd < 1000 else 2)
        torch.cuda.synchronize()
        st, dev = qb.qnn_device_status()
        assert st == 0 and dev == 0
        assert np.array_equal(decode_out(out.cpu().numpy(), out_fmt, case.out_bits, npix, case.OC, False), want)
    d = conv_desc(qb, case, INT8, INT8, pitch)
    raw = qb.qconv(d, Wp, x, None).clone()
    monkeypatch.setenv("QNN_CONV_EXPLICIT", "1")
    n0 = qb.qnn_launch_count()
    raw_explicit = qb.qconv(d, Wp, x, None)
    assert qb.qnn_launch_count() - n0 == 2            # lowering + GEMM
    torch.cuda.synchronize()
    assert torch.equal(raw, raw_explicit)
    acc = np.frombuffer(raw.cpu().numpy().tobytes(), dtype=np.int32).reshape(npix, case.OC)
    assert np.array_equal(acc, orc.conv_direct(case.In, case.Wt, case.stride, case.pad).reshape(npix, case.OC))


@pytest.mark.parametrize("shape", [
    # B, H, W, C, OC, KH, KW, stride, pad, w_bits, a_bits
    (2, 20, 21, 3, 40, 5, 5, 2, 0, 1, 2),         # runs of 15 bytes: one pad column per filter row
    (3, 9, 9, 5, 17, 3, 3, 1, 0, 1, 2),           # runs of 15 bytes
    (2, 11, 10, 20, 64, 3, 3, 1, 0, 1, 4),        # runs of 60 bytes
    (1, 12, 12, 16, 32, 3, 3, 1, 0, 1, 2),        # C a multiple of 16: no pad columns at all
])
def test_bipolar_weights_with_unaligned_runs(qb, monkeypatch, shape):
    """Bipolar weights have no zero: the pad columns that close each filter row's run hold -1 after
    packing.  The unmasked in-kernel lowering (which leaves image bytes opposite those columns)
    must therefore not be chosen for such a layer; whatever route the library takes, the codes and
    accumulators equal the direct convolution and the explicit route."""
    case = synth.conv_case(1500 + shape[3] + shape[5], *shape)
    assert case.w_enc == synth.BIPOLAR
    x, pitch = device_map(qb, case, INT8, in_pitch=case.C)
    Wp = device_weights(qb, case, INT8)
    npix = case.B * case.OH * case.OW
    thr = torch.from_numpy(case.thr).cuda()
    want = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
    want_acc = orc.conv_direct(case.In, case.Wt, case.stride, case.pad).reshape(npix, case.OC)
    for out_fmt in (INT8, BITPLANES):
        d = conv_desc(qb, case, INT8, out_fmt, pitch)
        out = qb.qconv(d, Wp, x, thr)
        torch.cuda.synchronize()
        assert np.array_equal(decode_out(out.cpu().numpy(), out_fmt, case.out_bits, npix, case.OC, False), want)
    d = conv_desc(qb, case, INT8, INT8, pitch)
    raw = qb.qconv(d, Wp, x, None).clone()
    acc = np.frombuffer(raw.cpu().numpy().tobytes(), dtype=np.int32).reshape(npix, case.OC)
    assert np.array_equal(acc, want_acc)
    monkeypatch.setenv("QNN_CONV_EXPLICIT", "1")
    raw_explicit = qb.qconv(d, Wp, x, None)
    torch.cuda.synchronize()
    assert torch.equal(raw, raw_explicit)
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0


@pytest.mark.parametrize("shape,fits", [
    # B, H, W, C, OC, KH, KW, stride, pad, w_bits, a_bits; fits: the staged image rows fit shared memory
    ((2, 27, 27, 96, 256, 5, 5, 1, 2, 1, 2), True),       # conv2 shape: runs of 480 bytes, padding 2
    ((3, 12, 12, 32, 64, 3, 3, 2, 0, 1, 2), True),        # stride 2, no padding
    ((2, 23, 17, 16, 48, 5, 3, 3, 2, 2, 2), True),        # stride 3 with padding, rectangular filter and image
    ((5, 6, 7, 48, 40, 3, 2, 1, 0, 2, 2), True),          # ragged everything
    ((200, 4, 4, 16, 70, 2, 2, 1, 1, 4, 4), True),        # many small images: a tile spans eight of them
    ((1, 5, 5, 272, 33, 5, 5, 1, 4, 3, 3), True),         # padding of four around a 5 x 5 map, 17 pieces per pixel
    ((1, 6, 40, 128, 130, 3, 3, 1, 1, 1, 2), True),       # a full 128-byte channel chunk
    ((1, 9, 9, 32, 300, 3, 3, 1, 1, 2, 2), True),         # two channel tiles of 256
    ((4, 9, 9, 128, 130, 3, 3, 2, 1, 1, 2), False),       # 55 image rows of 1152 bytes per tile: another route
])
def test_aligned_convolution_lowered_inside_the_kernel(qb, monkeypatch, shape, fits):
    """8-bit maps with contiguous pixels and C a multiple of 16: the lowering warps copy aligned
    16-byte pieces (zeros for taps outside the image), weights stream through the ring.  Forced
    here (the library picks this route for many tiles and C not a multiple of 128); against the
    direct convolution, the tensor-map loader and the explicit lowering."""
    monkeypatch.setenv("QNN_CONV_LOWER", "1")
    case = synth.conv_case(1400 + shape[3] + shape[7], *shape)
    x, pitch = device_map(qb, case, INT8)
    assert pitch == case.C
    Wp = device_weights(qb, case, INT8)
    npix = case.B * case.OH * case.OW
    thr = torch.from_numpy(case.thr).cuda()
    want = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
    for out_fmt in (INT8, BITPLANES):
        d = conv_desc(qb, case, INT8, out_fmt, pitch)
        n0 = qb.qnn_launch_count()
        out = qb.qconv(d, Wp, x, thr)
        if fits:
            assert qb.qnn_launch_count() - n0 == 1
        torch.cuda.synchronize()
        st, dev = qb.qnn_device_status()
        assert st == 0 and dev == 0
        assert np.array_equal(decode_out(out.cpu().numpy(), out_fmt, case.out_bits, npix, case.OC, False), want)
    d = conv_desc(qb, case, INT8, INT8, pitch)
    raw = qb.qconv(d, Wp, x, None).clone()
    monkeypatch.delenv("QNN_CONV_LOWER")
    monkeypatch.setenv("QNN_CONV_IMPLICIT", "1")
    raw_tma = qb.qconv(d, Wp, x, None).clone()
    monkeypatch.setenv("QNN_CONV_EXPLICIT", "1")
    raw_explicit = qb.qconv(d, Wp, x, None)
    torch.cuda.synchronize()
    assert torch.equal(raw, raw_explicit) and torch.equal(raw_tma, raw_explicit)
