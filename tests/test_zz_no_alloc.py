"""qnn_qconv_static: the convolution entry point for callers that cannot supply a workspace.

Some users of this library never get to allocate device memory: a plug-in whose host
application owns every byte of the GPU and passes in only the layer's input and output
tensors, or a latency-bound loop where cudaMalloc is banned because it may stall the
device.  For them the lowered matrix sits in a fixed 16 MiB array inside the library.
This file checks, through the C ABI, that the entry point gives exactly what qnn_qconv
gives (integer results: the tolerance is zero) on two calls in a row that share the array,
that both equal the CPU oracle's direct convolution, and that it refuses a problem whose
lowered matrix does not fit.

The file name makes pytest collect it after every other test file.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1709_04060_b200 import synth
from qnn_testutil import decode_out

pytestmark = pytest.mark.gpu

BITPLANES, INT8 = 0, 1


@pytest.fixture(scope="module")
def qb():
    from paper_1709_04060_b200 import binding
    return binding


def _setup(qb, case, fmt):
    """Device feature map, packed weights and descriptor for one convolution."""
    B, H, Wd, C = case.In.shape
    OC, KH, KW, _ = case.Wt.shape
    if fmt == BITPLANES:
        x = qb.pack(qb.to_device_logical(case.In.reshape(B * H * Wd, C), case.a_enc),
                    case.a_bits, case.a_enc, BITPLANES)
        cp = (C + 31) // 32 * 32
        Wl = np.zeros((OC, KH * KW, cp), dtype=np.int32)
        Wl[:, :, :C] = case.Wt.reshape(OC, KH * KW, C)
        pitch = 0
    else:
        pitch = (C + 15) // 16 * 16
        m = np.zeros((B, H, Wd, pitch), dtype=np.uint8)
        m[..., :C] = case.In.astype(np.uint8)
        x = torch.from_numpy(m).cuda()
        if C % 16 == 0:
            Wl = case.Wt
        else:                   # 8-bit maps with other channel counts: one zero-padded run per filter row
            Wl = np.zeros((OC, KH, (KW * C + 15) // 16 * 16), dtype=np.int32)
            Wl[:, :, :KW * C] = case.Wt.reshape(OC, KH, KW * C)
    Wp = qb.pack(qb.to_device_logical(Wl.reshape(OC, -1), case.w_enc), case.w_bits, case.w_enc, fmt)
    d = qb.qnn_conv_desc(B, H, Wd, C, pitch, OC, KH, KW, case.stride, case.pad, case.w_bits,
                         case.a_bits, case.out_bits, case.w_enc, case.a_enc, fmt, INT8, 0)
    return d, Wp, x, torch.from_numpy(case.thr).cuda()


def _both(qb, d, Wp, x, thr):
    """(output of qnn_qconv with a caller workspace, output of qnn_qconv_static)."""
    nbytes = qb.qnn_conv_out_bytes(d, thr is not None)
    want = qb.qconv(d, Wp, x, thr)
    got = torch.full((nbytes,), 0xEE, dtype=torch.uint8, device="cuda")
    qb.check(qb.qnn_qconv_static(d, Wp, x, thr, got))
    torch.cuda.synchronize()
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    return want.cpu().numpy()[:nbytes], got.cpu().numpy()


@pytest.mark.parametrize("fmt", [INT8, BITPLANES])
def test_two_calls_in_a_row_match_qconv(qb, fmt):
    # first call: conv2-shaped W1A2 layer, two images (lowered matrix 3.5 MB as bytes);
    # second call: a smaller, differently shaped layer, so that the array still holds most
    # of the first call's lowered matrix when the second one runs.
    first = synth.conv2_alexnet_case(2, seed=31)
    second = synth.conv_case(32, 1, 13, 11, 40, 33, 3, 3, 1, 1, 2, 2)
    for case in (first, second):
        d, Wp, x, thr = _setup(qb, case, fmt)
        assert qb.qnn_conv_workspace_bytes(d) <= qb.QNN_QCONV_STATIC_MAX_BYTES
        want, got = _both(qb, d, Wp, x, thr)
        assert np.array_equal(got, want)
        want_raw, got_raw = _both(qb, d, Wp, x, None)          # raw int32 accumulators
        assert np.array_equal(got_raw, want_raw)
        # and against the oracle's direct convolution (codes and accumulators)
        npix = case.B * case.OH * case.OW
        ref = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
        assert np.array_equal(decode_out(got, INT8, case.out_bits, npix, case.OC, False), ref)
        ref_acc = orc.conv_direct(case.In, case.Wt, case.stride, case.pad).reshape(npix, case.OC)
        assert np.array_equal(decode_out(got_raw, INT8, 0, npix, case.OC, True), ref_acc)


@pytest.mark.parametrize("C", [3, 5, 20])
def test_bipolar_weights_small_channel_counts(qb, C):
    """Bipolar (+-1) filters over an 8-bit map whose channel count is not a multiple of 16:
    the pad columns of the packed weight rows are -1, not 0, so the result depends on the
    lowered matrix being zero there.  Against the oracle and against qnn_qconv."""
    case = synth.conv_case(40 + C, 2, 14, 13, C, 24, 3, 3, 1, 0, 1, 2)
    d, Wp, x, thr = _setup(qb, case, INT8)
    want, got = _both(qb, d, Wp, x, thr)
    assert np.array_equal(got, want)
    npix = case.B * case.OH * case.OW
    ref = orc.qconv(case.In, case.Wt, case.thr, case.stride, case.pad).reshape(npix, case.OC)
    assert np.array_equal(decode_out(got, INT8, case.out_bits, npix, case.OC, False), ref)


def test_problem_larger_than_the_array_is_refused(qb):
    case = synth.conv2_alexnet_case(1, seed=33)
    d, Wp, x, thr = _setup(qb, case, INT8)
    d.B = 64                                   # lowered matrix 112 MB > 16 MiB; nothing is launched
    assert qb.qnn_conv_workspace_bytes(d) > qb.QNN_QCONV_STATIC_MAX_BYTES
    out = torch.empty(16, dtype=torch.uint8, device="cuda")
    launches = qb.qnn_launch_count()
    assert qb.qnn_qconv_static(d, Wp, x, thr, out) == qb.QNN_ERR_WORKSPACE
    assert qb.qnn_launch_count() == launches
