"""GPU parity of the plane-skipping product (descriptor field skip_planes; the paper's conclusion:
approximate computing from the higher-order bit planes) against the plane-skipping oracle:
the kernels must equal the truncated sum exactly, for every encoding, on the tiled and the
few-column bit-serial kernels, with and without the threshold activation."""
import itertools

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from oracle import planeskip as ps
from paper_1709_04060_b200 import synth
from qnn_testutil import decode_out

pytestmark = pytest.mark.gpu

BITPLANES, INT8 = 0, 1


@pytest.fixture(scope="module")
def qb():
    from paper_1709_04060_b200 import binding
    return binding


def run_skip(qb, case, skip, out_fmt, raw):
    Wp = qb.pack(qb.to_device_logical(case.W, case.w_enc), case.w_bits, case.w_enc, BITPLANES)
    Ap = qb.pack(qb.to_device_logical(case.At, case.a_enc), case.a_bits, case.a_enc, BITPLANES)
    thr = None if raw else torch.from_numpy(case.thr).cuda()
    d = qb.gemm_desc(case.M, case.N, case.K, case.w_bits, case.a_bits, case.out_bits,
                     case.w_enc, case.a_enc, BITPLANES, out_fmt, 0, skip)
    out = qb.qgemm(d, Wp, Ap, thr)
    torch.cuda.synchronize()
    got = decode_out(out.cpu().numpy().view(np.uint8).reshape(-1), out_fmt, case.out_bits, case.N, case.M, raw)
    acc = ps.gemm(case.W, case.At, case.w_bits, case.a_bits, case.w_enc, case.a_enc, skip)
    want = (acc if raw else orc.threshold(acc, case.thr)).T
    assert np.array_equal(got, want), f"skip {skip}: {(got != want).sum()} mismatches"
    return acc


@pytest.mark.parametrize("w,a", [(1, 1), (1, 2), (2, 1), (2, 2), (3, 2), (4, 4), (2, 4)])
def test_tiled_kernel_every_encoding(qb, w, a):
    """197 x 301 x 1100 (several tiles, ragged tails) on the tiled AND/POPC kernel."""
    w_encs = [synth.SIGNED, synth.UNSIGNED] + ([synth.BIPOLAR] if w == 1 else [])
    a_encs = [synth.UNSIGNED, synth.SIGNED] + ([synth.BIPOLAR] if a == 1 else [])
    for w_enc, a_enc in itertools.product(w_encs, a_encs):
        case = synth.gemm_case(8000 + 10 * w + a, 197, 301, 1100, w, a, w_enc, a_enc, out_bits=2)
        exact = orc.gemm(case.W, case.At)
        nw = 1 if w_enc == synth.BIPOLAR else w
        na = 1 if a_enc == synth.BIPOLAR else a
        for skip in range(0, nw + na):
            acc = run_skip(qb, case, skip, INT8, raw=True)
            run_skip(qb, case, skip, BITPLANES, raw=False)
            assert np.abs(exact - acc).max() <= ps.error_bound(1100, w, a, w_enc, a_enc, skip)
            if skip == 0:
                assert np.array_equal(acc, exact)


@pytest.mark.parametrize("w,a,w_enc,a_enc", [(2, 2, 1, 0), (4, 4, 1, 0), (1, 2, 2, 0), (3, 1, 1, 2), (1, 1, 2, 2)])
def test_few_column_kernel(qb, w, a, w_enc, a_enc):
    """N <= 16: the one-warp-per-row kernel, vector and scalar depth loops."""
    for (M, N, K) in ((1000, 3, 4096), (333, 16, 1000)):
        case = synth.gemm_case(8100 + w + a, M, N, K, w, a, w_enc, a_enc, out_bits=2)
        nw = 1 if w_enc == synth.BIPOLAR else w
        na = 1 if a_enc == synth.BIPOLAR else a
        for skip in range(0, nw + na):
            run_skip(qb, case, skip, INT8, raw=True)
            run_skip(qb, case, skip, INT8, raw=False)


def test_skipping_is_refused_where_it_has_no_meaning(qb):
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    n0 = qb.qnn_launch_count()
    d = qb.gemm_desc(64, 64, 256, 2, 2, 2, 1, 0, INT8, INT8, 0, 1)          # 8-bit containers
    assert qb.qnn_qgemm(d, buf, buf, None, buf) == qb.QNN_ERR_UNSUPPORTED
    d = qb.gemm_desc(64, 64, 256, 2, 2, 2, 1, 0, BITPLANES, INT8, 0, -1)
    assert qb.qnn_qgemm(d, buf, buf, None, buf) == qb.QNN_ERR_INVALID_ARG
    assert qb.qnn_launch_count() == n0


def test_skipping_saves_time_on_the_bit_serial_kernel(qb):
    """W4A4 at 1024^3: leaving out the pairs with i + j < 3 drops 6 of 16 AND/POPC passes; the
    kernel must get faster, not just differ (timed with CUDA events, generous margin)."""
    case = synth.gemm_case(8200, 1024, 1024, 1024, 4, 4)
    Wp = qb.pack(qb.to_device_logical(case.W, case.w_enc), 4, case.w_enc, BITPLANES)
    Ap = qb.pack(qb.to_device_logical(case.At, case.a_enc), 4, case.a_enc, BITPLANES)
    thr = torch.from_numpy(case.thr).cuda()
    times = {}
    for skip in (0, 3):
        d = qb.gemm_desc(1024, 1024, 1024, 4, 4, 4, case.w_enc, case.a_enc, BITPLANES, INT8, 0, skip)
        out = qb.qgemm(d, Wp, Ap, thr)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            qb.qgemm(d, Wp, Ap, thr, out)
        e1.record()
        torch.cuda.synchronize()
        times[skip] = e0.elapsed_time(e1)
    assert times[3] < 0.85 * times[0], times
