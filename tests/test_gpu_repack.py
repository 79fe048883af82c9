"""Bit-plane operands widened to 8-bit containers on the device (qnn_planes_to_int8): the planes
are packed on the host by the tests' own numpy packer, the containers are decoded on the host, and
the logical values must come back unchanged, pad bytes zero; the bytes must also equal what the
packer writes from the logical values directly."""
import numpy as np
import pytest
import torch

from paper_1709_04060_b200 import synth
from qnn_testutil import host_pack_planes, unpack_int8, round_up

pytestmark = pytest.mark.gpu

BITPLANES, INT8 = 0, 1


@pytest.fixture(scope="module")
def qb():
    from paper_1709_04060_b200 import binding
    return binding


@pytest.mark.parametrize("bits,enc", [(1, synth.UNSIGNED), (1, synth.SIGNED), (1, synth.BIPOLAR), (2, synth.UNSIGNED),
                                      (2, synth.SIGNED), (3, synth.UNSIGNED), (3, synth.SIGNED), (4, synth.UNSIGNED),
                                      (4, synth.SIGNED), (8, synth.UNSIGNED), (8, synth.SIGNED)])
def test_planes_to_containers(qb, bits, enc):
    rng = np.random.default_rng(40 + 3 * bits + enc)
    for (rows, K) in ((1, 1), (3, 15), (5, 16), (7, 17), (33, 31), (9, 32), (11, 33), (130, 1000), (64, 4096), (257, 2049)):
        X = synth.draw_operand(rng, (rows, K), bits, enc)
        planes = torch.from_numpy(host_pack_planes(X, 1 if enc == synth.BIPOLAR else bits, enc)).cuda()
        d = qb.qnn_pack_desc(rows, K, bits, enc, BITPLANES)
        out = torch.full((rows * round_up(K, 16) + 16,), 0xEE, dtype=torch.uint8, device="cuda")
        n0 = qb.qnn_launch_count()
        qb.check(qb.qnn_planes_to_int8(d, planes, out))
        assert qb.qnn_launch_count() - n0 == 1
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.array_equal(unpack_int8(got, rows, K, enc), X), (rows, K)        # also: pad bytes zero
        assert (got[rows * round_up(K, 16):] == 0xEE).all()                         # nothing past the matrix
        direct = qb.pack(qb.to_device_logical(X, enc), bits, enc, INT8).cpu().numpy()
        assert np.array_equal(got[: rows * round_up(K, 16)], direct[: rows * round_up(K, 16)])


def test_arguments_are_checked_before_launch(qb):
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    n0 = qb.qnn_launch_count()
    assert qb.qnn_planes_to_int8(qb.qnn_pack_desc(4, 64, 2, 0, INT8), buf, buf) == qb.QNN_ERR_INVALID_ARG
    assert qb.qnn_planes_to_int8(qb.qnn_pack_desc(4, 64, 9, 0, BITPLANES), buf, buf) == qb.QNN_ERR_INVALID_ARG
    assert qb.qnn_planes_to_int8(qb.qnn_pack_desc(4, 64, 2, 2, BITPLANES), buf, buf) == qb.QNN_ERR_UNSUPPORTED
    assert qb.qnn_planes_to_int8(qb.qnn_pack_desc(4, 64, 2, 0, BITPLANES), buf[4:], buf) == qb.QNN_ERR_ALIGNMENT
    assert qb.qnn_planes_to_int8(qb.qnn_pack_desc(0, 64, 2, 0, BITPLANES), buf, buf) == qb.QNN_ERR_INVALID_ARG
    assert qb.qnn_launch_count() == n0


@pytest.mark.parametrize("w,a", [(1, 2), (2, 1), (3, 3), (4, 4)])
def test_packed_in_packed_out_pipeline(qb, w, a):
    """The benchmark's end-to-end leg at a size the oracle finishes: activations packed as bit planes
    on the host (the tests' own packer), widened on the device, multiplied on the tensor cores with
    the threshold epilogue writing bit planes, unpacked on the host: every code against the oracle."""
    from oracle import oracle as orc
    from qnn_testutil import decode_out
    M, N, K = 300, 700, 1100
    case = synth.gemm_case(9100 + 10 * w + a, M, N, K, w, a)
    planes = torch.from_numpy(host_pack_planes(case.At, 1 if case.a_enc == synth.BIPOLAR else a, case.a_enc)).cuda()
    containers = torch.empty(N * round_up(K, 16), dtype=torch.uint8, device="cuda")
    qb.check(qb.qnn_planes_to_int8(qb.qnn_pack_desc(N, K, a, case.a_enc, BITPLANES), planes, containers))
    Wp = qb.pack(qb.to_device_logical(case.W, case.w_enc), w, case.w_enc, INT8)
    d = qb.gemm_desc(M, N, K, w, a, case.out_bits, case.w_enc, case.a_enc, INT8, BITPLANES)
    out = qb.qgemm(d, Wp, containers, torch.from_numpy(case.thr).cuda())
    torch.cuda.synchronize()
    got = decode_out(out.cpu().numpy().view(np.uint8).reshape(-1), BITPLANES, case.out_bits, N, M, False)
    assert np.array_equal(got, orc.qgemm(case.W, case.At, case.thr).T)
