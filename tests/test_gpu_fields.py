"""GPU parity of the few-column kernels on packed w-bit weights (QNN_FMT_FIELDS weights, 8-bit
activation containers, N <= 16) through the C ABI against the CPU oracle: bit-exact on every
element, every output layout, every weight encoding and field width.  Every test runs three times:
with the library's own choice between its two kernels (byte dot products on the CUDA cores for a
few columns, the tensor-core form beyond) and with each of them forced."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1709_04060_b200 import synth
from qnn_testutil import unpack_operand, decode_out

pytestmark = pytest.mark.gpu

BITPLANES, INT8, FIELDS = 0, 1, 2


@pytest.fixture(scope="module")
def qb():
    from paper_1709_04060_b200 import binding
    return binding


@pytest.fixture(autouse=True, params=["auto", "dp4a", "tensor"])
def fields_kernel(request, monkeypatch):
    if request.param == "auto":
        monkeypatch.delenv("QNN_FIELDS_KERNEL", raising=False)
    else:
        monkeypatch.setenv("QNN_FIELDS_KERNEL", request.param)
    return request.param


def run_fields(qb, case, out_fmt, raw=False, check_pack=False):
    Wp = qb.pack(qb.to_device_logical(case.W, case.w_enc), case.w_bits, case.w_enc, FIELDS)
    Ap = qb.pack(qb.to_device_logical(case.At, case.a_enc), case.a_bits, case.a_enc, INT8)
    if check_pack:
        back = unpack_operand(Wp.cpu().numpy(), FIELDS, case.w_bits, case.M, case.K, case.w_enc)
        assert np.array_equal(back, case.W)
    thr = None if raw else torch.from_numpy(case.thr).cuda()
    d = qb.qnn_gemm_desc(case.M, case.N, case.K, case.w_bits, case.a_bits, case.out_bits,
                         case.w_enc, case.a_enc, FIELDS, INT8, out_fmt, 0)
    nbytes = qb.qnn_gemm_out_bytes(d, not raw)
    out = torch.full((max(nbytes, 16),), 0xEE, dtype=torch.uint8, device="cuda")
    n0 = qb.qnn_launch_count()
    qb.check(qb.qnn_qgemm(d, Wp, Ap, thr, out))
    # one fused kernel (the byte-dot-product kernel clears a bit-plane output first)
    assert qb.qnn_launch_count() - n0 <= (2 if out_fmt == BITPLANES and not raw else 1)
    torch.cuda.synchronize()
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    got = decode_out(out.cpu().numpy()[:nbytes], out_fmt, case.out_bits, case.N, case.M, raw)
    want = orc.qgemm(case.W, case.At, None if raw else case.thr).T
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{len(bad)} mismatches, first at (n,m)={bad[0]}: got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}"


@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("N", [1, 4, 16])
def test_config5_skinny_fc_packed_weights(qb, bits, N):
    """M = K = 8192, W2A2 and W4A4, signed weights, N in {1, 4, 16}: every output, all three
    output layouts (the same seeded problems as the other operand formats' test)."""
    case = synth.gemm_case(5000 + 10 * bits + N, 8192, N, 8192, bits, bits)
    run_fields(qb, case, INT8, check_pack=(N == 1))
    run_fields(qb, case, BITPLANES)
    run_fields(qb, case, INT8, raw=True)


@pytest.mark.parametrize("w_bits,w_enc", [(1, 2), (1, 0), (1, 1), (2, 0), (2, 1), (3, 0), (3, 1), (4, 0), (4, 1)])
def test_every_width_and_encoding_ragged(qb, w_bits, w_enc):
    """Every field width and weight encoding on shapes with ragged tails: rows not a multiple of
    the block, depth not a multiple of a stage or of a 32-byte group, one to sixteen columns,
    signed and unsigned activations of 2, 4 and 8 bits, 1 to 15 thresholds."""
    shapes = [(333, 3, 9216, 2, 0, 2), (70, 16, 1000, 4, 1, 3), (4096, 1, 4100, 8, 0, 4), (5, 7, 33, 3, 1, 1),
              (1000, 5, 4096, 2, 0, 2), (129, 2, 31, 2, 0, 2), (2050, 9, 700, 4, 0, 4)]
    for (M, N, K, a_bits, a_enc, out_bits) in shapes:
        case = synth.gemm_case(6100 + M + 7 * w_bits + w_enc, M, N, K, w_bits, a_bits, w_enc, a_enc, out_bits=out_bits)
        run_fields(qb, case, INT8, check_pack=True)
        run_fields(qb, case, BITPLANES)
        run_fields(qb, case, INT8, raw=True)


def test_alexnet_fc_shapes_batch_1_to_16(qb):
    """fc6 / fc7 of the AlexNet-shaped network (bipolar weights, 2-bit activations; Table 3)."""
    for (M, K) in ((4096, 9216), (4096, 4096)):
        for N in (1, 16):
            case = synth.gemm_case(6300 + K + N, M, N, K, 1, 2)
            run_fields(qb, case, INT8)
            run_fields(qb, case, BITPLANES)


def test_extreme_values_and_thresholds(qb):
    """Every operand at the end of its range, thresholds at and next to the resulting sums,
    INT32 sentinels, unsorted thresholds."""
    K = 8192
    W = np.full((200, K), -8, dtype=np.int32); W[::3] = 7; W[5] = 0
    At = np.full((16, K), 15, dtype=np.int32); At[::5] = 0; At[3, ::2] = 1
    thr = np.sort(np.random.default_rng(9).integers(-983040, 983041, size=(200, 15)), axis=1).astype(np.int32)
    thr[0] = -983040; thr[1] = 983040 - 122880
    thr[2] = thr[2][::-1]                                   # unsorted: the counting rule still holds
    thr[4, :7] = -(2 ** 31); thr[4, 7:] = 2 ** 31 - 1
    case = synth.GemmCase(200, 16, K, 4, 4, synth.SIGNED, synth.UNSIGNED, 4, W, At, thr)
    run_fields(qb, case, INT8)
    run_fields(qb, case, BITPLANES)
    run_fields(qb, case, INT8, raw=True)


def test_unsupported_shapes_are_refused_before_launch(qb):
    """More than 16 columns, bit-plane activations, a forced bit-serial path, 8-bit weights."""
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    n0 = qb.qnn_launch_count()
    for d in (qb.qnn_gemm_desc(64, 17, 256, 2, 2, 2, 1, 0, FIELDS, INT8, INT8, 0),
              qb.qnn_gemm_desc(64, 4, 256, 2, 2, 2, 1, 0, FIELDS, BITPLANES, INT8, 0),
              qb.qnn_gemm_desc(64, 4, 256, 2, 2, 2, 1, 0, FIELDS, INT8, INT8, 1),
              qb.qnn_gemm_desc(64, 4, 256, 8, 2, 2, 1, 0, FIELDS, INT8, INT8, 0)):
        assert qb.qnn_qgemm(d, buf, buf, None, buf) == qb.QNN_ERR_UNSUPPORTED
    assert qb.qnn_launch_count() == n0
