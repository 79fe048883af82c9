"""GPU parity: packer and fused GEMM+threshold through the C ABI vs the CPU oracle.
Bit-exact on every element (integer results are unique)."""
import itertools

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_1709_04060_b200 import synth
from qnn_testutil import unpack_operand, decode_out

pytestmark = pytest.mark.gpu

BITPLANES, INT8 = 0, 1


@pytest.fixture(scope="module")
def qb():
    from paper_1709_04060_b200 import binding
    return binding


def run_case(qb, case, fmt, out_fmt, raw=False, path=0, check_pack=False):
    Wd = qb.to_device_logical(case.W, case.w_enc)
    Ad = qb.to_device_logical(case.At, case.a_enc)
    Wp = qb.pack(Wd, case.w_bits, case.w_enc, fmt)
    Ap = qb.pack(Ad, case.a_bits, case.a_enc, fmt)
    if check_pack:
        w_back = unpack_operand(Wp.cpu().numpy(), fmt, case.w_bits, case.M, case.K, case.w_enc)
        a_back = unpack_operand(Ap.cpu().numpy(), fmt, case.a_bits, case.N, case.K, case.a_enc)
        assert np.array_equal(w_back, case.W) and np.array_equal(a_back, case.At)
    thr = None if raw else torch.from_numpy(case.thr).cuda()
    d = qb.gemm_desc(case.M, case.N, case.K, case.w_bits, case.a_bits, case.out_bits,
                     case.w_enc, case.a_enc, fmt, out_fmt, path)
    out = qb.qgemm(d, Wp, Ap, thr)
    torch.cuda.synchronize()
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    got = decode_out(out.cpu().numpy().view(np.uint8).reshape(-1), out_fmt, case.out_bits,
                     case.N, case.M, raw)
    want = orc.qgemm(case.W, case.At, None if raw else case.thr).T
    assert got.shape == want.shape
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{len(bad)} mismatches, first at (n,m)={bad[0]}: got {got[tuple(bad[0])]} want {want[tuple(bad[0])]}"


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("out_fmt,raw", [(INT8, False), (BITPLANES, False), (INT8, True)])
def test_config1_w1a2(qb, fmt, out_fmt, raw):
    """Single W1A2 GEMM+threshold: M=64, K=576 bipolar weights, N=256 2-bit activations."""
    case = synth.gemm_case(1, 64, 256, 576, 1, 2)
    run_case(qb, case, fmt, out_fmt, raw, check_pack=True)


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
def test_config1_full_range_thresholds_with_ties(qb, fmt):
    """Thresholds over the whole +-1728 accumulator range, duplicates, and values
    that accumulators hit exactly (ties count as passed)."""
    case = synth.gemm_case(1, 64, 256, 576, 1, 2, spread=38.5)
    acc = orc.gemm(case.W, case.At)
    thr = case.thr.copy()
    thr[0] = [acc[0, 0], acc[0, 0], acc[0, 1]]
    thr[0].sort()
    thr[1] = [-1728, 0, 1728]
    thr[2] = [-(2**31), -(2**31), 2**31 - 1]
    thr[3] = [int(acc[3].min()), int(np.median(acc[3])), int(acc[3].max())]
    case.thr = thr
    run_case(qb, case, fmt, INT8)
    run_case(qb, case, fmt, BITPLANES)


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("w_bits,a_bits", list(itertools.product((1, 2, 3, 4), repeat=2)))
def test_all_widths_ragged(qb, fmt, w_bits, a_bits):
    """Every (w, a) pair with each encoding, on sizes that span several tiles of
    both kernels and leave ragged tails in M, N and K."""
    w_encs = [synth.SIGNED, synth.UNSIGNED] + ([synth.BIPOLAR] if w_bits == 1 else [])
    a_encs = [synth.UNSIGNED, synth.SIGNED] + ([synth.BIPOLAR] if a_bits == 1 else [])
    seed = 200 + 10 * w_bits + a_bits
    for w_enc, a_enc in itertools.product(w_encs, a_encs):
        case = synth.gemm_case(seed, 197, 301, 1100, w_bits, a_bits, w_enc, a_enc, out_bits=a_bits)
        out_fmt = BITPLANES if (w_enc + a_enc) % 2 else INT8
        run_case(qb, case, fmt, out_fmt, check_pack=True)


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (1, 7, 33), (129, 1, 31), (130, 257, 129),
                                   (64, 513, 4100), (300, 40, 16)])
def test_edge_shapes(qb, fmt, M, N, K):
    case = synth.gemm_case(300 + M + N, M, N, K, 2, 2)
    run_case(qb, case, fmt, INT8, check_pack=True)
    run_case(qb, case, fmt, BITPLANES)
    run_case(qb, case, fmt, INT8, raw=True)
    if fmt == INT8:            # few columns go to the byte dot-product kernel: also force the tensor cores
        run_case(qb, case, fmt, INT8, path=2)
        run_case(qb, case, fmt, BITPLANES, path=2)
        run_case(qb, case, fmt, INT8, raw=True, path=2)


@pytest.mark.parametrize("out_bits", [1, 2, 3, 4])
def test_out_bits_independent_of_a_bits(qb, out_bits):
    for fmt in (BITPLANES, INT8):
        case = synth.gemm_case(400 + out_bits, 150, 200, 640, 2, 3, out_bits=out_bits)
        run_case(qb, case, fmt, INT8)
        run_case(qb, case, fmt, BITPLANES)


def test_eight_bit_layers_tensor_path(qb):
    """8-bit first/last layer shapes (Section 4.2): s8 x u8 with K=363 (not a
    multiple of 16) and thresholds; s8 x 2-bit codes with raw int32 output."""
    c1 = synth.gemm_case(500, 96, 3025, 363, 8, 8, synth.SIGNED, synth.UNSIGNED, out_bits=2)
    run_case(qb, c1, INT8, INT8, check_pack=True)
    c8 = synth.gemm_case(501, 1000, 5, 4096, 8, 2, synth.SIGNED, synth.UNSIGNED, out_bits=2)
    run_case(qb, c8, INT8, INT8, raw=True)            # few columns: byte dot-product kernel
    run_case(qb, c8, INT8, INT8, raw=True, path=2)    # the same on the tensor cores


def test_unsorted_thresholds_follow_counting_rule(qb):
    case = synth.gemm_case(600, 70, 90, 256, 2, 2)
    case.thr = case.thr[:, ::-1].copy()
    for fmt in (BITPLANES, INT8):
        run_case(qb, case, fmt, INT8)
    st, bad = qb.qnn_validate_thresholds(torch.from_numpy(case.thr).cuda(), 70, 3)
    assert st == 0 and bad == int((np.diff(case.thr, axis=1) < 0).any(axis=1).sum())
    st, bad = qb.qnn_validate_thresholds(torch.from_numpy(np.sort(case.thr, axis=1)).cuda(), 70, 3)
    assert st == 0 and bad == 0


def test_outputs_monotone_in_accumulator(qb):
    """Codes are non-decreasing in the raw accumulator (property, any size)."""
    case = synth.gemm_case(700, 256, 512, 2048, 1, 2)
    Wd = qb.to_device_logical(case.W, case.w_enc)
    Ad = qb.to_device_logical(case.At, case.a_enc)
    Wp, Ap = qb.pack(Wd, 1, case.w_enc, INT8), qb.pack(Ad, 2, case.a_enc, INT8)
    d = qb.gemm_desc(256, 512, 2048, 1, 2, 2, case.w_enc, case.a_enc, INT8, INT8)
    codes = qb.qgemm(d, Wp, Ap, torch.from_numpy(case.thr).cuda()).cpu().numpy()[: 512 * 256].reshape(512, 256)
    acc = qb.qgemm(d, Wp, Ap, None).cpu().numpy()
    for m in range(0, 256, 17):
        order = np.argsort(acc[:, m], kind="stable")
        assert np.all(np.diff(codes[order, m].astype(np.int32)) >= 0)


@pytest.fixture
def force_tc_kernel(monkeypatch):
    def _set(which):
        monkeypatch.setenv("QNN_TC_KERNEL", which)
    return _set


@pytest.mark.parametrize("which", ["single", "pair"])
@pytest.mark.parametrize("M,N,K,w,a", [
    (64, 256, 576, 1, 2), (197, 301, 1100, 2, 2), (512, 768, 2048, 1, 2), (300, 1000, 4100, 4, 4),
    (256, 256, 128, 3, 3), (1, 1, 1, 2, 2), (129, 257, 129, 2, 3), (640, 520, 16, 4, 1),
])
def test_both_tensor_core_kernels(qb, force_tc_kernel, which, M, N, K, w, a):
    """The one-CTA and the CTA-pair (cta_group::2) kernels on the same problems,
    every output mode, incl. sizes with ragged M/N/K tails and fewer tiles than SMs."""
    force_tc_kernel(which)
    case = synth.gemm_case(1000 + M + N + K, M, N, K, w, a)
    run_case(qb, case, INT8, INT8, path=2)
    run_case(qb, case, INT8, BITPLANES, path=2)
    run_case(qb, case, INT8, INT8, raw=True, path=2)


@pytest.mark.parametrize("M,N,K,w,a", [
    (250, 19195, 256, 1, 2),     # 150 tiles on 148 SMs: the last 2 are shared, 1 + 1 k-blocks
    (512, 10240, 160, 2, 4),     # 160 tiles: the last 12 are shared (two k-blocks, the second ragged)
    (768, 8440, 1100, 4, 3),     # 198 tiles: the last 50 are shared, 5 + 4 k-blocks
])
def test_partial_last_round_is_shared_by_cta_pairs(qb, monkeypatch, M, N, K, w, a):
    """Tile counts just above a multiple of the SM count: the kernel runs as two-CTA clusters
    and each tile of the last round is computed by the two CTAs of a cluster, half of the
    depth each; the odd CTA hands its int32 partial sums to the even one through distributed
    shared memory before the threshold epilogue.  Every output is checked, and the same
    problem with sharing switched off must give identical bytes."""
    monkeypatch.setenv("QNN_TC_KERNEL", "single")     # the larger shapes would otherwise take the CTA-pair kernel
    case = synth.gemm_case(1200 + M, M, N, K, w, a)
    run_case(qb, case, INT8, INT8)
    run_case(qb, case, INT8, BITPLANES)
    run_case(qb, case, INT8, INT8, raw=True)
    d = qb.gemm_desc(M, N, K, w, a, case.out_bits, case.w_enc, case.a_enc, INT8, INT8)
    Wp = qb.pack(qb.to_device_logical(case.W, case.w_enc), w, case.w_enc, INT8)
    Ap = qb.pack(qb.to_device_logical(case.At, case.a_enc), a, case.a_enc, INT8)
    thr = torch.from_numpy(case.thr).cuda()
    shared = qb.qgemm(d, Wp, Ap, thr).clone()
    monkeypatch.setenv("QNN_TC_NO_SHARE", "1")
    whole = qb.qgemm(d, Wp, Ap, thr)
    torch.cuda.synchronize()
    assert torch.equal(shared, whole)


@pytest.mark.parametrize("M,N,K,w,a", [
    (512, 11520, 512, 1, 2),     # 90 tiles on 74 SM pairs: the last 16 are split, 2 + 2 k-blocks
    (480, 11520, 384, 2, 3),     # ragged last channel tile (224 of 256), 1 + 2 k-blocks, bisection epilogue
    (320, 12800, 700, 4, 4),     # second channel tile holds 64 channels: three column groups have no owner
    (768, 8448, 272, 1, 1),      # 99 tiles: 25 split, the second half of the depth is a ragged k-block
    (512, 11400, 640, 2, 2),     # the last tile of pixels is ragged (136 of 256) and is among the split ones
])
def test_pair_kernel_split_last_round(qb, monkeypatch, M, N, K, w, a):
    """CTA-pair kernel with a workspace: the tiles of a last round that would keep at most half of the
    SM pairs busy are each run by two neighbouring pairs, one per half of the depth, which exchange
    int32 partial sums through the workspace.  Every output against the oracle, every output mode;
    the same bytes as without a workspace; the workspace's flag words are zero again afterwards, so
    that a second call on the same workspace works."""
    monkeypatch.setenv("QNN_TC_KERNEL", "pair")
    case = synth.gemm_case(1300 + M + K, M, N, K, w, a)
    d = qb.gemm_desc(M, N, K, w, a, case.out_bits, case.w_enc, case.a_enc, INT8, INT8)
    ws_bytes = qb.qnn_gemm_workspace_bytes(d)
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert ws_bytes > 0
    if ws_bytes == 0:
        pytest.skip("this GPU's SM count gives the shape no half-empty last round")
    run_case(qb, case, INT8, INT8)
    run_case(qb, case, INT8, BITPLANES)
    run_case(qb, case, INT8, INT8, raw=True)
    Wp = qb.pack(qb.to_device_logical(case.W, case.w_enc), w, case.w_enc, INT8)
    Ap = qb.pack(qb.to_device_logical(case.At, case.a_enc), a, case.a_enc, INT8)
    thr = torch.from_numpy(case.thr).cuda()
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(3):                              # the same workspace three times in a row
        out = torch.empty(qb.qnn_gemm_out_bytes(d, True), dtype=torch.uint8, device="cuda")
        qb.check(qb.qnn_qgemm(d, Wp, Ap, thr, out, ws, ws_bytes))
        outs.append(out)
    whole = torch.empty_like(outs[0])
    qb.check(qb.qnn_qgemm(d, Wp, Ap, thr, whole, None, 0))       # no workspace: nothing is split
    torch.cuda.synchronize()
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    for out in outs:
        assert torch.equal(out, whole)
    assert int(ws[:8192].view(torch.int32).abs().sum()) == 0


@pytest.mark.parametrize("which", ["single", "pair"])
def test_integer_count_path_for_large_accumulators(qb, force_tc_kernel, which):
    """8-bit x 8-bit with K large enough that |acc| can exceed 2^24: the epilogue must
    count thresholds in integer arithmetic; thresholds beyond +-2^24 included."""
    force_tc_kernel(which)
    case = synth.gemm_case(1100, 200, 300, 1024, 8, 8, synth.SIGNED, synth.UNSIGNED, out_bits=3)
    case.thr[0] = [-(2**31), -(2**24) - 5, -(2**24), 0, 2**24, 2**24 + 7, 2**31 - 1]
    run_case(qb, case, INT8, INT8)
    small = synth.gemm_case(1101, 200, 300, 512, 4, 4, out_bits=3)
    small.thr[0] = [-(2**31), -(2**24) - 5, -(2**24), 0, 2**24, 2**24 + 7, 2**31 - 1]
    small.thr[1] = [-16777215, -16777214, -1, 0, 1, 16777215, 16777216]
    run_case(qb, small, INT8, INT8)
    run_case(qb, small, BITPLANES, INT8)


def _sample_indices(rng, M, N, count, edges):
    rows = np.concatenate([rng.integers(0, M, count), [e % M for e in edges]])
    cols = np.concatenate([rng.integers(0, N, count), [e % N for e in reversed(edges)]])
    return rows, cols


@pytest.mark.parametrize("w,a", list(itertools.product((1, 2, 3, 4), repeat=2)))
def test_full_size_4096_sampled(qb, w, a):
    """Every problem of the benchmark's sweep in the benchmark's own launch configuration
    (M = N = K = 4096, 8-bit containers in and out, the library's kernel choice, 2^a - 1
    thresholds): sampled accumulators and codes against oracle dot products, plus one whole
    weight row and one whole column.  A bit-plane output of the same problem is decoded and
    compared with the byte output element by element."""
    case = synth.gemm_case(2000 + 10 * w + a, 4096, 4096, 4096, w, a)
    Wd = qb.to_device_logical(case.W, case.w_enc)
    Ad = qb.to_device_logical(case.At, case.a_enc)
    Wp, Ap = qb.pack(Wd, w, case.w_enc, INT8), qb.pack(Ad, a, case.a_enc, INT8)
    d = qb.gemm_desc(4096, 4096, 4096, w, a, a, case.w_enc, case.a_enc, INT8, INT8)
    thr = torch.from_numpy(case.thr).cuda()
    codes = qb.qgemm(d, Wp, Ap, thr).cpu().numpy().reshape(4096, 4096)
    raw = qb.qgemm(d, Wp, Ap, None).cpu().numpy()
    rng = np.random.default_rng(7)
    rows, cols = _sample_indices(rng, 4096, 4096, 3000, [0, 4095, 127, 128, 255, 256, 4095])
    acc = orc.dot_at(case.W, case.At, rows, cols)
    assert np.array_equal(raw[cols, rows].astype(np.int64), acc)
    want = (acc[:, None] >= case.thr[rows]).sum(axis=1)
    assert np.array_equal(codes[cols, rows].astype(np.int64), want)
    # one full weight row and one full column through the oracle GEMM
    full_row = orc.qgemm(case.W[777:778], case.At, case.thr[777:778])[0]
    assert np.array_equal(codes[:, 777].astype(np.int64), full_row)
    full_col = orc.qgemm(case.W, case.At[1234:1235], case.thr)[:, 0]
    assert np.array_equal(codes[1234, :].astype(np.int64), full_col)
    # the raw accumulators decide every code: all 16.8 M codes against the counting rule
    # applied on the host to the device's own accumulators (whose samples the oracle confirmed)
    recount = np.zeros(raw.shape, dtype=np.uint8)
    for q in range(case.thr.shape[1]):
        recount += raw >= case.thr[None, :, q]
    assert np.array_equal(codes, recount)
    # qb.qgemm hands the library its optional workspace (a split last round of tiles on GPUs whose
    # SM count leaves one); the same call without a workspace must give the same bytes
    whole = torch.empty(qb.qnn_gemm_out_bytes(d, True), dtype=torch.uint8, device="cuda")
    qb.check(qb.qnn_qgemm(d, Wp, Ap, thr, whole, None, 0))
    assert np.array_equal(whole.cpu().numpy().reshape(4096, 4096), codes)
    dp = qb.gemm_desc(4096, 4096, 4096, w, a, a, case.w_enc, case.a_enc, INT8, BITPLANES)
    planes = qb.qgemm(dp, Wp, Ap, thr).cpu().numpy()
    assert np.array_equal(decode_out(planes, BITPLANES, a, 4096, 4096, False), codes.astype(np.int64))
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0


@pytest.mark.parametrize("out_bits", [1, 2, 3, 4])
def test_pair_kernel_many_rounds_every_threshold_count(qb, force_tc_kernel, out_bits):
    """The CTA-pair kernel over several rounds of its persistent loop (2 x 157 = 314 tiles of
    256 x 256 on 74 SM pairs: the tensor-memory and threshold double buffers wrap twice, the
    last round is partial), for 1, 3, 7 and 15 thresholds and both output layouts: every
    output against the oracle."""
    force_tc_kernel("pair")
    M, N, K = 512, 40000, 256
    case = synth.gemm_case(1700 + out_bits, M, N, K, 2, out_bits, out_bits=out_bits)
    run_case(qb, case, INT8, INT8, path=2)
    run_case(qb, case, INT8, BITPLANES, path=2)
    run_case(qb, case, INT8, INT8, raw=True, path=2)


@pytest.mark.parametrize("fmt", [BITPLANES, INT8])
@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("N", [1, 4, 16])
def test_config5_skinny_fc(qb, fmt, bits, N):
    """Large fully connected layer at small batch (M = K = 8192, N in {1, 4, 16}), W2A2 and
    W4A4, signed weights: every output against the oracle, both operand formats."""
    case = synth.gemm_case(5000 + 10 * bits + N, 8192, N, 8192, bits, bits)
    run_case(qb, case, fmt, INT8)
    run_case(qb, case, fmt, BITPLANES)
    run_case(qb, case, fmt, INT8, raw=True)


@pytest.mark.parametrize("w_enc,a_enc,w,a", [(2, 0, 1, 2), (1, 2, 3, 1), (2, 2, 1, 1), (0, 1, 4, 3)])
def test_skinny_bit_serial_encodings(qb, w_enc, a_enc, w, a):
    """The few-column bit-serial kernel with bipolar / signed / unsigned operands, depths that
    are and are not a multiple of 128 (vector and scalar loads), ragged M."""
    for K, M, N in ((9216, 333, 3), (1000, 70, 16), (4096, 4096, 1)):
        case = synth.gemm_case(5100 + K + w, M, N, K, w, a, w_enc, a_enc, out_bits=2)
        run_case(qb, case, BITPLANES, INT8, check_pack=True)
        run_case(qb, case, BITPLANES, BITPLANES)
        run_case(qb, case, BITPLANES, INT8, raw=True)


@pytest.mark.parametrize("bits", [2, 4])
def test_config5_square_8192_sampled(qb, bits):
    """M = N = K = 8192 (compute bound) on the tensor-core path: sampled accumulators and codes."""
    case = synth.gemm_case(5200 + bits, 8192, 8192, 8192, bits, bits)
    Wp = qb.pack(qb.to_device_logical(case.W, case.w_enc), bits, case.w_enc, INT8)
    Ap = qb.pack(qb.to_device_logical(case.At, case.a_enc), bits, case.a_enc, INT8)
    d = qb.gemm_desc(8192, 8192, 8192, bits, bits, bits, case.w_enc, case.a_enc, INT8, INT8)
    codes = qb.qgemm(d, Wp, Ap, torch.from_numpy(case.thr).cuda()).cpu().numpy().reshape(8192, 8192)
    raw = qb.qgemm(d, Wp, Ap, None).cpu().numpy()
    rng = np.random.default_rng(11)
    rows = np.concatenate([rng.integers(0, 8192, 2000), [0, 8191, 255, 256]])
    cols = np.concatenate([rng.integers(0, 8192, 2000), [0, 8191, 127, 128]])
    acc = orc.dot_at(case.W, case.At, rows, cols)
    assert np.array_equal(raw[cols, rows].astype(np.int64), acc)
    want = (acc[:, None] >= case.thr[rows]).sum(axis=1)
    assert np.array_equal(codes[cols, rows].astype(np.int64), want)
    full_col = orc.qgemm(case.W, case.At[4321:4322], case.thr)[:, 0]
    assert np.array_equal(codes[4321, :].astype(np.int64), full_col)


@pytest.mark.parametrize("w_enc,a_enc,w,a", [(1, 0, 8, 8), (1, 1, 4, 8), (0, 0, 3, 2), (0, 1, 2, 4), (2, 0, 1, 2)])
def test_skinny_byte_kernel_encodings(qb, w_enc, a_enc, w, a):
    """The few-column kernel on 8-bit containers (4-way byte dot products) with every
    signedness pair, depths that are not a multiple of 16, ragged M, every output mode."""
    for K, M, N in ((4100, 333, 3), (1000, 70, 8), (8192, 1000, 1), (33, 5, 7)):
        case = synth.gemm_case(5300 + K + w, M, N, K, w, a, w_enc, a_enc, out_bits=3)
        run_case(qb, case, INT8, INT8, check_pack=True)
        run_case(qb, case, INT8, BITPLANES)
        run_case(qb, case, INT8, INT8, raw=True)


def test_streamlined_layer_end_to_end(qb):
    """Section 2.1 end to end: float alpha / batch-norm / quantizer parameters of a W1A2 layer
    are absorbed into integer thresholds by the library's host tool (rows with a negative
    collapsed slope are negated), the fused GEMM+threshold kernel runs on integers only, and its
    codes equal the float forward pass of the un-streamlined layer evaluated by the oracle."""
    from oracle import streamline as ref
    case = synth.gemm_case(7000, 64, 256, 576, 1, 2)
    rng = np.random.default_rng(7000)
    chans = [ref.random_params(rng, int(case.W[m].sum()), 45.0) for m in range(64)]
    st, thr, neg = qb.qnn_streamline(
        [(c.a_prev, c.b_prev, c.alpha, c.gamma, c.beta, c.mu, c.sigma, c.row_sum) for c in chans],
        ref.HWGQ_THRESHOLDS, -1728, 1728)
    assert st == 0 and any(neg)
    W_dev = case.W.copy()
    W_dev[np.array(neg, dtype=bool)] *= -1                       # bipolar rows: a sign flip
    acc = orc.gemm(case.W, case.At)                              # accumulators of the original layer
    want = np.array([[ref.float_forward(int(acc[m, n]), chans[m], ref.HWGQ_THRESHOLDS)
                      for m in range(64)] for n in range(256)])
    for fmt in (INT8, BITPLANES):
        Wp = qb.pack(qb.to_device_logical(W_dev, case.w_enc), 1, case.w_enc, fmt)
        Ap = qb.pack(qb.to_device_logical(case.At, case.a_enc), 2, case.a_enc, fmt)
        d = qb.gemm_desc(64, 256, 576, 1, 2, 2, case.w_enc, case.a_enc, fmt, INT8)
        out = qb.qgemm(d, Wp, Ap, torch.tensor(thr, dtype=torch.int32).cuda())
        torch.cuda.synchronize()
        got = decode_out(out.cpu().numpy(), INT8, 2, 256, 64, False)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("path", [0, 2])
def test_extreme_operands_and_accumulators(qb, path):
    """Degenerate and extreme inputs: every operand at the end of its range, so that every
    accumulator sits at the analytic bound K * max|w| * max|a| (here up to 1.07e9, close to
    the int32 limit the library accepts), with thresholds at and next to those values."""
    K = 32768
    for wv, av in ((-128, 255), (127, 255), (-128, 0)):
        W = np.full((130, K), wv, dtype=np.int32)
        W[7] = 0; W[8, ::2] = -wv - 1 if wv < 0 else -wv          # a zero row and a mixed row
        At = np.full((70, K), av, dtype=np.int32)
        At[3] = 0; At[4, : K // 2] = 1
        acc = int(wv) * int(av) * K
        thr = np.sort(np.array([[acc - 1, acc, acc + 1, 0, -1, 1, 2**31 - 1]] * 130, dtype=np.int64), axis=1)
        thr = np.clip(thr, -2**31, 2**31 - 1).astype(np.int32)
        case = synth.GemmCase(130, 70, K, 8, 8, synth.SIGNED, synth.UNSIGNED, 3, W, At, thr)
        run_case(qb, case, INT8, INT8, path=path)
        run_case(qb, case, INT8, INT8, raw=True, path=path)
    # few-bit containers and bit planes at their extremes (W4A4: -8 x 15)
    W = np.full((100, 8192), -8, dtype=np.int32); W[::3] = 7
    At = np.full((40, 8192), 15, dtype=np.int32); At[::5] = 0
    thr = np.sort(np.random.default_rng(9).integers(-983040, 983041, size=(100, 15)), axis=1).astype(np.int32)
    thr[0] = -983040; thr[1] = 983040 - 122880                   # exactly the extreme accumulators
    case = synth.GemmCase(100, 40, 8192, 4, 4, synth.SIGNED, synth.UNSIGNED, 4, W, At, thr)
    run_case(qb, case, INT8, INT8, path=path)
    if path == 0:
        run_case(qb, case, BITPLANES, INT8)
        run_case(qb, case, BITPLANES, BITPLANES)


def test_accumulator_range_is_checked_on_the_host(qb):
    """K * max|w| * max|a| >= 2^31 cannot be accumulated in int32: refused before any launch."""
    K = 65808                                   # 65808 * 128 * 255 = 2^31 + 489472
    d = qb.gemm_desc(64, 64, K, 8, 8, 2, qb.QNN_ENC_SIGNED, qb.QNN_ENC_UNSIGNED, INT8, INT8)
    buf = torch.zeros(64 * K, dtype=torch.uint8, device="cuda")
    out = torch.zeros(64 * 64, dtype=torch.uint8, device="cuda")
    n0 = qb.qnn_launch_count()
    assert qb.qnn_qgemm(d, buf, buf, None, out) == qb.QNN_ERR_UNSUPPORTED
    assert qb.qnn_launch_count() == n0
