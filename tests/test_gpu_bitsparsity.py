"""Bit-level sparsity on the tiled AND/POPC kernel (the paper's conclusion names it beside the
approximate product): plane tiles without a set bit are skipped, which must not change a single
output -- every case is compared with the exact CPU oracle -- and must save time where the
high-order planes of an operand are empty over whole tiles."""
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


def run_planes(qb, W, At, thr, w_bits, a_bits, w_enc, a_enc, out_bits, out_fmt=INT8, raw=False):
    M, K = W.shape
    N = At.shape[0]
    Wp = qb.pack(qb.to_device_logical(W, w_enc), w_bits, w_enc, BITPLANES)
    Ap = qb.pack(qb.to_device_logical(At, a_enc), a_bits, a_enc, BITPLANES)
    d = qb.gemm_desc(M, N, K, w_bits, a_bits, out_bits, w_enc, a_enc, BITPLANES, out_fmt)
    assert qb.qnn_qgemm_kernel(d, not raw) == qb.QNN_KERNEL_PLANES_TILED
    out = qb.qgemm(d, Wp, Ap, None if raw else torch.from_numpy(thr).cuda())
    torch.cuda.synchronize()
    got = decode_out(out.cpu().numpy().view(np.uint8).reshape(-1), out_fmt, out_bits, N, M, raw)
    want = orc.qgemm(W, At, None if raw else thr).T
    bad = np.argwhere(got != want)
    assert bad.size == 0, f"{len(bad)} mismatches, first at (n,m)={bad[0]}"


def _thresholds(rng, acc, out_bits):
    lo, hi = int(acc.min()), int(acc.max())
    return np.sort(rng.integers(lo, hi + 1, size=(acc.shape[0], (1 << out_bits) - 1)), axis=1).astype(np.int32)


@pytest.mark.parametrize("w_bits,a_bits,w_enc,a_enc", [
    (4, 4, synth.UNSIGNED, synth.UNSIGNED), (4, 4, synth.SIGNED, synth.UNSIGNED),
    (3, 4, synth.SIGNED, synth.SIGNED), (1, 4, synth.BIPOLAR, synth.UNSIGNED),
    (4, 1, synth.UNSIGNED, synth.BIPOLAR), (2, 3, synth.UNSIGNED, synth.SIGNED)])
def test_empty_planes_and_empty_blocks_change_nothing(qb, w_bits, a_bits, w_enc, a_enc):
    """Operands built so that many 64-row x 512-bit plane tiles are empty in different patterns:
    small values in wide containers (high planes empty everywhere), all-zero blocks of rows and of
    depth, a single set bit in an otherwise empty tile, negative values (every plane set) next to
    them.  Several tiles in both directions and ragged tails; all three output layouts."""
    rng = np.random.default_rng(900 + 16 * w_bits + a_bits + w_enc + 3 * a_enc)
    M, N, K = 197, 301, 2100
    wl, wh = synth.value_range(w_bits, w_enc)
    al, ah = synth.value_range(a_bits, a_enc)
    W = synth.draw_operand(rng, (M, K), w_bits, w_enc)
    At = synth.draw_operand(rng, (N, K), a_bits, a_enc)
    if w_enc != synth.BIPOLAR:
        W[:64] = np.clip(W[:64], 0, 1)                 # rows 0-63: only plane 0 occupied
        W[64:128, 512:1536] = 0                        # two empty depth steps for a row block
        W[128:, 1024:1536] = 0
        W[130, 1100] = wh                              # one value in an otherwise empty tile
    if a_enc != synth.BIPOLAR:
        At[:, :512] = np.clip(At[:, :512], 0, 1)       # first depth step: plane 0 only
        At[64:192] = 0                                 # two empty column blocks
        At[100, 2099] = al if al < 0 else ah           # ... but for one element (all planes when negative)
        At[256:, 1536:2048] = 0
    acc = orc.gemm(W, At)
    thr = _thresholds(rng, acc, 2)
    run_planes(qb, W, At, thr, w_bits, a_bits, w_enc, a_enc, 2, INT8)
    run_planes(qb, W, At, thr, w_bits, a_bits, w_enc, a_enc, 2, BITPLANES)
    run_planes(qb, W, At, thr, w_bits, a_bits, w_enc, a_enc, 2, INT8, raw=True)


def test_all_zero_operands(qb):
    """Every tile empty: nothing is multiplied at all, the thresholds still count."""
    M, N, K = 130, 70, 1000
    W = np.zeros((M, K), dtype=np.int32)
    At = np.zeros((N, K), dtype=np.int32)
    thr = np.tile(np.array([-1, 0, 1], dtype=np.int32), (M, 1))
    run_planes(qb, W, At, thr, 2, 2, synth.SIGNED, synth.UNSIGNED, 2)
    run_planes(qb, W, np.ones((N, K), dtype=np.int32), thr, 2, 2, synth.SIGNED, synth.UNSIGNED, 2)


def test_empty_high_planes_save_time(qb):
    """W4A4 at 1024^3: with activations below 4 two of the four activation planes are empty in every
    tile, so half of the 16 AND/POPC passes fall away; timed with CUDA events, generous margin.
    The results of both runs are exact (sampled against the oracle's dot products)."""
    rng = np.random.default_rng(77)
    W = synth.draw_operand(rng, (1024, 1024), 4, synth.SIGNED)
    dense = synth.draw_operand(rng, (1024, 1024), 4, synth.UNSIGNED)
    small = dense & 3
    Wp = qb.pack(qb.to_device_logical(W, synth.SIGNED), 4, synth.SIGNED, BITPLANES)
    d = qb.gemm_desc(1024, 1024, 1024, 4, 4, 4, synth.SIGNED, synth.UNSIGNED, BITPLANES, INT8)
    rows, cols = rng.integers(0, 1024, 500), rng.integers(0, 1024, 500)
    times = {}
    for name, At in (("dense", dense), ("small", small)):
        Ap = qb.pack(qb.to_device_logical(At, synth.UNSIGNED), 4, synth.UNSIGNED, BITPLANES)
        raw = qb.qgemm(d, Wp, Ap, None)
        torch.cuda.synchronize()
        assert np.array_equal(raw.cpu().numpy()[cols, rows].astype(np.int64), orc.dot_at(W, At, rows, cols))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            qb.qgemm(d, Wp, Ap, None, raw.view(torch.uint8).view(-1))
        e1.record()
        torch.cuda.synchronize()
        times[name] = e0.elapsed_time(e1)
    assert times["small"] < 0.75 * times["dense"], times
