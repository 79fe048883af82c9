"""Pins for the GEMM oracle: library routine, brute force, closed forms, and the
paper's bit-serial identities (Section 3.1, Algorithms 1 and 2)."""
import itertools

import numpy as np
import pytest

from oracle import oracle as orc
from oracle import bitserial as bs
from paper_1709_04060_b200 import synth

ENCS = {synth.UNSIGNED: "u", synth.SIGNED: "s", synth.BIPOLAR: "b"}


def _enc_choices(bits):
    return [synth.UNSIGNED, synth.SIGNED] + ([synth.BIPOLAR] if bits == 1 else [])


def test_against_numpy_matmul():
    rng = np.random.default_rng(1)
    for (M, N, K) in [(1, 1, 1), (3, 5, 7), (64, 33, 576), (17, 4, 130)]:
        W = rng.integers(-8, 8, size=(M, K), dtype=np.int32)
        At = rng.integers(0, 16, size=(N, K), dtype=np.int32)
        want = W.astype(np.int64) @ At.astype(np.int64).T
        got = orc.gemm(W, At)
        assert got.dtype == np.int64 and np.array_equal(got, want)


def test_not_symmetric_in_operands():
    # a transposed operand or swapped roles must change the result
    W = np.array([[1, 2, 3], [4, 5, 6]], dtype=np.int32)        # M=2, K=3
    At = np.array([[1, 0, 0], [0, 1, 0], [0, 0, 1], [1, 1, 1]], dtype=np.int32)  # N=4
    got = orc.gemm(W, At)
    assert got.tolist() == [[1, 2, 3, 6], [4, 5, 6, 15]]


def test_brute_force_all_values_small_depth():
    """Every operand value combination for K <= 2 at each width/encoding."""
    for w_bits, a_bits in itertools.product((1, 2, 3, 4), repeat=2):
        for w_enc in _enc_choices(w_bits):
            for a_enc in _enc_choices(a_bits):
                wl, wh = synth.value_range(w_bits, w_enc)
                al, ah = synth.value_range(a_bits, a_enc)
                wv = [-1, 1] if w_enc == synth.BIPOLAR else list(range(wl, wh + 1))
                av = [-1, 1] if a_enc == synth.BIPOLAR else list(range(al, ah + 1))
                K = 2 if len(wv) * len(av) <= 64 else 1
                Wrows = list(itertools.product(wv, repeat=K))
                Arows = list(itertools.product(av, repeat=K))
                got = orc.gemm(np.array(Wrows, dtype=np.int32), np.array(Arows, dtype=np.int32))
                for r, wr in enumerate(Wrows):
                    for c, ar in enumerate(Arows):
                        assert got[r, c] == sum(x * y for x, y in zip(wr, ar))


def test_closed_forms():
    K = 100
    ones = np.ones((3, K), dtype=np.int32)
    At = np.full((2, K), 3, dtype=np.int32)
    assert np.all(orc.gemm(ones, At) == 3 * K)
    # identity / permutation weights copy rows of A
    rng = np.random.default_rng(2)
    At = rng.integers(0, 4, size=(5, 8), dtype=np.int32)
    perm = rng.permutation(8)
    P = np.zeros((8, 8), dtype=np.int32)
    P[np.arange(8), perm] = 1
    assert np.array_equal(orc.gemm(P, At), At[:, perm].T)
    # single non-zero element
    W = np.zeros((4, 9), dtype=np.int32)
    W[2, 5] = -7
    At = rng.integers(0, 16, size=(3, 9), dtype=np.int32)
    want = np.zeros((4, 3), dtype=np.int64)
    want[2, :] = -7 * At[:, 5]
    assert np.array_equal(orc.gemm(W, At), want)
    # extreme values hit the analytic range bound K * 8 * 15
    K = 8192
    W = np.full((1, K), -8, dtype=np.int32)
    At = np.full((1, K), 15, dtype=np.int32)
    assert orc.gemm(W, At)[0, 0] == -K * 8 * 15 == -983040


def test_dot_at_matches_full():
    rng = np.random.default_rng(3)
    W = rng.integers(-2, 2, size=(9, 70), dtype=np.int32)
    At = rng.integers(0, 4, size=(11, 70), dtype=np.int32)
    full = orc.gemm(W, At)
    rows = rng.integers(0, 9, size=20)
    cols = rng.integers(0, 11, size=20)
    assert np.array_equal(orc.dot_at(W, At, rows, cols), full[rows, cols])


@pytest.mark.parametrize("w_bits,a_bits", list(itertools.product((1, 2, 3, 4), repeat=2)))
def test_bitserial_identity(w_bits, a_bits):
    """Sum over bit-plane pairs (Algorithm 2, with per-operand sign rules and the
    bipolar forms) equals the direct product, including K not a multiple of 32."""
    rng = np.random.default_rng(100 + 4 * w_bits + a_bits)
    for w_enc in _enc_choices(w_bits):
        for a_enc in _enc_choices(a_bits):
            for (M, N, K) in [(2, 3, 1), (3, 2, 31), (2, 2, 32), (4, 3, 70)]:
                W = synth.draw_operand(rng, (M, K), w_bits, w_enc)
                At = synth.draw_operand(rng, (N, K), a_bits, a_enc)
                direct = orc.gemm(W, At)
                serial = bs.bitserial_gemm(W.tolist(), At.tolist(), w_bits, a_bits, w_enc, a_enc)
                assert direct.tolist() == serial, (ENCS[w_enc], ENCS[a_enc], M, N, K)


def test_bipolar_xnor_popcount_closed_form():
    """dot of +-1 vectors = K - 2 * popcount(a xor b) (Section 3.1)."""
    rng = np.random.default_rng(5)
    for K in (1, 7, 32, 33, 95):
        a = rng.integers(0, 2, size=K)
        b = rng.integers(0, 2, size=K)
        va = (2 * a - 1).astype(np.int32)[None, :]
        vb = (2 * b - 1).astype(np.int32)[None, :]
        ia = int("".join(map(str, a[::-1])), 2)
        ib = int("".join(map(str, b[::-1])), 2)
        assert orc.gemm(va, vb)[0, 0] == K - 2 * bin(ia ^ ib).count("1")


def test_bipolar_times_unsigned_and_popcount_form():
    """w = 2b - 1: w.a = 2 * sum_j 2^j popc(b & a[j]) - sum_j 2^j popc(a[j])."""
    rng = np.random.default_rng(6)
    K = 77
    b = rng.integers(0, 2, size=K)
    a = rng.integers(0, 4, size=K)
    bw = int("".join(map(str, b[::-1])), 2)
    planes = [int("".join(map(str, ((a >> j) & 1)[::-1])), 2) for j in range(2)]
    want = 2 * sum((1 << j) * bin(bw & planes[j]).count("1") for j in range(2)) \
        - sum((1 << j) * bin(planes[j]).count("1") for j in range(2))
    got = orc.gemm((2 * b - 1).astype(np.int32)[None, :], a.astype(np.int32)[None, :])[0, 0]
    assert got == want


def test_planted_mistake_is_caught():
    """A dropped sign on the MSB plane must break the identity (the pin bites)."""
    W = np.array([[-2, 1, -1]], dtype=np.int32)
    At = np.array([[3, 1, 2]], dtype=np.int32)
    wrong = bs.bitserial_gemm(W.tolist(), At.tolist(), 2, 2, synth.UNSIGNED, synth.UNSIGNED)
    assert wrong != orc.gemm(W, At).tolist()


def test_config1_accumulator_range():
    case = synth.gemm_case(1, 64, 256, 576, 1, 2)
    acc = orc.gemm(case.W, case.At)
    assert acc.shape == (64, 256)
    assert np.abs(acc).max() <= 576 * 3
    # parity of a bipolar accumulator: sum of +-a_k has the parity of sum(a_k)
    assert np.array_equal(acc % 2, (case.At.sum(axis=1) % 2)[None, :].repeat(64, 0))
