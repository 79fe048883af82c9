"""Pins for the threshold oracle and the streamlining identity (Section 2.1)."""
import math
import os

import numpy as np

from oracle import oracle as orc
from oracle import streamline as sl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _hwgq_rows():
    rows = []
    with open(os.path.join(GOLDEN, "hwgq_quantizer.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                x, level, code = line.split()
                rows.append((float(x), float(level), int(code)))
    return rows


def test_hwgq_worked_example_float():
    for x, level, code in _hwgq_rows():
        got = sl.successive_threshold(x, sl.HWGQ_THRESHOLDS)
        assert got == code
        assert abs(sl.HWGQ_STEP * got - level) < 1e-12


def test_hwgq_worked_example_integer_oracle():
    """The same table through the integer oracle, on a 1/1000 fixed-point grid."""
    rows = _hwgq_rows()
    acc = np.array([[int(round(x * 1000)) for x, _, _ in rows]], dtype=np.int64)
    thr = np.array([[0, 807, 1345]], dtype=np.int32)
    # non-tie points only, except x=0.001 -> 1 which is above t0=0
    got = orc.threshold(acc, thr)[0]
    assert got.tolist() == [c for _, _, c in rows]


def test_tie_counts_as_passed():
    acc = np.array([[-1, 0, 1, 4, 5, 6]], dtype=np.int64)
    thr = np.array([[0, 5, 5]], dtype=np.int32)
    assert orc.threshold(acc, thr)[0].tolist() == [0, 1, 1, 1, 3, 3]


def test_monotone_and_range():
    rng = np.random.default_rng(0)
    for n_thr in (1, 3, 7, 15):
        thr = np.sort(rng.integers(-50, 50, size=(4, n_thr)), axis=1).astype(np.int32)
        acc = np.tile(np.arange(-80, 80, dtype=np.int64), (4, 1))
        out = orc.threshold(acc, thr)
        assert out.min() >= 0 and out.max() <= n_thr
        assert np.all(np.diff(out, axis=1) >= 0)
        assert np.all(out[:, 0] == 0) and np.all(out[:, -1] == n_thr)
        # brute force
        for r in range(4):
            for c in range(0, 160, 7):
                assert out[r, c] == sum(1 for t in thr[r] if t <= acc[r, c])


def test_per_row_thresholds_are_per_row():
    acc = np.array([[5, 5], [5, 5]], dtype=np.int64)
    thr = np.array([[0, 1, 2], [6, 7, 8]], dtype=np.int32)
    assert orc.threshold(acc, thr).tolist() == [[3, 3], [0, 0]]


def test_sentinels_and_repeated_thresholds():
    acc = np.array([[-2**31 + 1, 0, 2**31 - 2]], dtype=np.int64)
    thr = np.array([[sl.INT32_MIN, sl.INT32_MIN, sl.INT32_MAX]], dtype=np.int32)
    assert orc.threshold(acc, thr)[0].tolist() == [2, 2, 2]
    thr = np.array([[7, 7, 7]], dtype=np.int32)
    assert orc.threshold(np.array([[6, 7, 8]], dtype=np.int64), thr)[0].tolist() == [0, 3, 3]


def test_nhwc_variant_matches_row_variant():
    rng = np.random.default_rng(1)
    acc = rng.integers(-100, 100, size=(2, 3, 4, 5), dtype=np.int64)   # [B][H][W][OC]
    thr = np.sort(rng.integers(-60, 60, size=(5, 3)), axis=1).astype(np.int32)
    got = orc.threshold_nhwc(acc, thr)
    want = orc.threshold(acc.reshape(-1, 5).T.copy(), thr).T.reshape(acc.shape)
    assert np.array_equal(got, want)


def test_threshold_equals_bn_then_quantize_exhaustive():
    """Streamlined integer thresholds reproduce float BN+quantizer over the WHOLE
    accumulator range of a depth-576 bipolar x 2-bit layer (+-1728), including
    channels with negative and zero collapsed scale."""
    rng = np.random.default_rng(7)
    lo, hi = -1728, 1728
    accs = np.arange(lo, hi + 1, dtype=np.int64)
    seen_neg = seen_pos = 0
    for ch in range(40):
        p = sl.random_params(rng, row_sum=int(rng.integers(-100, 100)), scale=45.0)
        if ch == 5:
            p.gamma = 0.0
        thr, negate = sl.streamline(p, sl.HWGQ_THRESHOLDS, lo, hi)
        assert thr == sorted(thr)
        seen_neg += negate
        seen_pos += (not negate)
        x = -accs if negate else accs
        got = orc.threshold(x[None, :], np.array([thr], dtype=np.int32))[0]
        want = [sl.float_forward(int(a), p, sl.HWGQ_THRESHOLDS) for a in accs]
        assert got.tolist() == want
    assert seen_neg > 0 and seen_pos > 0


def test_closed_form_ceil_on_exact_parameters():
    """ceil((t - B)/A) with dyadic-rational parameters (fp64 exact), incl. integer ties."""
    p = sl.ChannelParams(a_prev=0.5, b_prev=0.25, alpha=0.125, gamma=2.0, beta=0.5,
                         mu=1.0, sigma=4.0, row_sum=12)
    qthr = (0.0, 0.75, 1.5, 0.53125)
    A, B = sl.collapse(p)
    assert A == 2.0 * 0.125 * 0.5 / 4.0
    closed = sl.closed_form_thresholds(p, sorted(qthr))
    searched, negate = sl.streamline(p, sorted(qthr), -10000, 10000)
    assert not negate and closed == searched
    # (t-B)/A integer for t=0.53125 -> x == threshold must count (tie rule)
    t_int = (0.53125 - B) / A
    assert t_int == math.floor(t_int)
    assert sl.float_forward(int(t_int), p, [0.53125]) == 1
    assert sl.float_forward(int(t_int) - 1, p, [0.53125]) == 0


def test_collapse_matches_sequential_forward():
    rng = np.random.default_rng(8)
    for _ in range(20):
        p = sl.random_params(rng, row_sum=int(rng.integers(-50, 50)), scale=30.0)
        A, B = sl.collapse(p)
        for acc in (-100, -1, 0, 3, 250):
            z = p.alpha * (p.a_prev * acc + p.b_prev * p.row_sum)
            y = p.gamma * (z - p.mu) / p.sigma + p.beta
            assert abs((A * acc + B) - y) <= 1e-9 * max(1.0, abs(y))
