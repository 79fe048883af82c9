"""The library's host-side streamlining tool (qnn_streamline) against the fp64 reference in
oracle/streamline.py (written independently: bisection there, closed form + correction here)
and against the float forward pass itself, exhaustively over the accumulator range."""
import numpy as np
import pytest

from oracle import streamline as ref


@pytest.fixture(scope="module")
def qb():
    import __graft_entry__ as ge
    ge.build()
    from paper_1709_04060_b200 import binding
    return binding


def _as_tuple(p):
    return (p.a_prev, p.b_prev, p.alpha, p.gamma, p.beta, p.mu, p.sigma, p.row_sum)


def test_matches_reference_on_random_channels(qb):
    rng = np.random.default_rng(20)
    lo, hi = -1728, 1728                       # accumulator range of the 576-deep W1A2 layer
    chans = [ref.random_params(rng, int(rng.integers(-200, 200)), 45.0) for _ in range(300)]
    chans[5].gamma = 0.0                        # zero slope: constant code
    chans[6].alpha = 0.0
    st, thr, neg = qb.qnn_streamline([_as_tuple(c) for c in chans], ref.HWGQ_THRESHOLDS, lo, hi)
    assert st == 0
    assert any(neg) and not all(neg)
    for c, t, n in zip(chans, thr, neg):
        want_t, want_n = ref.streamline(c, ref.HWGQ_THRESHOLDS, lo, hi)
        assert t == want_t and bool(n) == want_n


def test_thresholds_reproduce_the_float_forward_pass_exhaustively(qb):
    rng = np.random.default_rng(21)
    lo, hi = -300, 300
    qthr = (-0.5, 0.0, 0.25, 0.8, 1.3, 2.0, 2.2)           # a 3-bit quantizer
    chans = [ref.random_params(rng, int(rng.integers(-50, 50)), 20.0) for _ in range(40)]
    st, thr, neg = qb.qnn_streamline([_as_tuple(c) for c in chans], qthr, lo, hi)
    assert st == 0
    for c, t, n in zip(chans, thr, neg):
        assert t == sorted(t)
        for x in range(lo, hi + 1):
            u = -x if n else x
            assert sum(1 for ti in t if u >= ti) == ref.float_forward(x, c, qthr)


def test_closed_form_on_exact_parameters(qb):
    # dyadic parameters: y = 0.5 * x - 1.25, thresholds {0, 0.75, 1.5} -> ceil((t + 1.25) / 0.5)
    ch = (1.0, 0.0, 0.5, 1.0, -1.25, 0.0, 1.0, 0)
    st, thr, neg = qb.qnn_streamline([ch], (0.0, 0.75, 1.5), -100, 100)
    assert st == 0 and neg == [0] and thr == [[3, 4, 6]]
    # a tie counts as passed: x = 4 gives y = 0.75 exactly -> code 2
    assert sum(1 for t in thr[0] if 4 >= t) == 2


def test_argument_errors(qb):
    ch = (1.0, 0.0, 1.0, 1.0, 0.0, 0.0, 1.0, 0)
    assert qb.qnn_streamline([ch], (1.0, 0.5), -10, 10)[0] == qb.QNN_ERR_INVALID_ARG      # not ascending
    assert qb.qnn_streamline([ch], (0.5,), 10, -10)[0] == qb.QNN_ERR_INVALID_ARG          # empty range
    bad = (1.0, 0.0, 1.0, 1.0, 0.0, 0.0, 0.0, 0)
    assert qb.qnn_streamline([bad], (0.5,), -10, 10)[0] == qb.QNN_ERR_INVALID_ARG         # sigma == 0
