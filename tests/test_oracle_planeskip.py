"""Pins of the plane-skipping oracle (the paper's conclusion: approximate products from the
higher-order bit planes only): the exact product at skip = 0 (the C oracle, an independent
routine), closed forms, brute force over all operand values, and the error bound."""
import itertools

import numpy as np
import pytest

from oracle import oracle as orc
from oracle import planeskip as ps
from paper_1709_04060_b200 import synth

ENCS = {"u": synth.UNSIGNED, "s": synth.SIGNED, "b": synth.BIPOLAR}


def _case(seed, M, N, K, w, a, w_enc, a_enc):
    return synth.gemm_case(seed, M, N, K, w, a, w_enc, a_enc)


@pytest.mark.parametrize("w,a", list(itertools.product((1, 2, 3, 4), repeat=2)))
def test_skip_zero_is_the_exact_product(w, a):
    for w_enc, a_enc in itertools.product((0, 1), repeat=2):
        c = _case(900 + 10 * w + a, 7, 5, 70, w, a, w_enc, a_enc)
        assert np.array_equal(ps.gemm(c.W, c.At, w, a, w_enc, a_enc, 0), orc.gemm(c.W, c.At))
    if w == 1:
        c = _case(950 + a, 6, 4, 45, 1, a, synth.BIPOLAR, synth.UNSIGNED)
        assert np.array_equal(ps.gemm(c.W, c.At, 1, a, synth.BIPOLAR, synth.UNSIGNED, 0), orc.gemm(c.W, c.At))


def test_everything_skipped_gives_zero():
    c = _case(960, 4, 3, 33, 3, 2, synth.SIGNED, synth.UNSIGNED)
    assert not ps.gemm(c.W, c.At, 3, 2, synth.SIGNED, synth.UNSIGNED, 4).any()       # max i + j = 3
    assert ps.gemm(c.W, c.At, 3, 2, synth.SIGNED, synth.UNSIGNED, 3).any()


@pytest.mark.parametrize("w_enc", [synth.UNSIGNED, synth.BIPOLAR])
@pytest.mark.parametrize("a_bits,a_enc", [(2, 0), (4, 0), (3, 1), (4, 1)])
def test_one_weight_plane_is_the_product_with_truncated_activations(w_enc, a_bits, a_enc):
    """With a single weight plane only the activation's plane index counts, so the result is the
    exact product with the activations' low `skip` bits cleared (floor to a multiple of 2^skip,
    also for negative two's-complement values)."""
    c = _case(970 + a_bits, 9, 6, 100, 1, a_bits, w_enc, a_enc)
    for skip in range(a_bits + 1):
        # all planes gone: zero (the floor form would keep the sign of a negative value)
        trunc = (c.At >> skip) << skip if skip < a_bits else np.zeros_like(c.At)
        assert np.array_equal(ps.gemm(c.W, c.At, 1, a_bits, w_enc, a_enc, skip), orc.gemm(c.W, trunc))
        # and with the roles exchanged
        assert np.array_equal(ps.gemm(c.At, c.W, a_bits, 1, a_enc, w_enc, skip), orc.gemm(trunc, c.W))


@pytest.mark.parametrize("w,a", [(2, 2), (3, 2), (2, 4)])
def test_brute_force_over_all_scalar_operands(w, a):
    """K = 1: every pair of operand values against the double loop over their bits."""
    for w_enc, a_enc in itertools.product((0, 1), repeat=2):
        wl, wh = synth.value_range(w, w_enc)
        al, ah = synth.value_range(a, a_enc)
        for skip in range(w + a):
            for x, y in itertools.product(range(wl, wh + 1), range(al, ah + 1)):
                want = 0
                for i in range(w):
                    for j in range(a):
                        if i + j < skip:
                            continue
                        ci = -1 if (w_enc == 1 and i == w - 1) else 1
                        cj = -1 if (a_enc == 1 and j == a - 1) else 1
                        want += ci * cj * (((x >> i) & 1) * ((y >> j) & 1) << (i + j))
                got = ps.gemm([[x]], [[y]], w, a, w_enc, a_enc, skip)[0, 0]
                assert got == want, (w_enc, a_enc, skip, x, y)


def test_error_bound_holds_and_is_attained_by_all_ones():
    K = 200
    for (w, a) in ((2, 2), (4, 4), (3, 1)):
        c = _case(980 + w, 8, 8, K, w, a, synth.SIGNED, synth.UNSIGNED)
        exact = orc.gemm(c.W, c.At)
        for skip in range(w + a):
            bound = ps.error_bound(K, w, a, synth.SIGNED, synth.UNSIGNED, skip)
            err = np.abs(exact - ps.gemm(c.W, c.At, w, a, synth.SIGNED, synth.UNSIGNED, skip))
            assert err.max() <= bound
        W1 = np.full((3, K), (1 << w) - 1); A1 = np.full((2, K), (1 << a) - 1)
        for skip in range(w + a):
            err = orc.gemm(W1, A1) - ps.gemm(W1, A1, w, a, 0, 0, skip)
            assert (err == ps.error_bound(K, w, a, 0, 0, skip)).all()


def test_a_planted_mistake_is_caught():
    """Using i + j > skip instead of >= changes results the pins above would reject."""
    c = _case(990, 5, 5, 64, 2, 2, synth.UNSIGNED, synth.UNSIGNED)
    right = ps.gemm(c.W, c.At, 2, 2, 0, 0, 1)
    wrong = np.zeros_like(right)
    for i, (cw, Wi) in enumerate(ps.planes(c.W, 2, 0)):
        for j, (ca, Aj) in enumerate(ps.planes(c.At, 2, 0)):
            if i + j > 1:
                wrong += cw * ca * (Wi @ Aj.T)
    assert not np.array_equal(right, wrong)
