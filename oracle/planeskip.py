"""Bit-plane products that leave out the low-order plane pairs (TEST INFRASTRUCTURE ONLY).

The paper's conclusion names, as future work, approximate computing that considers only the
contributions of the higher-order bits.  With the bit-plane identity of Section 3.1,

    W . A = sum_i sum_j c_i c_j 2^(i+j) W[i] . A[j],

that is the same sum restricted to the pairs with i + j >= skip:

    approx(W, A; skip) = sum_{i + j >= skip} c_i c_j 2^(i+j) W[i] . A[j].

Planes: an UNSIGNED or SIGNED operand of b bits has planes 0..b-1 of 0/1 values (bit i of the
two's-complement pattern), with c = -1 on the top plane of a SIGNED operand and +1 elsewhere
(Algorithm 2's sgnW, sgnA); a BIPOLAR operand is one plane (index 0) of -1/+1 values, c = +1.
skip = 0 is the exact product.  What is left out is bounded by

    |W . A - approx| <= K * sum_{i + j < skip} 2^(i+j)      (every plane product is at most K),

with equality for all-ones UNSIGNED operands.

Each plane product is a numpy int64 matrix product; nothing is packed, blocked or reordered.
"""
import numpy as np

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2


def planes(X, bits: int, enc: int):
    """[(coefficient c_i * 2^i, plane matrix int64)] of a logical integer matrix."""
    X = np.asarray(X, dtype=np.int64)
    if enc == BIPOLAR:
        assert bits == 1 and np.isin(X, (-1, 1)).all()
        return [(1, X)]
    out = []
    for i in range(bits):
        sign = -1 if (enc == SIGNED and i == bits - 1) else 1
        out.append((sign * (1 << i), (X >> i) & 1))          # >> on negative int64 is arithmetic: two's complement bits
    return out


def gemm(W, At, w_bits, a_bits, w_enc, a_enc, skip: int) -> np.ndarray:
    """approx(W, A; skip)[m][n] in int64; W[M][K], At[N][K]."""
    W = np.asarray(W, dtype=np.int64)
    At = np.asarray(At, dtype=np.int64)
    acc = np.zeros((W.shape[0], At.shape[0]), dtype=np.int64)
    for i, (cw, Wi) in enumerate(planes(W, w_bits, w_enc)):
        for j, (ca, Aj) in enumerate(planes(At, a_bits, a_enc)):
            if i + j >= skip:
                acc += cw * ca * (Wi @ Aj.T)
    return acc


def error_bound(K: int, w_bits, a_bits, w_enc, a_enc, skip: int) -> int:
    """K * sum of 2^(i+j) over the pairs left out."""
    nw = 1 if w_enc == BIPOLAR else w_bits
    na = 1 if a_enc == BIPOLAR else a_bits
    return K * sum(1 << (i + j) for i in range(nw) for j in range(na) if i + j < skip)
