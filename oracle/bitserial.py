"""The bit-plane identity of Section 3.1 on Python integers (TEST INFRASTRUCTURE ONLY).

Section 3.1 (Algorithms 1-2) states that a few-bit integer product is a weighted sum of binary
products of bit planes, each binary product being a population count of an AND along the depth:

    W . A = sum_i sum_j c_i^W c_j^A * popcount(W[i] row  AND  A[j] column).

This module restates that identity for tiny matrices so that the plain integer GEMM oracle can be
pinned to it.  It is organised around the identity, not around a kernel: every row of a plane is
ONE arbitrary-precision Python integer (bit k = element k), so a binary dot product is a single
``popcount(x & y)`` with no word loop, and the plane weights come from a small table.  It also
spells out the reading of the encodings the paper leaves open:

* UNSIGNED operand of b bits: planes 0..b-1, weight +2^i each.
* SIGNED (two's complement): the same planes, the top one with weight -2^(b-1) (the sign rule of
  Algorithm 2).
* BIPOLAR (1 bit, bit 1 -> +1, bit 0 -> -1): x = 2 beta - 1 with beta the bit, so
  x . y = 2 (beta . y) - sum(y); two bipolar operands give the XNOR-popcount form
  K - 2 popcount(beta_x xor beta_y) quoted in Section 3.1.
"""

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2


def popcount(x: int) -> int:
    return bin(x).count("1")


def plane_weights(bits: int, enc: int):
    """Weight of each bit plane of an operand (a BIPOLAR operand has its bit as only plane)."""
    if enc == BIPOLAR:
        return [1]
    return [(-(1 << i) if (enc == SIGNED and i == bits - 1) else (1 << i)) for i in range(bits)]


def row_planes(row, bits: int, enc: int):
    """One Python integer per plane: bit k of plane i is bit i of element k (the bit itself for a
    BIPOLAR element: +1 -> 1, -1 -> 0)."""
    n_planes = 1 if enc == BIPOLAR else bits
    out = [0] * n_planes
    for k, v in enumerate(row):
        v = int(v)
        if enc == BIPOLAR:
            assert v in (-1, 1)
            out[0] |= (1 if v == 1 else 0) << k
        else:
            for i in range(bits):
                out[i] |= ((v >> i) & 1) << k            # >> on a negative int: two's-complement bits
    return out


def bitserial_dot(w_planes, a_planes, cw, ca, w_enc, a_enc, K: int, a_sum: int, w_sum: int) -> int:
    """One accumulator from the planes of a weight row and of an activation column."""
    if w_enc == BIPOLAR and a_enc == BIPOLAR:
        return K - 2 * popcount(w_planes[0] ^ a_planes[0])
    if w_enc == BIPOLAR:                                  # (2 beta - 1) . a = 2 (beta . a) - sum(a)
        return 2 * sum(c * popcount(w_planes[0] & aj) for c, aj in zip(ca, a_planes)) - a_sum
    if a_enc == BIPOLAR:
        return 2 * sum(c * popcount(wi & a_planes[0]) for c, wi in zip(cw, w_planes)) - w_sum
    return sum(ci * cj * popcount(wi & aj) for ci, wi in zip(cw, w_planes) for cj, aj in zip(ca, a_planes))


def bitserial_gemm(W, At, w_bits, a_bits, w_enc, a_enc):
    """acc[m][n] by the bit-plane identity.  W[M][K], At[N][K]: lists of rows of logical ints."""
    K = len(W[0]) if W else 0
    cw, ca = plane_weights(w_bits, w_enc), plane_weights(a_bits, a_enc)
    Wp = [row_planes(r, w_bits, w_enc) for r in W]
    Ap = [row_planes(r, a_bits, a_enc) for r in At]
    w_sums = [sum(int(v) for v in r) for r in W]
    a_sums = [sum(int(v) for v in r) for r in At]
    return [[bitserial_dot(Wp[m], Ap[n], cw, ca, w_enc, a_enc, K, a_sums[n], w_sums[m])
             for n in range(len(At))] for m in range(len(W))]
