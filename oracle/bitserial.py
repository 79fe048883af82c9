"""Algorithms 1 and 2 of the paper on Python integers (TEST INFRASTRUCTURE ONLY).

A slow restatement, for tiny matrices, of the bit-serial formulation of
Section 3.1: operands are split into bit planes, each plane is packed into
words along the depth dimension, and every pair of planes contributes
``+-2^(i+j) * popcount(W(r,d) & A(c,d))``.  It exists to pin the plain integer
GEMM oracle to the identity the paper states, and to spell out the reading of
the encodings the paper leaves open:

* UNSIGNED operand: every plane has weight +2^i.
* SIGNED (two's complement) operand: the most significant plane has weight
  -2^(bits-1) (Algorithm 2's sgnW / sgnA).
* BIPOLAR operand (1 bit, bit 1 -> +1, bit 0 -> -1): w = 2b - 1, so
  ``w.a = 2*(b.a) - sum(a)``; two bipolar operands give the XNOR-popcount form
  ``K - 2*popcount(a xor b)`` quoted in Section 3.1.
"""

WORDSIZE = 32

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2


def popcount(x: int) -> int:
    return bin(x).count("1")


def pack_planes(X, bits: int, enc: int):
    """X: list of rows of logical ints -> planes[i][row][d] of WORDSIZE-bit words.

    Element k of a row lands in word k // WORDSIZE at bit k % WORDSIZE; the
    last word is padded with zero bits."""
    planes = []
    for i in range(bits):
        plane = []
        for row in X:
            nwords = (len(row) + WORDSIZE - 1) // WORDSIZE
            words = [0] * nwords
            for k, v in enumerate(row):
                if enc == BIPOLAR:
                    assert v in (-1, 1)
                    bit = 1 if v == 1 else 0
                else:
                    bit = (int(v) >> i) & 1  # two's complement bit i
                words[k // WORDSIZE] |= bit << (k % WORDSIZE)
            plane.append(words)
        planes.append(plane)
    return planes


def binary_gemm(Wp, Ap, res, alpha: int):
    """Algorithm 1: res[r][c] += alpha * popcount(W(r,d) & A(c,d)) over depth words."""
    rows, cols = len(Wp), len(Ap)
    for r in range(rows):
        for c in range(cols):
            for d in range(len(Wp[r])):
                res[r][c] += alpha * popcount(Wp[r][d] & Ap[c][d])


def bitserial_gemm(W, At, w_bits, a_bits, w_enc, a_enc):
    """Algorithm 2 generalised to per-operand encodings. W[M][K], At[N][K] lists."""
    M, N = len(W), len(At)
    K = len(W[0]) if M else 0
    res = [[0] * N for _ in range(M)]

    if w_enc == BIPOLAR and a_enc == BIPOLAR:
        wp = pack_planes(W, 1, BIPOLAR)[0]
        ap = pack_planes(At, 1, BIPOLAR)[0]
        for r in range(M):
            for c in range(N):
                diff = sum(popcount(wp[r][d] ^ ap[c][d]) for d in range(len(wp[r])))
                res[r][c] = K - 2 * diff
        return res

    if w_enc == BIPOLAR or a_enc == BIPOLAR:
        # x = 2b - 1 on the bipolar side: x.y = 2*(b.y) - sum(y)
        if w_enc == BIPOLAR:
            Bp = pack_planes(W, 1, BIPOLAR)
            Op = pack_planes(At, a_bits, a_enc)
            o_bits, o_enc, other = a_bits, a_enc, At
        else:
            Bp = pack_planes(At, 1, BIPOLAR)
            Op = pack_planes(W, w_bits, w_enc)
            o_bits, o_enc, other = w_bits, w_enc, W
        for j in range(o_bits):
            sgn = -1 if (o_enc == SIGNED and j == o_bits - 1) else 1
            if w_enc == BIPOLAR:
                binary_gemm(Bp[0], Op[j], res, 2 * sgn * (1 << j))
            else:
                binary_gemm(Op[j], Bp[0], res, 2 * sgn * (1 << j))
        sums = [sum(int(v) for v in row) for row in other]
        for r in range(M):
            for c in range(N):
                res[r][c] -= sums[c] if w_enc == BIPOLAR else sums[r]
        return res

    Wp = pack_planes(W, w_bits, w_enc)
    Ap = pack_planes(At, a_bits, a_enc)
    for i in range(w_bits):
        for j in range(a_bits):
            sgn_w = -1 if (w_enc == SIGNED and i == w_bits - 1) else 1
            sgn_a = -1 if (a_enc == SIGNED and j == a_bits - 1) else 1
            binary_gemm(Wp[i], Ap[j], res, sgn_w * sgn_a * (1 << (i + j)))
    return res
