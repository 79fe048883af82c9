"""Host-side decoding of the library's packed formats, written independently of
both the CUDA kernels and the oracle (numpy only), so that parity is checked on
logical values."""
import numpy as np

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2


def round_up(x, m):
    return (x + m - 1) // m * m


def unpack_planes(buf: np.ndarray, bits: int, rows: int, K: int, enc: int) -> np.ndarray:
    """uint32 [bits][rows][ceil(K/32)] -> logical int32 [rows][K]; also checks zero pad bits."""
    kw = (K + 31) // 32
    words = buf.view(np.uint32)[: bits * rows * kw].reshape(bits, rows, kw)
    shifts = np.arange(32, dtype=np.uint32)
    allbits = ((words[..., None] >> shifts) & 1).reshape(bits, rows, kw * 32)
    assert not allbits[:, :, K:].any(), "pad bits must be zero"
    b = allbits[:, :, :K].astype(np.int32)
    if enc == BIPOLAR:
        return 2 * b[0] - 1
    val = np.zeros((rows, K), dtype=np.int32)
    for i in range(bits):
        wgt = -(1 << i) if (enc == SIGNED and i == bits - 1) else (1 << i)
        val += wgt * b[i]
    return val


def unpack_int8(buf: np.ndarray, rows: int, K: int, enc: int) -> np.ndarray:
    ld = round_up(K, 16)
    m = buf.view(np.uint8)[: rows * ld].reshape(rows, ld)
    assert not m[:, K:].any(), "pad bytes must be zero"
    m = m[:, :K]
    return (m if enc == UNSIGNED else m.view(np.int8)).astype(np.int32)


def unpack_fields(buf: np.ndarray, bits: int, rows: int, K: int, enc: int) -> np.ndarray:
    """QNN_FMT_FIELDS [rows][ldf] bytes -> logical int32 [rows][K]; also checks zero pad fields.
    Element k sits in byte 32 g + j at bit f s, g = k // (32 S), s = (k % (32 S)) // 32, j = k % 32."""
    f = 1 if bits == 1 else (2 if bits == 2 else 4)
    S = 8 // f
    groups = (K + 32 * S - 1) // (32 * S)
    ldf = 32 * groups
    m = buf.view(np.uint8)[: rows * ldf].reshape(rows, groups, 32).astype(np.int32)
    fields = np.stack([(m >> (f * s)) & ((1 << f) - 1) for s in range(S)], axis=2)     # [rows][g][s][j]
    u = fields.reshape(rows, groups * 32 * S)
    assert not u[:, K:].any(), "pad fields must be zero"
    u = u[:, :K]
    if enc == BIPOLAR:
        return 2 * u - 1
    if enc == SIGNED:
        return u - (1 << (bits - 1))
    return u


def unpack_operand(buf, fmt, bits, rows, K, enc):
    if fmt == 2:
        return unpack_fields(buf, bits, rows, K, enc)
    return unpack_planes(buf, bits, rows, K, enc) if fmt == 0 else unpack_int8(buf, rows, K, enc)


def decode_out(buf: np.ndarray, out_fmt, out_bits: int, N: int, M: int, raw: bool) -> np.ndarray:
    """Library output -> logical [N][M] int64."""
    if raw:
        return buf.view(np.int32)[: N * M].reshape(N, M).astype(np.int64)
    if out_fmt == 1:
        return unpack_int8(buf, N, M, UNSIGNED).astype(np.int64)
    return unpack_planes(buf, out_bits, N, M, UNSIGNED).astype(np.int64)


def host_pack_planes(X: np.ndarray, bits: int, enc: int) -> np.ndarray:
    """logical [rows][K] -> uint32 [bits][rows][ceil(K/32)] (test-side packer)."""
    rows, K = X.shape
    kw = (K + 31) // 32
    out = np.zeros((bits, rows, kw), dtype=np.uint32)
    padded = np.zeros((rows, kw * 32), dtype=np.int64)
    padded[:, :K] = X
    for i in range(bits):
        if enc == BIPOLAR:
            b = np.zeros((rows, kw * 32), dtype=np.uint32)
            b[:, :K] = (X > 0)
        else:
            b = ((padded >> i) & 1).astype(np.uint32)
            b[:, K:] = 0
        out[i] = (b.reshape(rows, kw, 32) << np.arange(32, dtype=np.uint32)).sum(-1).astype(np.uint32)
    return out
