"""ctypes access to the plain-C oracle (TEST INFRASTRUCTURE ONLY).

All arrays are LOGICAL integers (numpy int32, one element per value); packed
formats never reach the oracle, so the device-side packers are tested too.

Shapes follow the paper's (rows, depth, cols) = (M, K, N) convention of
Section 4.1, with the activation matrix held transposed as in Algorithm 1:
``W[M][K]``, ``At[N][K]``.
"""
import ctypes
import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        i64 = ctypes.c_int64
        p = ctypes.c_void_p
        lib.orc_num_threads.restype = ctypes.c_int
        lib.orc_dot_i64.restype = i64
        lib.orc_dot_i64.argtypes = [p, p, i64]
        lib.orc_gemm_i64.argtypes = [p, p, i64, i64, i64, p]
        lib.orc_threshold.argtypes = [p, p, i64, i64, i64, p]
        lib.orc_threshold_nhwc.argtypes = [p, p, i64, i64, i64, p]
        lib.orc_conv_direct.argtypes = [p, p] + [i64] * 9 + [p]
        lib.orc_maxpool.argtypes = [p] + [i64] * 6 + [p]
        for f in (lib.orc_gemm_i64, lib.orc_threshold, lib.orc_threshold_nhwc,
                  lib.orc_conv_direct, lib.orc_maxpool):
            f.restype = None
        _lib = lib
    return _lib


def _i32(x):
    x = np.ascontiguousarray(x, dtype=np.int32)
    return x


def _ptr(x):
    return x.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    """Threads the C oracle uses (OpenMP over output rows)."""
    return int(_load().orc_num_threads())


def gemm(W, At) -> np.ndarray:
    """acc[m][n] = sum_k W[m][k] * At[n][k] in int64 (Section 3.1)."""
    W, At = _i32(W), _i32(At)
    M, K = W.shape
    N, K2 = At.shape
    assert K == K2
    acc = np.empty((M, N), dtype=np.int64)
    _load().orc_gemm_i64(_ptr(W), _ptr(At), M, N, K, _ptr(acc))
    return acc


def dot_at(W, At, rows, cols) -> np.ndarray:
    """Accumulators at sampled (row, col) positions, one dot product each."""
    W, At = _i32(W), _i32(At)
    K = W.shape[1]
    lib = _load()
    out = np.empty(len(rows), dtype=np.int64)
    for i, (m, n) in enumerate(zip(rows, cols)):
        out[i] = lib.orc_dot_i64(_ptr(W[int(m)]), _ptr(At[int(n)]), K)
    return out


def threshold(acc, thr) -> np.ndarray:
    """codes[m][n] = #{i : thr[m][i] <= acc[m][n]} (Section 2.1.1)."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    thr = _i32(thr)
    M, N = acc.shape
    assert thr.shape[0] == M
    out = np.empty((M, N), dtype=np.int32)
    _load().orc_threshold(_ptr(acc), _ptr(thr), M, N, thr.shape[1], _ptr(out))
    return out


def qgemm(W, At, thr=None) -> np.ndarray:
    """Few-bit GEMM followed by the per-row threshold activation.

    Returns codes [M][N] (int32), or the raw accumulators (int64, checked to
    fit int32) when ``thr`` is None."""
    acc = gemm(W, At)
    assert acc.size == 0 or (acc.min() >= -2**31 and acc.max() < 2**31)
    if thr is None:
        return acc
    return threshold(acc, thr)


def conv_direct(In, Wt, stride: int, pad: int) -> np.ndarray:
    """Direct convolution on channels-last tensors, int64 accumulators.

    In [B][H][W][C], Wt [OC][KH][KW][C] -> acc [B][OH][OW][OC]."""
    In, Wt = _i32(In), _i32(Wt)
    B, H, Wd, C = In.shape
    OC, KH, KW, C2 = Wt.shape
    assert C == C2
    OH = (H + 2 * pad - KH) // stride + 1
    OW = (Wd + 2 * pad - KW) // stride + 1
    acc = np.empty((B, OH, OW, OC), dtype=np.int64)
    _load().orc_conv_direct(_ptr(In), _ptr(Wt), B, H, Wd, C, OC, KH, KW,
                            stride, pad, _ptr(acc))
    return acc


def threshold_nhwc(acc, thr) -> np.ndarray:
    """Per-channel T(x, t) on a channels-last accumulator tensor [..., OC]."""
    acc = np.ascontiguousarray(acc, dtype=np.int64)
    thr = _i32(thr)
    OC = acc.shape[-1]
    assert thr.shape[0] == OC
    P = acc.size // OC if OC else 0
    out = np.empty(acc.shape, dtype=np.int32)
    _load().orc_threshold_nhwc(_ptr(acc), _ptr(thr), P, OC, thr.shape[1], _ptr(out))
    return out


def qconv(In, Wt, thr, stride: int, pad: int) -> np.ndarray:
    """Convolution + per-channel threshold activation; raw int64 if thr is None."""
    acc = conv_direct(In, Wt, stride, pad)
    assert acc.size == 0 or (acc.min() >= -2**31 and acc.max() < 2**31)
    if thr is None:
        return acc
    return threshold_nhwc(acc, thr)


def maxpool(In, k: int, s: int) -> np.ndarray:
    """k x k / stride s max-pool, no padding, floor; channels-last int32."""
    In = _i32(In)
    B, H, Wd, C = In.shape
    OH = (H - k) // s + 1
    OW = (Wd - k) // s + 1
    out = np.empty((B, OH, OW, C), dtype=np.int32)
    _load().orc_maxpool(_ptr(In), B, H, Wd, C, k, s, _ptr(out))
    return out
