"""ctypes binding of the C ABI in ``include/qnn.h`` (argument marshalling only).

The ``qnn_*`` functions mirror the C entry points one to one and return the
status code.  Pointer arguments accept a ``torch.Tensor`` (its ``data_ptr()``
is passed; the tensor must be contiguous and live on the GPU), an ``int``
address, or ``None``.  ``stream=None`` means torch's current CUDA stream.

The helpers below them (``pack``, ``qgemm``, ``qconv``, ...) only allocate the
output tensor with torch, build the descriptor and call the entry point; every
step of the computation runs in the library's kernels.  There is no fallback:
if the shared library is missing, importing this module raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqnn_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build it with `python -m paper_1709_04060_b200.build` "
        "(there is no CPU fallback)")
_lib = ctypes.CDLL(LIB_PATH)

QNN_OK = 0
QNN_ERR_INVALID_ARG, QNN_ERR_UNSUPPORTED, QNN_ERR_ALIGNMENT = -1, -2, -3
QNN_ERR_WORKSPACE, QNN_ERR_CUDA, QNN_ERR_DEVICE_TIMEOUT = -4, -5, -6
QNN_ENC_UNSIGNED, QNN_ENC_SIGNED, QNN_ENC_BIPOLAR = 0, 1, 2
QNN_FMT_BITPLANES, QNN_FMT_INT8, QNN_FMT_FIELDS = 0, 1, 2
QNN_PATH_AUTO, QNN_PATH_BITSERIAL, QNN_PATH_TCGEN05_I8 = 0, 1, 2

EXPORTS = (
    "qnn_packed_ld", "qnn_packed_bytes", "qnn_pack", "qnn_planes_to_int8", "qnn_gemm_workspace_bytes",
    "qnn_gemm_out_bytes", "qnn_qgemm", "qnn_qgemm_kernel", "qnn_conv_out_h", "qnn_conv_out_w",
    "qnn_conv_lowered_k", "qnn_conv_lowered_bytes", "qnn_conv_workspace_bytes",
    "qnn_conv_out_bytes", "qnn_im2col", "qnn_qconv", "qnn_qconv_static", "qnn_maxpool",
    "qnn_streamline", "qnn_peak_mma_i8", "qnn_peak_popc", "qnn_peak_popc_sink_bytes", "qnn_validate_thresholds", "qnn_device_status", "qnn_launch_count",
    "qnn_status_string", "qnn_version",
)


class qnn_pack_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("rows", "K", "bits", "enc", "fmt")]


class qnn_gemm_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "M", "N", "K", "w_bits", "a_bits", "out_bits", "w_enc", "a_enc",
        "w_fmt", "a_fmt", "out_fmt", "path", "skip_planes")]


class qnn_conv_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "B", "H", "W", "C", "in_pitch", "OC", "KH", "KW", "stride", "pad",
        "w_bits", "a_bits", "out_bits", "w_enc", "a_enc", "fmt", "out_fmt", "path")]


class qnn_channel_params(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("a_prev", "b_prev", "alpha", "gamma", "beta", "mu", "sigma")] + \
               [("row_sum", ctypes.c_longlong)]


class qnn_pool_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("B", "H", "W", "C", "k", "stride", "bits", "fmt")]


_vp, _sz, _ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
_P = ctypes.POINTER
_lib.qnn_packed_ld.restype = _sz
_lib.qnn_packed_ld.argtypes = [_ci, _ci]
_lib.qnn_packed_bytes.restype = _sz
_lib.qnn_packed_bytes.argtypes = [_P(qnn_pack_desc)]
_lib.qnn_pack.restype = _ci
_lib.qnn_pack.argtypes = [_P(qnn_pack_desc), _vp, _vp, _vp]
_lib.qnn_planes_to_int8.argtypes = [_P(qnn_pack_desc), _vp, _vp, _vp]
_lib.qnn_planes_to_int8.restype = _ci
_lib.qnn_gemm_workspace_bytes.restype = _sz
_lib.qnn_gemm_workspace_bytes.argtypes = [_P(qnn_gemm_desc)]
_lib.qnn_gemm_out_bytes.restype = _sz
_lib.qnn_gemm_out_bytes.argtypes = [_P(qnn_gemm_desc), _ci]
_lib.qnn_qgemm_kernel.restype = _ci
_lib.qnn_qgemm_kernel.argtypes = [_P(qnn_gemm_desc), _ci]
_lib.qnn_qgemm.restype = _ci
_lib.qnn_qgemm.argtypes = [_P(qnn_gemm_desc), _vp, _vp, _vp, _vp, _vp, _sz, _vp]
for _n in ("qnn_conv_out_h", "qnn_conv_out_w", "qnn_conv_lowered_k"):
    getattr(_lib, _n).restype = _ci
    getattr(_lib, _n).argtypes = [_P(qnn_conv_desc)]
for _n in ("qnn_conv_lowered_bytes", "qnn_conv_workspace_bytes"):
    getattr(_lib, _n).restype = _sz
    getattr(_lib, _n).argtypes = [_P(qnn_conv_desc)]
_lib.qnn_conv_out_bytes.restype = _sz
_lib.qnn_conv_out_bytes.argtypes = [_P(qnn_conv_desc), _ci]
_lib.qnn_im2col.restype = _ci
_lib.qnn_im2col.argtypes = [_P(qnn_conv_desc), _vp, _vp, _vp]
_lib.qnn_qconv.restype = _ci
_lib.qnn_qconv.argtypes = [_P(qnn_conv_desc), _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.qnn_qconv_static.restype = _ci
_lib.qnn_qconv_static.argtypes = [_P(qnn_conv_desc), _vp, _vp, _vp, _vp, _vp]
_lib.qnn_maxpool.restype = _ci
_lib.qnn_maxpool.argtypes = [_P(qnn_pool_desc), _vp, _vp, _vp]
_lib.qnn_streamline.restype = _ci
_lib.qnn_streamline.argtypes = [_P(qnn_channel_params), _ci, _P(ctypes.c_double), _ci, ctypes.c_longlong,
                                ctypes.c_longlong, _P(ctypes.c_int32), _P(ctypes.c_uint8)]
_lib.qnn_peak_mma_i8.restype = _ci
_lib.qnn_peak_mma_i8.argtypes = [_ci, _ci, _ci, _P(ctypes.c_double), _vp]
_lib.qnn_peak_popc.restype = _ci
_lib.qnn_peak_popc.argtypes = [_ci, _vp, _sz, _P(ctypes.c_double), _vp]
_lib.qnn_peak_popc_sink_bytes.restype = _sz
_lib.qnn_peak_popc_sink_bytes.argtypes = []
_lib.qnn_validate_thresholds.restype = _ci
_lib.qnn_validate_thresholds.argtypes = [_vp, _ci, _ci, _P(_ci), _vp]
_lib.qnn_device_status.restype = _ci
_lib.qnn_device_status.argtypes = [_P(_ci)]
_lib.qnn_launch_count.restype = ctypes.c_ulonglong
_lib.qnn_launch_count.argtypes = []
_lib.qnn_status_string.restype = ctypes.c_char_p
_lib.qnn_status_string.argtypes = [_ci]
_lib.qnn_version.restype = _ci
_lib.qnn_version.argtypes = []


class QnnError(RuntimeError):
    def __init__(self, status):
        self.status = status
        super().__init__(f"qnn status {status}: {qnn_status_string(status)}")


def check(status: int) -> None:
    if status != QNN_OK:
        raise QnnError(status)


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, torch.Tensor):
        assert x.is_contiguous(), "device buffers must be contiguous"
        return x.data_ptr()
    raise TypeError(type(x))


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return int(stream)


# ---- one-to-one entry points -------------------------------------------------
def qnn_version() -> int:
    return _lib.qnn_version()


def qnn_status_string(s: int) -> str:
    return _lib.qnn_status_string(s).decode()


def qnn_launch_count() -> int:
    return int(_lib.qnn_launch_count())


def qnn_packed_ld(K: int, fmt: int) -> int:
    return int(_lib.qnn_packed_ld(K, fmt))


def qnn_packed_bytes(d: qnn_pack_desc) -> int:
    return int(_lib.qnn_packed_bytes(ctypes.byref(d)))


def qnn_pack(d, logical, packed, stream=None) -> int:
    return _lib.qnn_pack(ctypes.byref(d), _ptr(logical), _ptr(packed), _stream(stream))


def qnn_planes_to_int8(d, planes, containers, stream=None) -> int:
    return _lib.qnn_planes_to_int8(ctypes.byref(d), _ptr(planes), _ptr(containers), _stream(stream))


def qnn_gemm_workspace_bytes(d) -> int:
    return int(_lib.qnn_gemm_workspace_bytes(ctypes.byref(d)))


def qnn_gemm_out_bytes(d, has_thresholds: bool) -> int:
    return int(_lib.qnn_gemm_out_bytes(ctypes.byref(d), int(has_thresholds)))


QNN_KERNEL_TENSOR, QNN_KERNEL_TENSOR_CTA_PAIR, QNN_KERNEL_BYTES_FEW_COLUMNS = 1, 2, 3
QNN_KERNEL_PLANES_FEW_COLUMNS, QNN_KERNEL_PLANES_TILED, QNN_KERNEL_FIELDS_FEW_COLUMNS = 4, 5, 6


def qnn_qgemm_kernel(d, has_thresholds: bool = True) -> int:
    """The kernel qnn_qgemm would run for this problem (a QNN_KERNEL_* value, or a negative status)."""
    return _lib.qnn_qgemm_kernel(ctypes.byref(d), int(has_thresholds))


def qnn_qgemm(d, W, A, thr, out, workspace=None, workspace_bytes=0, stream=None) -> int:
    return _lib.qnn_qgemm(ctypes.byref(d), _ptr(W), _ptr(A), _ptr(thr), _ptr(out),
                          _ptr(workspace), workspace_bytes, _stream(stream))


def qnn_conv_out_h(d) -> int:
    return _lib.qnn_conv_out_h(ctypes.byref(d))


def qnn_conv_out_w(d) -> int:
    return _lib.qnn_conv_out_w(ctypes.byref(d))


def qnn_conv_lowered_k(d) -> int:
    return _lib.qnn_conv_lowered_k(ctypes.byref(d))


def qnn_conv_lowered_bytes(d) -> int:
    return int(_lib.qnn_conv_lowered_bytes(ctypes.byref(d)))


def qnn_conv_workspace_bytes(d) -> int:
    return int(_lib.qnn_conv_workspace_bytes(ctypes.byref(d)))


def qnn_conv_out_bytes(d, has_thresholds: bool) -> int:
    return int(_lib.qnn_conv_out_bytes(ctypes.byref(d), int(has_thresholds)))


def qnn_im2col(d, inp, lowered, stream=None) -> int:
    return _lib.qnn_im2col(ctypes.byref(d), _ptr(inp), _ptr(lowered), _stream(stream))


def qnn_qconv(d, Wpacked, inp, thr, out, workspace, workspace_bytes, stream=None) -> int:
    return _lib.qnn_qconv(ctypes.byref(d), _ptr(Wpacked), _ptr(inp), _ptr(thr), _ptr(out),
                          _ptr(workspace), workspace_bytes, _stream(stream))


QNN_QCONV_STATIC_MAX_BYTES = 16 << 20


def qnn_qconv_static(d, Wpacked, inp, thr, out, stream=None) -> int:
    """qnn_qconv without a workspace argument: the lowered matrix goes into a fixed
    array inside the library, so the call allocates nothing (see include/qnn.h)."""
    return _lib.qnn_qconv_static(ctypes.byref(d), _ptr(Wpacked), _ptr(inp), _ptr(thr), _ptr(out),
                                 _stream(stream))


def qnn_maxpool(d, inp, out, stream=None) -> int:
    return _lib.qnn_maxpool(ctypes.byref(d), _ptr(inp), _ptr(out), _stream(stream))


def qnn_streamline(channels, qthr, acc_lo: int, acc_hi: int):
    """Host-only.  channels: sequence of qnn_channel_params (or 8-tuples in field order);
    qthr: the quantizer's float thresholds.  Returns (status, thresholds [channels][n_thr] as
    nested lists of ints, negate flags)."""
    arr = (qnn_channel_params * len(channels))(*[c if isinstance(c, qnn_channel_params) else qnn_channel_params(*c)
                                                  for c in channels])
    n = len(qthr)
    q = (ctypes.c_double * n)(*[float(t) for t in qthr])
    out = (ctypes.c_int32 * (len(channels) * n))()
    neg = (ctypes.c_uint8 * len(channels))()
    st = _lib.qnn_streamline(arr, len(channels), q, n, int(acc_lo), int(acc_hi), out, neg)
    thr = [[out[c * n + i] for i in range(n)] for c in range(len(channels))]
    return st, thr, [int(v) for v in neg]


def qnn_peak_mma_i8(pair: int, n: int, mmas_per_cta: int, stream=None):
    """Launches the tensor-pipe issue-rate microbenchmark; returns (status, integer ops of the launch)."""
    ops = ctypes.c_double(0.0)
    st = _lib.qnn_peak_mma_i8(int(pair), int(n), int(mmas_per_cta), ctypes.byref(ops), _stream(stream))
    return st, ops.value


def qnn_peak_popc_sink_bytes() -> int:
    return int(_lib.qnn_peak_popc_sink_bytes())


def qnn_peak_popc(iters: int, sink, stream=None):
    """Launches the POPC issue-rate microbenchmark; returns (status, population counts of the launch)."""
    n = ctypes.c_double(0.0)
    st = _lib.qnn_peak_popc(int(iters), _ptr(sink), sink.numel() * sink.element_size(), ctypes.byref(n),
                            _stream(stream))
    return st, n.value


def qnn_validate_thresholds(thr, M: int, n_thr: int, stream=None):
    """Returns (status, number of unsorted rows).  Synchronises the stream."""
    n_bad = _ci(0)
    st = _lib.qnn_validate_thresholds(_ptr(thr), M, n_thr, ctypes.byref(n_bad), _stream(stream))
    return st, n_bad.value


def qnn_device_status():
    """Returns (status, device status word).  Synchronises the device."""
    v = _ci(0)
    st = _lib.qnn_device_status(ctypes.byref(v))
    return st, v.value


# ---- allocation helpers (marshalling only) -----------------------------------
def _dev_bytes(n: int) -> torch.Tensor:
    return torch.empty(max(int(n), 16), dtype=torch.uint8, device="cuda")


def to_device_logical(x, enc: int) -> torch.Tensor:
    """numpy/torch logical integers -> contiguous device bytes (uint8 for
    UNSIGNED, int8 otherwise), the packer's input format."""
    t = torch.as_tensor(x)
    t = t.to(torch.uint8 if enc == QNN_ENC_UNSIGNED else torch.int8)
    return t.contiguous().cuda()


def pack(logical: torch.Tensor, bits: int, enc: int, fmt: int, stream=None) -> torch.Tensor:
    """Pack a [rows][K] device byte matrix; returns the packed device buffer (uint8 view)."""
    rows, K = logical.shape
    d = qnn_pack_desc(rows, K, bits, enc, fmt)
    out = _dev_bytes(qnn_packed_bytes(d))
    check(qnn_pack(d, logical, out, stream))
    return out


def gemm_desc(M, N, K, w_bits, a_bits, out_bits, w_enc, a_enc, fmt, out_fmt,
              path=QNN_PATH_AUTO, skip_planes=0) -> qnn_gemm_desc:
    return qnn_gemm_desc(M, N, K, w_bits, a_bits, out_bits, w_enc, a_enc, fmt, fmt, out_fmt, path, skip_planes)


def qgemm(d: qnn_gemm_desc, W, A, thr, out=None, stream=None) -> torch.Tensor:
    """Fused GEMM + threshold; returns the output buffer (uint8 view, or int32
    [N][M] when thr is None)."""
    if out is None:
        out = _dev_bytes(qnn_gemm_out_bytes(d, thr is not None))
    # the optional workspace starts with flag words that must be zero before the first call
    ws_bytes = qnn_gemm_workspace_bytes(d)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None
    check(qnn_qgemm(d, W, A, thr, out, ws, ws_bytes, stream))
    if thr is None:
        return out[: d.N * d.M * 4].view(torch.int32).view(d.N, d.M)
    return out


def conv_weight_rows(d: qnn_conv_desc, Wt):
    """Logical filters [OC][KH][KW][C] (numpy) laid out as the rows [OC][qnn_conv_lowered_k]
    that `pack` expects for this convolution: per-pixel padding to 32 channels for bit planes,
    per-filter-row padding to 16 bytes for 8-bit maps whose C is not a multiple of 16."""
    import numpy as np
    OC, KH, KW, C = Wt.shape
    K = qnn_conv_lowered_k(d)
    if d.fmt == QNN_FMT_BITPLANES:
        cp = (C + 31) // 32 * 32
        rows = np.zeros((OC, KH * KW, cp), dtype=Wt.dtype)
        rows[:, :, :C] = Wt.reshape(OC, KH * KW, C)
    elif C % 16 == 0:
        rows = Wt
    else:
        rows = np.zeros((OC, KH, K // KH), dtype=Wt.dtype)
        rows[:, :, :KW * C] = Wt.reshape(OC, KH, KW * C)
    return np.ascontiguousarray(rows.reshape(OC, K))


def qconv(d: qnn_conv_desc, Wpacked, inp, thr, out=None, workspace=None, stream=None) -> torch.Tensor:
    if out is None:
        out = _dev_bytes(qnn_conv_out_bytes(d, thr is not None))
    ws_bytes = qnn_conv_workspace_bytes(d)
    if workspace is None:
        workspace = _dev_bytes(ws_bytes)
    check(qnn_qconv(d, Wpacked, inp, thr, out, workspace, workspace.numel(), stream))
    return out
