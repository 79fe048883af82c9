"""CPU-side checks of the C ABI: the shared library loads, exports every symbol the
header declares, and its host-only logic (size queries, argument validation)
behaves as documented.  No kernel is launched here."""
import ctypes
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def qb():
    import __graft_entry__ as ge
    ge.build()
    from paper_1709_04060_b200 import binding
    return binding


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "qnn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qnn_[a-z0-9_]+)\s*\(", text)))


def test_exports_match_header(qb):
    declared = _declared_functions()
    assert len(declared) >= 20
    lib = ctypes.CDLL(qb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in qnn.h but not exported"
    assert sorted(qb.EXPORTS) == [d for d in declared if d in qb.EXPORTS]
    missing_in_binding = [d for d in declared if d not in qb.EXPORTS]
    assert missing_in_binding == [], missing_in_binding
    for name in declared:
        assert hasattr(qb, name), f"binding lacks {name}"


def test_no_oracle_or_cpu_fallback_in_product():
    """The product package must not reference the oracle."""
    pkg = os.path.join(ROOT, "paper_1709_04060_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src, f
                assert "qnn_oracle" not in src, f


def test_version_and_status_strings(qb):
    assert qb.qnn_version() >= 100
    assert qb.qnn_status_string(0) == "ok"
    for s in range(-6, 0):
        assert qb.qnn_status_string(s) not in ("ok", "unknown status")


def test_packed_sizes(qb):
    assert qb.qnn_packed_ld(576, qb.QNN_FMT_BITPLANES) == 18
    assert qb.qnn_packed_ld(577, qb.QNN_FMT_BITPLANES) == 19
    assert qb.qnn_packed_ld(363, qb.QNN_FMT_INT8) == 368
    # config-1 operand sizes: W 1 x 64 x 18 words, A 2 x 256 x 18 words
    assert qb.qnn_packed_bytes(qb.qnn_pack_desc(64, 576, 1, 2, 0)) == 4608
    assert qb.qnn_packed_bytes(qb.qnn_pack_desc(256, 576, 2, 0, 0)) == 36864
    assert qb.qnn_packed_bytes(qb.qnn_pack_desc(256, 576, 2, 0, 1)) == 256 * 576
    assert qb.qnn_packed_bytes(qb.qnn_pack_desc(0, 576, 2, 0, 1)) == 0


def test_gemm_out_sizes(qb):
    d = qb.gemm_desc(64, 256, 576, 1, 2, 2, 2, 0, 0, qb.QNN_FMT_INT8)
    assert qb.qnn_gemm_out_bytes(d, True) == 256 * 64
    assert qb.qnn_gemm_out_bytes(d, False) == 256 * 64 * 4
    d = qb.gemm_desc(70, 10, 64, 1, 2, 2, 2, 0, 0, qb.QNN_FMT_BITPLANES)
    assert qb.qnn_gemm_out_bytes(d, True) == 2 * 10 * 3 * 4
    d = qb.gemm_desc(70, 10, 64, 1, 2, 2, 2, 0, 0, qb.QNN_FMT_INT8)
    assert qb.qnn_gemm_out_bytes(d, True) == 10 * 80


def test_conv_geometry(qb):
    # AlexNet conv2: 27x27x96, 5x5 pad 2 -> lowered (256, 2400, 729)
    d = qb.qnn_conv_desc(1, 27, 27, 96, 0, 256, 5, 5, 1, 2, 1, 2, 2, 2, 0, 0, 1, 0)
    assert qb.qnn_conv_out_h(d) == 27 and qb.qnn_conv_out_w(d) == 27
    assert qb.qnn_conv_lowered_k(d) == 2400
    assert qb.qnn_conv_lowered_bytes(d) == 2 * 729 * 75 * 4
    d.fmt = 1
    assert qb.qnn_conv_lowered_k(d) == 2400
    assert qb.qnn_conv_lowered_bytes(d) == 729 * 2400
    # conv1: 227x227x3, 11x11 stride 4 -> (96, 363, 3025); each filter row (33 bytes) is a
    # run padded to 48 bytes, so the lowered depth is 11 * 48
    d = qb.qnn_conv_desc(1, 227, 227, 3, 3, 96, 11, 11, 4, 0, 8, 8, 2, 1, 0, 1, 1, 0)
    assert qb.qnn_conv_out_h(d) == 55
    assert qb.qnn_conv_lowered_k(d) == 11 * 48
    assert qb.qnn_conv_lowered_bytes(d) == 3025 * 528
    # channel count not a multiple of 32: every pixel is padded to whole words
    d = qb.qnn_conv_desc(1, 8, 8, 40, 0, 16, 3, 3, 1, 1, 1, 2, 2, 2, 0, 0, 1, 0)
    assert qb.qnn_conv_lowered_k(d) == 32 * 9 * 2


def test_argument_validation_without_launch(qb):
    """Errors are detected on the host before any CUDA call (fake aligned addresses)."""
    P = 0x10000
    ok = dict(M=64, N=256, K=576, w_bits=1, a_bits=2, out_bits=2, w_enc=2, a_enc=0,
              fmt=0, out_fmt=1)

    def call(**kw):
        a = dict(ok); a.update(kw)
        ptrs = a.pop("ptrs", (P, P, P, P))
        path = a.pop("path", 0)
        d = qb.gemm_desc(a["M"], a["N"], a["K"], a["w_bits"], a["a_bits"], a["out_bits"],
                         a["w_enc"], a["a_enc"], a["fmt"], a["out_fmt"], path)
        if "a_fmt" in a:
            d.a_fmt = a["a_fmt"]
        return qb.qnn_qgemm(d, ptrs[0], ptrs[1], ptrs[2], ptrs[3], None, 0, stream=0)

    assert call(M=0) == qb.QNN_ERR_INVALID_ARG
    assert call(K=-1) == qb.QNN_ERR_INVALID_ARG
    assert call(w_bits=9) == qb.QNN_ERR_INVALID_ARG
    assert call(out_bits=5) == qb.QNN_ERR_INVALID_ARG
    assert call(w_enc=3) == qb.QNN_ERR_INVALID_ARG
    assert call(w_bits=2) == qb.QNN_ERR_UNSUPPORTED            # bipolar needs 1 bit
    assert call(a_fmt=1) == qb.QNN_ERR_UNSUPPORTED             # mixed operand formats
    assert call(path=qb.QNN_PATH_TCGEN05_I8) == qb.QNN_ERR_UNSUPPORTED   # planes on tensor path
    assert call(fmt=0, w_enc=1, w_bits=8, a_bits=8) == qb.QNN_ERR_UNSUPPORTED  # bit-serial > 4 bits
    assert call(ptrs=(None, P, P, P)) == qb.QNN_ERR_INVALID_ARG
    assert call(ptrs=(P, P, P, None)) == qb.QNN_ERR_INVALID_ARG
    assert call(ptrs=(P + 4, P, P, P)) == qb.QNN_ERR_ALIGNMENT
    assert call(ptrs=(P, P, P + 2, P)) == qb.QNN_ERR_ALIGNMENT

    pd = qb.qnn_pack_desc(4, 64, 2, qb.QNN_ENC_BIPOLAR, 0)
    assert qb.qnn_pack(pd, P, P, stream=0) == qb.QNN_ERR_UNSUPPORTED
    pd = qb.qnn_pack_desc(4, 64, 0, 0, 0)
    assert qb.qnn_pack(pd, P, P, stream=0) == qb.QNN_ERR_INVALID_ARG
    pd = qb.qnn_pack_desc(4, 64, 2, 0, 0)
    assert qb.qnn_pack(pd, P + 1, P, stream=0) == qb.QNN_ERR_ALIGNMENT

    cd = qb.qnn_conv_desc(1, 27, 27, 96, 0, 256, 5, 5, 1, 2, 1, 2, 2, 2, 0, 0, 1, 0)
    assert qb.qnn_qconv(cd, P, P, P, P, None, 0, stream=0) == qb.QNN_ERR_WORKSPACE
    assert qb.qnn_qconv(cd, P, P, P, P, P, 16, stream=0) == qb.QNN_ERR_WORKSPACE
    cd.a_enc, cd.a_bits = qb.QNN_ENC_BIPOLAR, 1
    assert qb.qnn_im2col(cd, P, P, stream=0) == qb.QNN_ERR_UNSUPPORTED    # zero pad not representable
    cd = qb.qnn_conv_desc(1, 3, 3, 96, 0, 256, 5, 5, 1, 0, 1, 2, 2, 2, 0, 0, 1, 0)
    assert qb.qnn_im2col(cd, P, P, stream=0) == qb.QNN_ERR_INVALID_ARG    # filter larger than image

    pl = qb.qnn_pool_desc(1, 2, 2, 16, 3, 2, 2, 1)
    assert qb.qnn_maxpool(pl, P, P, stream=0) == qb.QNN_ERR_INVALID_ARG


def test_gemm_workspace_size_rule(qb):
    """qnn_gemm_workspace_bytes (host only; 148 SMs assumed when there is no GPU): non-zero exactly
    where the CTA-pair kernel would leave a last round of tiles at most half full -- 8192 bytes of
    flags plus 256 KB per tile of that round."""
    if torch.cuda.is_available() and torch.cuda.get_device_properties(0).multi_processor_count != 148:
        pytest.skip("the expected sizes are those of 74 SM pairs")
    I8, PL = qb.QNN_FMT_INT8, qb.QNN_FMT_BITPLANES

    def ws(M, N, K, fmt=I8):
        return qb.qnn_gemm_workspace_bytes(qb.qnn_gemm_desc(M, N, K, 1, 2, 2, 2, 0, fmt, fmt, I8, 0, 0))

    assert ws(4096, 4096, 4096) == 8192 + 34 * 256 * 1024     # 256 tiles on 74 pairs: 3 rounds + 34
    assert ws(5120, 5120, 5120) == 8192 + 30 * 256 * 1024     # 400 tiles: 5 rounds + 30
    assert ws(8192, 8192, 8192) == 0                          # 1024 tiles: the last round holds 62 of 74
    assert ws(4096, 4096, 128) == 0                           # one k-block: nothing to split
    assert ws(4096, 1024, 4096) == 0                          # not the CTA-pair kernel
    assert ws(64, 256, 576) == 0
    assert ws(4096, 4096, 4096, PL) == 0                      # bit planes: another path


def test_kernel_choice_follows_the_documented_rule(qb):
    """qnn_qgemm_kernel (host only): the shape-driven choice documented in qnn.h -- the operand
    format is the caller's, the kernel follows from the shape (size sweep of Section 4.1.2)."""
    I8, PL, FL = qb.QNN_FMT_INT8, qb.QNN_FMT_BITPLANES, qb.QNN_FMT_FIELDS

    def k(M, N, K, w_fmt, a_fmt, path=0, w=2, a=2):
        d = qb.qnn_gemm_desc(M, N, K, w, a, 2, 1, 0, w_fmt, a_fmt, I8, path, 0)
        return qb.qnn_qgemm_kernel(d, True)

    assert k(4096, 4096, 4096, I8, I8) == qb.QNN_KERNEL_TENSOR_CTA_PAIR
    assert k(8192, 8192, 8192, I8, I8) == qb.QNN_KERNEL_TENSOR_CTA_PAIR
    assert k(4096, 1024, 4096, I8, I8) == qb.QNN_KERNEL_TENSOR            # fewer than 2048 columns
    assert k(128, 4096, 4096, I8, I8) == qb.QNN_KERNEL_TENSOR             # fewer than 256 channels
    assert k(64, 256, 576, I8, I8) == qb.QNN_KERNEL_TENSOR                # config 1
    assert k(8192, 1, 8192, I8, I8) == qb.QNN_KERNEL_BYTES_FEW_COLUMNS
    assert k(8192, 8, 8192, I8, I8) == qb.QNN_KERNEL_BYTES_FEW_COLUMNS
    assert k(8192, 16, 8192, I8, I8) == qb.QNN_KERNEL_TENSOR
    assert k(8192, 8, 8192, I8, I8, path=2) == qb.QNN_KERNEL_TENSOR       # path forced
    assert k(8192, 16, 8192, PL, PL) == qb.QNN_KERNEL_PLANES_FEW_COLUMNS
    assert k(8192, 17, 8192, PL, PL) == qb.QNN_KERNEL_PLANES_TILED
    assert k(64, 256, 576, PL, PL) == qb.QNN_KERNEL_PLANES_TILED
    assert k(8192, 16, 8192, FL, I8) == qb.QNN_KERNEL_FIELDS_FEW_COLUMNS
    assert k(8192, 17, 8192, FL, I8) == qb.QNN_ERR_UNSUPPORTED
    assert k(64, 64, 64, I8, PL) == qb.QNN_ERR_UNSUPPORTED                # mixed formats
