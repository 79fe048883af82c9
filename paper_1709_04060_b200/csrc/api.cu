// C ABI entry points: host-side validation, size queries and dispatch.
// Every step of the path itself runs in the kernels of the sibling files.
#include <stdlib.h>

#include "common.cuh"

namespace qnn {

std::atomic<unsigned long long> g_launches{0};

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

static bool valid_fmt(int fmt) { return fmt == QNN_FMT_BITPLANES || fmt == QNN_FMT_INT8; }
static int field_bits(int bits) { return bits == 1 ? 1 : (bits == 2 ? 2 : 4); }

static qnn_status check_gemm_desc(const qnn_gemm_desc *d, bool has_thr, int *path_out) {
    if (!d) return QNN_ERR_INVALID_ARG;
    if (d->M <= 0 || d->N <= 0 || d->K <= 0) return QNN_ERR_INVALID_ARG;
    if (d->w_bits < 1 || d->w_bits > 8 || d->a_bits < 1 || d->a_bits > 8) return QNN_ERR_INVALID_ARG;
    if (!(valid_fmt(d->w_fmt) || d->w_fmt == QNN_FMT_FIELDS) || !valid_fmt(d->a_fmt)) return QNN_ERR_INVALID_ARG;
    if (d->w_enc < 0 || d->w_enc > 2 || d->a_enc < 0 || d->a_enc > 2) return QNN_ERR_INVALID_ARG;
    if (d->path < QNN_PATH_AUTO || d->path > QNN_PATH_TCGEN05_I8) return QNN_ERR_INVALID_ARG;
    if (d->skip_planes < 0) return QNN_ERR_INVALID_ARG;
    // leaving plane pairs out is a notion of the bit-plane formulation only
    if (d->skip_planes > 0 && (d->w_fmt != QNN_FMT_BITPLANES || d->a_fmt != QNN_FMT_BITPLANES)) return QNN_ERR_UNSUPPORTED;
    if (has_thr) {
        if (d->out_bits < 1 || d->out_bits > 4) return QNN_ERR_INVALID_ARG;
        if (!valid_fmt(d->out_fmt)) return QNN_ERR_INVALID_ARG;
    }
    if (!valid_enc(d->w_enc, d->w_bits) || !valid_enc(d->a_enc, d->a_bits)) return QNN_ERR_UNSUPPORTED;
    if (d->w_fmt == QNN_FMT_FIELDS) {
        // packed w-bit weights against 8-bit activation containers: the few-column kernel only
        if (d->a_fmt != QNN_FMT_INT8 || d->path == QNN_PATH_BITSERIAL) return QNN_ERR_UNSUPPORTED;
        if (!gemv_fields_dp4a_fits(d) && !gemv_fields_fits(d, has_thr)) return QNN_ERR_UNSUPPORTED;
        if (path_out) *path_out = QNN_PATH_TCGEN05_I8;
        return QNN_OK;
    }
    if (d->w_fmt != d->a_fmt) return QNN_ERR_UNSUPPORTED;
    int path = d->path;
    if (path == QNN_PATH_AUTO)
        path = d->w_fmt == QNN_FMT_INT8 ? QNN_PATH_TCGEN05_I8 : QNN_PATH_BITSERIAL;
    if (path == QNN_PATH_TCGEN05_I8 && d->w_fmt != QNN_FMT_INT8) return QNN_ERR_UNSUPPORTED;
    if (path == QNN_PATH_BITSERIAL) {
        if (d->w_fmt != QNN_FMT_BITPLANES) return QNN_ERR_UNSUPPORTED;
        if (d->w_bits > 4 || d->a_bits > 4) return QNN_ERR_UNSUPPORTED;
    }
    // int32 accumulator range: K * max|w| * max|a| must stay below 2^31
    const double wmax = d->w_enc == QNN_ENC_BIPOLAR ? 1.0
                        : (d->w_enc == QNN_ENC_SIGNED ? double(1 << (d->w_bits - 1)) : double((1 << d->w_bits) - 1));
    const double amax = d->a_enc == QNN_ENC_BIPOLAR ? 1.0
                        : (d->a_enc == QNN_ENC_SIGNED ? double(1 << (d->a_bits - 1)) : double((1 << d->a_bits) - 1));
    if (double(d->K) * wmax * amax >= 2147483648.0) return QNN_ERR_UNSUPPORTED;
    if (path_out) *path_out = path;
    return QNN_OK;
}

static qnn_status check_conv_desc(const qnn_conv_desc *d) {
    if (!d) return QNN_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->OC <= 0 || d->KH <= 0 || d->KW <= 0)
        return QNN_ERR_INVALID_ARG;
    if (d->stride <= 0 || d->pad < 0 || d->in_pitch < 0) return QNN_ERR_INVALID_ARG;
    if (!valid_fmt(d->fmt)) return QNN_ERR_INVALID_ARG;
    if (d->a_bits < 1 || d->a_bits > 8) return QNN_ERR_INVALID_ARG;
    if (d->H + 2 * d->pad < d->KH || d->W + 2 * d->pad < d->KW) return QNN_ERR_INVALID_ARG;
    // the lowered GEMM's column count B*OH*OW and the map's pixel count are ints
    const long long oh = (d->H + 2 * d->pad - d->KH) / d->stride + 1, ow = (d->W + 2 * d->pad - d->KW) / d->stride + 1;
    if ((long long)d->B * oh * ow > 0x7fffffffll || (long long)d->B * d->H * d->W > 0x7fffffffll)
        return QNN_ERR_UNSUPPORTED;
    if (d->fmt == QNN_FMT_INT8 && d->in_pitch != 0 && d->in_pitch < d->C) return QNN_ERR_INVALID_ARG;
    if (d->a_enc == QNN_ENC_BIPOLAR && d->pad > 0) return QNN_ERR_UNSUPPORTED;
    // per-pixel pad bits would read as -1 for a bipolar operand
    if (d->fmt == QNN_FMT_BITPLANES && (d->C % 32) != 0 &&
        (d->a_enc == QNN_ENC_BIPOLAR || d->w_enc == QNN_ENC_BIPOLAR) &&
        (d->a_enc == QNN_ENC_BIPOLAR) == (d->w_enc == QNN_ENC_BIPOLAR))
        return QNN_ERR_UNSUPPORTED;
    return QNN_OK;
}

static void conv_to_gemm(const qnn_conv_desc *d, qnn_gemm_desc *g) {
    g->M = d->OC;
    g->N = d->B * qnn_conv_out_h(d) * qnn_conv_out_w(d);
    g->K = qnn_conv_lowered_k(d);
    g->w_bits = d->w_bits; g->a_bits = d->a_bits; g->out_bits = d->out_bits;
    g->w_enc = d->w_enc; g->a_enc = d->a_enc;
    g->w_fmt = d->fmt; g->a_fmt = d->fmt; g->out_fmt = d->out_fmt;
    g->path = d->path;
    g->skip_planes = 0;
}

}  // namespace qnn

using namespace qnn;

extern "C" {

int qnn_version(void) { return 100; }

const char *qnn_status_string(qnn_status s) {
    switch (s) {
        case QNN_OK: return "ok";
        case QNN_ERR_INVALID_ARG: return "invalid argument";
        case QNN_ERR_UNSUPPORTED: return "unsupported combination";
        case QNN_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case QNN_ERR_WORKSPACE: return "workspace missing or too small";
        case QNN_ERR_CUDA: return "CUDA call failed";
        case QNN_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

unsigned long long qnn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t qnn_packed_ld(int K, int fmt) {
    if (K <= 0) return 0;
    if (fmt == QNN_FMT_BITPLANES) return (size_t)ceil_div(K, 32);
    if (fmt == QNN_FMT_INT8) return (size_t)round_up(K, 16);
    return 0;           // QNN_FMT_FIELDS: the pitch depends on the bit width, see qnn_packed_bytes
}

size_t qnn_packed_bytes(const qnn_pack_desc *d) {
    if (!d || d->rows <= 0 || d->K <= 0 || d->bits < 1 || d->bits > 8) return 0;
    if (d->fmt == QNN_FMT_BITPLANES) return (size_t)d->bits * d->rows * qnn_packed_ld(d->K, d->fmt) * 4;
    if (d->fmt == QNN_FMT_INT8) return (size_t)d->rows * qnn_packed_ld(d->K, d->fmt);
    if (d->fmt == QNN_FMT_FIELDS && d->bits <= 4)
        return (size_t)d->rows * 32 * ceil_div(d->K, 32 * (8 / field_bits(d->bits)));
    return 0;
}

qnn_status qnn_pack(const qnn_pack_desc *d, const void *logical, void *packed, void *stream) {
    if (!d || !logical || !packed) return QNN_ERR_INVALID_ARG;
    if (d->rows <= 0 || d->K <= 0 || d->bits < 1 || d->bits > 8) return QNN_ERR_INVALID_ARG;
    if (!(valid_fmt(d->fmt) || d->fmt == QNN_FMT_FIELDS) || d->enc < 0 || d->enc > 2) return QNN_ERR_INVALID_ARG;
    if (!valid_enc(d->enc, d->bits)) return QNN_ERR_UNSUPPORTED;
    if (d->fmt == QNN_FMT_FIELDS && d->bits > 4) return QNN_ERR_UNSUPPORTED;
    if (!aligned16(logical) || !aligned16(packed)) return QNN_ERR_ALIGNMENT;
    return pack_launch(d, logical, packed, (cudaStream_t)stream);
}

qnn_status qnn_planes_to_int8(const qnn_pack_desc *d, const void *planes, void *containers, void *stream) {
    if (!d || !planes || !containers) return QNN_ERR_INVALID_ARG;
    if (d->rows <= 0 || d->K <= 0 || d->bits < 1 || d->bits > 8) return QNN_ERR_INVALID_ARG;
    if (d->fmt != QNN_FMT_BITPLANES || d->enc < 0 || d->enc > 2) return QNN_ERR_INVALID_ARG;
    if (!valid_enc(d->enc, d->bits)) return QNN_ERR_UNSUPPORTED;
    if (!aligned16(planes) || !aligned16(containers)) return QNN_ERR_ALIGNMENT;
    return planes_to_int8_launch(d, planes, containers, (cudaStream_t)stream);
}

size_t qnn_gemm_workspace_bytes(const qnn_gemm_desc *d) {
    int path = 0;
    if (check_gemm_desc(d, true, &path) != QNN_OK) return 0;
    if (d->w_fmt != QNN_FMT_INT8 || path != QNN_PATH_TCGEN05_I8) return 0;
    if (d->path == QNN_PATH_AUTO && gemv_i8_fits(d)) return 0;
    return gemm_tc_workspace_bytes(d);
}

size_t qnn_gemm_out_bytes(const qnn_gemm_desc *d, int has_thresholds) {
    if (!d || d->M <= 0 || d->N <= 0) return 0;
    if (!has_thresholds) return (size_t)d->N * d->M * 4;
    if (d->out_fmt == QNN_FMT_INT8) return (size_t)d->N * round_up(d->M, 16);
    if (d->out_fmt == QNN_FMT_BITPLANES) return (size_t)d->out_bits * d->N * ceil_div(d->M, 32) * 4;
    return 0;
}

int qnn_qgemm_kernel(const qnn_gemm_desc *d, int has_thresholds) {
    int path = 0;
    const qnn_status st = check_gemm_desc(d, has_thresholds != 0, &path);
    if (st != QNN_OK) return (int)st;
    if (d->w_fmt == QNN_FMT_FIELDS) return QNN_KERNEL_FIELDS_FEW_COLUMNS;
    if (d->path == QNN_PATH_AUTO && d->w_fmt == QNN_FMT_INT8 && gemv_i8_fits(d)) return QNN_KERNEL_BYTES_FEW_COLUMNS;
    if (path == QNN_PATH_TCGEN05_I8) return gemm_tc_uses_pair_kernel(d) ? QNN_KERNEL_TENSOR_CTA_PAIR : QNN_KERNEL_TENSOR;
    if (gemv_planes_fits(d)) return QNN_KERNEL_PLANES_FEW_COLUMNS;
    return QNN_KERNEL_PLANES_TILED;
}

qnn_status qnn_qgemm(const qnn_gemm_desc *d, const void *W, const void *A, const int32_t *thr,
                     void *out, void *workspace, size_t workspace_bytes, void *stream) {
    int path = 0;
    qnn_status st = check_gemm_desc(d, thr != nullptr, &path);
    if (st != QNN_OK) return st;
    if (!W || !A || !out) return QNN_ERR_INVALID_ARG;
    if (!aligned16(W) || !aligned16(A) || !aligned16(out) || (thr && (reinterpret_cast<uintptr_t>(thr) & 3u)))
        return QNN_ERR_ALIGNMENT;
    if (d->w_fmt == QNN_FMT_FIELDS) {
        // a few columns: byte dot products on the CUDA cores; more: the tensor-core form
        if (gemv_fields_dp4a_fits(d)) return gemv_fields_dp4a_launch(d, W, A, thr, out, (cudaStream_t)stream);
        return gemv_fields_launch(d, W, A, thr, out, (cudaStream_t)stream);
    }
    // 8-bit containers with a handful of columns and no path forced: byte dot products,
    // one warp per weight row (a tensor-core tile would be almost empty)
    if (d->path == QNN_PATH_AUTO && d->w_fmt == QNN_FMT_INT8 && gemv_i8_fits(d))
        return gemv_i8_launch(d, W, A, thr, out, (cudaStream_t)stream);
    if (path == QNN_PATH_TCGEN05_I8) {
        // the workspace is optional (see the header): used only when given, large enough and aligned
        const bool ws_ok = workspace && aligned16(workspace);
        return gemm_tc_launch(d, W, A, thr, out, ws_ok ? workspace : nullptr, ws_ok ? workspace_bytes : 0,
                              (cudaStream_t)stream);
    }
    // a handful of columns: stream the weight planes once, one warp per row
    if (gemv_planes_fits(d)) return gemv_planes_launch(d, W, A, thr, out, (cudaStream_t)stream);
    return gemm_bitserial_launch(d, W, A, thr, out, (cudaStream_t)stream);
}

int qnn_conv_out_h(const qnn_conv_desc *d) {
    return d ? (d->H + 2 * d->pad - d->KH) / d->stride + 1 : 0;
}
int qnn_conv_out_w(const qnn_conv_desc *d) {
    return d ? (d->W + 2 * d->pad - d->KW) / d->stride + 1 : 0;
}

int qnn_conv_lowered_k(const qnn_conv_desc *d) {
    if (!d) return 0;
    if (d->fmt == QNN_FMT_BITPLANES) return 32 * d->KH * d->KW * ceil_div(d->C, 32);
    if (d->C % 16 == 0) return d->KH * d->KW * d->C;
    return d->KH * round_up(d->KW * d->C, 16);       // one zero-padded run per filter row
}

size_t qnn_conv_lowered_bytes(const qnn_conv_desc *d) {
    if (check_conv_desc(d) != QNN_OK) return 0;
    qnn_pack_desc p;
    p.rows = d->B * qnn_conv_out_h(d) * qnn_conv_out_w(d);
    p.K = qnn_conv_lowered_k(d);
    p.bits = d->a_bits; p.enc = d->a_enc; p.fmt = d->fmt;
    return qnn_packed_bytes(&p);
}

size_t qnn_conv_workspace_bytes(const qnn_conv_desc *d) {
    size_t b = qnn_conv_lowered_bytes(d);
    return (b + 255) / 256 * 256;
}

size_t qnn_conv_out_bytes(const qnn_conv_desc *d, int has_thresholds) {
    if (check_conv_desc(d) != QNN_OK) return 0;
    qnn_gemm_desc g;
    conv_to_gemm(d, &g);
    return qnn_gemm_out_bytes(&g, has_thresholds);
}

qnn_status qnn_im2col(const qnn_conv_desc *d, const void *in, void *lowered, void *stream) {
    qnn_status st = check_conv_desc(d);
    if (st != QNN_OK) return st;
    if (!in || !lowered) return QNN_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(lowered)) return QNN_ERR_ALIGNMENT;
    return im2col_launch(d, in, lowered, (cudaStream_t)stream);
}

qnn_status qnn_qconv(const qnn_conv_desc *d, const void *Wpacked, const void *in, const int32_t *thr,
                     void *out, void *workspace, size_t workspace_bytes, void *stream) {
    qnn_status st = check_conv_desc(d);
    if (st != QNN_OK) return st;
    qnn_gemm_desc g;
    conv_to_gemm(d, &g);
    int path = 0;
    st = check_gemm_desc(&g, thr != nullptr, &path);
    if (st != QNN_OK) return st;
    if (!Wpacked || !in || !out) return QNN_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < qnn_conv_workspace_bytes(d)) return QNN_ERR_WORKSPACE;
    if (!aligned16(Wpacked) || !aligned16(in) || !aligned16(out) || !aligned16(workspace))
        return QNN_ERR_ALIGNMENT;
    // 8-bit maps on the tensor-core path: the GEMM's loader does the lowering itself (im2col
    // tensor map) where the shape allows; QNN_CONV_EXPLICIT=1 in the environment keeps the
    // lowered matrix (measurements, tests)
    const char *explicit_env = getenv("QNN_CONV_EXPLICIT");
    if (path == QNN_PATH_TCGEN05_I8 && !(explicit_env && explicit_env[0] == '1')) {
        // lowering warps inside the kernel where the tensor-map loader does not apply (few
        // channels: the first layer) or would waste k-blocks (channel count not a multiple of 128)
        st = gemm_tc_lower_launch(d, &g, Wpacked, in, thr, out, (cudaStream_t)stream);
        if (st != QNN_ERR_UNSUPPORTED) return st;
        st = gemm_tc_conv_launch(d, &g, Wpacked, in, thr, out, (cudaStream_t)stream);
        if (st != QNN_ERR_UNSUPPORTED) return st;
    }
    // bit-plane maps on the tiled bit-serial kernel: its staging code lowers on the fly (a handful
    // of output pixels goes through the lowered matrix and the few-column kernel instead)
    if (path == QNN_PATH_BITSERIAL && !(explicit_env && explicit_env[0] == '1') && !gemv_planes_fits(&g)) {
        st = gemm_bitserial_conv_launch(d, &g, Wpacked, in, thr, out, (cudaStream_t)stream);
        if (st != QNN_ERR_UNSUPPORTED) return st;
    }
    st = im2col_launch(d, in, workspace, (cudaStream_t)stream);
    if (st != QNN_OK) return st;
    return qnn_qgemm(&g, Wpacked, workspace, thr, out, nullptr, 0, stream);
}

// Lowered-matrix storage of qnn_qconv_static.  In host code this name is only a
// handle for cudaGetSymbolAddress; the kernels get the address that call returns.
static __device__ __align__(256) unsigned char g_static_lowered[QNN_QCONV_STATIC_MAX_BYTES];

// Device address of g_static_lowered on the current device, looked up once per device.
static qnn_status static_lowered_ptr(void **ptr) {
    static void *cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return QNN_ERR_CUDA;
    if (!cached[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_lowered) != cudaSuccess || !p) return QNN_ERR_CUDA;
        cached[dev] = p;
    }
    *ptr = cached[dev];
    return QNN_OK;
}

qnn_status qnn_qconv_static(const qnn_conv_desc *d, const void *Wpacked, const void *in, const int32_t *thr,
                            void *out, void *stream) {
    qnn_status st = check_conv_desc(d);
    if (st != QNN_OK) return st;
    qnn_gemm_desc g;
    conv_to_gemm(d, &g);
    st = check_gemm_desc(&g, thr != nullptr, nullptr);
    if (st != QNN_OK) return st;
    if (qnn_conv_workspace_bytes(d) > (size_t)QNN_QCONV_STATIC_MAX_BYTES) return QNN_ERR_WORKSPACE;
    if (!Wpacked || !in || !out) return QNN_ERR_INVALID_ARG;
    if (!aligned16(Wpacked) || !aligned16(in) || !aligned16(out)) return QNN_ERR_ALIGNMENT;
    void *lowered = nullptr;
    st = static_lowered_ptr(&lowered);
    if (st != QNN_OK) return st;
    st = im2col_launch(d, in, lowered, (cudaStream_t)stream);
    if (st != QNN_OK) return st;
    return qnn_qgemm(&g, Wpacked, lowered, thr, out, nullptr, 0, stream);
}

qnn_status qnn_maxpool(const qnn_pool_desc *d, const void *in, void *out, void *stream) {
    if (!d || !in || !out) return QNN_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->k <= 0 || d->stride <= 0)
        return QNN_ERR_INVALID_ARG;
    if (d->k > d->H || d->k > d->W) return QNN_ERR_INVALID_ARG;
    if (d->bits < 1 || d->bits > 8 || !valid_fmt(d->fmt)) return QNN_ERR_INVALID_ARG;
    if (d->fmt == QNN_FMT_BITPLANES && d->bits > 4) return QNN_ERR_UNSUPPORTED;
    if (!aligned16(in) || !aligned16(out)) return QNN_ERR_ALIGNMENT;
    return maxpool_launch(d, in, out, (cudaStream_t)stream);
}

qnn_status qnn_validate_thresholds(const int32_t *thr, int M, int n_thr, int *n_bad_rows, void *stream) {
    if (!thr || !n_bad_rows || M <= 0 || n_thr <= 0) return QNN_ERR_INVALID_ARG;
    return validate_thresholds_launch(thr, M, n_thr, n_bad_rows, (cudaStream_t)stream);
}

qnn_status qnn_device_status(int *status) {
    if (!status) return QNN_ERR_INVALID_ARG;
    return device_status_read(status);
}

}  // extern "C"
