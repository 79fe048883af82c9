/*
 * qnn.h -- C ABI of the B200 (sm_100a) hot path of streamlined few-bit QNN
 * inference: few-bit integer GEMM WwAa fused with the per-output-channel
 * multi-threshold activation, fed by channel-interleaved lowering.
 *
 * General conventions
 * -------------------
 *  - Shapes follow the paper's (rows, depth, cols) = (M, K, N) of Section 4.1:
 *    M output channels (weight rows), K depth, N columns (pixels x batch).
 *    Both operands are indexed (row-or-column, depth) as in Algorithm 1, i.e.
 *    the activation matrix is held transposed: W is [M][K], A is [N][K].
 *  - Every data pointer is a DEVICE pointer owned by the caller; descriptors
 *    are host structs read during the call.  The library allocates no device
 *    memory: scratch is sized by a *_workspace_bytes query and passed in.
 *  - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on
 *    that stream; they never synchronise (the two functions that return a
 *    value read back from the device say so).
 *  - Errors are return codes.  Argument errors are detected on the host before
 *    anything is launched.  Device code never traps: a bounded wait that runs
 *    out records QNN_ERR_DEVICE_TIMEOUT in a device status word that
 *    qnn_device_status() reads.
 *  - All results are exact integers; there is no CPU fallback and no other
 *    backend.
 *
 * Encodings (Section 3.1; the paper's Algorithm 2 is the SIGNED x SIGNED case)
 *   QNN_ENC_UNSIGNED  b bits, value in [0, 2^b - 1]
 *   QNN_ENC_SIGNED    b bits two's complement, value in [-2^(b-1), 2^(b-1)-1]
 *   QNN_ENC_BIPOLAR   1 bit, bit 1 -> +1, bit 0 -> -1
 *
 * Environment switches (read at call time; for measurements and tests only)
 *   QNN_TC_KERNEL=single|pair  one-CTA or CTA-pair tensor-core kernel (default: the pair
 *                              kernel for large problems, the one-CTA kernel otherwise)
 *   QNN_TC_NO_SHARE=1          never split a tile's depth between two CTAs
 *   QNN_CONV_EXPLICIT=1        qnn_qconv always goes through the lowered matrix
 *   QNN_CONV_IMPLICIT=1        qnn_qconv lowers inside the GEMM wherever it can
 *   QNN_CONV_LOWER=1|0         qnn_qconv uses the aligned lowering warps wherever they
 *                              apply | never
 *   QNN_FIELDS_KERNEL=dp4a|tensor  packed (FIELDS) weights: byte dot products on the CUDA
 *                              cores for up to 16 columns | always the tensor-core form
 *
 * Operand formats
 *   QNN_FMT_BITPLANES  uint32 [bits][rows][kw], kw = ceil(K/32): plane i holds
 *                      bit i of every element (Section 3.1), element k of a row
 *                      in word k/32 at bit k%32, pad bits zero.  This is the
 *                      paper's depth-packed binary matrix (Algorithm 1) and, for
 *                      activations, its channel-interleaved layout (Section 3.2).
 *   QNN_FMT_INT8       one byte per element [rows][ld], ld = K rounded up to a
 *                      multiple of 16, pad bytes zero: int8 for SIGNED/BIPOLAR,
 *                      uint8 for UNSIGNED (the 8-bit formulation of Section 3:
 *                      few-bit values held in 8-bit containers); the tensor-core
 *                      path consumes this.
 *   QNN_FMT_FIELDS     weights only: w-bit fields packed along the depth, f = 1, 2 or 4
 *                      bits per field (3-bit values take 4-bit fields), S = 8/f fields
 *                      per byte, [rows][ldf] bytes with ldf = 32 * ceil(K / (32 S)).
 *                      Element k of a row lies in byte 32 g + j at bits [f s, f s + f),
 *                      where g = k / (32 S), s = (k mod 32 S) / 32, j = k mod 32: the 32
 *                      elements at field position s of 32 consecutive bytes are 32
 *                      consecutive depth indices.  A field holds the value minus the
 *                      encoding's minimum (UNSIGNED: the value, SIGNED: value + 2^(b-1),
 *                      BIPOLAR: the bit); fields past K are zero.  This is the paper's
 *                      packed weight storage (Section 4.2: fully connected layers gain
 *                      from the cut in memory traffic) in a form that expands to 8-bit
 *                      values with one AND per word; qnn_qgemm takes it with INT8
 *                      activations and N <= 16 columns.
 */
#ifndef QNN_H_
#define QNN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QNN_OK = 0,
    QNN_ERR_INVALID_ARG = -1,     /* null pointer, non-positive size, bad enum */
    QNN_ERR_UNSUPPORTED = -2,     /* legal but not implemented combination    */
    QNN_ERR_ALIGNMENT = -3,       /* a device pointer is not 16-byte aligned   */
    QNN_ERR_WORKSPACE = -4,       /* workspace missing or too small            */
    QNN_ERR_CUDA = -5,            /* a CUDA runtime/driver call failed         */
    QNN_ERR_DEVICE_TIMEOUT = -6   /* a bounded device-side wait ran out        */
} qnn_status;

typedef enum { QNN_ENC_UNSIGNED = 0, QNN_ENC_SIGNED = 1, QNN_ENC_BIPOLAR = 2 } qnn_enc;
typedef enum { QNN_FMT_BITPLANES = 0, QNN_FMT_INT8 = 1, QNN_FMT_FIELDS = 2 } qnn_fmt;
typedef enum { QNN_PATH_AUTO = 0, QNN_PATH_BITSERIAL = 1, QNN_PATH_TCGEN05_I8 = 2 } qnn_path;

/* ---- packer (Section 3.1 bit planes; Section 3 8-bit containers) ---------- */

typedef struct {
    int rows;        /* M for weights, N for activations                      */
    int K;           /* depth                                                 */
    int bits;        /* 1..8; BIPOLAR requires 1                              */
    int enc;         /* qnn_enc                                               */
    int fmt;         /* qnn_fmt of the packed result (FIELDS: bits <= 4)      */
} qnn_pack_desc;

/* Row pitch of a packed operand: 32-bit words per row and plane for BITPLANES
 * (ceil(K/32)), bytes per row for INT8 (K rounded up to 16); 0 for FIELDS, whose pitch
 * depends on the bit width (qnn_packed_bytes / rows).  Host only. */
size_t qnn_packed_ld(int K, int fmt);

/* Bytes of a packed operand.  Host only; 0 on invalid arguments. */
size_t qnn_packed_bytes(const qnn_pack_desc *d);

/* logical: one byte per element, dense [rows][K] (uint8 for UNSIGNED, int8
 * for SIGNED and BIPOLAR); values outside the encoding's range are truncated
 * to their low `bits` bits (BIPOLAR: value > 0 -> bit 1).  packed: written in
 * full, padding included.  Both 16-byte aligned. */
qnn_status qnn_pack(const qnn_pack_desc *d, const void *logical, void *packed, void *stream);

/* A BITPLANES operand widened to INT8 containers of the same values (Section 3.1's planes to
 * Section 3's 8-bit operands): d describes the source (d->fmt must be QNN_FMT_BITPLANES; rows, K,
 * bits, enc); planes: uint32 [bits][rows][ceil(K/32)]; containers: [rows][K rounded up to 16],
 * written in full, pad bytes zero.  For data that is stored or shipped packed -- `bits` instead of
 * 8 bits per element over the host link -- and multiplied on the tensor cores.  Both pointers
 * 16-byte aligned. */
qnn_status qnn_planes_to_int8(const qnn_pack_desc *d, const void *planes, void *containers, void *stream);

/* ---- fused GEMM + threshold (Sections 3.1 and 2.1.1) ---------------------- */

typedef struct {
    int M, N, K;
    int w_bits, a_bits;   /* 1..8 (tensor path) / 1..4 (bit-serial path)      */
    int out_bits;         /* 1..4: 2^out_bits - 1 thresholds per row; ignored
                             when thr == NULL                                 */
    int w_enc, a_enc;     /* qnn_enc                                          */
    int w_fmt, a_fmt;     /* qnn_fmt; both operands must use the same format,
                             except w_fmt FIELDS, which goes with a_fmt INT8     */
    int out_fmt;          /* qnn_fmt of the output codes; ignored if thr==NULL*/
    int path;             /* qnn_path; AUTO selects by operand format, and for a
                             handful of columns (N <= 16 bit planes, N <= 8
                             bytes) the one-warp-per-weight-row kernels       */
    int skip_planes;      /* 0: the exact product.  s > 0 (BITPLANES operands only):
                             the bit-plane pairs (i, j) with i + j < s are left out
                             of sum_i sum_j +-2^(i+j) W[i].A[j] -- the approximate
                             product from the higher-order bits that the paper's
                             conclusion names; it differs from the exact one by at
                             most K * sum_{i+j<s} 2^(i+j), and the bit-serial kernels
                             skip the AND/POPC work of those pairs.  A BIPOLAR
                             operand counts as one plane (index 0).  (Apart from
                             this, and exactly: the tiled bit-plane kernel skips a
                             plane pair wherever one of its 64-row x 512-bit plane
                             tiles holds no set bit -- the bit-level sparsity the
                             same sentence of the paper names.)                   */
} qnn_gemm_desc;

/* Scratch bytes qnn_qgemm can use for this problem (0: none).  The workspace is OPTIONAL:
 * without it (NULL, or fewer bytes) the call computes the same result.  With it, the CTA-pair
 * tensor-core kernel splits a last round of 256 x 256 tiles that would keep at most half of the
 * SM pairs busy: two neighbouring pairs take one half of the depth each and exchange int32
 * partial sums through the workspace (Section 4.1 of the paper measures exactly such large square
 * products; the split is worth 2-4 % there).  Contract: 16-byte aligned; its first 8192 bytes
 * are flag words that must be ZERO before the first call that uses the workspace; the kernel
 * leaves them zero, so the same workspace serves call after call (after a call that ended in
 * QNN_ERR_DEVICE_TIMEOUT, zero them again).  Calls that may run concurrently (different streams)
 * need different workspaces, and a call that uses one should have the GPU's SMs to itself apart
 * from kernels that do not wait on others: the two pairs of a split tile wait for each other (a
 * bounded wait, ending in QNN_ERR_DEVICE_TIMEOUT).  Host only. */
size_t qnn_gemm_workspace_bytes(const qnn_gemm_desc *d);

/* Bytes of the output buffer for this problem (see qnn_qgemm).  Host only. */
size_t qnn_gemm_out_bytes(const qnn_gemm_desc *d, int has_thresholds);

/* acc[m][n] = sum_k W[m][k] * A[n][k], exact in int32 (Section 3.1), then
 *   out[n][m] = #{ i : thr[m][i] <= acc[m][n] }      (Section 2.1.1, T(x, t)).
 * thr: int32 [M][2^out_bits - 1], expected sorted non-decreasing per row (the
 * counting rule is well defined either way).  Output, column(pixel)-major with
 * channels fastest so that it is directly the next layer's activation operand:
 *   out_fmt INT8       uint8  [N][ld], ld = M rounded up to 16, pad bytes 0
 *   out_fmt BITPLANES  uint32 [out_bits][N][ceil(M/32)], pad bits 0
 *   thr == NULL        int32  [N][M] raw accumulators
 * The accumulators never reach global memory on the fused path.
 * w_fmt FIELDS (with a_fmt INT8): N <= 16, w_bits <= 4; the packed weights are read
 * from memory once and expanded inside the kernel.
 * Errors: INVALID_ARG, UNSUPPORTED (mixed formats, bits out of range for the
 * path, BIPOLAR with bits != 1, FIELDS with more than 16 columns or a depth slice that
 * does not fit shared memory), ALIGNMENT, WORKSPACE, CUDA. */
qnn_status qnn_qgemm(const qnn_gemm_desc *d, const void *W, const void *A,
                     const int32_t *thr, void *out,
                     void *workspace, size_t workspace_bytes, void *stream);

/* Which kernel qnn_qgemm runs for this problem (Section 4.1.2 of the paper: the engine is
 * chosen per layer shape).  The operand format is the caller's choice; on this GPU 8-bit
 * containers on the tensor cores are faster than bit planes for every size from 64 to 4096 per
 * dimension and every (w, a), so AUTO never converts between formats, it picks by shape:
 *   INT8 operands       N <= 8: byte dot products, one warp per weight row;
 *                       M >= 256, N >= 2048 and at least a round and a half of 256 x 256 tiles
 *                       on the SM pairs: the CTA-pair tensor-core kernel; else the one-CTA
 *                       tensor-core kernel
 *   BITPLANES operands  N <= 16: one warp per weight row over the planes; else the tiled
 *                       AND/POPC kernel
 *   FIELDS weights      N <= 16 only: one or two columns: one warp per
 *                       packed weight row, an AND and a 4-way byte dot product per word and
 *                       field position; more columns: packed weights expanded inside a
 *                       tensor-core kernel
 * Returns a qnn_kernel value, or the (negative) qnn_status qnn_qgemm would return.  Host only. */
typedef enum {
    QNN_KERNEL_TENSOR = 1, QNN_KERNEL_TENSOR_CTA_PAIR = 2, QNN_KERNEL_BYTES_FEW_COLUMNS = 3,
    QNN_KERNEL_PLANES_FEW_COLUMNS = 4, QNN_KERNEL_PLANES_TILED = 5, QNN_KERNEL_FIELDS_FEW_COLUMNS = 6
} qnn_kernel;
int qnn_qgemm_kernel(const qnn_gemm_desc *d, int has_thresholds);

/* ---- lowering and convolution (Section 3.2) ------------------------------- */

typedef struct {
    int B, H, W, C;          /* input feature map, channels-last               */
    int in_pitch;            /* INT8 only: bytes between consecutive pixels of
                                the input map; 0 = C rounded up to 16          */
    int OC, KH, KW;          /* filters                                        */
    int stride, pad;         /* same in both spatial dimensions                */
    int w_bits, a_bits, out_bits;
    int w_enc, a_enc;
    int fmt;                 /* qnn_fmt of input map, weights and lowered matrix */
    int out_fmt;             /* qnn_fmt of the output map                      */
    int path;                /* qnn_path                                       */
} qnn_conv_desc;

/* Output spatial size: (H + 2*pad - KH)/stride + 1.  Host only. */
int qnn_conv_out_h(const qnn_conv_desc *d);
int qnn_conv_out_w(const qnn_conv_desc *d);

/* Depth of the lowered GEMM.  BITPLANES: 32 * KH*KW*ceil(C/32) (each pixel is
 * padded to whole words, Section 3.2).  INT8: KH*KW*C when C is a multiple of
 * 16; otherwise KH * (KW*C rounded up to 16): the KW*C bytes of each filter row
 * form one run, zero padded to a 16-byte boundary.  The weight operand passed
 * to qnn_qconv must be packed with this K and the same padding (zeros):
 * logical weight row = (kh, kw, c) with c fastest.  Host only. */
int qnn_conv_lowered_k(const qnn_conv_desc *d);

/* Bytes of the lowered matrix / of qnn_qconv's workspace.  Host only. */
size_t qnn_conv_lowered_bytes(const qnn_conv_desc *d);
size_t qnn_conv_workspace_bytes(const qnn_conv_desc *d);
size_t qnn_conv_out_bytes(const qnn_conv_desc *d, int has_thresholds);

/* Interleaved lowering (Section 3.2): for every activation bit plane j and
 * output pixel (b, oh, ow), concatenate over (kh, kw) in raster order the
 * ceil(C/32) words of input pixel (oh*stride - pad + kh, ow*stride - pad + kw);
 * pixels outside the image contribute zero words.
 *   fmt BITPLANES: in uint32 [a_bits][B][H][W][ceil(C/32)]
 *                  -> lowered uint32 [a_bits][B*OH*OW][KH*KW*ceil(C/32)]
 *   fmt INT8:      in uint8 [B][H][W][in_pitch] (the first C bytes of a pixel
 *                  are its channels; in_pitch a multiple of 16 when C is)
 *                  -> lowered uint8 [B*OH*OW][qnn_conv_lowered_k], pad bytes zero.
 * The lowered matrix is the activation operand A of qnn_qgemm (N = B*OH*OW). */
qnn_status qnn_im2col(const qnn_conv_desc *d, const void *in, void *lowered, void *stream);

/* Convolution by lowering + fused GEMM/threshold.  Wpacked: the [OC][K_lowered]
 * weight operand in format d->fmt.  Output: as qnn_qgemm with N = B*OH*OW,
 * M = OC, i.e. a channels-last feature map [B][OH][OW][...].  BIPOLAR
 * activations with pad > 0 are UNSUPPORTED (zero is not representable).
 * The lowered matrix of Section 3.2 is written to `workspace` only where the GEMM
 * kernel cannot form its tiles itself.  Bit-plane maps are lowered on the fly by the
 * staging code of the tiled AND/POPC kernel (word-granular, as in Section 3.2).
 * 8-bit maps are lowered inside the tensor-core kernel: by its tensor-map loader
 * when C and in_pitch are multiples of 16 (the CTA-pair kernel for large layers,
 * the one-CTA kernel otherwise); by lowering warps when pixels are contiguous and
 * either C is not a multiple of 16, pad == 0, OC <= 128 and the weights are not
 * BIPOLAR, or C is a multiple of 16 but not of 128, the layer has many tiles and
 * the CTA-pair kernel does not apply.  All routes give the same integer results.
 * The pad columns of the weight rows (see qnn_conv_lowered_k) must be zero bytes
 * for the lowering warps' unmasked route: it leaves image bytes,
 * not zeros, opposite them.  The workspace must be given in every case. */
qnn_status qnn_qconv(const qnn_conv_desc *d, const void *Wpacked, const void *in,
                     const int32_t *thr, void *out,
                     void *workspace, size_t workspace_bytes, void *stream);

/* Largest lowered matrix, in bytes, that qnn_qconv_static accepts. */
#define QNN_QCONV_STATIC_MAX_BYTES (16u << 20)

/* Convolution for callers that have no device memory to give as workspace and no
 * means of getting any.  (The paper has no counterpart; this is a deployment aid.)
 * Typical cases: a layer plug-in inside an inference server that carves up all
 * device memory at start-up and hands the plug-in nothing but its input and
 * output tensors; a control loop with a latency bound, where cudaMalloc may not
 * be called because it can stall on the whole device.  Same computation, arguments, output and error codes as
 * qnn_qconv, minus the workspace: the lowered matrix lives in an array that is
 * part of the library image (QNN_QCONV_STATIC_MAX_BYTES of device memory on
 * every GPU that loads the library, held until the process exits).  The call
 * allocates and frees nothing, on the device or through any library.
 *  - Problems whose lowered matrix (qnn_conv_workspace_bytes) is larger than
 *    QNN_QCONV_STATIC_MAX_BYTES are refused with QNN_ERR_WORKSPACE before
 *    anything is launched.
 *  - The first call on each device looks up the array's device address (with
 *    that device current); make that first call before any stream capture
 *    begins on the device.
 *  - All calls on a device share the one array, and it keeps whatever the
 *    previous call left in it.  Nothing in it has to start at zero: every call
 *    rewrites, padding included, all of the lowered matrix it reads.  Two calls
 *    whose kernels can overlap on the GPU (different streams, no dependency)
 *    race on the array; order them on one stream or with events. */
qnn_status qnn_qconv_static(const qnn_conv_desc *d, const void *Wpacked, const void *in,
                            const int32_t *thr, void *out, void *stream);

/* ---- integer max-pool on activation codes (Section 4.2) ------------------- */

typedef struct {
    int B, H, W, C;      /* input map, channels-last                          */
    int k, stride;       /* window and stride; no padding, floor              */
    int bits;            /* code width (BITPLANES: number of planes)          */
    int fmt;             /* INT8: uint8 [B][H][W][Cp], Cp = C rounded up to 16;
                            BITPLANES: uint32 [bits][B][H][W][ceil(C/32)]     */
} qnn_pool_desc;

/* out has the same format with H, W replaced by (H-k)/stride+1, (W-k)/stride+1. */
qnn_status qnn_maxpool(const qnn_pool_desc *d, const void *in, void *out, void *stream);

/* ---- streamlining (Section 2.1), host only -------------------------------- */

/* Float parameters around one output channel of a quantized matrix layer. */
typedef struct {
    double a_prev, b_prev;     /* previous layer's activation value = a_prev * code + b_prev
                                  (quantizer as thresholding + affine map, Section 2.1.1) */
    double alpha;              /* alpha-scaling of this channel's weight row (Section 2) */
    double gamma, beta;        /* batch normalisation: gamma * (z - mu) / sigma + beta     */
    double mu, sigma;
    long long row_sum;         /* sum of the channel's integer weights: the W.b term of
                                  W.(a x + b) = a (W.x) + W.b (Section 2.1.2)              */
} qnn_channel_params;

/* Absorbs the float operations between the integer accumulator and the activation
 * quantizer into integer thresholds (Sections 2.1.2 and 2.1.3).  qthr: the quantizer's
 * n_thr float thresholds, ascending (e.g. {0, 0.807, 1.345} for the 2-bit HWGQ quantizer);
 * [acc_lo, acc_hi]: range of the accumulator (|.| < 2^31).  thr_out [channels][n_thr]:
 * threshold i is the smallest integer accumulator whose float forward pass reaches code
 * i + 1, INT32_MIN if every accumulator does, INT32_MAX if none does; a tie (accumulator
 * maps exactly onto a float threshold) counts as passed.  negate_out [channels]: 1 where
 * the collapsed slope is negative -- that channel's thresholds are for the NEGATED
 * accumulator, i.e. the caller negates the channel's weight row.  All pointers are host
 * pointers; nothing is launched.  Errors: INVALID_ARG. */
qnn_status qnn_streamline(const qnn_channel_params *ch, int channels, const double *qthr, int n_thr,
                          long long acc_lo, long long acc_hi, int32_t *thr_out, uint8_t *negate_out);

/* ---- roofline denominators (Section 4.1.1 reports against the machine's peak) -- */

/* Launches the tensor-pipe issue-rate microbenchmark on `stream`: every SM (mode 0; one
 * CTA each; mode 2: the same with the 128-row operand read from tensor memory, n <= 128) or
 * every pair of SMs (mode 1; tcgen05 cta_group::2) issues mmas_per_cta
 * back-to-back tcgen05.mma kind::i8 instructions of 128 (256 for a pair) x n x 32 on operand
 * tiles of pseudo-random bytes resident in shared memory: no loads, no epilogue.  n: a
 * multiple of 16 (32 for a pair) in [16, 256].  *ops (host) receives the integer operations (2 per multiply-
 * accumulate) the launch performs; the caller times the launch with events.  The peak of
 * the dense int8 tensor path is ops / time.  Errors: INVALID_ARG, CUDA. */
qnn_status qnn_peak_mma_i8(int mode, int n, int mmas_per_cta, double *ops, void *stream);

/* Launches the POPC issue-rate microbenchmark (chains of XOR + POPC in registers, the inner
 * operation of Algorithm 1): *popcs (host) receives the number of 32-bit population counts
 * the launch executes; 32 x popcs / time is the peak of the bit-serial path in binary
 * multiply-accumulates per second.  sink: device scratch of at least
 * qnn_peak_popc_sink_bytes() bytes, 16-byte aligned (each thread stores one word there).
 * Errors: INVALID_ARG, WORKSPACE, ALIGNMENT, CUDA. */
qnn_status qnn_peak_popc(int iters, void *sink, size_t sink_bytes, double *popcs, void *stream);
size_t qnn_peak_popc_sink_bytes(void);

/* ---- utilities ------------------------------------------------------------ */

/* Checks on the device that every row of thr [M][n_thr] is sorted
 * non-decreasing; *n_bad_rows receives the number of unsorted rows.
 * SYNCHRONISES the stream. */
qnn_status qnn_validate_thresholds(const int32_t *thr, int M, int n_thr,
                                   int *n_bad_rows, void *stream);

/* Reads and clears the device status word of the current device
 * (QNN_OK or QNN_ERR_DEVICE_TIMEOUT).  SYNCHRONISES the device. */
qnn_status qnn_device_status(int *status);

/* Number of kernels this library has launched since it was loaded (host
 * counter; used by benchmarks to report launches per step). */
unsigned long long qnn_launch_count(void);

const char *qnn_status_string(qnn_status s);
int qnn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* QNN_H_ */
