// Bit-serial few-bit GEMM (Section 3.1, Algorithms 1 and 2) fused with the
// threshold activation T(x, t) of Section 2.1.1.
//
// acc[m][n] = sum_i sum_j c_w[i] c_a[j] sum_d popc(W[i](m,d) & A[j](n,d)),
// c[i] = +-2^i with the minus sign on the top plane of a SIGNED operand.
// A BIPOLAR operand x = 2b - 1 is handled with b as its single plane:
//   W bipolar:     acc = sum_j c_a[j] (2 popc(b & A[j]) - popc(A[j]))
//   A bipolar:     acc = sum_i c_w[i] (2 popc(W[i] & b) - popc(W[i]))
//   both bipolar:  acc = K - 2 popc(b_w ^ b_a)          (XNOR-popcount form)
// The popc(A[j]) / popc(W[i]) correction sums are gathered while the tiles are
// staged into shared memory, so they cost 1/64 of the main loop.
//
// Bit-level sparsity (named with the approximate product in the paper's conclusion; this half of
// it is exact): while a 64 x 512-bit tile of a plane is staged the CTA notes whether it holds any
// set bit, and the AND/POPC work of a plane pair is skipped for that depth step when either tile
// is all zero (popc(0 & x) = 0).  Operands whose high-order planes are empty over whole tiles --
// small activations in a wide container, pruned weight blocks -- then cost only their occupied
// planes.  The XNOR form of two bipolar operands has no such zero and is never skipped, and
// kernels with fewer than four plane pairs do not look (the bookkeeping costs 1-2 % of a dense
// product with 4 to 16 pairs, but 6 % of one with two).
//
// Tiling: one CTA (8 warps) per 64 x 64 output tile, depth staged 16 words at a
// time.  Lanes run along the output-channel dimension (rows m0+lane, m0+32+lane)
// so that (a) weight words are read conflict-free from a 17-word-pitch tile while
// activation words are warp-wide broadcasts, and (b) a warp ballot over the
// bits of the 32 lanes' codes is exactly one word of the channel-interleaved
// bit-plane layout of Section 3.2 that the next layer consumes.
#include "common.cuh"

namespace qnn {

constexpr int BS_BM = 64, BS_BN = 64, BS_KT = 16, BS_PITCH = BS_KT + 1, BS_THREADS = 256;
constexpr int BS_TN = 8;   // columns per warp

struct BsParams {
    const uint32_t *W;     // [WB][M][kw]
    const uint32_t *A;     // [AB][N][kw]
    const int32_t *thr;    // [M][n_thr] or null
    void *out;
    int M, N, K, kw;
    int out_bits, out_fmt, ld_out;
    int coef[4][4];        // multiplier of popc(W[i] op A[j])
    int corr[4];           // multiplier of the correction popcounts (modes 1, 2)
    // Implicit convolution (conv != 0): A is the channel-interleaved bit-plane map
    // [AB][B][H][W][cw] itself, and the staging code does the lowering of Section 3.2 on the fly:
    // depth word c of output pixel n is word c % cw of input pixel (oh*stride - pad + kh,
    // ow*stride - pad + kw), (kh, kw) = tap c / cw in raster order; zero outside the image.
    int conv, cv_H, cv_W, cv_cw, cv_KW, cv_stride, cv_pad, cv_OW, cv_OHW;
    long long cv_plane;    // words per plane of the map: B*H*W*cw
};

enum { BS_REGULAR = 0, BS_W_BIPOLAR = 1, BS_A_BIPOLAR = 2, BS_BOTH_BIPOLAR = 3 };

template <int WB, int AB, int MODE>
__global__ void __launch_bounds__(BS_THREADS)
qgemm_bitserial_kernel(const BsParams p) {
    __shared__ uint32_t Ws[WB][BS_BM][BS_PITCH];
    __shared__ uint32_t As[AB][BS_BN][BS_PITCH];
    __shared__ int corr_s[64];
    __shared__ unsigned nz_s[2][2];              // [depth step parity][W, A]: planes with a set bit in the staged tile

    constexpr bool SPARSE = WB * AB >= 4 && MODE != BS_BOTH_BIPOLAR;     // look for empty plane tiles
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m0 = blockIdx.y * BS_BM, n0 = blockIdx.x * BS_BN;
    const int lc = tid & 15, lr = tid >> 4;      // staging: word column, first row

    int acc[2][BS_TN];
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int nn = 0; nn < BS_TN; ++nn) acc[t][nn] = 0;
    int corr_part[4] = {0, 0, 0, 0};             // rows lr, lr+16, lr+32, lr+48
    if (tid < 4) (&nz_s[0][0])[tid] = 0u;
    __syncthreads();

    // implicit convolution: first tap of the four output pixels this thread stages
    int cv_ih0[4], cv_iw0[4];
    long long cv_img[4];
    if (p.conv) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int n = min(n0 + lr + 16 * q, p.N - 1);
            const int b = n / p.cv_OHW, rem = n - b * p.cv_OHW, oh = rem / p.cv_OW, ow = rem - oh * p.cv_OW;
            cv_ih0[q] = oh * p.cv_stride - p.cv_pad;
            cv_iw0[q] = ow * p.cv_stride - p.cv_pad;
            cv_img[q] = (long long)b * p.cv_H * p.cv_W * p.cv_cw;
        }
    }

    for (int kw0 = 0, step = 0; kw0 < p.kw; kw0 += BS_KT, ++step) {
        const int par = step & 1;
        unsigned w_nz = 0, a_nz = 0;             // planes of which this thread staged a non-zero word
        const int c = kw0 + lc;
        const bool c_ok = c < p.kw;
        int cv_kh = 0, cv_kw = 0, cv_word = 0;
        if (p.conv) {
            const int tap = c / p.cv_cw;
            cv_word = c - tap * p.cv_cw;
            cv_kh = tap / p.cv_KW;
            cv_kw = tap - cv_kh * p.cv_KW;
        }
#pragma unroll
        for (int i = 0; i < WB; ++i)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = lr + 16 * q, m = m0 + r;
                uint32_t v = 0;
                if (c_ok && m < p.M) v = p.W[((size_t)i * p.M + m) * p.kw + c];
                Ws[i][r][lc] = v;
                if (SPARSE) w_nz |= v ? (1u << i) : 0u;
                if (MODE == BS_A_BIPOLAR) corr_part[q] += p.corr[i] * __popc(v);
            }
#pragma unroll
        for (int j = 0; j < AB; ++j)
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int r = lr + 16 * q, n = n0 + r;
                uint32_t v = 0;
                if (p.conv) {
                    const int ih = cv_ih0[q] + cv_kh, iw = cv_iw0[q] + cv_kw;
                    if (c_ok && n < p.N && (unsigned)ih < (unsigned)p.cv_H && (unsigned)iw < (unsigned)p.cv_W)
                        v = p.A[(size_t)j * p.cv_plane + cv_img[q] + ((size_t)ih * p.cv_W + iw) * p.cv_cw + cv_word];
                } else if (c_ok && n < p.N) {
                    v = p.A[((size_t)j * p.N + n) * p.kw + c];
                }
                As[j][r][lc] = v;
                if (SPARSE) a_nz |= v ? (1u << j) : 0u;
                if (MODE == BS_W_BIPOLAR) corr_part[q] += p.corr[j] * __popc(v);
            }
        if (SPARSE) {
            w_nz = __reduce_or_sync(0xffffffffu, w_nz);
            a_nz = __reduce_or_sync(0xffffffffu, a_nz);
            if (lane == 0) {
                if (w_nz) atomicOr(&nz_s[par][0], w_nz);
                if (a_nz) atomicOr(&nz_s[par][1], a_nz);
            }
        }
        __syncthreads();
        // plane pairs to run in this depth step: coefficient not zero, both tiles occupied
        unsigned live = 0, wanted = 0;
#pragma unroll
        for (int i = 0; i < WB; ++i)
#pragma unroll
            for (int j = 0; j < AB; ++j) {
                if (p.coef[i][j] == 0) continue;
                wanted |= 1u << (4 * i + j);
                if (!SPARSE || (((nz_s[par][0] >> i) & 1u) && ((nz_s[par][1] >> j) & 1u)))
                    live |= 1u << (4 * i + j);
            }
        if (SPARSE && tid < 2) nz_s[par ^ 1][tid] = 0u;    // the other parity's flags: last read a step ago, next written a step ahead

        // Two copies of the depth step: when every pair with a coefficient runs (dense operands)
        // the loop carries no per-pair test, so it costs what it did without the skipping.
#define QNN_BS_STEP(SKIP_TEST)                                                                         \
        _Pragma("unroll 2")                                                                            \
        for (int cc = 0; cc < BS_KT; ++cc) {                                                           \
            uint32_t wv[2][WB], av[BS_TN][AB];                                                         \
            _Pragma("unroll")                                                                          \
            for (int t = 0; t < 2; ++t)                                                                \
                _Pragma("unroll")                                                                      \
                for (int i = 0; i < WB; ++i) wv[t][i] = Ws[i][lane + 32 * t][cc];                      \
            _Pragma("unroll")                                                                          \
            for (int nn = 0; nn < BS_TN; ++nn)                                                         \
                _Pragma("unroll")                                                                      \
                for (int j = 0; j < AB; ++j) av[nn][j] = As[j][warp * BS_TN + nn][cc];                 \
            /* plane pair outermost: a pair that is left out (uniform) costs one branch */             \
            _Pragma("unroll")                                                                          \
            for (int i = 0; i < WB; ++i)                                                               \
                _Pragma("unroll")                                                                      \
                for (int j = 0; j < AB; ++j) {                                                         \
                    const int cf = p.coef[i][j];                                                       \
                    if (SKIP_TEST) continue;                                                           \
                    _Pragma("unroll")                                                                  \
                    for (int nn = 0; nn < BS_TN; ++nn)                                                 \
                        _Pragma("unroll")                                                              \
                        for (int t = 0; t < 2; ++t) {                                                  \
                            const uint32_t x = (MODE == BS_BOTH_BIPOLAR) ? (wv[t][i] ^ av[nn][j])      \
                                                                          : (wv[t][i] & av[nn][j]);    \
                            acc[t][nn] += cf * __popc(x);                                              \
                        }                                                                              \
                }                                                                                      \
        }
        if (!SPARSE || live == wanted) {
            QNN_BS_STEP(cf == 0)
        } else {
            QNN_BS_STEP(!((live >> (4 * i + j)) & 1u))
        }
#undef QNN_BS_STEP
        __syncthreads();
    }

    pdl_trigger();          // main loop done: the next kernel may start placing its CTAs

    // correction sums: reduce the 16 staging threads that share a row
    if (MODE == BS_W_BIPOLAR || MODE == BS_A_BIPOLAR) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int v = corr_part[q];
#pragma unroll
            for (int off = 8; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (lc == 0) corr_s[lr + 16 * q] = v;
        }
        __syncthreads();
    }

    // epilogue: correction, threshold count, store
    const int n_thr = p.thr ? (1 << p.out_bits) - 1 : 0;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int m = m0 + lane + 32 * t;
        const bool m_ok = m < p.M;
        int thr_r[15];
#pragma unroll
        for (int q = 0; q < 15; ++q)
            thr_r[q] = (m_ok && q < n_thr) ? p.thr[(size_t)m * n_thr + q] : 0x7fffffff;
#pragma unroll
        for (int nn = 0; nn < BS_TN; ++nn) {
            const int nl = warp * BS_TN + nn, n = n0 + nl;
            int a = acc[t][nn];
            if (MODE == BS_W_BIPOLAR) a -= corr_s[nl];
            if (MODE == BS_A_BIPOLAR) a -= corr_s[lane + 32 * t];
            if (MODE == BS_BOTH_BIPOLAR) a += p.K;
            if (n >= p.N) continue;                       // warp-uniform
            if (!p.thr) {
                if (m_ok) reinterpret_cast<int32_t *>(p.out)[(size_t)n * p.M + m] = a;
                continue;
            }
            int code = 0;
#pragma unroll
            for (int q = 0; q < 15; ++q) code += (a >= thr_r[q]) ? 1 : 0;   // pads are INT32_MAX
            if (!m_ok) code = 0;
            if (p.out_fmt == QNN_FMT_INT8) {
                if (m < p.ld_out) reinterpret_cast<uint8_t *>(p.out)[(size_t)n * p.ld_out + m] = (uint8_t)code;
            } else {
                const int mw = (p.M + 31) >> 5, word = (m0 >> 5) + t;
                for (int b = 0; b < p.out_bits; ++b) {
                    const uint32_t bits = __ballot_sync(0xffffffffu, (code >> b) & 1);
                    if (lane == 0 && word < mw)
                        reinterpret_cast<uint32_t *>(p.out)[((size_t)b * p.N + n) * mw + word] = bits;
                }
            }
        }
    }
}

template <int WB, int AB, int MODE>
static void launch_one(const BsParams &p, cudaStream_t s) {
    dim3 grid(ceil_div(p.N, BS_BN), ceil_div(p.M, BS_BM));
    qgemm_bitserial_kernel<WB, AB, MODE><<<grid, BS_THREADS, 0, s>>>(p);
}

template <int MODE>
static bool dispatch_bits(int wb, int ab, const BsParams &p, cudaStream_t s) {
#define QNN_BS_CASE(W_, A_) if (wb == W_ && ab == A_) { launch_one<W_, A_, MODE>(p, s); return true; }
    if (MODE == BS_REGULAR) {
        QNN_BS_CASE(1, 1) QNN_BS_CASE(1, 2) QNN_BS_CASE(1, 3) QNN_BS_CASE(1, 4)
        QNN_BS_CASE(2, 1) QNN_BS_CASE(2, 2) QNN_BS_CASE(2, 3) QNN_BS_CASE(2, 4)
        QNN_BS_CASE(3, 1) QNN_BS_CASE(3, 2) QNN_BS_CASE(3, 3) QNN_BS_CASE(3, 4)
        QNN_BS_CASE(4, 1) QNN_BS_CASE(4, 2) QNN_BS_CASE(4, 3) QNN_BS_CASE(4, 4)
    } else if (MODE == BS_W_BIPOLAR) {
        QNN_BS_CASE(1, 1) QNN_BS_CASE(1, 2) QNN_BS_CASE(1, 3) QNN_BS_CASE(1, 4)
    } else if (MODE == BS_A_BIPOLAR) {
        QNN_BS_CASE(1, 1) QNN_BS_CASE(2, 1) QNN_BS_CASE(3, 1) QNN_BS_CASE(4, 1)
    } else {
        QNN_BS_CASE(1, 1)
    }
#undef QNN_BS_CASE
    return false;
}

// Plane weights: +2^i, minus on the top plane of a SIGNED operand (Algorithm 2).
static void plane_coef(int bits, int enc, int *c) {
    for (int i = 0; i < 4; ++i) c[i] = 0;
    for (int i = 0; i < bits; ++i) c[i] = (enc == QNN_ENC_SIGNED && i == bits - 1) ? -(1 << i) : (1 << i);
}

static qnn_status bs_launch(const qnn_gemm_desc *d, const qnn_conv_desc *cv, const void *W, const void *A,
                            const int32_t *thr, void *out, cudaStream_t s) {
    BsParams p;
    p.W = (const uint32_t *)W; p.A = (const uint32_t *)A; p.thr = thr; p.out = out;
    p.conv = 0; p.cv_H = p.cv_W = p.cv_cw = p.cv_KW = p.cv_stride = p.cv_OW = p.cv_OHW = 1; p.cv_pad = 0; p.cv_plane = 0;
    if (cv) {
        p.conv = 1; p.cv_H = cv->H; p.cv_W = cv->W; p.cv_cw = ceil_div(cv->C, 32); p.cv_KW = cv->KW;
        p.cv_stride = cv->stride; p.cv_pad = cv->pad;
        p.cv_OW = qnn_conv_out_w(cv); p.cv_OHW = qnn_conv_out_h(cv) * p.cv_OW;
        p.cv_plane = (long long)cv->B * cv->H * cv->W * p.cv_cw;
    }
    p.M = d->M; p.N = d->N; p.K = d->K; p.kw = ceil_div(d->K, 32);
    p.out_bits = thr ? d->out_bits : 0;
    p.out_fmt = d->out_fmt;
    p.ld_out = round_up(d->M, 16);
    int cw[4], ca[4];
    plane_coef(d->w_bits, d->w_enc, cw);
    plane_coef(d->a_bits, d->a_enc, ca);
    const bool wb = d->w_enc == QNN_ENC_BIPOLAR, ab = d->a_enc == QNN_ENC_BIPOLAR;
    for (int i = 0; i < 4; ++i) p.corr[i] = 0;
    for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j) p.coef[i][j] = cw[i] * ca[j];
    // plane pairs (i, j) with i + j < skip_planes are left out (a bipolar operand is plane 0)
    const int skip = d->skip_planes;
    for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j)
            if (i + j < skip) p.coef[i][j] = 0;
    bool ok;
    if (wb && ab) {
        p.coef[0][0] = skip > 0 ? 0 : -2;
        if (skip > 0) p.K = 0;                       // the pair's K - 2 popc(xor) goes as a whole
        ok = dispatch_bits<BS_BOTH_BIPOLAR>(1, 1, p, s);
    } else if (wb) {
        for (int j = 0; j < 4; ++j) { p.coef[0][j] = j < skip ? 0 : 2 * ca[j]; p.corr[j] = j < skip ? 0 : ca[j]; }
        ok = dispatch_bits<BS_W_BIPOLAR>(1, d->a_bits, p, s);
    } else if (ab) {
        for (int i = 0; i < 4; ++i) { p.coef[i][0] = i < skip ? 0 : 2 * cw[i]; p.corr[i] = i < skip ? 0 : cw[i]; }
        ok = dispatch_bits<BS_A_BIPOLAR>(d->w_bits, 1, p, s);
    } else {
        ok = dispatch_bits<BS_REGULAR>(d->w_bits, d->a_bits, p, s);
    }
    if (!ok) return QNN_ERR_UNSUPPORTED;
    count_launch();
    return launch_status();
}

qnn_status gemm_bitserial_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                                 const int32_t *thr, void *out, cudaStream_t s) {
    return bs_launch(d, nullptr, W, A, thr, out, s);
}

// Convolution on bit-plane maps without a lowered matrix: the tiled kernel's staging code reads
// the map through the lowering's index arithmetic.  g: the lowered GEMM (N = B*OH*OW,
// K = 32*KH*KW*ceil(C/32)).
qnn_status gemm_bitserial_conv_launch(const qnn_conv_desc *cv, const qnn_gemm_desc *g, const void *W,
                                      const void *in, const int32_t *thr, void *out, cudaStream_t s) {
    if (cv->fmt != QNN_FMT_BITPLANES) return QNN_ERR_UNSUPPORTED;
    return bs_launch(g, cv, W, in, thr, out, s);
}

}  // namespace qnn
