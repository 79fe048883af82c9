/*
 * CPU oracle for streamlined few-bit QNN inference.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product (CUDA) path may include, link or call this file.
 *
 * Every function is the plain definition of the quantity, written as direct
 * loops on LOGICAL integer values (one int32 per element, never packed):
 * no blocking, no bit tricks, no SIMD intrinsics.  OpenMP is used only as a
 * `parallel for` over independent output rows.
 *
 * The paper's bit-serial GEMM (Section 3.1, Algorithms 1 and 2) is an exact
 * identity for the integer matrix product  W.A = sum_i sum_j 2^(i+j) W[i].A[j],
 * so the oracle for it is the integer matrix product itself.
 *
 * Layout conventions (the paper's Algorithm 1 indexes both operands as
 * (row-or-column, depth), i.e. the activation matrix is held transposed):
 *   W   int32 [M][K]   rows x depth
 *   At  int32 [N][K]   cols x depth   (A transposed, depth contiguous)
 *   acc int64 [M][N]
 */
#include <stdint.h>
#include <stddef.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One accumulator: acc = sum_k W[m][k] * A[k][n].  Section 3.1: the result the
 * weighted sum over bit-plane pairs must reproduce. */
int64_t orc_dot_i64(const int32_t *w_row, const int32_t *a_col, int64_t K)
{
    int64_t s = 0;
    for (int64_t k = 0; k < K; ++k)
        s += (int64_t)w_row[k] * (int64_t)a_col[k];
    return s;
}

/* Integer matrix product, triple loop in the order of Algorithm 1
 * (rows, cols, depth).  Section 3.1. */
void orc_gemm_i64(const int32_t *W, const int32_t *At,
                  int64_t M, int64_t N, int64_t K, int64_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < M; ++r)
        for (int64_t c = 0; c < N; ++c) {
            int64_t s = 0;
            for (int64_t d = 0; d < K; ++d)
                s += (int64_t)W[r * K + d] * (int64_t)At[c * K + d];
            acc[r * N + c] = s;
        }
}

/* Successive thresholding T(x, t), Section 2.1.1: the returned integer is the
 * number of thresholds that x is greater than or equal to.  thr is
 * [M][n_thr] (one threshold set per output row / channel), out is [M][N]. */
void orc_threshold(const int64_t *acc, const int32_t *thr,
                   int64_t M, int64_t N, int64_t n_thr, int32_t *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < M; ++r)
        for (int64_t c = 0; c < N; ++c) {
            int32_t cnt = 0;
            for (int64_t i = 0; i < n_thr; ++i)
                if (acc[r * N + c] >= (int64_t)thr[r * n_thr + i])
                    ++cnt;
            out[r * N + c] = cnt;
        }
}

/* Direct convolution (no lowering), the definition that the lowered GEMM of
 * Section 3.2 must reproduce.  Channels-last ("channel-interleaved") tensors:
 *   In  int32 [B][H][Wd][C]
 *   Wt  int32 [OC][KH][KW][C]
 *   acc int64 [B][OH][OW][OC],  OH = (H + 2*pad - KH)/stride + 1
 * Taps that fall outside the image contribute zero. */
void orc_conv_direct(const int32_t *In, const int32_t *Wt,
                     int64_t B, int64_t H, int64_t Wd, int64_t C,
                     int64_t OC, int64_t KH, int64_t KW,
                     int64_t stride, int64_t pad, int64_t *acc)
{
    const int64_t OH = (H + 2 * pad - KH) / stride + 1;
    const int64_t OW = (Wd + 2 * pad - KW) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t oh = 0; oh < OH; ++oh)
            for (int64_t ow = 0; ow < OW; ++ow)
                for (int64_t oc = 0; oc < OC; ++oc) {
                    int64_t s = 0;
                    for (int64_t kh = 0; kh < KH; ++kh) {
                        const int64_t ih = oh * stride - pad + kh;
                        if (ih < 0 || ih >= H) continue;
                        for (int64_t kw = 0; kw < KW; ++kw) {
                            const int64_t iw = ow * stride - pad + kw;
                            if (iw < 0 || iw >= Wd) continue;
                            const int32_t *px = In + ((b * H + ih) * Wd + iw) * C;
                            const int32_t *wt = Wt + ((oc * KH + kh) * KW + kw) * C;
                            for (int64_t c = 0; c < C; ++c)
                                s += (int64_t)wt[c] * (int64_t)px[c];
                        }
                    }
                    acc[((b * OH + oh) * OW + ow) * OC + oc] = s;
                }
}

/* Per-channel thresholding of a channels-last accumulator tensor:
 * acc [P][OC] (P = B*OH*OW pixels), thr [OC][n_thr], out [P][OC].
 * Same T(x, t) as orc_threshold, Section 2.1.1. */
void orc_threshold_nhwc(const int64_t *acc, const int32_t *thr,
                        int64_t P, int64_t OC, int64_t n_thr, int32_t *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p)
        for (int64_t oc = 0; oc < OC; ++oc) {
            int32_t cnt = 0;
            for (int64_t i = 0; i < n_thr; ++i)
                if (acc[p * OC + oc] >= (int64_t)thr[oc * n_thr + i])
                    ++cnt;
            out[p * OC + oc] = cnt;
        }
}

/* Max-pooling on integer activations (Section 4.2 lists it among the cheap
 * non-matrix layers): window k x k, stride s, no padding, floor:
 * OH = (H - k)/s + 1.  In/out are channels-last int32. */
void orc_maxpool(const int32_t *In, int64_t B, int64_t H, int64_t Wd, int64_t C,
                 int64_t k, int64_t s, int32_t *out)
{
    const int64_t OH = (H - k) / s + 1;
    const int64_t OW = (Wd - k) / s + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t oh = 0; oh < OH; ++oh)
            for (int64_t ow = 0; ow < OW; ++ow)
                for (int64_t c = 0; c < C; ++c) {
                    int32_t best = In[((b * H + oh * s) * Wd + ow * s) * C + c];
                    for (int64_t i = 0; i < k; ++i)
                        for (int64_t j = 0; j < k; ++j) {
                            const int32_t v =
                                In[((b * H + oh * s + i) * Wd + ow * s + j) * C + c];
                            if (v > best) best = v;
                        }
                    out[((b * OH + oh) * OW + ow) * C + c] = best;
                }
}
