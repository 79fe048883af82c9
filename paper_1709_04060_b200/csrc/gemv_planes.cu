// Bit-serial GEMM for a handful of activation columns (N <= 16), fused with the
// threshold activation.  This is the fully connected layer at small batch of
// Section 4.2 (matrix-vector products, where the paper's packed weights cut the
// memory traffic): the weight bit planes are streamed from HBM exactly once with
// 16-byte loads, the few activation columns sit in shared memory, and
//   acc[m][n] = sum_i sum_j c_w[i] c_a[j] sum_d popc(W[i](m,d) & A[j](n,d))
// (Section 3.1, Algorithms 1 and 2; bipolar operands as in the tiled kernel).
//
// One warp per weight row: lanes stride over the depth words, partial sums meet in
// a shuffle reduction, then lane n counts the thresholds of column n (Section 2.1.1).
// Columns are handled four at a time (blockIdx.y); more than four columns re-read
// the weights from L2.
#include "common.cuh"

namespace qnn {

constexpr int GV_THREADS = 256;
constexpr int GV_COLS = 4;          // columns per CTA

struct GvParams {
    const uint32_t *W;     // [WB][M][kw]
    const uint32_t *A;     // [AB][N][kw]
    const int32_t *thr;    // [M][n_thr] or null
    void *out;
    int M, N, K, kw, kw_pad;   // kw_pad: kw rounded up to 4 (shared-memory row pitch)
    int out_bits, out_fmt, ld_out;
    int coef[4][4];
    int corr[4];
};

enum { GV_REGULAR = 0, GV_W_BIPOLAR = 1, GV_A_BIPOLAR = 2, GV_BOTH_BIPOLAR = 3 };

// At most 36 registers, so that 7 CTAs share an SM: the 1024 CTAs of an 8192-row layer are then
// resident in a single wave (with more registers it took 1.4 waves, i.e. twice the latency chain).
template <int WB, int AB, int MODE, bool VEC>
__global__ void __launch_bounds__(GV_THREADS, 7)
gemv_planes_kernel(const GvParams p) {
    extern __shared__ uint32_t gv_smem[];          // [AB][GV_COLS][kw_pad] activation words
    __shared__ int corr_s[GV_COLS];
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n0 = blockIdx.y * GV_COLS;
    const int ncols = min(GV_COLS, p.N - n0);

    // stage this CTA's activation columns (zero padded) and their correction sums
    if (threadIdx.x < GV_COLS) corr_s[threadIdx.x] = 0;
    __syncthreads();
    for (int j = 0; j < AB; ++j)
        for (int c = 0; c < ncols; ++c) {                 // only the columns in use
            int part = 0;
            for (int d = threadIdx.x; d < p.kw_pad; d += GV_THREADS) {
                uint32_t v = 0;
                if (d < p.kw) v = p.A[((size_t)j * p.N + n0 + c) * p.kw + d];
                gv_smem[(j * GV_COLS + c) * p.kw_pad + d] = v;
                part += p.corr[j] * __popc(v);
            }
            if (MODE == GV_W_BIPOLAR) {
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                if (lane == 0 && part != 0) atomicAdd(&corr_s[c], part);
            }
        }
    __syncthreads();

    const int n_thr = p.thr ? (1 << p.out_bits) - 1 : 0;
    const int rows_per_grid = gridDim.x * (GV_THREADS / 32);
    for (int m = blockIdx.x * (GV_THREADS / 32) + warp; m < p.M; m += rows_per_grid) {
        int acc[GV_COLS];
#pragma unroll
        for (int c = 0; c < GV_COLS; ++c) acc[c] = 0;
        int wcorr = 0;                              // A bipolar: sum_i corr[i] * popc(W[i] row)

        if (VEC) {
            // kw a multiple of 4: a lane takes 4 consecutive words per step
            const int steps = p.kw >> 2;
#pragma unroll 2
            for (int q = lane; q < steps; q += 32) {
                uint4 wv[WB];
#pragma unroll
                for (int i = 0; i < WB; ++i)
                    wv[i] = __ldcs(reinterpret_cast<const uint4 *>(p.W + ((size_t)i * p.M + m) * p.kw) + q);
                if (MODE == GV_A_BIPOLAR) {
#pragma unroll
                    for (int i = 0; i < WB; ++i)
                        wcorr += p.corr[i] * (__popc(wv[i].x) + __popc(wv[i].y) + __popc(wv[i].z) + __popc(wv[i].w));
                }
#pragma unroll
                for (int c = 0; c < GV_COLS; ++c) {
                    if (c < ncols) {
#pragma unroll
                        for (int j = 0; j < AB; ++j) {
                            const uint4 av = *reinterpret_cast<const uint4 *>(
                                gv_smem + (j * GV_COLS + c) * p.kw_pad + 4 * q);
#pragma unroll
                            for (int i = 0; i < WB; ++i) {
                                if (p.coef[i][j] == 0) continue;   // a plane pair that is left out (uniform)
                                int cnt;
                                if (MODE == GV_BOTH_BIPOLAR)
                                    cnt = __popc(wv[i].x ^ av.x) + __popc(wv[i].y ^ av.y) +
                                          __popc(wv[i].z ^ av.z) + __popc(wv[i].w ^ av.w);
                                else
                                    cnt = __popc(wv[i].x & av.x) + __popc(wv[i].y & av.y) +
                                          __popc(wv[i].z & av.z) + __popc(wv[i].w & av.w);
                                acc[c] += p.coef[i][j] * cnt;
                            }
                        }
                    }
                }
            }
        } else {
            for (int d = lane; d < p.kw; d += 32) {
                uint32_t wv[WB];
#pragma unroll
                for (int i = 0; i < WB; ++i) wv[i] = p.W[((size_t)i * p.M + m) * p.kw + d];
                if (MODE == GV_A_BIPOLAR) {
#pragma unroll
                    for (int i = 0; i < WB; ++i) wcorr += p.corr[i] * __popc(wv[i]);
                }
#pragma unroll
                for (int c = 0; c < GV_COLS; ++c) {
                    if (c < ncols) {
#pragma unroll
                        for (int j = 0; j < AB; ++j) {
                            const uint32_t av = gv_smem[(j * GV_COLS + c) * p.kw_pad + d];
#pragma unroll
                            for (int i = 0; i < WB; ++i) {
                                if (p.coef[i][j] == 0) continue;
                                const uint32_t x = (MODE == GV_BOTH_BIPOLAR) ? (wv[i] ^ av) : (wv[i] & av);
                                acc[c] += p.coef[i][j] * __popc(x);
                            }
                        }
                    }
                }
            }
        }

        // warp reduction; afterwards every lane holds the full sums
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
#pragma unroll
            for (int c = 0; c < GV_COLS; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], off);
            if (MODE == GV_A_BIPOLAR) wcorr += __shfl_xor_sync(0xffffffffu, wcorr, off);
        }

        // lane c finishes column n0 + c
        int a = 0;
#pragma unroll
        for (int c = 0; c < GV_COLS; ++c)
            if (lane == c) a = acc[c];
        if (lane < ncols) {
            const int n = n0 + lane;
            if (MODE == GV_W_BIPOLAR) a -= corr_s[lane];
            if (MODE == GV_A_BIPOLAR) a -= wcorr;
            if (MODE == GV_BOTH_BIPOLAR) a += p.K;
            if (!p.thr) {
                reinterpret_cast<int32_t *>(p.out)[(size_t)n * p.M + m] = a;
            } else {
                int code = 0;
                for (int q = 0; q < n_thr; ++q) code += (a >= __ldg(p.thr + (size_t)m * n_thr + q)) ? 1 : 0;
                if (p.out_fmt == QNN_FMT_INT8) {
                    reinterpret_cast<uint8_t *>(p.out)[(size_t)n * p.ld_out + m] = (uint8_t)code;
                } else {
                    // bit-plane words are shared by 32 rows that other warps own: set single bits
                    const int mw = (p.M + 31) >> 5;
                    for (int b = 0; b < p.out_bits; ++b)
                        if ((code >> b) & 1)
                            atomicOr(reinterpret_cast<uint32_t *>(p.out) + ((size_t)b * p.N + n) * mw + (m >> 5),
                                     1u << (m & 31));
                }
            }
        }
    }
    pdl_trigger();
}

// Clears the output before the kernel sets bits (bit-plane output) or leaves pad
// bytes untouched (8-bit output: pad bytes of a row are zeroed here).
__global__ void gemv_clear_kernel(uint32_t *out, long long words) {
    pdl_enter();
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < words;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0u;
}

template <int WB, int AB, int MODE>
static void gv_launch_one(const GvParams &p, dim3 grid, size_t smem, cudaStream_t s) {
    if ((p.kw & 3) == 0) gemv_planes_kernel<WB, AB, MODE, true><<<grid, GV_THREADS, smem, s>>>(p);
    else gemv_planes_kernel<WB, AB, MODE, false><<<grid, GV_THREADS, smem, s>>>(p);
}

template <int MODE>
static bool gv_dispatch(int wb, int ab, const GvParams &p, dim3 grid, size_t smem, cudaStream_t s) {
#define QNN_GV_CASE(W_, A_) if (wb == W_ && ab == A_) { gv_launch_one<W_, A_, MODE>(p, grid, smem, s); return true; }
    if (MODE == GV_REGULAR) {
        QNN_GV_CASE(1, 1) QNN_GV_CASE(1, 2) QNN_GV_CASE(1, 3) QNN_GV_CASE(1, 4)
        QNN_GV_CASE(2, 1) QNN_GV_CASE(2, 2) QNN_GV_CASE(2, 3) QNN_GV_CASE(2, 4)
        QNN_GV_CASE(3, 1) QNN_GV_CASE(3, 2) QNN_GV_CASE(3, 3) QNN_GV_CASE(3, 4)
        QNN_GV_CASE(4, 1) QNN_GV_CASE(4, 2) QNN_GV_CASE(4, 3) QNN_GV_CASE(4, 4)
    } else if (MODE == GV_W_BIPOLAR) {
        QNN_GV_CASE(1, 1) QNN_GV_CASE(1, 2) QNN_GV_CASE(1, 3) QNN_GV_CASE(1, 4)
    } else if (MODE == GV_A_BIPOLAR) {
        QNN_GV_CASE(1, 1) QNN_GV_CASE(2, 1) QNN_GV_CASE(3, 1) QNN_GV_CASE(4, 1)
    } else {
        QNN_GV_CASE(1, 1)
    }
#undef QNN_GV_CASE
    return false;
}

// N <= 16 and the activation columns of one CTA fit the default 48 KB of shared memory.
bool gemv_planes_fits(const qnn_gemm_desc *d) {
    const int kw_pad = round_up(ceil_div(d->K, 32), 4);
    return d->N <= 16 && (size_t)d->a_bits * GV_COLS * kw_pad * 4 <= 48 * 1024;
}

qnn_status gemv_planes_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                              const int32_t *thr, void *out, cudaStream_t s) {
    GvParams p;
    p.W = (const uint32_t *)W; p.A = (const uint32_t *)A; p.thr = thr; p.out = out;
    p.M = d->M; p.N = d->N; p.K = d->K; p.kw = ceil_div(d->K, 32); p.kw_pad = round_up(p.kw, 4);
    p.out_bits = thr ? d->out_bits : 0;
    p.out_fmt = d->out_fmt;
    p.ld_out = round_up(d->M, 16);
    int cw[4], ca[4];
    for (int i = 0; i < 4; ++i) {
        cw[i] = i < d->w_bits ? ((d->w_enc == QNN_ENC_SIGNED && i == d->w_bits - 1) ? -(1 << i) : (1 << i)) : 0;
        ca[i] = i < d->a_bits ? ((d->a_enc == QNN_ENC_SIGNED && i == d->a_bits - 1) ? -(1 << i) : (1 << i)) : 0;
        p.corr[i] = 0;
    }
    for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j) p.coef[i][j] = cw[i] * ca[j];
    const bool wb = d->w_enc == QNN_ENC_BIPOLAR, ab = d->a_enc == QNN_ENC_BIPOLAR;

    // outputs that are only partly written by the main kernel are cleared first
    int launches = 1;
    if (thr) {
        long long words = 0;
        if (d->out_fmt == QNN_FMT_BITPLANES) words = (long long)d->out_bits * d->N * ceil_div(d->M, 32);
        else if (p.ld_out != d->M) words = (long long)d->N * p.ld_out / 4;
        if (words > 0) {
            const long long blocks = (words + 255) / 256;
            gemv_clear_kernel<<<(unsigned)(blocks < 1184 ? blocks : 1184), 256, 0, s>>>((uint32_t *)out, words);
            ++launches;
        }
    }

    const size_t smem = (size_t)d->a_bits * GV_COLS * p.kw_pad * 4;     // [plane][column slot][word]
    const int row_blocks = ceil_div(d->M, GV_THREADS / 32);
    const int max_blocks = sm_count() * 8;
    dim3 grid(row_blocks < max_blocks ? row_blocks : max_blocks, ceil_div(d->N, GV_COLS));
    // plane pairs (i, j) with i + j < skip_planes are left out (a bipolar operand is plane 0)
    const int skip = d->skip_planes;
    for (int i = 0; i < 4; ++i)
        for (int j = 0; j < 4; ++j)
            if (i + j < skip) p.coef[i][j] = 0;
    bool ok;
    if (wb && ab) {
        p.coef[0][0] = skip > 0 ? 0 : -2;
        if (skip > 0) p.K = 0;                       // the pair's K - 2 popc(xor) goes as a whole
        ok = gv_dispatch<GV_BOTH_BIPOLAR>(1, 1, p, grid, smem, s);
    } else if (wb) {
        for (int j = 0; j < 4; ++j) { p.coef[0][j] = j < skip ? 0 : 2 * ca[j]; p.corr[j] = j < skip ? 0 : ca[j]; }
        ok = gv_dispatch<GV_W_BIPOLAR>(1, d->a_bits, p, grid, smem, s);
    } else if (ab) {
        for (int i = 0; i < 4; ++i) { p.coef[i][0] = i < skip ? 0 : 2 * cw[i]; p.corr[i] = i < skip ? 0 : cw[i]; }
        ok = gv_dispatch<GV_A_BIPOLAR>(d->w_bits, 1, p, grid, smem, s);
    } else {
        ok = gv_dispatch<GV_REGULAR>(d->w_bits, d->a_bits, p, grid, smem, s);
    }
    if (!ok) return QNN_ERR_UNSUPPORTED;
    count_launch(launches);
    return launch_status();
}

}  // namespace qnn
