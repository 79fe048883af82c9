// GEMM for a handful of activation columns (N <= 8) on 8-bit containers, fused with the
// threshold activation: the fully connected layer at small batch of Section 4.2 when the
// operands are held as bytes (the 8-bit last layer, or few-bit values in 8-bit containers
// as in Section 3).  With so few columns a 128-pixel tensor-core tile would be almost
// empty and its depth loop is one long serial chain, so here one warp owns a weight row,
// streams it once with 16-byte loads and multiplies with 4-way byte dot products (dp4a)
// against the columns held in shared memory; a shuffle reduction and the threshold count
// T(x, t) of Section 2.1.1 finish the row.  Columns are handled four at a time
// (blockIdx.y).  The result is the exact int32 product of Section 3.1.
#include "common.cuh"

namespace qnn {

constexpr int G8_THREADS = 256;
constexpr int G8_COLS = 4;

struct G8Params {
    const uint8_t *W;      // [M][ld]
    const uint8_t *A;      // [N][ld]
    const int32_t *thr;    // [M][n_thr] or null
    void *out;
    int M, N, ld;          // ld: K rounded up to 16, pad bytes zero in both operands
    int out_bits, out_fmt, ld_out;
};

template <bool W_SIGNED, bool A_SIGNED>
__device__ __forceinline__ int dot4(uint32_t w, uint32_t a, int c) {
    int d;
    if (W_SIGNED && A_SIGNED) asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(a), "r"(c));
    else if (W_SIGNED) asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(a), "r"(c));
    else if (A_SIGNED) asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(a), "r"(c));
    else asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(a), "r"(c));
    return d;
}

// At most 36 registers, so that 7 CTAs share an SM and the 1024 CTAs of an 8192-row layer are
// resident in a single wave.
template <bool W_SIGNED, bool A_SIGNED, int V>
__global__ void __launch_bounds__(G8_THREADS, 7)
gemv_i8_kernel(const G8Params p) {
    extern __shared__ __align__(16) uint8_t g8_smem[];     // [G8_COLS][ld] activation bytes
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n0 = blockIdx.y * G8_COLS;
    const int ncols = min(G8_COLS, p.N - n0);
    const int steps = p.ld >> 4;                           // 16-byte steps per row

    for (int idx = threadIdx.x; idx < ncols * steps; idx += G8_THREADS) {      // only the columns in use
        const int c = idx / steps, q = idx - c * steps;
        reinterpret_cast<uint4 *>(g8_smem)[idx] = reinterpret_cast<const uint4 *>(p.A + (size_t)(n0 + c) * p.ld)[q];
    }
    __syncthreads();

    const int n_thr = p.thr ? (1 << p.out_bits) - 1 : 0;
    const int rows_per_grid = gridDim.x * (G8_THREADS / 32);
    for (int m = blockIdx.x * (G8_THREADS / 32) + warp; m < p.M; m += rows_per_grid) {
        int acc[G8_COLS];
#pragma unroll
        for (int c = 0; c < G8_COLS; ++c) acc[c] = 0;
        const uint4 *wrow = reinterpret_cast<const uint4 *>(p.W + (size_t)m * p.ld);
        // a lane takes V consecutive 16-byte units per step (whole sectors; a warp 512 V bytes)
        const int groups = steps / V;
#pragma unroll 2
        for (int q = lane; q < groups; q += 32) {
            uint4 w[V];
#pragma unroll
            for (int v = 0; v < V; ++v) w[v] = __ldcs(wrow + V * q + v);
#pragma unroll
            for (int c = 0; c < G8_COLS; ++c) {
                if (c < ncols) {
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const uint4 a = reinterpret_cast<const uint4 *>(g8_smem)[c * steps + V * q + v];
                        acc[c] = dot4<W_SIGNED, A_SIGNED>(w[v].x, a.x, acc[c]);
                        acc[c] = dot4<W_SIGNED, A_SIGNED>(w[v].y, a.y, acc[c]);
                        acc[c] = dot4<W_SIGNED, A_SIGNED>(w[v].z, a.z, acc[c]);
                        acc[c] = dot4<W_SIGNED, A_SIGNED>(w[v].w, a.w, acc[c]);
                    }
                }
            }
        }
        for (int q = groups * V + lane; q < steps; q += 32) {      // what is left of the row
            const uint4 w = __ldcs(wrow + q);
#pragma unroll
            for (int c = 0; c < G8_COLS; ++c) {
                if (c < ncols) {
                    const uint4 a = reinterpret_cast<const uint4 *>(g8_smem)[c * steps + q];
                    acc[c] = dot4<W_SIGNED, A_SIGNED>(w.x, a.x, acc[c]);
                    acc[c] = dot4<W_SIGNED, A_SIGNED>(w.y, a.y, acc[c]);
                    acc[c] = dot4<W_SIGNED, A_SIGNED>(w.z, a.z, acc[c]);
                    acc[c] = dot4<W_SIGNED, A_SIGNED>(w.w, a.w, acc[c]);
                }
            }
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1)
#pragma unroll
            for (int c = 0; c < G8_COLS; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], off);

        int a = 0;                                         // lane c finishes column n0 + c
#pragma unroll
        for (int c = 0; c < G8_COLS; ++c)
            if (lane == c) a = acc[c];
        if (lane < ncols) {
            const int n = n0 + lane;
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

__global__ void gemv_i8_clear_kernel(uint32_t *out, long long words) {
    pdl_enter();
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < words;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0u;
}

// N <= 8 (beyond that the shared-memory reads of the columns cost more than an almost
// empty tensor-core tile) and four activation columns fit the default 48 KB of shared memory.
bool gemv_i8_fits(const qnn_gemm_desc *d) {
    return d->N <= 8 && (size_t)G8_COLS * round_up(d->K, 16) <= 48 * 1024;
}

qnn_status gemv_i8_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                          const int32_t *thr, void *out, cudaStream_t s) {
    G8Params p;
    p.W = (const uint8_t *)W; p.A = (const uint8_t *)A; p.thr = thr; p.out = out;
    p.M = d->M; p.N = d->N; p.ld = round_up(d->K, 16);
    p.out_bits = thr ? d->out_bits : 0;
    p.out_fmt = d->out_fmt;
    p.ld_out = round_up(d->M, 16);

    // outputs that the main kernel writes only in part are cleared first
    int launches = 1;
    if (thr) {
        long long words = 0;
        if (d->out_fmt == QNN_FMT_BITPLANES) words = (long long)d->out_bits * d->N * ceil_div(d->M, 32);
        else if (p.ld_out != d->M) words = (long long)d->N * p.ld_out / 4;
        if (words > 0) {
            const long long blocks = (words + 255) / 256;
            gemv_i8_clear_kernel<<<(unsigned)(blocks < 1184 ? blocks : 1184), 256, 0, s>>>((uint32_t *)out, words);
            ++launches;
        }
    }
    const size_t smem = (size_t)(d->N < G8_COLS ? d->N : G8_COLS) * p.ld;    // only the columns in use
    const int row_blocks = ceil_div(d->M, G8_THREADS / 32);
    const int max_blocks = sm_count() * 8;
    dim3 grid(row_blocks < max_blocks ? row_blocks : max_blocks, ceil_div(d->N, G8_COLS));
    const bool ws = d->w_enc != QNN_ENC_UNSIGNED, as = d->a_enc != QNN_ENC_UNSIGNED;
    // measured at 8192 x 8192: one column is fastest with 32 bytes per lane and step (16.0 us
    // against 20.5 with 16 and 21.2 with 64), several columns with 16
#define QNN_G8_LAUNCH(WS_, AS_)                                                                 \
    do {                                                                                        \
        if (d->N == 1) gemv_i8_kernel<WS_, AS_, 2><<<grid, G8_THREADS, smem, s>>>(p);           \
        else gemv_i8_kernel<WS_, AS_, 1><<<grid, G8_THREADS, smem, s>>>(p);                     \
    } while (0)
    if (ws && as) QNN_G8_LAUNCH(true, true);
    else if (ws) QNN_G8_LAUNCH(true, false);
    else if (as) QNN_G8_LAUNCH(false, true);
    else QNN_G8_LAUNCH(false, false);
#undef QNN_G8_LAUNCH
    count_launch(launches);
    return launch_status();
}

}  // namespace qnn
