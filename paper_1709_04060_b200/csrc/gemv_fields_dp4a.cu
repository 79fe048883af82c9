// Packed w-bit weights (QNN_FMT_FIELDS) times a handful of activation columns on the CUDA cores,
// fused with the threshold activation: the fully connected layer at small batch of Section 4.2,
// whose gain the paper attributes to the cut in memory traffic that packed weights bring.
//
// One warp owns a weight row and streams its packed bytes once with 16-byte loads.  A 32-bit word
// of packed weights ANDed with the mask of field position s is four 8-bit values, each the field
// times 2^(f s), that belong to four consecutive depth indices (that is what the FIELDS layout is
// for), so one AND and one 4-way byte dot product (dp4a) per word, field position and column do the
// work; every field position has its own accumulator, which holds an exact multiple of 2^(f s) and
// is shifted back before the warp's shuffle reduction.  The activation columns (8-bit containers)
// sit in shared memory, laid out with 32 pad bytes per group of 32 S depth indices so that the
// 16-byte reads of a warp (lanes 16 packed bytes apart = 16 S depth indices apart per field
// position) fall into different banks.  Fields hold value minus the encoding's minimum; the
// column sums that the correction needs are taken while the columns are staged.  Exact int32
// results (Section 3.1), thresholds counted as T(x, t) of Section 2.1.1.
//
// Against the tensor-core form of the same product (gemv_fields.cu) this kernel has no serial
// per-SM pipeline to fill, but every further column adds its shared-memory reads and dot products
// to each warp's dependent chain (about 4 us per column at 8192 x 8192; the counters show load
// latency, global and shared, not a saturated pipe), so it is the faster one for one column
// (7.0 / 9.4 us against 12.5 / 14.7 us at 8192 x 8192 with 2- / 4-bit fields) and for two
// (11.2 / 11.7 us against 12.7 / 15.0 us).
#include <stdlib.h>

#include "common.cuh"

namespace qnn {

constexpr int FD_THREADS = 256;
constexpr int FD_COLS = 4;            // most columns per CTA (blockIdx.y picks the block of columns)
constexpr int FD_MAX_N = 2;           // more columns: the tensor-core form

struct FdParams {
    const uint8_t *W;      // [M][ldf] packed fields
    const uint8_t *A;      // [N][lda] 8-bit containers
    const int32_t *thr;    // [M][n_thr] or null
    void *out;
    int M, N, K;
    int ldf, lda;          // bytes per packed weight row, per activation column
    int steps;             // 16-byte units per packed row (ldf / 16)
    int col_bytes;         // shared-memory bytes per staged column (depth + pads)
    int cols_alloc;        // columns that shared memory has room for (min(N, FD_COLS))
    int w_scale, w_off;    // true weight = w_scale * field + w_off
    int out_bits, out_fmt, ld_out;
};

// Rows a warp takes at a time: two (measured faster) for 2-bit fields x 1 column and 4-bit fields x 2.
__host__ __device__ constexpr int fd_rows_at_a_time(int F, int NC) { return (8 / F) * NC == 4 ? 2 : 1; }

template <bool A_SIGNED>
__device__ __forceinline__ int fd_dot4(uint32_t w, uint32_t a, int c) {
    int d;
    if (A_SIGNED) asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(a), "r"(c));
    else asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(w), "r"(a), "r"(c));
    return d;
}

// F: bits per field (1, 2, 4); S = 8 / F field positions per byte; NC: columns per CTA (1, 2, 4:
// fewer columns, fewer registers, more warps per SM with loads in flight).  Shared memory:
// [cols_alloc][col_bytes] columns, then FD_COLS column sums.
template <int F, bool A_SIGNED, int NC>
__global__ void __launch_bounds__(FD_THREADS, 4)
gemv_fields_dp4a_kernel(const FdParams p) {
    constexpr int S = 8 / F;
    constexpr int R = fd_rows_at_a_time(F, NC);
    constexpr uint32_t MASK = (F == 1 ? 0x01010101u : (F == 2 ? 0x03030303u : 0x0f0f0f0fu));
    constexpr int GROUP = 32 * S;                 // depth indices per 32 packed bytes
    constexpr int GSTRIDE = GROUP + 32;           // their stride in shared memory
    extern __shared__ __align__(16) uint8_t fd_smem[];
    int *colsum = reinterpret_cast<int *>(fd_smem + (size_t)p.cols_alloc * p.col_bytes);
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n0 = blockIdx.y * NC;
    const int ncols = min(NC, p.N - n0);
    const int rows_per_grid = gridDim.x * (FD_THREADS / 32);
    const int m_first = blockIdx.x * (FD_THREADS / 32) + warp;
    // the first row's packed bytes are requested before the columns are staged
    uint4 w_first = make_uint4(0, 0, 0, 0);
    if (m_first < p.M && lane < p.steps) w_first = __ldcs(reinterpret_cast<const uint4 *>(p.W + (size_t)m_first * p.ldf) + lane);

    // ---- stage the columns (depth index k at k + 32 * (k / GROUP); zeros past the column's bytes)
    if (threadIdx.x < FD_COLS) colsum[threadIdx.x] = 0;
    __syncthreads();
    {
        const int units = p.steps * S;                               // 16-byte units of depth that the packed rows cover
        for (int c = 0; c < ncols; ++c) {
            int sum = 0;
            for (int u = threadIdx.x; u < units; u += FD_THREADS) {
                const int k = 16 * u;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (k < p.lda) v = *reinterpret_cast<const uint4 *>(p.A + (size_t)(n0 + c) * p.lda + k);
                *reinterpret_cast<uint4 *>(fd_smem + (size_t)c * p.col_bytes + k + 32 * (k / GROUP)) = v;
                sum = fd_dot4<A_SIGNED>(0x01010101u, v.x, sum);
                sum = fd_dot4<A_SIGNED>(0x01010101u, v.y, sum);
                sum = fd_dot4<A_SIGNED>(0x01010101u, v.z, sum);
                sum = fd_dot4<A_SIGNED>(0x01010101u, v.w, sum);
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            if (lane == 0) atomicAdd(&colsum[c], sum);
        }
    }
    __syncthreads();

    const int n_thr = p.thr ? (1 << p.out_bits) - 1 : 0;
    // R rows at a time: their loads are in flight together and they share the reads of the columns
    for (int m = m_first; m < p.M; m += R * rows_per_grid) {
        int acc[R][NC][S];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int c = 0; c < NC; ++c)
#pragma unroll
                for (int s = 0; s < S; ++s) acc[r][c][s] = 0;
        const uint4 *wrow[R];
        bool row_ok[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            row_ok[r] = m + r * rows_per_grid < p.M;
            wrow[r] = reinterpret_cast<const uint4 *>(p.W + (size_t)(row_ok[r] ? m + r * rows_per_grid : m) * p.ldf);
        }
#pragma unroll 4
        for (int q = lane; q < p.steps; q += 32) {
            uint4 w[R];
#pragma unroll
            for (int r = 0; r < R; ++r) w[r] = (r == 0 && m == m_first && q == lane) ? w_first : __ldcs(wrow[r] + q);
            // 16 packed bytes = one half (q & 1) of group q / 2: field position s of these bytes is
            // depth GROUP * (q / 2) + 32 s + 16 (q & 1) .. + 15
            const uint8_t *a0 = fd_smem + (q >> 1) * GSTRIDE + 16 * (q & 1);
#pragma unroll
            for (int s = 0; s < S; ++s) {
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    if (NC == 1 || c < ncols) {
                        const uint4 a = *reinterpret_cast<const uint4 *>(a0 + (size_t)c * p.col_bytes + 32 * s);
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            acc[r][c][s] = fd_dot4<A_SIGNED>(w[r].x & (MASK << (F * s)), a.x, acc[r][c][s]);
                            acc[r][c][s] = fd_dot4<A_SIGNED>(w[r].y & (MASK << (F * s)), a.y, acc[r][c][s]);
                            acc[r][c][s] = fd_dot4<A_SIGNED>(w[r].z & (MASK << (F * s)), a.z, acc[r][c][s]);
                            acc[r][c][s] = fd_dot4<A_SIGNED>(w[r].w & (MASK << (F * s)), a.w, acc[r][c][s]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (!row_ok[r]) continue;                      // warp-uniform
            const int mr = m + r * rows_per_grid;
            int tot[NC];
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                tot[c] = 0;
#pragma unroll
                for (int s = 0; s < S; ++s) tot[c] += acc[r][c][s] >> (F * s);       // exact: a multiple of 2^(F s)
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1)
#pragma unroll
                for (int c = 0; c < NC; ++c) tot[c] += __shfl_xor_sync(0xffffffffu, tot[c], off);

            int a = 0;                                     // lane c finishes column n0 + c
#pragma unroll
            for (int c = 0; c < NC; ++c)
                if (lane == c) a = tot[c];
            if (lane < ncols) {
                a = p.w_scale * a + p.w_off * colsum[lane];
                const int n = n0 + lane;
                if (!p.thr) {
                    reinterpret_cast<int32_t *>(p.out)[(size_t)n * p.M + mr] = a;
                } else {
                    int code = 0;
                    for (int q = 0; q < n_thr; ++q) code += (a >= __ldg(p.thr + (size_t)mr * n_thr + q)) ? 1 : 0;
                    if (p.out_fmt == QNN_FMT_INT8) {
                        uint8_t *o = reinterpret_cast<uint8_t *>(p.out) + (size_t)n * p.ld_out;
                        o[mr] = (uint8_t)code;
                        if (mr == p.M - 1)                     // the pad bytes of the column
                            for (int mm = p.M; mm < p.ld_out; ++mm) o[mm] = 0;
                    } else {
                        // bit-plane words are shared by 32 rows that other warps own: set single bits
                        const int mw = (p.M + 31) >> 5;
                        for (int b = 0; b < p.out_bits; ++b)
                            if ((code >> b) & 1)
                                atomicOr(reinterpret_cast<uint32_t *>(p.out) + ((size_t)b * p.N + n) * mw + (mr >> 5),
                                         1u << (mr & 31));
                    }
                }
            }
        }
    }
    pdl_trigger();
}

__global__ void gemv_fields_clear_kernel(uint32_t *out, long long words) {
    pdl_enter();
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < words;
         i += (long long)gridDim.x * blockDim.x)
        out[i] = 0u;
}

static int fd_field_bits(int bits) { return bits == 1 ? 1 : (bits == 2 ? 2 : 4); }
static int fd_cols_per_cta(int N) { return N == 1 ? 1 : (N == 2 ? 2 : FD_COLS); }

// Shared memory of one CTA: the columns in use (depth rounded up to what the packed rows cover,
// plus 32 pad bytes per group) and their sums.
static size_t fd_smem_bytes(const qnn_gemm_desc *d, int *col_bytes_out) {
    const int F = fd_field_bits(d->w_bits), S = 8 / F;
    const long long groups = ceil_div(d->K, 32 * S);
    const long long col_bytes = groups * (32 * S + 32);
    if (col_bytes_out) *col_bytes_out = (int)col_bytes;
    return (size_t)fd_cols_per_cta(d->N) * (size_t)col_bytes + FD_COLS * sizeof(int);
}

// One or two columns whose staged form fits shared memory, and accumulators
// that cannot overflow (a field position's partial sum is at most 2^8 * |a|max * K).
// QNN_FIELDS_KERNEL=tensor in the environment keeps the tensor-core form, =dp4a widens this one to
// 16 columns (tests).
bool gemv_fields_dp4a_fits(const qnn_gemm_desc *d) {
    if (d->w_fmt != QNN_FMT_FIELDS || d->a_fmt != QNN_FMT_INT8 || d->w_bits > 4) return false;
    const char *force = getenv("QNN_FIELDS_KERNEL");
    if (force && force[0] == 't') return false;
    const int max_n = (force && force[0] == 'd') ? 16 : FD_MAX_N;
    if (d->N > max_n) return false;
    if ((long long)ceil_div(d->K, 32 * (8 / fd_field_bits(d->w_bits))) * (32 * (8 / fd_field_bits(d->w_bits)) + 32) > (48 << 10))
        return false;                                       // a column's staged form: at most 48 KB
    if (fd_smem_bytes(d, nullptr) > (size_t)200 * 1024) return false;
    const double amax = d->a_enc == QNN_ENC_SIGNED ? double(1 << (d->a_bits - 1)) : double((1 << d->a_bits) - 1);
    return 256.0 * amax * double(d->K) < 2147483648.0;
}

qnn_status gemv_fields_dp4a_launch(const qnn_gemm_desc *d, const void *W, const void *A, const int32_t *thr,
                                   void *out, cudaStream_t s) {
    const int F = fd_field_bits(d->w_bits), S = 8 / F;
    FdParams p;
    p.W = (const uint8_t *)W; p.A = (const uint8_t *)A; p.thr = thr; p.out = out;
    p.M = d->M; p.N = d->N; p.K = d->K;
    p.ldf = 32 * ceil_div(d->K, 32 * S);
    p.lda = round_up(d->K, 16);
    p.steps = p.ldf / 16;
    const size_t smem = fd_smem_bytes(d, &p.col_bytes);
    const int nc = fd_cols_per_cta(d->N);
    p.cols_alloc = nc;
    if (d->w_enc == QNN_ENC_BIPOLAR) { p.w_scale = 2; p.w_off = -1; }
    else if (d->w_enc == QNN_ENC_SIGNED) { p.w_scale = 1; p.w_off = -(1 << (d->w_bits - 1)); }
    else { p.w_scale = 1; p.w_off = 0; }
    p.out_bits = thr ? d->out_bits : 0;
    p.out_fmt = d->out_fmt;
    p.ld_out = round_up(d->M, 16);

    // bit-plane outputs, which the main kernel sets bit by bit, are cleared first
    int launches = 1;
    if (thr) {
        long long words = 0;
        if (d->out_fmt == QNN_FMT_BITPLANES) words = (long long)d->out_bits * d->N * ceil_div(d->M, 32);
        if (words > 0) {
            const long long blocks = (words + 255) / 256;
            gemv_fields_clear_kernel<<<(unsigned)(blocks < 1184 ? blocks : 1184), 256, 0, s>>>((uint32_t *)out, words);
            ++launches;
        }
    }
    const bool as = d->a_enc != QNN_ENC_UNSIGNED;
    const void *fn = nullptr;
#define QNN_FD_PICK(F_)                                                                                       \
    do {                                                                                                      \
        if (nc == 1) fn = as ? (const void *)gemv_fields_dp4a_kernel<F_, true, 1> : (const void *)gemv_fields_dp4a_kernel<F_, false, 1>; \
        else if (nc == 2) fn = as ? (const void *)gemv_fields_dp4a_kernel<F_, true, 2> : (const void *)gemv_fields_dp4a_kernel<F_, false, 2>; \
        else fn = as ? (const void *)gemv_fields_dp4a_kernel<F_, true, 4> : (const void *)gemv_fields_dp4a_kernel<F_, false, 4>; \
    } while (0)
    if (F == 1) QNN_FD_PICK(1);
    else if (F == 2) QNN_FD_PICK(2);
    else QNN_FD_PICK(4);
#undef QNN_FD_PICK
    const int dev = current_device();
    if (dev < 0) return QNN_ERR_CUDA;
    static size_t attr_smem[18][QNN_MAX_DEVICES] = {{0}};
    const int fi = ((F == 1 ? 0 : (F == 2 ? 1 : 2)) * 2 + (as ? 1 : 0)) * 3 + (nc == 1 ? 0 : (nc == 2 ? 1 : 2));
    if (smem > 48 * 1024 && smem > attr_smem[fi][dev]) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return QNN_ERR_CUDA;
        attr_smem[fi][dev] = smem;
    }
    // a persistent grid: as many CTAs as are resident at once, each staging its columns once and
    // then taking row blocks in turn
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, FD_THREADS, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int row_blocks = ceil_div(ceil_div(d->M, FD_THREADS / 32), fd_rows_at_a_time(F, nc));
    const int max_blocks = sm_count() * per_sm;
    dim3 grid(row_blocks < max_blocks ? row_blocks : max_blocks, ceil_div(d->N, nc));
    void *args[] = {(void *)&p};
    if (cudaLaunchKernel(fn, grid, dim3(FD_THREADS), args, smem, s) != cudaSuccess) return QNN_ERR_CUDA;
    count_launch(launches);
    return launch_status();
}

}  // namespace qnn
