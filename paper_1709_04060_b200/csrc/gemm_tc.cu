// Tensor-core few-bit GEMM fused with the threshold activation.
//
// The few-bit operands sit in 8-bit containers (Section 3 of the paper: "casting
// all operands to 8-bit integers"); on B200 the fifth-generation tensor cores
// multiply them exactly (tcgen05.mma kind::i8, int32 accumulators in tensor
// memory), which reproduces the integer product that the bit-serial sum of
// Section 3.1 equals.  The epilogue applies T(x, t) of Section 2.1.1 to the
// accumulators straight out of tensor memory, so they never reach HBM.
//
// Kernel structure (persistent, one CTA per SM, 192 threads):
//   warp 0     TMA producer: 128-byte-swizzled K-major tiles of W (128 rows)
//              and A (BN rows) into a STAGES-deep shared-memory ring
//   warp 1     allocates tensor memory; one lane issues the MMAs
//              (M = 128, N = BN, K = 32 per instruction) and commits to mbarriers
//   warps 2-5  epilogue: tcgen05.ld of a 32-lane x 32-column block, threshold
//              count with the row's thresholds in registers, store.
// Output channels (weight rows) lie on the 128 tensor-memory lanes, so each
// epilogue thread owns one channel, and a warp ballot over code bits yields one
// word of the channel-interleaved bit-plane layout of Section 3.2.
// Two accumulator buffers in tensor memory let the epilogue of tile t overlap the
// main loop of tile t+1.  Every wait is bounded; on expiry the CTA records
// QNN_ERR_DEVICE_TIMEOUT in the device status word, drains and exits.
#include <cuda.h>

#include "common.cuh"

namespace qnn {

__device__ int g_dev_status;   // QNN_OK or QNN_ERR_DEVICE_TIMEOUT

constexpr int TC_BM = 128;          // weight rows per tile = tensor-memory lanes
constexpr int TC_BK = 128;          // depth bytes per stage = one 128B swizzle row
constexpr int TC_THREADS = 192;
constexpr long long TC_WAIT_CYCLES = 2000000000ll;   // ~1 s

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the limit ran out or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > TC_WAIT_CYCLES) {
            *abort_flag = 1;
            atomicExch(&g_dev_status, (int)QNN_ERR_DEVICE_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
                 "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}

// K-major operand tile, rows at a 128-byte pitch, 128B swizzle (what TMA writes
// with CU_TENSOR_MAP_SWIZZLE_128B): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);          // start address
    d |= (uint64_t)1 << 16;                            // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset: 8 rows x 128 B
    d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                            // 128-byte swizzle
    return d;
}

struct TcParams {
    const int32_t *thr;    // [M][n_thr] or null
    void *out;
    int M, N, K;
    int tiles_m, tiles_n, num_kb;
    int ld_out;            // INT8 output row pitch
    uint32_t idesc;
};

enum { OUT_RAW = 0, OUT_U8 = 1, OUT_PLANES = 2 };

template <int BN, int STAGES>
struct TcSmem {
    alignas(1024) uint8_t w[STAGES][TC_BM * TC_BK];
    alignas(1024) uint8_t a[STAGES][BN * TC_BK];
    alignas(8) uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

template <int BN, int STAGES, int OUT_MODE, int OUT_BITS>
__global__ void __launch_bounds__(TC_THREADS, 1)
qgemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_a,
                const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    using Smem = TcSmem<BN, STAGES>;
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr uint32_t TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;
    constexpr uint32_t STAGE_BYTES = (TC_BM + BN) * TC_BK;
    constexpr int N_THR = (1 << OUT_BITS) - 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sm.abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&sm.tmem_full[b], 1); mbar_init(&sm.tmem_empty[b], 128); }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&sm.tmem_base, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm.tmem_base;
    const int num_tiles = p.tiles_m * p.tiles_n;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int m0 = (tile % p.tiles_m) * TC_BM, n0 = (tile / p.tiles_m) * BN;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!(ok = mbar_wait(&sm.empty[s], ph ^ 1, abort_flag))) break;
                    mbar_arrive_expect_tx(&sm.full[s], STAGE_BYTES);
                    tma_load_2d(sm.w[s], &map_w, &sm.full[s], kb * TC_BK, m0);
                    tma_load_2d(sm.a[s], &map_a, &sm.full[s], kb * TC_BK, n0);
                }
            }
            if (!ok) {
                // gave up: let the copies already issued land before the CTA exits
                const uint32_t last = it - 1;
                if (it > 0) mbar_wait(&sm.full[last % STAGES], (last / STAGES) & 1, abort_flag);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++tcount) {
                const uint32_t buf = tcount & 1, acc_ph = (tcount >> 1) & 1;
                if (!(ok = mbar_wait(&sm.tmem_empty[buf], acc_ph ^ 1, abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!(ok = mbar_wait(&sm.full[s], ph, abort_flag))) break;
                    tc_fence_after();
                    const uint64_t dw = umma_smem_desc(smem_u32(sm.w[s]));
                    const uint64_t da = umma_smem_desc(smem_u32(sm.a[s]));
#pragma unroll
                    for (int kk = 0; kk < TC_BK / 32; ++kk)   // 32 depth bytes per MMA: +2 in 16-byte units
                        umma_i8(d_tmem, dw + 2 * kk, da + 2 * kk, p.idesc, (kb | kk) != 0);
                    umma_commit(&sm.empty[s]);
                }
                if (ok) umma_commit(&sm.tmem_full[buf]);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------ epilogue
        const int quad = warp & 3;                       // tensor-memory lane group of this warp
        uint32_t tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++tcount) {
            const int m0 = (tile % p.tiles_m) * TC_BM, n0 = (tile / p.tiles_m) * BN;
            const uint32_t buf = tcount & 1, acc_ph = (tcount >> 1) & 1;
            const int m = m0 + quad * 32 + lane;
            const bool m_ok = m < p.M;
            int thr_r[N_THR > 0 ? N_THR : 1];
            if (OUT_MODE != OUT_RAW) {
#pragma unroll
                for (int q = 0; q < N_THR; ++q) thr_r[q] = m_ok ? p.thr[(size_t)m * N_THR + q] : 0x7fffffff;
            }
            ok = mbar_wait(&sm.tmem_full[buf], acc_ph, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (n0 + c0 >= p.N) break;               // warp-uniform: nothing left in this tile
                int acc[32];
                tmem_ld32(t_row + c0, acc);
                if (OUT_MODE == OUT_RAW) {
                    int32_t *o = reinterpret_cast<int32_t *>(p.out);
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int n = n0 + c0 + j;
                        if (m_ok && n < p.N) o[(size_t)n * p.M + m] = acc[j];
                    }
                } else {
                    uint32_t keep[OUT_BITS > 0 ? OUT_BITS : 1];
#pragma unroll
                    for (int b = 0; b < OUT_BITS; ++b) keep[b] = 0;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        int code = 0;
#pragma unroll
                        for (int q = 0; q < N_THR; ++q) code += (acc[j] >= thr_r[q]) ? 1 : 0;
                        if (!m_ok) code = 0;
                        const int n = n0 + c0 + j;
                        if (OUT_MODE == OUT_U8) {
                            if (n < p.N && m < p.ld_out)
                                reinterpret_cast<uint8_t *>(p.out)[(size_t)n * p.ld_out + m] = (uint8_t)code;
                        } else {
#pragma unroll
                            for (int b = 0; b < OUT_BITS; ++b) {
                                const uint32_t w = __ballot_sync(0xffffffffu, (code >> b) & 1);
                                if (lane == j) keep[b] = w;    // lane j keeps column j's word
                            }
                        }
                    }
                    if (OUT_MODE == OUT_PLANES) {
                        const int mw = (p.M + 31) >> 5, word = (m0 >> 5) + quad, n = n0 + c0 + lane;
                        if (n < p.N && word < mw) {
#pragma unroll
                            for (int b = 0; b < OUT_BITS; ++b)
                                reinterpret_cast<uint32_t *>(p.out)[((size_t)b * p.N + n) * mw + word] = keep[b];
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&sm.tmem_empty[buf]);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// [rows][K] bytes at pitch ld; box = 128 depth bytes x box_rows rows; out-of-range reads give zeros.
static bool make_map(CUtensorMap *map, const void *base, int rows, int K, int ld, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int STAGES, int OUT_MODE, int OUT_BITS>
static qnn_status launch_cfg(const CUtensorMap &mw, const CUtensorMap &ma, const TcParams &p, cudaStream_t s) {
    auto kern = qgemm_tc_kernel<BN, STAGES, OUT_MODE, OUT_BITS>;
    const size_t smem = sizeof(TcSmem<BN, STAGES>) + 1024;
    static bool attr_done = false;        // per instantiation
    if (!attr_done) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return QNN_ERR_CUDA;
        attr_done = true;
    }
    const int tiles = p.tiles_m * p.tiles_n;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    kern<<<grid, TC_THREADS, smem, s>>>(mw, ma, p);
    count_launch();
    return launch_status();
}

template <int BN, int STAGES>
static qnn_status launch_out(int mode, int out_bits, const CUtensorMap &mw, const CUtensorMap &ma,
                             const TcParams &p, cudaStream_t s) {
    if (mode == OUT_RAW) return launch_cfg<BN, STAGES, OUT_RAW, 0>(mw, ma, p, s);
#define QNN_TC_CASE(B_)                                                                   \
    if (out_bits == B_)                                                                   \
        return mode == OUT_U8 ? launch_cfg<BN, STAGES, OUT_U8, B_>(mw, ma, p, s)         \
                              : launch_cfg<BN, STAGES, OUT_PLANES, B_>(mw, ma, p, s);
    QNN_TC_CASE(1) QNN_TC_CASE(2) QNN_TC_CASE(3) QNN_TC_CASE(4)
#undef QNN_TC_CASE
    return QNN_ERR_UNSUPPORTED;
}

qnn_status gemm_tc_launch(const qnn_gemm_desc *d, const void *W, const void *A, const int32_t *thr,
                          void *out, cudaStream_t s) {
    const int ld = round_up(d->K, 16);
    // column tile: the widest that still gives every SM a tile
    const int sms = sm_count();
    const int tiles_m = ceil_div(d->M, TC_BM);
    int bn = 256;
    while (bn > 32 && (long long)tiles_m * ceil_div(d->N, bn) < sms) bn >>= 1;
    if (bn == 64) bn = 32;

    CUtensorMap mw, ma;
    if (!make_map(&mw, W, d->M, d->K, ld, TC_BM) || !make_map(&ma, A, d->N, d->K, ld, bn)) return QNN_ERR_CUDA;

    TcParams p;
    p.thr = thr; p.out = out; p.M = d->M; p.N = d->N; p.K = d->K;
    p.tiles_m = tiles_m; p.tiles_n = ceil_div(d->N, bn); p.num_kb = ceil_div(d->K, TC_BK);
    p.ld_out = round_up(d->M, 16);
    const uint32_t w_s8 = d->w_enc == QNN_ENC_UNSIGNED ? 0u : 1u;
    const uint32_t a_s8 = d->a_enc == QNN_ENC_UNSIGNED ? 0u : 1u;
    p.idesc = (2u << 4)                 // accumulator format: s32
              | (w_s8 << 7)             // A-operand (weights) format: 0 = u8, 1 = s8
              | (a_s8 << 10)            // B-operand (activations) format
              | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);   // both K-major
    const int mode = !thr ? OUT_RAW : (d->out_fmt == QNN_FMT_INT8 ? OUT_U8 : OUT_PLANES);
    switch (bn) {
        case 256: return launch_out<256, 4>(mode, d->out_bits, mw, ma, p, s);
        case 128: return launch_out<128, 6>(mode, d->out_bits, mw, ma, p, s);
        default:  return launch_out<32, 8>(mode, d->out_bits, mw, ma, p, s);
    }
}

qnn_status device_status_read(int *status) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_dev_status, sizeof(int)) != cudaSuccess) return QNN_ERR_CUDA;
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_dev_status, &zero, sizeof(int)) != cudaSuccess) return QNN_ERR_CUDA;
    *status = v;
    return QNN_OK;
}

}  // namespace qnn
