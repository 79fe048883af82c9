// Issue-rate microbenchmarks that give the roofline denominators of the two GEMM paths
// (the paper reports its kernels against the peak of the machine's binary-operation
// throughput, Section 4.1.1; these are the same two peaks for this GPU):
//
//  * tensor path:  tcgen05.mma kind::i8 issued back to back on operand tiles that already sit in
//    shared memory (or, for the 128-row operand, in tensor memory) -- no loads, no epilogue,
//    nothing to wait for but the tensor pipe itself;
//  * bit-serial path: chains of XOR + POPC, the inner operation of Algorithm 1, in registers.
//
// Both kernels touch no global memory besides one result word per thread (POPC) and are timed
// by the caller with CUDA events.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace qnn {

constexpr int PK_BK = 128;            // depth bytes of one operand tile (one 128-byte swizzle row)
constexpr int PK_STAGES = 2;          // distinct operand tiles the MMAs rotate through

struct PeakSmem {
    alignas(1024) uint8_t a[PK_STAGES][128 * PK_BK];
    alignas(1024) uint8_t b[PK_STAGES][256 * PK_BK];    // up to 256 rows (pair: this CTA's half, 128)
    alignas(8) uint64_t done;
    uint32_t tmem_base;
    int abort_flag;
};

// A operand (128 rows x 32 depth bytes) taken from tensor memory instead of shared memory.
__device__ __forceinline__ void umma_i8_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

enum { PK_SINGLE = 0, PK_PAIR = 1, PK_TMEM_A = 2 };

// MODE PK_SINGLE: every CTA issues `mmas` MMAs of 128 x n x 32; PK_PAIR: the leader of every CTA
// pair issues `mmas` MMAs of 256 x n x 32 (cta_group::2) that read both CTAs' tiles; PK_TMEM_A: as
// PK_SINGLE with the 128-row operand read from tensor memory.
template <int MODE>
__global__ void __launch_bounds__(128, 1) peak_mma_i8_kernel(int n, int mmas, int *status_word) {
    constexpr bool PAIR = MODE == PK_PAIR;
    extern __shared__ uint8_t pk_raw[];
    PeakSmem &sm = *reinterpret_cast<PeakSmem *>(pk_raw + ((1024u - (smem_u32(pk_raw) & 1023u)) & 1023u));
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    volatile int *abort_flag = &sm.abort_flag;

    // operand values do not change the instruction rate, but they do change the power drawn (and
    // with it the clock under the power cap): pseudo-random bytes, as a real GEMM would see; the
    // int32 accumulators simply wrap
    uint32_t h = 0x9E3779B9u * (uint32_t)(blockIdx.x * blockDim.x + threadIdx.x + 1);
    for (int i = threadIdx.x; i < (int)((sizeof(sm.a) + sizeof(sm.b)) / 4); i += blockDim.x) {
        h = h * 1664525u + 1013904223u;
        reinterpret_cast<uint32_t *>(sm.a)[i] = h ^ (h >> 15);        // a and b are adjacent
    }
    if (threadIdx.x == 0) {
        mbar_init(&sm.done, 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == 1) {
        if (PAIR) tmem_alloc_pair(&sm.tmem_base, 512);
        else tmem_alloc(&sm.tmem_base, 512);
    }
    tc_fence_before();
    if (PAIR) cluster_sync_all(); else __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm.tmem_base;

    if (threadIdx.x == 0 && rank == 0) {
        const uint32_t idesc = (2u << 4) | (1u << 10) | ((uint32_t)(n >> 3) << 17) |
                               ((uint32_t)((PAIR ? 256 : 128) >> 4) << 24);      // s32 += u8 x s8, both K-major
        for (int i = 0; i < mmas; ++i) {
            const int st = (i >> 2) % PK_STAGES, kk = i & 3;
            const uint64_t da = umma_smem_desc(smem_u32(sm.a[st])) + 2 * kk;
            const uint64_t db = umma_smem_desc(smem_u32(sm.b[st])) + 2 * kk;
            // two accumulators, 128 MMAs each in turn (PK_TMEM_A: n <= 128, columns 384.. hold the operand)
            const uint32_t d = tmem_base + (uint32_t)(((i >> 7) & 1) * (MODE == PK_TMEM_A ? 128 : 256));
            if (PAIR) umma_i8_pair(d, da, db, idesc, 1u);
            else if (MODE == PK_TMEM_A) umma_i8_tmem_a(d, tmem_base + 384u + (uint32_t)(8 * (i & 7)), db, idesc, 1u);
            else umma_i8(d, da, db, idesc, 1u);
        }
        if (PAIR) umma_commit_pair(map_to_cta(smem_u32(&sm.done), 0));
        else umma_commit(&sm.done);
        mbar_wait(&sm.done, 0, abort_flag, status_word);
    }
    tc_fence_before();
    if (PAIR) cluster_sync_all(); else __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, 512);
        else tmem_dealloc(tmem_base, 512);
    }
}

// Every thread runs CHAINS independent chains x = popc(x ^ c) + k for `iters` steps: one POPC
// and one LOP3 (+ one add) per step and chain, so the POPC pipe is the limit.
constexpr int PK_CHAINS = 8;
__global__ void __launch_bounds__(1024, 1) peak_popc_kernel(int iters, uint32_t seed, uint32_t *sink) {
    uint32_t x[PK_CHAINS], c[PK_CHAINS];
#pragma unroll
    for (int j = 0; j < PK_CHAINS; ++j) {
        x[j] = seed * (uint32_t)(threadIdx.x + 1) + 0x9E3779B9u * (uint32_t)j;
        c[j] = (seed ^ 0xA5A5A5A5u) + 0x85EBCA6Bu * (uint32_t)(j + blockIdx.x);
    }
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int j = 0; j < PK_CHAINS; ++j) x[j] = (uint32_t)__popc(x[j] ^ c[j]) + c[j];
    }
    uint32_t r = 0;
#pragma unroll
    for (int j = 0; j < PK_CHAINS; ++j) r ^= x[j];
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = r;
}

}  // namespace qnn

using namespace qnn;

extern "C" {

qnn_status qnn_peak_mma_i8(int mode, int n, int mmas_per_cta, double *ops, void *stream) {
    if (!ops || mmas_per_cta <= 0 || n < 16 || n > 256 || (n % 16) != 0 || mode < 0 || mode > 2 ||
        (mode == PK_PAIR && (n % 32) != 0) || (mode == PK_TMEM_A && n > 128))
        return QNN_ERR_INVALID_ARG;
    const bool pair = mode == PK_PAIR;
    int *status = device_status_word();
    if (!status) return QNN_ERR_CUDA;
    const int sms = sm_count();
    const size_t smem = sizeof(PeakSmem) + 1024;
    const int dev = current_device();
    if (dev < 0) return QNN_ERR_CUDA;
    static bool attr_done[3][QNN_MAX_DEVICES] = {{false}};
    if (!attr_done[mode][dev]) {
        const void *fn = mode == PK_PAIR ? (const void *)peak_mma_i8_kernel<PK_PAIR>
                         : (mode == PK_TMEM_A ? (const void *)peak_mma_i8_kernel<PK_TMEM_A>
                                              : (const void *)peak_mma_i8_kernel<PK_SINGLE>);
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return QNN_ERR_CUDA;
        attr_done[mode][dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem; cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[1];
    cfg.attrs = attr; cfg.numAttrs = 0;
    cudaError_t e;
    if (pair) {
        cfg.gridDim = dim3(sms / 2 * 2);
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, peak_mma_i8_kernel<PK_PAIR>, n, mmas_per_cta, status);
        *ops = 2.0 * 256.0 * n * 32.0 * (double)mmas_per_cta * (sms / 2);
    } else {
        cfg.gridDim = dim3(sms);
        e = mode == PK_TMEM_A ? cudaLaunchKernelEx(&cfg, peak_mma_i8_kernel<PK_TMEM_A>, n, mmas_per_cta, status)
                              : cudaLaunchKernelEx(&cfg, peak_mma_i8_kernel<PK_SINGLE>, n, mmas_per_cta, status);
        *ops = 2.0 * 128.0 * n * 32.0 * (double)mmas_per_cta * sms;
    }
    if (e != cudaSuccess) return QNN_ERR_CUDA;
    count_launch();
    return launch_status();
}

qnn_status qnn_peak_popc(int iters, void *sink, size_t sink_bytes, double *popcs, void *stream) {
    if (!sink || !popcs || iters <= 0) return QNN_ERR_INVALID_ARG;
    const int blocks = 2 * sm_count(), threads = 1024;
    if (sink_bytes < (size_t)blocks * threads * 4) return QNN_ERR_WORKSPACE;
    if (!aligned16(sink)) return QNN_ERR_ALIGNMENT;
    peak_popc_kernel<<<blocks, threads, 0, (cudaStream_t)stream>>>(iters, 0x1234567u, (uint32_t *)sink);
    *popcs = (double)blocks * threads * (double)iters * PK_CHAINS;
    count_launch();
    return launch_status();
}

size_t qnn_peak_popc_sink_bytes(void) { return (size_t)2 * sm_count() * 1024 * 4; }

}  // extern "C"
