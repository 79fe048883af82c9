// Few-column GEMM (N <= 16) on w-bit packed weights, fused with the threshold activation:
// the fully connected layer at small batch of Section 4.2, whose speed-up in the paper comes
// from the packed weights cutting the memory traffic.  The weights are streamed from HBM
// exactly once in their packed form (w bits per element, QNN_FMT_FIELDS), expanded to
// 8-bit values inside the SM, and multiplied exactly by the tensor cores (tcgen05.mma
// kind::i8), which reproduces the integer product that the bit-serial sum of Section 3.1
// equals; T(x, t) of Section 2.1.1 is applied to the int32 sums before anything is stored.
//
// Orientation: weight rows are the MMA's 128-row operand and sit on the 128 tensor-memory
// lanes; the (at most 16) activation columns are the MMA's N side.  A thread that owns a
// lane therefore owns one output channel: it expands that row's packed bytes, and in the
// epilogue counts that row's thresholds for every column.
//
// Expansion without shifts: a packed byte holds S = 8 / f fields of f bits (f = 1, 2 or 4).
// Masking a packed word with the field-s mask leaves, in every byte, field s scaled by
// 2^(f s) -- still an 8-bit unsigned value.  The masked words are written to tensor memory as
// the MMA's row operand (tcgen05.st), one accumulator per field position s collects
// sum_k 2^(f s) u_k a_k over the elements stored at that position, and the epilogue adds the
// S accumulators after an exact right shift by f s.  The field layout (see qnn.h) is chosen
// so that the 32 elements at position s of 32 consecutive packed bytes are 32 consecutive
// depth indices: the activation operand is the plain [N][K] byte matrix, untouched.
// Fields hold the value minus the encoding's minimum (u = v - vmin >= 0), or the bit of a
// bipolar weight (v = 2u - 1): sum_k v_k a_k = scale * sum_k u_k a_k + offset * sum_k a_k,
// and the column sums of the activations come out of the same MMAs: the first tensor-memory lane
// past the block's rows holds a row of ones.
//
// CTA = one block of up to 128 weight rows x one slice of the depth; the CTAs of a cluster
// split the depth of the same rows and hand their int32 partial sums to the cluster's first
// CTA through distributed shared memory before the thresholds are counted.  Warp roles:
//   warp 0       producer: TMA loads of the packed weight stages (rows x 128 bytes, 128-byte
//                swizzle) into a ring
//   warp 1       allocates tensor memory; one lane issues the MMAs (128 x 16 x 32 per
//                instruction, row operand from tensor memory, activations from shared memory)
//   warps 2-9    expansion, two groups of four warps (one warp per lane quarter) that take the
//                chunks in turn and fill the three operand buffers in tensor memory round
//                robin; group 0 then runs the epilogue
//   warp 10      TMA loads of the slice's activation k-blocks (16 rows x 128 bytes each, all
//                resident)
// Every wait is bounded; on expiry the CTA records QNN_ERR_DEVICE_TIMEOUT and drains.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace qnn {

constexpr int GF_NPAD = 16;                 // MMA N: activation columns, zero padded
constexpr int GF_STAGE_ROW_BYTES = 128;     // packed bytes per row and stage (one swizzle row)
constexpr int GF_NS = 6;                    // weight stages in the ring
constexpr int GF_MAX_ST = 32;               // stages per depth slice (one barrier each)
constexpr int GF_ACT_KB_BYTES = GF_NPAD * 128;       // one activation k-block in shared memory
constexpr int GF_ACT_MAX_BYTES = 100 * 1024;
constexpr int GF_MAX_SPLIT = 4;
constexpr int GF_THREADS = 32 * 11;
constexpr int GF_NB = 3;                    // operand buffers in tensor memory (128 columns apart)
constexpr uint32_t GF_TMEM_COLS = 512;
constexpr uint32_t GF_ACC_COL = 128 * GF_NB;         // accumulators behind the operand buffers

enum { GF_OUT_RAW = 0, GF_OUT_U8 = 1, GF_OUT_PLANES = 2 };

struct GfParams {
    const int32_t *thr;     // [M][n_thr] or null
    void *out;
    int *status;            // device status word
    int M, N;
    int R;                  // weight rows per block (<= 128)
    int sk;                 // CTAs per cluster = slices of the depth
    int nst, st_per;        // 128-byte stages per packed row; stages per slice
    int out_mode, out_bits, ld_out;
    int w_scale, w_off;     // weight value = w_scale * field + w_off
    int a_signed;
    uint32_t idesc;
};

struct GfBars {
    alignas(8) uint64_t full[GF_NS];
    uint64_t empty[GF_NS];
    uint64_t a_full[GF_NB];
    uint64_t a_empty[GF_NB];
    uint64_t act_full[GF_MAX_ST];
    uint64_t acc_full;
    int colsum[GF_NPAD];
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ void umma_i8_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t *r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t *r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_fence() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, int (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr));
    return v;
}
__device__ __forceinline__ bool gf_warp_wait(uint64_t *bar, uint32_t parity, int lane, volatile int *abort_flag,
                                             int *status) {
    bool ok = true;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, status);
    return __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
}

// F: field width in bits (1, 2 or 4).
template <int F>
__global__ void __launch_bounds__(GF_THREADS, 1)
gemv_fields_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_act,
                   const GfParams p) {
    constexpr int S = 8 / F;                       // fields per byte = accumulators
    constexpr int CG = 16 / S;                     // 32-byte groups per operand buffer fill ("chunk"): 128 columns
    constexpr int GPS = 4;                         // groups per stage (128 packed bytes per row)
    constexpr uint32_t FMASK = F == 1 ? 0x01010101u : (F == 2 ? 0x03030303u : 0x0F0F0F0Fu);
    extern __shared__ uint8_t gf_raw[];
    uint8_t *base = gf_raw + ((1024u - (smem_u32(gf_raw) & 1023u)) & 1023u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = p.sk > 1 ? cluster_ctarank() : 0u;
    const int block = blockIdx.x / p.sk;
    const int m0 = block * p.R;
    const int st0 = (int)rank * p.st_per;
    const int nst_local = min(p.nst, st0 + p.st_per) - st0;          // >= 1 by construction
    const int nchunks = (nst_local * GPS + CG - 1) / CG;
    const uint32_t stage_bytes = (uint32_t)p.R * GF_STAGE_ROW_BYTES;
    // The blocks walk the stages of their slice in rotated orders (integer sums do not care): all
    // blocks read the same activation bytes, and in lock step they would all ask for the same
    // lines of L2 at the same time.
    const int rot = block % nst_local;

    uint8_t *ring = base;                                                       // [GF_NS][128 rows x 128 B]
    uint8_t *act = ring + GF_NS * 128 * GF_STAGE_ROW_BYTES;                     // [st_per * S][16 x 128 B]
    int *red = reinterpret_cast<int *>(act + (size_t)p.st_per * S * GF_ACT_KB_BYTES);   // [sk - 1][128][16]
    GfBars &bar = *reinterpret_cast<GfBars *>(reinterpret_cast<uint8_t *>(red) +
                                              (size_t)(p.sk - 1) * 128 * GF_NPAD * 4);
    volatile int *abort_flag = &bar.abort_flag;

    if (threadIdx.x == 0) {
        // a stage is read by the four warps of every group that has a chunk (or part of one) in it
        for (int s = 0; s < GF_NS; ++s) { mbar_init(&bar.full[s], 1); mbar_init(&bar.empty[s], CG < GPS ? 8 : 4); }
        for (int b = 0; b < GF_NB; ++b) { mbar_init(&bar.a_full[b], 4); mbar_init(&bar.a_empty[b], 1); }
        for (int j = 0; j < GF_MAX_ST; ++j) mbar_init(&bar.act_full[j], 1);
        mbar_init(&bar.acc_full, 1);
        bar.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < GF_NPAD) bar.colsum[threadIdx.x] = 0;
    if (warp == 1) tmem_alloc(&bar.tmem_base, GF_TMEM_COLS);
    tc_fence_before();
    if (p.sk > 1) cluster_sync_all(); else __syncthreads();
    tc_fence_after();
    pdl_enter();
    const uint32_t tmem_base = bar.tmem_base;

    // state the row-owning threads (expansion group 0) carry from the main loop into the epilogue
    const int h = (warp >= 2 && warp < 10) ? (warp - 2) >> 2 : -1, q = warp & 3;
    const int r = q * 32 + lane;                                     // weight row of this thread = lane of tensor memory
    const int m = m0 + r;
    const int n_thr = p.out_mode == GF_OUT_RAW ? 0 : (1 << p.out_bits) - 1;
    int acc[GF_NPAD], t[15];
#pragma unroll
    for (int n = 0; n < GF_NPAD; ++n) acc[n] = 0;

    if (warp == 0) {
        // ------------------------------------------------- producer of the packed weight stages
        if (lane == 0) {
            for (int j = 0; j < nst_local; ++j) {
                const int slot = j % GF_NS;
                if (!mbar_wait(&bar.empty[slot], ((j / GF_NS) & 1) ^ 1, abort_flag, p.status)) break;
                mbar_arrive_expect_tx(&bar.full[slot], stage_bytes);
                tma_load_2d(ring + (size_t)slot * 128 * GF_STAGE_ROW_BYTES, &map_w, &bar.full[slot],
                            (st0 + (j + rot) % nst_local) * GF_STAGE_ROW_BYTES, m0);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        // A 128 x 16 x 32 MMA keeps the tensor pipe busy for 64 cycles only and the pipe's queue is
        // short, so whatever this thread does between two MMAs (a barrier poll costs about 150
        // cycles while the pipe reads shared memory) shows up as idle pipe: one poll per chunk,
        // placed where half of the chunk's MMAs are queued, and no other work in the loop.
        if (lane == 0) {
            // act_ok: stages whose activation k-blocks are known to have landed
            bool ok = true;
            int act_ok = 0;
            const int first_stages = min(nst_local, (CG + GPS - 1) / GPS);
            for (; ok && act_ok < first_stages; ++act_ok) ok = mbar_wait_spin(&bar.act_full[act_ok], 0, abort_flag, p.status);
            if (ok) ok = mbar_wait_spin(&bar.a_full[0], 0, abort_flag, p.status);
            tc_fence_after();
            uint64_t db_chunk = umma_smem_desc(smem_u32(act));       // first activation slice of the chunk
            uint32_t buf = 0, use = 0;                               // operand buffer of the chunk, its use count
            for (int c = 0; ok && c < nchunks; ++c) {
                const uint32_t a_tmem = tmem_base + buf * 128u;
                uint32_t nbuf = buf + 1, nuse = use;
                if (nbuf == GF_NB) { nbuf = 0; ++nuse; }
                // a chunk is MPC MMAs unless the slice ends inside it
                const int groups = min(CG, 4 * nst_local - c * CG);
#pragma unroll
                for (int gl = 0; gl < CG; ++gl) {
                    if (gl < groups) {
#pragma unroll
                        for (int s = 0; s < S; ++s) {
                            const int rel = gl * S + s;              // slice within the chunk (compile time)
                            umma_i8_a_tmem(tmem_base + GF_ACC_COL + (uint32_t)(s * GF_NPAD), a_tmem + (uint32_t)(rel * 8),
                                           db_chunk + (uint64_t)((rel >> 2) * 128 + (rel & 3) * 2), p.idesc,
                                           (c | gl) != 0);
                        }
                    }
                    if (gl == CG / 2 - 1 && c + 1 < nchunks) {
                        // the next chunk never depends on this one's completion
                        const int need = min(nst_local, ((c + 2) * CG + GPS - 1) / GPS);     // stages up to its end
                        for (; ok && act_ok < need; ++act_ok) ok = mbar_wait_spin(&bar.act_full[act_ok], 0, abort_flag, p.status);
                        if (ok) ok = mbar_wait_spin(&bar.a_full[nbuf], nuse & 1u, abort_flag, p.status);
                        tc_fence_after();
                        if (!ok) break;
                    }
                }
                if (!ok) break;
                umma_commit(&bar.a_empty[buf]);
                db_chunk += (uint64_t)(S * CG / 4) * 128u;           // S * CG slices = S * CG / 4 k-blocks
                buf = nbuf; use = nuse;
            }
            if (ok) umma_commit(&bar.acc_full);
        }
        __syncwarp();
    } else if (warp == 10) {
        // -------------------------- activations: all k-blocks of the slice stay resident
        if (lane == 0) {
            for (int j = 0; j < nst_local; ++j) {
                mbar_arrive_expect_tx(&bar.act_full[j], (uint32_t)S * GF_ACT_KB_BYTES);
                for (int s = 0; s < S; ++s)
                    tma_load_2d(act + (size_t)(j * S + s) * GF_ACT_KB_BYTES, &map_act, &bar.act_full[j],
                                ((st0 + (j + rot) % nst_local) * S + s) * 128, 0);
            }
        }
        __syncwarp();
    } else {
        // -------------------------------------------------------- expansion, then epilogue
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        if (h == 0) {
            // thresholds of this thread's row: in registers long before they are needed
#pragma unroll
            for (int i = 0; i < 15; ++i)
                t[i] = (i < n_thr && m < p.M && r < p.R) ? __ldg(p.thr + (size_t)m * n_thr + i) : 0x7fffffff;
        }
        // Lane R of tensor memory (the first one past the block's rows) carries a row of ones: its
        // accumulators collect sum_k a[n][k], the column sums that the weight encoding's offset
        // multiplies, at no extra cost.
        const bool ones_row = r == p.R;
        const uint32_t fill = ones_row ? 0xFFFFFFFFu : 0u;           // ones row: every field mask sees all bits ...
        uint32_t fmask[S];
#pragma unroll
        for (int s = 0; s < S; ++s) fmask[s] = ones_row ? 0x01010101u : (FMASK << (F * s));    // ... and keeps a 1
        bool ok = true;
        for (int c = h; c < nchunks; c += 2) {
            const int buf = c % GF_NB;
            const int g_first = c * CG;                              // first 32-byte group of the chunk (slice-relative)
            const int groups = min(CG, GPS * nst_local - g_first);
            const int j_first = g_first / GPS, j_last = (g_first + groups - 1) / GPS;
            if (lane == 0) {
                ok = mbar_wait_spin(&bar.a_empty[buf], (uint32_t)(((c / GF_NB) & 1) ^ 1), abort_flag, p.status);
                for (int j = j_first; ok && j <= j_last; ++j)
                    ok = mbar_wait_spin(&bar.full[j % GF_NS], (j / GF_NS) & 1, abort_flag, p.status);
            }
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int gl = 0; gl < CG; ++gl) {
                if (gl < groups) {
                    const int gg = g_first + gl, j = gg / GPS, g = gg % GPS;
                    const uint32_t row = smem_u32(ring + (size_t)(j % GF_NS) * 128 * GF_STAGE_ROW_BYTES) + (uint32_t)r * 128u;
                    const uint4 lo = lds128(row + (uint32_t)(((2 * g) ^ (r & 7)) << 4));
                    const uint4 hi = lds128(row + (uint32_t)(((2 * g + 1) ^ (r & 7)) << 4));
                    const uint32_t x[8] = {lo.x | fill, lo.y | fill, lo.z | fill, lo.w | fill,
                                           hi.x | fill, hi.y | fill, hi.z | fill, hi.w | fill};
                    uint32_t y[8 * S];
#pragma unroll
                    for (int s = 0; s < S; ++s)
#pragma unroll
                        for (int i = 0; i < 8; ++i) y[8 * s + i] = x[i] & fmask[s];
                    const uint32_t taddr = tmem_base + lane_addr + (uint32_t)buf * 128u + (uint32_t)(gl * S * 8);
                    if (S == 2) {
                        tmem_st16(taddr, y);
                    } else {
#pragma unroll
                        for (int v = 0; v < S / 4; ++v) tmem_st32(taddr + 32u * v, y + 32 * v);
                    }
                }
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&bar.a_full[buf]);
                // this warp has read its part of these stages (its only visit to them)
                for (int j = j_first; j <= j_last; ++j) mbar_arrive(&bar.empty[j % GF_NS]);
            }
        }

        if (h == 0) {
            if (lane == 0 && ok) ok = mbar_wait_spin(&bar.acc_full, 0, abort_flag, p.status);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (ok) {
                tc_fence_after();
                // the S accumulators of this row, four at a time
                int ones[GF_NPAD];
#pragma unroll
                for (int n = 0; n < GF_NPAD; ++n) ones[n] = 0;
#pragma unroll
                for (int s0 = 0; s0 < S; s0 += 4) {
                    int d[4][GF_NPAD];
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        if (s0 + s < S) tmem_ld16_issue(tmem_base + lane_addr + GF_ACC_COL + (uint32_t)((s0 + s) * GF_NPAD), d[s]);
                    tmem_ld_fence();
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        if (s0 + s < S) {
#pragma unroll
                            for (int n = 0; n < GF_NPAD; ++n) {
                                acc[n] += d[s][n] >> (F * (s0 + s));     // exact: a multiple of 2^(F s)
                                ones[n] += d[s][n];                      // the row of ones is not scaled
                            }
                        }
                }
                if (ones_row) {
#pragma unroll
                    for (int n = 0; n < GF_NPAD; ++n) bar.colsum[n] = ones[n];
                }
            }
            // the four epilogue warps meet: the column sums are in shared memory
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ok) {
#pragma unroll
                for (int n = 0; n < GF_NPAD; ++n) acc[n] = p.w_scale * acc[n] + p.w_off * bar.colsum[n];
                if (rank != 0) {
                    // partial sums of this depth slice go to the cluster's first CTA
                    const uint32_t dst = map_to_cta(smem_u32(red + ((size_t)(rank - 1) * 128 + r) * GF_NPAD), 0);
#pragma unroll
                    for (int v = 0; v < GF_NPAD / 4; ++v)
                        asm volatile("st.shared::cluster.v4.s32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(dst + 16u * v), "r"(acc[4 * v]), "r"(acc[4 * v + 1]), "r"(acc[4 * v + 2]),
                                       "r"(acc[4 * v + 3]) : "memory");
                }
            }
        }
    }

    // partial sums have reached the first CTA of the cluster; tensor memory is no longer read
    tc_fence_before();
    if (p.sk > 1) cluster_sync_all(); else __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, GF_TMEM_COLS);
    }
    if (h == 0 && rank == 0 && !*abort_flag) {
        for (int k = 0; k < p.sk - 1; ++k) {
            const int4 *src = reinterpret_cast<const int4 *>(red + ((size_t)k * 128 + r) * GF_NPAD);
#pragma unroll
            for (int v = 0; v < GF_NPAD / 4; ++v) {
                const int4 d = src[v];
                acc[4 * v] += d.x; acc[4 * v + 1] += d.y; acc[4 * v + 2] += d.z; acc[4 * v + 3] += d.w;
            }
        }
        const bool row_ok = r < p.R && m < p.M;
        const int mw = (p.M + 31) >> 5, word = (m0 >> 5) + q;
#pragma unroll
        for (int n = 0; n < GF_NPAD; ++n) {
            if (n >= p.N) break;                                     // uniform
            if (p.out_mode == GF_OUT_RAW) {
                if (row_ok) reinterpret_cast<int32_t *>(p.out)[(size_t)n * p.M + m] = acc[n];
                continue;
            }
            // T(x, t): thresholds past the row's count hold INT32_MAX and are not looked at
            const int x = acc[n];
            int code = (x >= t[0]) ? 1 : 0;
            if (p.out_bits >= 2) code += ((x >= t[1]) ? 1 : 0) + ((x >= t[2]) ? 1 : 0);
            if (p.out_bits >= 3) code += ((x >= t[3]) ? 1 : 0) + ((x >= t[4]) ? 1 : 0) + ((x >= t[5]) ? 1 : 0) + ((x >= t[6]) ? 1 : 0);
            if (p.out_bits >= 4) {
                int c2 = 0;
#pragma unroll
                for (int i = 7; i < 15; ++i) c2 += (x >= t[i]) ? 1 : 0;
                code += c2;
            }
            if (!row_ok) code = 0;
            if (p.out_mode == GF_OUT_U8) {
                // pad bytes of an output row (m in [M, ld_out)) are written as zeros
                if (r < p.R && m < p.ld_out) reinterpret_cast<uint8_t *>(p.out)[(size_t)n * p.ld_out + m] = (uint8_t)code;
            } else {
                // 32 rows of a warp are one word of the channel-interleaved layout (R is a multiple of 32)
                for (int b = 0; b < p.out_bits; ++b) {
                    const uint32_t bits = __ballot_sync(0xffffffffu, (code >> b) & 1);
                    if (lane == 0 && q * 32 < p.R && word < mw)
                        reinterpret_cast<uint32_t *>(p.out)[((size_t)b * p.N + n) * mw + word] = bits;
                }
            }
        }
    }
    pdl_trigger();
}

// ------------------------------------------------------------------- host side
struct GfPlan { int F, S, ldf, nst, sk, st_per, R, nblocks; };

static int gf_field_bits(int w_bits) { return w_bits == 1 ? 1 : (w_bits == 2 ? 2 : 4); }

static bool gf_plan(const qnn_gemm_desc *d, bool has_thr, GfPlan *pl) {
    if (d->w_fmt != QNN_FMT_FIELDS || d->a_fmt != QNN_FMT_INT8) return false;
    if (d->N > GF_NPAD || d->w_bits > 4) return false;
    pl->F = gf_field_bits(d->w_bits); pl->S = 8 / pl->F;
    pl->ldf = 32 * ceil_div(d->K, 32 * pl->S);
    pl->nst = ceil_div(pl->ldf, GF_STAGE_ROW_BYTES);
    // every sub-accumulator must fit int32: fields scaled to at most 240, activations to 255
    const double amax = d->a_enc == QNN_ENC_BIPOLAR ? 1.0
                        : (d->a_enc == QNN_ENC_SIGNED ? double(1 << (d->a_bits - 1)) : double((1 << d->a_bits) - 1));
    if (double(d->K) * 240.0 * amax >= 2147483648.0) return false;
    const int gran = !has_thr ? 8 : (d->out_fmt == QNN_FMT_INT8 ? 16 : 32);
    const int cover = (has_thr && d->out_fmt == QNN_FMT_INT8) ? round_up(d->M, 16) : d->M;
    const int sms = sm_count();
    double best = 0.0;
    bool found = false;
    for (int sk = 1; sk <= GF_MAX_SPLIT; sk *= 2) {
        const int st_per = ceil_div(pl->nst, sk);
        if ((sk - 1) * st_per >= pl->nst) continue;                       // a slice would be empty
        if (st_per > GF_MAX_ST || (size_t)st_per * pl->S * GF_ACT_KB_BYTES > (size_t)GF_ACT_MAX_BYTES) continue;
        const int target = sms / sk > 0 ? sms / sk : 1;
        int R = round_up(ceil_div(cover, target), gran);
        if (R > 128 - gran) R = 128 - gran;                                // one lane is left for the row of ones
        const int nblocks = ceil_div(cover, R);
        const long long ctas = (long long)nblocks * sk;
        const double waves = (double)((ctas + sms - 1) / sms);
        // time of a CTA ~ its packed bytes plus a fixed cost worth about 24 KB of streaming
        const double cost = waves * ((double)R * st_per * GF_STAGE_ROW_BYTES + 24.0 * 1024.0 * (1.0 + 0.25 * (sk - 1)));
        if (!found || cost < best) {
            found = true; best = cost;
            pl->sk = sk; pl->st_per = st_per; pl->R = R; pl->nblocks = nblocks;
        }
    }
    return found;
}

bool gemv_fields_fits(const qnn_gemm_desc *d, bool has_thr) {
    GfPlan pl;
    return gf_plan(d, has_thr, &pl);
}

qnn_status gemv_fields_launch(const qnn_gemm_desc *d, const void *W, const void *A, const int32_t *thr,
                              void *out, cudaStream_t s) {
    GfPlan pl;
    if (!gf_plan(d, thr != nullptr, &pl)) return QNN_ERR_UNSUPPORTED;
    GfParams p;
    p.thr = thr; p.out = out; p.status = device_status_word();
    if (!p.status) return QNN_ERR_CUDA;
    p.M = d->M; p.N = d->N; p.R = pl.R; p.sk = pl.sk; p.nst = pl.nst; p.st_per = pl.st_per;
    p.out_mode = !thr ? GF_OUT_RAW : (d->out_fmt == QNN_FMT_INT8 ? GF_OUT_U8 : GF_OUT_PLANES);
    p.out_bits = thr ? d->out_bits : 0;
    p.ld_out = round_up(d->M, 16);
    if (d->w_enc == QNN_ENC_BIPOLAR) { p.w_scale = 2; p.w_off = -1; }
    else if (d->w_enc == QNN_ENC_SIGNED) { p.w_scale = 1; p.w_off = -(1 << (d->w_bits - 1)); }
    else { p.w_scale = 1; p.w_off = 0; }
    p.a_signed = d->a_enc != QNN_ENC_UNSIGNED ? 1 : 0;
    p.idesc = (2u << 4) | ((uint32_t)p.a_signed << 10) | ((uint32_t)(GF_NPAD >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    CUtensorMap mw, ma;
    if (!tc_make_tile_map(&mw, W, d->M, pl.ldf, pl.ldf, pl.R)) return QNN_ERR_CUDA;
    if (!tc_make_tile_map(&ma, A, d->N, d->K, round_up(d->K, 16), GF_NPAD)) return QNN_ERR_CUDA;

    const size_t smem = 1024 + (size_t)GF_NS * 128 * GF_STAGE_ROW_BYTES + (size_t)pl.st_per * pl.S * GF_ACT_KB_BYTES +
                        (size_t)(pl.sk - 1) * 128 * GF_NPAD * 4 + sizeof(GfBars);
    const int dev = current_device();
    if (dev < 0) return QNN_ERR_CUDA;
    const void *fn = pl.F == 1 ? (const void *)gemv_fields_kernel<1>
                     : (pl.F == 2 ? (const void *)gemv_fields_kernel<2> : (const void *)gemv_fields_kernel<4>);
    static size_t attr_smem[3][QNN_MAX_DEVICES] = {{0}};
    const int fi = pl.F == 1 ? 0 : (pl.F == 2 ? 1 : 2);
    if (smem > attr_smem[fi][dev]) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return QNN_ERR_CUDA;
        attr_smem[fi][dev] = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(pl.nblocks * pl.sk)); cfg.blockDim = dim3(GF_THREADS);
    cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    // programmatic dependent launch: the CTAs set up (barriers, tensor memory) as SMs fall idle at
    // the end of the previous kernel and wait in griddepcontrol.wait before touching global memory
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
    if (pl.sk > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)pl.sk; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    cudaError_t e;
    if (pl.F == 1) e = cudaLaunchKernelEx(&cfg, gemv_fields_kernel<1>, mw, ma, p);
    else if (pl.F == 2) e = cudaLaunchKernelEx(&cfg, gemv_fields_kernel<2>, mw, ma, p);
    else e = cudaLaunchKernelEx(&cfg, gemv_fields_kernel<4>, mw, ma, p);
    if (e != cudaSuccess) return QNN_ERR_CUDA;
    count_launch();
    return launch_status();
}

}  // namespace qnn
