// Tensor-core few-bit GEMM fused with the threshold activation.
//
// The few-bit operands sit in 8-bit containers (the 8-bit formulation that Section 3
// of the paper starts from); on B200 the fifth-generation tensor cores
// multiply them exactly (tcgen05.mma kind::i8, int32 accumulators in tensor
// memory), which reproduces the integer product that the bit-serial sum of
// Section 3.1 equals.  The epilogue applies T(x, t) of Section 2.1.1 to the
// accumulators straight out of tensor memory, so they never reach HBM.
//
// Orientation: activation rows (pixels, the GEMM's N) are the MMA's M side and
// land on the 128 tensor-memory lanes; weight rows (output channels, the GEMM's
// M) are the MMA's N side and land on tensor-memory columns.  An epilogue thread
// therefore owns one pixel and reads 32 consecutive channels per tcgen05.ld,
// which is exactly the channels-fastest output layout: 32 codes leave as two
// 16-byte stores, and the 32 bits of one plane are one word of the
// channel-interleaved layout of Section 3.2.
//
// Kernel structure (persistent, one CTA per SM, 352 threads):
//   warp 0     TMA producer: 128-byte-swizzled K-major tiles of the activations
//              (128 rows) and weights (BN rows) into a shared-memory ring
//   warp 1     allocates tensor memory; one lane issues the MMAs
//              (M = 128, N = BN, K = 32 per instruction) and commits to mbarriers
//   warps 2-9  epilogue: warp e reads lanes 32*(e%4).. and the column half e/4
//   warp 10    threshold stager: loads the thresholds of the next work unit's
//              channels, sorts each channel's set (the count does not depend on
//              their order) and writes them to one of two shared-memory buffers
// Two accumulator buffers in tensor memory let the epilogue of tile t overlap the
// main loop of tile t+1.  Every wait is bounded; on expiry the CTA records
// QNN_ERR_DEVICE_TIMEOUT in the device status word, drains and exits.
//
// Work units: 128 x BN tiles dealt round-robin to the CTAs.  One MMA costs about the
// same time for every N (the 128 x 32-byte activation operand is the limit), so a
// narrower tile is no cheaper; what halves a tile's cost is half the depth.  When the
// last round would fill at most half of the GPU, the kernel is launched as clusters of
// two CTAs and each tile of that round is shared by the two CTAs of a cluster, one per
// half of the depth.  Each CTA then finishes one half of the tile's channels: it stages
// the int32 partial sums of the other half in its own (by then idle) operand ring and
// bulk-copies them, 4 KB per 32 x 32 chunk, into the peer's ring (distributed shared
// memory, completion counted on the peer's mbarriers), while its other four epilogue
// warps add what the peer sent to their own accumulators and run the threshold
// epilogue.  Nothing of it touches global memory, and both CTAs of a cluster are
// resident by construction, so neither can wait for one that is not running.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace qnn {

__device__ int g_dev_status;   // QNN_OK or QNN_ERR_DEVICE_TIMEOUT

#ifdef QNN_TC_TRACE
// Debug builds only: clock64() stamps of one CTA, [slot][unit round].  Slots 0-3: epilogue
// warp 2 (entry, thresholds ready, accumulators ready, done); 4: CTA start, set-up done, all
// roles done; 5-7: MMA issuer (accumulator buffer free, first stage landed, all issued);
// 8: %globaltimer (ns) next to the slot-4 stamps, to convert cycles to time.
__device__ long long g_trace[16 * 512];
__device__ int g_trace_cta;
#define QNN_TRACE(slot, idx) do { if (blockIdx.x == g_trace_cta && (idx) < 512) g_trace[(slot) * 512 + (idx)] = clock64(); } while (0)
#define QNN_TRACE_NS(idx) do { if (blockIdx.x == g_trace_cta) { long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_trace[8 * 512 + (idx)] = t_; } } while (0)
// per-CTA wall-clock stamp (slot indexed by CTA): shows how evenly the CTAs finish
#define QNN_TRACE_CTA(slot) do { if (threadIdx.x == 0 && blockIdx.x < 512) { long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); g_trace[(slot) * 512 + blockIdx.x] = t_; } } while (0)
#else
#define QNN_TRACE(slot, idx) do { } while (0)
#define QNN_TRACE_NS(idx) do { } while (0)
#define QNN_TRACE_CTA(slot) do { } while (0)
#endif

constexpr int TC_BP = 128;          // activation rows (pixels) per tile = tensor-memory lanes
constexpr int TC_BK = 128;          // depth bytes per stage = one 128B swizzle row

// Waits of this file report to the status word defined here.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
    return mbar_wait(bar, parity, abort_flag, &g_dev_status);
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
    return mbar_wait_cluster(bar, parity, abort_flag, &g_dev_status);
}

struct TcParams {
    const int32_t *thr;    // [M][n_thr] or null
    void *out;
    int M, N, K;           // channels (weight rows), pixels (activation rows), depth
    int tiles_p, tiles_c, num_kb;
    int ld_out;            // INT8 output row pitch
    int fp_count;          // 1: |acc| < 2^22, thresholds are counted on the FP32 pipe
    uint32_t idesc;
    // work units: [0, full_units) are whole tiles; unit full_units + 2r + h is half h of
    // the depth (k-blocks [0, kb_half) / [kb_half, num_kb)) of tile full_units + r
    int units, full_units, kb_half;
    int share;             // 1: launched as clusters of two CTAs that share the tiles of the last round
    // Implicit convolution (taps == 0: plain GEMM).  The activation operand is then the
    // channels-last feature map itself: k-block kb = (filter tap, 128-byte channel chunk), and
    // the 128 pixels x 128 bytes of a stage are fetched by one im2col-mode TMA load.
    int taps, cchunks, cv_C, cv_KW, cv_OW, cv_OHW, cv_stride, cv_pad;
    // Convolution lowered inside the kernel (LOWER kernels; 8-bit maps with contiguous pixels): the
    // map itself is the input, four lowering warps build the activation tiles in shared memory
    // from image rows staged there by bulk copies.  A lowered row is one run per filter row: the
    // KW*C bytes that row contributes, padded to a multiple of 16.  LOWER == 1: C not a multiple
    // of 16 (unaligned runs), no padding around the image, the whole weight matrix resident in
    // shared memory.  LOWER == 2: C a multiple of 16 (every 16-byte piece lies in one pixel and is
    // aligned), zero padding around the image, weights streamed through the ring.
    const uint8_t *lw_in;  // the map [B][H][W][C]
    long long lw_total;    // its size in bytes
    int lw_H, lw_KH;       // image rows, filter rows
    int lw_W, lw_cpp;      // LOWER == 2: image columns, 16-byte pieces per pixel (C / 16)
    int lw_rowbytes;       // W*C: bytes of an image row
    int lw_step;           // stride*C: bytes between the runs of neighbouring output pixels
    int lw_run, lw_vecs;   // bytes of a run (KW*C) and its 16-byte pieces
    int lw_stage_bytes;    // bytes of one staging buffer
    // CTA-pair kernel with a split last round (see qgemm_tc2_kernel): the depth of each of the last
    // split_rem tiles is shared by two neighbouring CTA pairs, which exchange int32 partial sums
    // through global memory.
    int split_rem;             // tiles of the last round (0: nothing is split)
    unsigned *split_flags;     // [split_rem][part][rank][epilogue warp]: 1 = that warp's partial sums are in its slab
    int4 *split_slabs;         // same index: 2 chunks x 32 lanes x 32 columns of int32
};

constexpr int LW_WARPS = 4;                    // lowering warps of the LOWER kernels
constexpr int LW_THREADS = 32 * LW_WARPS;      // = TC_BP: one thread per pixel of the tile

// Byte range [lo, hi) of the map that the runs of output pixels [p0, p1] touch (whole image rows),
// lo rounded down to 16.
__host__ __device__ inline void lw_range(const TcParams &p, int p0, int p1, long long *lo, long long *hi) {
    const int b0 = p0 / p.cv_OHW, oh0 = (p0 - b0 * p.cv_OHW) / p.cv_OW;
    const int b1 = p1 / p.cv_OHW, oh1 = (p1 - b1 * p.cv_OHW) / p.cv_OW;
    int r0 = oh0 * p.cv_stride - p.cv_pad, r1 = oh1 * p.cv_stride - p.cv_pad + p.lw_KH;   // rows of the image
    if (r0 < 0) r0 = 0;
    if (r1 > p.lw_H) r1 = p.lw_H;
    *lo = (((long long)b0 * p.lw_H + r0) * p.lw_rowbytes) & ~15ll;
    *hi = ((long long)b1 * p.lw_H + r1) * p.lw_rowbytes;
}

// What an epilogue warp needs for the exchange of a shared tile.  The weight ring holds,
// per lane quarter q, a landing slab (what the peer sends) and a staging slab (what this
// CTA sends), each [chunk][column / 4][lane] in 16-byte units.
struct TcExchange {
    uint32_t zone;         // shared-memory address of the weight ring
    uint64_t *ring_free;   // the peer's ring is idle (1 arrival from the peer)
    uint64_t *landed;      // [lane quarter][chunk]: bytes of one chunk from the peer
    uint32_t rank;         // CTA rank in the cluster = the half of the channels this CTA finishes
};

struct TcUnit { int p0, c0, kb0, kb1, shared; };   // shared: index of the shared tile, or -1

__device__ __forceinline__ TcUnit tc_unit(const TcParams &p, int u, int bn) {
    TcUnit r;
    int tile = u;
    r.kb0 = 0; r.kb1 = p.num_kb; r.shared = -1;
    if (u >= p.full_units) {
        const int j = u - p.full_units;
        r.shared = j >> 1;
        tile = p.full_units + r.shared;
        if (j & 1) r.kb0 = p.kb_half; else r.kb1 = p.kb_half;
    }
    r.p0 = (tile % p.tiles_p) * TC_BP;
    r.c0 = (tile / p.tiles_p) * bn;
    return r;
}

enum { OUT_RAW = 0, OUT_U8 = 1, OUT_PLANES = 2 };

// ------------------------------------------------------------------- epilogue
// T(x, t) = #{q : t_q <= x}.  When every |acc| is below 2^22 the count runs on the
// FP32 pipe (twice the int32 rate, no conversions): the int32 accumulator x is
// turned into the float 1.5*2^23 + x by one integer add on its bit pattern, each
// threshold is held as the float 1.5*2^23 + (t - 1), and for integers
// saturate((1.5*2^23 + x) - (1.5*2^23 + t - 1)) is exactly 1 if x >= t, else 0.
// Thresholds are clamped to [-2^22 + 1, 2^22] first, which cannot change a
// comparison with such an accumulator.  Counts of two neighbouring channels are
// accumulated in one float on top of 1.5*2^23 (the second scaled by 256), so the
// two codes are the low two bytes of the sum's bit pattern.
constexpr int EPI_WARPS = 8;
constexpr int STAGER_WARP = 2 + EPI_WARPS;
constexpr int TC_THREADS = 64 + 32 * EPI_WARPS + 32;
constexpr float FP_MAGIC = 12582912.0f;        // 1.5 * 2^23, bit pattern 0x4B400000
constexpr int FP_MAGIC_BITS = 0x4B400000;
constexpr int FP_LIMIT = 1 << 22;

// thresholds per channel in shared memory, padded to a multiple of four
__host__ __device__ constexpr int thr_slots(int out_bits) {
    return out_bits <= 0 ? 4 : (((1 << out_bits) - 1 + 3) / 4 * 4);
}

__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, int (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// Completes every tcgen05.ld issued so far; the registers pass through the statement so
// that no use of them can be scheduled ahead of it.
__device__ __forceinline__ void tmem_ld_wait(int (&r)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
        : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
          "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
          "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
          "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
        :: "memory");
}

// Bits b, 8+b, 16+b, 24+b of x gathered into the low nibble.
__device__ __forceinline__ uint32_t nibble_of_plane(uint32_t x, int b) {
    return (((x >> b) & 0x01010101u) * 0x01020408u) >> 24;
}

// Stage the thresholds of channels [c0, c0 + bn) in shared memory (one warp, a lane per
// channel).  Slots past the row's thresholds and channels past M hold a value no
// accumulator reaches.  Sets of 7 or 15 thresholds are sorted so that the epilogue can
// count by bisection (raw int32); sets of 1 or 3 are counted linearly, in float form
// when the FP count applies.
template <int OUT_BITS>
__device__ __forceinline__ void stage_thresholds(const TcParams &p, int *thr_s, int c0, int bn, int lane) {
    constexpr int N_THR = (1 << OUT_BITS) - 1, NT = thr_slots(OUT_BITS);
    for (int c = lane; c < bn; c += 32) {
        const int m = c0 + c;
        int t[NT];
#pragma unroll
        for (int q = 0; q < NT; ++q) t[q] = 0x7fffffff;
        if (m < p.M) {
#pragma unroll
            for (int q = 0; q < N_THR; ++q) t[q] = __ldg(p.thr + (size_t)m * N_THR + q);
        }
        if (OUT_BITS >= 3) {
            // odd-even transposition sort; the pads are the largest value and stay last
#pragma unroll
            for (int r = 0; r < NT; ++r)
#pragma unroll
                for (int i = r & 1; i + 1 < NT; i += 2) {
                    const int lo = min(t[i], t[i + 1]), hi = max(t[i], t[i + 1]);
                    t[i] = lo; t[i + 1] = hi;
                }
        } else if (p.fp_count) {
#pragma unroll
            for (int q = 0; q < NT; ++q) {
                const int tc = t[q] <= -FP_LIMIT ? -FP_LIMIT + 1 : (t[q] > FP_LIMIT ? FP_LIMIT : t[q]);
                t[q] = FP_MAGIC_BITS + (tc - 1);
            }
        }
#pragma unroll
        for (int v = 0; v < NT / 4; ++v)
            reinterpret_cast<int4 *>(thr_s + c * NT)[v] = make_int4(t[4 * v], t[4 * v + 1], t[4 * v + 2], t[4 * v + 3]);
    }
}

// One chunk: this thread's pixel n, channels mc .. mc+31 (accumulators acc[0..31]).
template <int OUT_MODE, int OUT_BITS>
__device__ __forceinline__ void epilogue_chunk(const TcParams &p, const int *thr_c, const int (&acc)[32],
                                               int n, bool n_ok, int mc) {
    constexpr int N_THR = (1 << OUT_BITS) - 1, NT = thr_slots(OUT_BITS);
    if (OUT_MODE == OUT_RAW) {
        if (!n_ok) return;
        int32_t *o = reinterpret_cast<int32_t *>(p.out) + (size_t)n * p.M + mc;
        if ((p.M & 3) == 0 && mc + 32 <= p.M) {
#pragma unroll
            for (int v = 0; v < 8; ++v)
                reinterpret_cast<int4 *>(o)[v] = make_int4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (mc + j < p.M) o[j] = acc[j];
        }
        return;
    }
    // Eight channels at a time, written so that the threshold loads of all eight are issued
    // before any of them is used (independent chains interleave instead of running one
    // after the other).
    uint32_t packed[8];                          // four codes per word, one byte each
    if (OUT_BITS >= 3) {
        // bisection over the channel's sorted thresholds: the row of NT words sits in NT
        // distinct banks, so lanes that look at different slots do not conflict
        // Sixteen channels' searches advance together: a probe's load takes 100+ cycles while the
        // tensor pipe reads shared memory, and only independent chains hide that.
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            // the search position is carried as a pointer (row + count): every probe is a load at a
            // constant offset from it, and a step is load, compare, conditional add
            const int *pos[16];
            int c[16], t[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) pos[e] = thr_c + (16 * g + e) * NT;
#pragma unroll
            for (int step = NT / 2; step >= 1; step >>= 1) {
#pragma unroll
                for (int e = 0; e < 16; ++e) t[e] = pos[e][step - 1];
#pragma unroll
                for (int e = 0; e < 16; ++e) pos[e] += (acc[16 * g + e] >= t[e]) ? step : 0;
            }
#pragma unroll
            for (int e = 0; e < 16; ++e) c[e] = (int)(pos[e] - (thr_c + (16 * g + e) * NT));
#pragma unroll
            for (int v = 0; v < 4; ++v)
                packed[4 * g + v] = (uint32_t)c[4 * v] | ((uint32_t)c[4 * v + 1] << 8) | ((uint32_t)c[4 * v + 2] << 16) |
                                    ((uint32_t)c[4 * v + 3] << 24);
        }
    } else if (p.fp_count) {
        // NT == 4: one float4 of thresholds per channel
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            float4 t[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) t[e] = *reinterpret_cast<const float4 *>(thr_c + (8 * g + e) * NT);
            uint32_t pr[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const float x0 = __int_as_float(acc[8 * g + 2 * h] + FP_MAGIC_BITS);
                const float x1 = __int_as_float(acc[8 * g + 2 * h + 1] + FP_MAGIC_BITS);
                const float4 t0 = t[2 * h], t1 = t[2 * h + 1];
                float s0 = __saturatef(x0 - t0.x), s1 = __saturatef(x1 - t1.x);
                if (N_THR > 1) {
                    s0 += __saturatef(x0 - t0.y); s1 += __saturatef(x1 - t1.y);
                    s0 += __saturatef(x0 - t0.z); s1 += __saturatef(x1 - t1.z);
                }
                pr[h] = (uint32_t)__float_as_int(fmaf(s1, 256.f, s0 + FP_MAGIC));
            }
            packed[2 * g] = __byte_perm(pr[0], pr[1], 0x5410);
            packed[2 * g + 1] = __byte_perm(pr[2], pr[3], 0x5410);
        }
    } else {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            int4 t[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) t[e] = *reinterpret_cast<const int4 *>(thr_c + (8 * g + e) * NT);
            int c[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int x = acc[8 * g + e];
                c[e] = (x >= t[e].x) ? 1 : 0;
                if (N_THR > 1) c[e] += ((x >= t[e].y) ? 1 : 0) + ((x >= t[e].z) ? 1 : 0);
            }
            packed[2 * g] = (uint32_t)c[0] | ((uint32_t)c[1] << 8) | ((uint32_t)c[2] << 16) | ((uint32_t)c[3] << 24);
            packed[2 * g + 1] = (uint32_t)c[4] | ((uint32_t)c[5] << 8) | ((uint32_t)c[6] << 16) | ((uint32_t)c[7] << 24);
        }
    }
    if (!n_ok) return;
    if (OUT_MODE == OUT_U8) {
        uint8_t *o = reinterpret_cast<uint8_t *>(p.out) + (size_t)n * p.ld_out + mc;
        const int valid = p.ld_out - mc;         // a multiple of 16
        if (valid >= 16) reinterpret_cast<uint4 *>(o)[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        if (valid >= 32) reinterpret_cast<uint4 *>(o)[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
    } else {
        const int mw = (p.M + 31) >> 5, word = mc >> 5;
#pragma unroll
        for (int b = 0; b < OUT_BITS; ++b) {
            uint32_t bits = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) bits |= nibble_of_plane(packed[k], b) << (4 * k);
            reinterpret_cast<uint32_t *>(p.out)[((size_t)b * p.N + n) * mw + word] = bits;
        }
    }
}

// Exchange of partial sums between the two CTAs of a cluster that share a tile (one per
// half of the depth); see TcExchange for the layout.
enum { XCH_NONE = 0, XCH_SEND = 1, XCH_ADD = 2 };
constexpr uint32_t XCH_CHUNK_BYTES = 32 * 32 * 4;

struct TcXchWarp {
    int mode;              // XCH_*
    uint32_t local;        // SEND: staging slab, ADD: landing slab (own shared memory)
    uint32_t remote;       // SEND: the peer's landing slab (shared::cluster address)
    uint32_t bars;         // SEND: the peer's landed[q][0] (shared::cluster), ADD: own landed[q][0]
    volatile int *abort_flag;
};

// Stage one chunk in own shared memory, then one lane bulk-copies it into the peer's ring;
// the copy's bytes complete on the peer's barrier of that chunk.
__device__ __forceinline__ void send_chunk(const TcXchWarp &x, int chunk, const int (&acc)[32], int lane) {
    const uint32_t src = x.local + (uint32_t)chunk * XCH_CHUNK_BYTES;
#pragma unroll
    for (int v = 0; v < 8; ++v)
        asm volatile("st.shared.v4.s32 [%0], {%1, %2, %3, %4};"
                     ::"r"(src + (uint32_t)(v * 32 + lane) * 16u), "r"(acc[4 * v]), "r"(acc[4 * v + 1]),
                       "r"(acc[4 * v + 2]), "r"(acc[4 * v + 3]) : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // visible to the copy engine
    __syncwarp();
    if (lane == 0)
        asm volatile(
            "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
            ::"r"(x.remote + (uint32_t)chunk * XCH_CHUNK_BYTES), "r"(src), "r"(XCH_CHUNK_BYTES),
              "r"(x.bars + (uint32_t)chunk * 8u) : "memory");
}
// Wait for the peer's chunk and add it.  Returns false if the wait ran out.
__device__ __forceinline__ bool add_chunk(const TcXchWarp &x, int chunk, int (&acc)[32], int lane) {
    bool ok = true;
    if (lane == 0)
        ok = mbar_wait_cluster(reinterpret_cast<uint64_t *>(__cvta_shared_to_generic(x.bars + (uint32_t)chunk * 8u)),
                               0, x.abort_flag);
    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    __syncwarp();
    if (!ok) return false;
    const uint32_t src = x.local + (uint32_t)chunk * XCH_CHUNK_BYTES;
#pragma unroll
    for (int v = 0; v < 8; ++v) {
        int a, b, c, d;
        asm volatile("ld.shared.v4.s32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(src + (uint32_t)(v * 32 + lane) * 16u) : "memory");
        acc[4 * v] += a; acc[4 * v + 1] += b; acc[4 * v + 2] += c; acc[4 * v + 3] += d;
    }
    return true;
}

// Columns [c_begin, c_end) of one accumulator tile for this thread's pixel.  The
// tensor-memory load of the next chunk is in flight while the current one is processed.
template <int OUT_MODE, int OUT_BITS>
__device__ __forceinline__ void epilogue_cols(const TcParams &p, const int *thr_s, uint32_t t_row,
                                              int c_begin, int c_end, int n, int m0, const TcXchWarp &x,
                                              int lane) {
    constexpr int NT = thr_slots(OUT_BITS);
    int c_stop = c_end;                                  // skip chunks wholly beyond M (warp-uniform)
    if (m0 + c_stop > p.M) c_stop = c_begin + ((p.M - m0 - c_begin + 31) & ~31);
    if (c_begin >= c_stop) return;
    const bool n_ok = n < p.N;
    int acc_a[32], acc_b[32];
    tmem_ld32_issue(t_row + c_begin, acc_a);
#pragma unroll 1
    for (int c0 = c_begin; c0 < c_stop; c0 += 64) {
        tmem_ld_wait(acc_a);
        const bool has_b = c0 + 32 < c_stop;
        if (has_b) tmem_ld32_issue(t_row + c0 + 32, acc_b);
        if (x.mode == XCH_SEND) {
            send_chunk(x, (c0 - c_begin) >> 5, acc_a, lane);
        } else {
            if (x.mode == XCH_ADD && !add_chunk(x, (c0 - c_begin) >> 5, acc_a, lane)) return;
            epilogue_chunk<OUT_MODE, OUT_BITS>(p, thr_s + c0 * NT, acc_a, n, n_ok, m0 + c0);
        }
        if (has_b) {
            tmem_ld_wait(acc_b);
            if (c0 + 64 < c_stop) tmem_ld32_issue(t_row + c0 + 64, acc_a);
            if (x.mode == XCH_SEND) {
                send_chunk(x, (c0 + 32 - c_begin) >> 5, acc_b, lane);
            } else {
                if (x.mode == XCH_ADD && !add_chunk(x, (c0 + 32 - c_begin) >> 5, acc_b, lane)) return;
                epilogue_chunk<OUT_MODE, OUT_BITS>(p, thr_s + (c0 + 32) * NT, acc_b, n, n_ok, m0 + c0 + 32);
            }
        }
    }
}

// One lane polls the barrier, the warp follows.
__device__ __forceinline__ bool warp_wait(uint64_t *bar, uint32_t parity, int lane, volatile int *abort_flag) {
    bool ok = true;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag);
    return __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
}

// Threshold stager (one warp): unit i of this CTA uses threshold buffer i & 1.
// `next_unit(i, c0, bn)` yields the channel range of the CTA's i-th unit, false past the end.
template <int OUT_BITS, int BN, typename NextUnit>
__device__ __forceinline__ void stager_loop(const TcParams &p, int *thr_s, uint64_t *thr_full, uint64_t *thr_empty,
                                            int lane, volatile int *abort_flag, NextUnit next_unit) {
    constexpr int NT = thr_slots(OUT_BITS);
    int c0, bn;
    for (uint32_t i = 0; next_unit(i, c0, bn); ++i) {
        const uint32_t b = i & 1, ph = (i >> 1) & 1;
        if (!warp_wait(&thr_empty[b], ph ^ 1, lane, abort_flag)) return;
        stage_thresholds<OUT_BITS>(p, thr_s + b * BN * NT, c0, bn, lane);
        __syncwarp();
        if (lane == 0) mbar_arrive(&thr_full[b]);
    }
}

// Per-unit epilogue shared by both kernels: waits for the unit's thresholds and for its
// accumulators, processes this warp's part, then releases the threshold buffer (the
// caller releases the accumulators).  Returns false if a wait ran out.
template <int OUT_MODE, int OUT_BITS>
__device__ __forceinline__ bool epilogue_tile(const TcParams &p, const int *thr_s, uint64_t *thr_full,
                                              uint64_t *thr_empty, uint32_t thr_parity,
                                              uint64_t *tmem_full, uint32_t full_parity,
                                              uint32_t t_acc, int bn, int p0, int c0, int shared,
                                              const TcExchange &x, int warp, int lane,
                                              volatile int *abort_flag, int full_parity_dbg = 0) {
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const bool tr = warp == 2 && lane == 0;
    if (tr) QNN_TRACE(0, full_parity_dbg);
    if (OUT_MODE != OUT_RAW && !warp_wait(thr_full, thr_parity, lane, abort_flag)) return false;
    if (tr) QNN_TRACE(1, full_parity_dbg);
    if (!warp_wait(tmem_full, full_parity, lane, abort_flag)) return false;
    if (tr) QNN_TRACE(2, full_parity_dbg);
    tc_fence_after();
    const int hcols = bn >= 64 ? bn / 2 : bn;
    const int c_begin = half * hcols, c_end = (bn >= 64 || half == 0) ? c_begin + hcols : c_begin;
    TcXchWarp xw;
    xw.mode = XCH_NONE; xw.local = xw.remote = xw.bars = 0; xw.abort_flag = abort_flag;
    if (shared >= 0) {
        // warps whose channel half equals the CTA's rank finish those channels; the others
        // send their half to the peer, whose rank it equals
        const uint32_t peer = x.rank ^ 1u;
        const uint32_t slab_bytes = (uint32_t)hcols * 128u;            // hcols columns x 32 lanes x 4 bytes
        const int chunks = hcols >> 5;
        // all MMAs of this CTA are complete: its operand ring may be overwritten
        if (warp == 2 && lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(x.ring_free), peer));
        if ((uint32_t)half == x.rank) {
            xw.mode = XCH_ADD;
            xw.local = x.zone + (uint32_t)quad * slab_bytes;
            xw.bars = smem_u32(&x.landed[quad * 4]);
            if (lane == 0)
                for (int c = 0; c < chunks; ++c) mbar_arrive_expect_tx(&x.landed[quad * 4 + c], XCH_CHUNK_BYTES);
        } else {
            bool ok = true;
            if (lane == 0) ok = mbar_wait_cluster(x.ring_free, 0, abort_flag);
            if (__shfl_sync(0xffffffffu, (int)ok, 0) == 0) return false;
            __syncwarp();
            xw.mode = XCH_SEND;
            xw.local = x.zone + (uint32_t)(4 + quad) * slab_bytes;
            xw.remote = map_to_cta(x.zone + (uint32_t)quad * slab_bytes, peer);
            xw.bars = map_to_cta(smem_u32(&x.landed[quad * 4]), peer);
        }
    }
    epilogue_cols<OUT_MODE, OUT_BITS>(p, thr_s, t_acc + ((uint32_t)(quad * 32) << 16), c_begin, c_end,
                                      p0 + quad * 32 + lane, c0, xw, lane);
    tc_fence_before();
    __syncwarp();
    if (OUT_MODE != OUT_RAW && lane == 0) mbar_arrive(thr_empty);
    if (tr) QNN_TRACE(3, full_parity_dbg);
    return true;
}

// ------------------------------------------------------- kernel A: one CTA per tile
template <int BN, int STAGES, int OUT_BITS>
struct TcSmem {
    alignas(1024) uint8_t act[STAGES][TC_BP * TC_BK];
    alignas(1024) uint8_t wgt[STAGES][BN * TC_BK];
    alignas(16) int thr[2][BN * thr_slots(OUT_BITS)];
    alignas(8) uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t thr_full[2];
    uint64_t thr_empty[2];
    uint64_t ring_free;
    uint64_t landed[4 * 4];
    uint64_t w_full;           // LOWER: the resident weights have landed
    uint64_t in_full[2];       // LOWER: image rows of a unit have landed in staging buffer b
    uint64_t in_empty[2];      // LOWER: the lowering warps are done with staging buffer b
    uint32_t tmem_base;
    int abort_flag;
};

template <int BN, int STAGES, int OUT_MODE, int OUT_BITS, int LOWER>
__global__ void __launch_bounds__(LOWER ? TC_THREADS + LW_THREADS : TC_THREADS, 1)
qgemm_tc_kernel(const __grid_constant__ CUtensorMap map_act, const __grid_constant__ CUtensorMap map_wgt,
                const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    using Smem = TcSmem<BN, STAGES, OUT_BITS>;
    // 1024-byte alignment by an offset into the array (not by rounding the pointer's integer
    // value), so that the compiler still knows these are shared-memory addresses
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    constexpr uint32_t TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;
    constexpr uint32_t STAGE_BYTES = (TC_BP + BN) * TC_BK;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sm.abort_flag;
    if (threadIdx.x == 0) { QNN_TRACE(4, 0); QNN_TRACE_NS(0); }

    if (threadIdx.x == 0) {
        // LOWER: a stage is full when every lowering thread has written its row of the activation tile
        for (int s = 0; s < STAGES; ++s) { mbar_init(&sm.full[s], LOWER == 1 ? LW_THREADS : (LOWER == 2 ? LW_THREADS + 1 : 1)); mbar_init(&sm.empty[s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.tmem_full[b], 1); mbar_init(&sm.tmem_empty[b], EPI_WARPS);
            mbar_init(&sm.thr_full[b], 1); mbar_init(&sm.thr_empty[b], EPI_WARPS);
            mbar_init(&sm.in_full[b], 1); mbar_init(&sm.in_empty[b], LW_WARPS);
        }
        mbar_init(&sm.w_full, 1);
        mbar_init(&sm.ring_free, 1);
        for (int e = 0; e < 16; ++e) mbar_init(&sm.landed[e], 1);
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&sm.tmem_base, TMEM_COLS);
    tc_fence_before();
    if (p.share) cluster_sync_all();       // the peer's barriers are initialised before anyone signals them
    else __syncthreads();
    tc_fence_after();
    // set-up done: a kernel queued behind this one may start placing CTAs as SMs fall idle, and
    // this one waits here for the kernel before it (no global memory has been touched yet)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t tmem_base = sm.tmem_base;
    if (threadIdx.x == 0) QNN_TRACE(4, 1);
    QNN_TRACE_CTA(10);

    // LOWER kernels: after the struct come weight k-blocks STAGES.. (k-blocks 0..STAGES-1 live in the
    // weight ring, which these kernels do not cycle: the whole weight matrix stays resident) and
    // the two staging buffers for image rows.
    uint8_t *const w_extra = reinterpret_cast<uint8_t *>(&sm) + ((sizeof(Smem) + 1023) & ~size_t(1023));
    uint8_t *const stage_in = w_extra + (LOWER == 1 && p.num_kb > STAGES ? (size_t)(p.num_kb - STAGES) * BN * TC_BK : 0);
    auto w_block = [&](int kb) -> uint8_t * { return kb < STAGES ? sm.wgt[kb] : w_extra + (size_t)(kb - STAGES) * BN * TC_BK; };
    if (LOWER && warp == 0) {
        // ------------------- producer of the LOWER kernels: the weights once, then image rows
        if (lane == 0) {
            uint32_t staged = 0;                               // staging copies issued
            // image rows of unit u into staging buffer n & 1 (n = the unit's index in this CTA)
            auto stage_rows = [&](int u, uint32_t n) -> bool {
                const uint32_t ib = n & 1;
                if (!mbar_wait(&sm.in_empty[ib], ((n >> 1) & 1) ^ 1, abort_flag)) return false;
                const TcUnit un = tc_unit(p, u, BN);
                long long lo, hi;
                lw_range(p, un.p0, min(un.p0 + TC_BP, p.N) - 1, &lo, &hi);
                uint8_t *dst = stage_in + (size_t)ib * p.lw_stage_bytes;
                // whole 16-byte units by one bulk copy; the copy stays inside the map, whose last
                // (fewer than 16) bytes are fetched by plain loads when the unit reaches them
                long long end = (hi + 15) & ~15ll;
                if (end > p.lw_total) {
                    end = p.lw_total & ~15ll;
                    for (long long q = end; q < p.lw_total; ++q) dst[q - lo] = p.lw_in[q];
                }
                const uint32_t bytes = (uint32_t)(end - lo);
                mbar_arrive_expect_tx(&sm.in_full[ib], bytes);
                asm volatile(
                    "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                    ::"r"(smem_u32(dst)), "l"(p.lw_in + lo), "r"(bytes), "r"(smem_u32(&sm.in_full[ib])) : "memory");
                staged = n + 1;
                return true;
            };
            bool ok = true;
            uint32_t n = 0, it = 0;
            if (LOWER == 1) {
                // the whole weight matrix once, then nothing but image rows
                mbar_arrive_expect_tx(&sm.w_full, (uint32_t)p.num_kb * BN * TC_BK);
                for (int kb = 0; kb < p.num_kb; ++kb) tma_load_2d(w_block(kb), &map_wgt, &sm.w_full, kb * TC_BK, 0);
                for (int u = blockIdx.x; ok && u < p.units; u += gridDim.x, ++n) ok = stage_rows(u, n);
            } else {
                // image rows one unit ahead, weights k-block by k-block through the ring
                if ((int)blockIdx.x < p.units) ok = stage_rows(blockIdx.x, 0);
                for (int u = blockIdx.x; ok && u < p.units; u += gridDim.x, ++n) {
                    const TcUnit un = tc_unit(p, u, BN);
                    if (u + (int)gridDim.x < p.units && !(ok = stage_rows(u + gridDim.x, n + 1))) break;
                    for (int kb = un.kb0; kb < un.kb1; ++kb, ++it) {
                        const int s = it % STAGES;
                        const uint32_t ph = (it / STAGES) & 1;
                        if (!(ok = mbar_wait(&sm.empty[s], ph ^ 1, abort_flag))) break;
                        mbar_arrive_expect_tx(&sm.full[s], BN * TC_BK);
                        tma_load_2d(sm.wgt[s], &map_wgt, &sm.full[s], kb * TC_BK, un.c0);
                    }
                }
            }
            // gave up: let the copies issued last land before the CTA exits
            if (!ok) {
                if (LOWER == 1) mbar_wait(&sm.w_full, 0, abort_flag);
                if (staged > 0) mbar_wait(&sm.in_full[(staged - 1) & 1], ((staged - 1) >> 1) & 1, abort_flag);
            }
        }
        __syncwarp();
    } else if (LOWER && warp > STAGER_WARP) {
        // ------------------------------------------------------------ lowering warps
        // Thread t builds row t of every activation tile: the 128 depth bytes of pixel p0 + t in
        // k-block kb are pieces 8*kb .. 8*kb+7 of its lowered row (piece V = 16 bytes of run
        // V / vecs at offset 16 * (V % vecs); a run is contiguous in the staged image row).  The
        // tile has the layout a 128-byte-swizzled tensor-map copy would give it: 16-byte piece c
        // of row r sits at piece position c ^ (r & 7).
        const int t = threadIdx.x - 32 * (STAGER_WARP + 1);
        uint32_t it = 0, ucount = 0;
        const int total_vecs = p.lw_KH * p.lw_vecs;
        for (int u = blockIdx.x; u < p.units; u += gridDim.x, ++ucount) {
            const TcUnit un = tc_unit(p, u, BN);
            const uint32_t ib = ucount & 1;
            const int pix = min(un.p0 + t, p.N - 1);
            const int b = pix / p.cv_OHW, r = pix - b * p.cv_OHW, oh = r / p.cv_OW, ow = r - oh * p.cv_OW;
            long long lo, hi;
            lw_range(p, un.p0, min(un.p0 + TC_BP, p.N) - 1, &lo, &hi);
            const int ih0 = oh * p.cv_stride - p.cv_pad, iw0 = ow * p.cv_stride - p.cv_pad;   // first tap
            const int off = (int)((((long long)b * p.lw_H + ih0) * p.lw_rowbytes + (long long)iw0 * p.cv_C) - lo);
            const int src_px = (int)ib * p.lw_stage_bytes + off;        // byte offset of this pixel's first run in stage_in
            if (!warp_wait(&sm.in_full[ib], (ucount >> 1) & 1, lane, abort_flag)) break;
            // Piece V = 8 * kb + c of the lowered row is piece v of run kh; `so` is its byte offset in
            // stage_in.  Branch-free (selects only), so that the eight pieces of a k-block form one
            // block of independent loads and shifts.
            int v = 0, so = src_px, vleft = total_vecs;
            int kh = 0, kw = 0, vp = 0;                        // LOWER == 2: filter row, tap in it, piece in the pixel
            bool ok = true;
            for (int kb = un.kb0; kb < un.kb1; ++kb, ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                if (!(ok = warp_wait(&sm.empty[s], ph ^ 1, lane, abort_flag))) break;
                const uint32_t row = (smem_u32(sm.act[s]) + (uint32_t)t * TC_BK) ^ (uint32_t)((t & 7) << 4);
                uint32_t o[TC_BK / 16][4];
                if (LOWER == 1) {
#pragma unroll
                    for (int c = 0; c < TC_BK / 16; ++c) {
                        const bool live = c < vleft, last = v == p.lw_vecs - 1;
                        // an unaligned 16-byte read: five aligned words and four funnel shifts
                        const int a = live ? so : src_px;
                        const uint32_t *w = reinterpret_cast<const uint32_t *>(stage_in) + (a >> 2);
                        const int sh = (a & 3) * 8;
                        uint32_t x[5];
#pragma unroll
                        for (int i = 0; i < 5; ++i) x[i] = w[i];
                        // No masking: the bytes past a run's end (and the pieces past the last run) meet
                        // weight bytes that are zero -- the pad columns of the weight rows, or depth
                        // positions past K, which the weight copy fills with zeros -- so whatever image
                        // bytes land there add nothing to the integer sums.
#pragma unroll
                        for (int i = 0; i < 4; ++i) o[c][i] = __funnelshift_r(x[i], x[i + 1], sh);
                        so += last ? p.lw_rowbytes - 16 * (p.lw_vecs - 1) : 16;
                        v = last ? 0 : v + 1;
                    }
                } else {
                    // aligned pieces, each inside one pixel: tap (kh, kw) outside the image reads as zero
#pragma unroll
                    for (int c = 0; c < TC_BK / 16; ++c) {
                        const bool last = v == p.lw_vecs - 1;
                        const bool inside = c < vleft && (unsigned)(ih0 + kh) < (unsigned)p.lw_H &&
                                            (unsigned)(iw0 + kw) < (unsigned)p.lw_W;
                        const uint4 d = *reinterpret_cast<const uint4 *>(stage_in + (inside ? so : (int)ib * p.lw_stage_bytes));
                        o[c][0] = inside ? d.x : 0u; o[c][1] = inside ? d.y : 0u;
                        o[c][2] = inside ? d.z : 0u; o[c][3] = inside ? d.w : 0u;
                        const bool px_end = vp == p.lw_cpp - 1;
                        so += last ? p.lw_rowbytes - 16 * (p.lw_vecs - 1) : 16;
                        kw = last ? 0 : (px_end ? kw + 1 : kw);
                        vp = (last || px_end) ? 0 : vp + 1;
                        kh += last ? 1 : 0;
                        v = last ? 0 : v + 1;
                    }
                }
                vleft -= TC_BK / 16;
#pragma unroll
                for (int c = 0; c < TC_BK / 16; ++c)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                 ::"r"(row ^ (uint32_t)(c << 4)), "r"(o[c][0]), "r"(o[c][1]), "r"(o[c][2]), "r"(o[c][3])
                                 : "memory");
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core's reads
                mbar_arrive(&sm.full[s]);
            }
            if (!ok) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.in_empty[ib]);
        }
    } else if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int u = blockIdx.x; ok && u < p.units; u += gridDim.x) {
                const TcUnit un = tc_unit(p, u, BN);
                int cv_w = 0, cv_h = 0, cv_n = 0;          // base pixel of the unit's first output pixel
                if (p.taps) {
                    cv_n = un.p0 / p.cv_OHW;
                    const int r = un.p0 - cv_n * p.cv_OHW, oh = r / p.cv_OW;
                    cv_h = oh * p.cv_stride - p.cv_pad;
                    cv_w = (r - oh * p.cv_OW) * p.cv_stride - p.cv_pad;
                }
                for (int kb = un.kb0; kb < un.kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    QNN_TRACE(14, it);
                    if (!(ok = mbar_wait(&sm.empty[s], ph ^ 1, abort_flag))) break;
                    QNN_TRACE(15, it);
                    mbar_arrive_expect_tx(&sm.full[s], STAGE_BYTES);
                    if (p.taps) {
                        const int tap = kb / p.cchunks, cc = kb - tap * p.cchunks;
                        const int kh = tap / p.cv_KW, kw = tap - kh * p.cv_KW;
                        tma_load_im2col(sm.act[s], &map_act, &sm.full[s], cc * TC_BK, cv_w, cv_h, cv_n,
                                        (uint16_t)kw, (uint16_t)kh);
                        tma_load_2d(sm.wgt[s], &map_wgt, &sm.full[s], tap * p.cv_C + cc * TC_BK, un.c0);
                    } else {
                        tma_load_2d(sm.act[s], &map_act, &sm.full[s], kb * TC_BK, un.p0);
                        tma_load_2d(sm.wgt[s], &map_wgt, &sm.full[s], kb * TC_BK, un.c0);
                    }
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
            // 32-byte slices with real data in a "tail" k-block (see below); 4: none is ever skipped
            const int tail_bytes = p.taps ? p.cv_C - (p.cchunks - 1) * TC_BK : (LOWER ? p.K - (p.num_kb - 1) * TC_BK : TC_BK);
            const int tail_kk = tail_bytes >= TC_BK ? TC_BK / 32 : (tail_bytes + 31) >> 5;
            if (LOWER == 1) ok = mbar_wait(&sm.w_full, 0, abort_flag);
            for (int u = blockIdx.x; ok && u < p.units; u += gridDim.x, ++tcount) {
                const uint32_t buf = tcount & 1, acc_ph = (tcount >> 1) & 1;
                const TcUnit un = tc_unit(p, u, BN);
                if (!(ok = mbar_wait(&sm.tmem_empty[buf], acc_ph ^ 1, abort_flag))) break;
                tc_fence_after();
                QNN_TRACE(5, tcount);
                const uint32_t d_tmem = tmem_base + buf * BN;
                int cc = p.taps ? un.kb0 % p.cchunks : 0;      // implicit convolution: channel chunk of the k-block
                for (int kb = un.kb0; kb < un.kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    QNN_TRACE(12, it);
                    if (!(ok = mbar_wait(&sm.full[s], ph, abort_flag))) break;
                    tc_fence_after();
                    QNN_TRACE(13, it);
                    if (kb == un.kb0) QNN_TRACE(6, tcount);
                    const uint64_t da = umma_smem_desc(smem_u32(sm.act[s]));
                    const uint64_t db = umma_smem_desc(smem_u32(LOWER == 1 ? w_block(kb) : sm.wgt[s]));
                    // A k-block that holds fewer than 128 real depth bytes (the last channel chunk of a
                    // filter tap; the end of a lowered row) skips its all-zero MMAs.  Everything else
                    // takes the loop of exactly four MMAs: this thread's instructions between MMAs are
                    // time during which the tensor pipe may run dry.
                    const bool tail = p.taps ? cc == p.cchunks - 1 : (LOWER != 0 && kb == p.num_kb - 1);
                    if (LOWER) {
                        // (the kernels with lowering warps are bound by those warps, and measured faster
                        // with the predicated form of the loop)
                        const int nk = tail ? tail_kk : TC_BK / 32;
#pragma unroll
                        for (int kk = 0; kk < TC_BK / 32; ++kk)
                            if (kk < nk) umma_i8(d_tmem, da + 2 * kk, db + 2 * kk, p.idesc, (kb > un.kb0) || kk != 0);
                    } else if (tail && tail_kk != TC_BK / 32) {
                        for (int kk = 0; kk < tail_kk; ++kk)
                            umma_i8(d_tmem, da + 2 * kk, db + 2 * kk, p.idesc, (kb > un.kb0) || kk != 0);
                    } else {
#pragma unroll
                        for (int kk = 0; kk < TC_BK / 32; ++kk)   // 32 depth bytes per MMA: +2 in 16-byte units
                            umma_i8(d_tmem, da + 2 * kk, db + 2 * kk, p.idesc, (kb > un.kb0) || kk != 0);
                    }
                    umma_commit(&sm.empty[s]);
                    if (p.taps && ++cc == p.cchunks) cc = 0;
                }
                if (ok) umma_commit(&sm.tmem_full[buf]);
                QNN_TRACE(7, tcount);
            }
        }
        __syncwarp();
    } else if (warp == STAGER_WARP) {
        // ---------------------------------------------------- threshold stager
        if (OUT_MODE != OUT_RAW)
            stager_loop<OUT_BITS, BN>(p, &sm.thr[0][0], sm.thr_full, sm.thr_empty, lane, abort_flag,
                                      [&](uint32_t i, int &c0, int &bn) {
                                          const long long u = blockIdx.x + (long long)i * gridDim.x;
                                          if (u >= p.units) return false;
                                          const TcUnit un = tc_unit(p, (int)u, BN);
                                          c0 = un.c0; bn = BN;
                                          return true;
                                      });
    } else {
        // ------------------------------------------------------------ epilogue
        uint32_t tcount = 0;
        TcExchange xc;
        xc.zone = smem_u32(&sm.wgt[0][0]);
        xc.ring_free = &sm.ring_free; xc.landed = sm.landed;
        xc.rank = p.share ? cluster_ctarank() : 0u;
        for (int u = blockIdx.x; u < p.units; u += gridDim.x, ++tcount) {
            const TcUnit un = tc_unit(p, u, BN);
            const uint32_t buf = tcount & 1, acc_ph = (tcount >> 1) & 1;
            if (!epilogue_tile<OUT_MODE, OUT_BITS>(p, sm.thr[buf], &sm.thr_full[buf], &sm.thr_empty[buf], acc_ph,
                                                   &sm.tmem_full[buf], acc_ph, tmem_base + buf * BN, BN,
                                                   un.p0, un.c0, un.shared, xc, warp, lane, abort_flag, (int)tcount))
                break;
            if (lane == 0) mbar_arrive(&sm.tmem_empty[buf]);     // one arrival per warp
        }
    }

    tc_fence_before();
    if (p.share) cluster_sync_all();       // the peer may still write this CTA's shared memory or barriers
    else __syncthreads();
    if (threadIdx.x == 0) { QNN_TRACE(4, 2); QNN_TRACE_NS(2); }
    QNN_TRACE_CTA(11);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------- kernel B: a CTA pair per 256 x 256 tile
// Two CTAs of a cluster (two SMs) share one tile: each stages 128 activation rows
// and 128 of the 256 weight rows, and the leader CTA issues cta_group::2 MMAs
// (M = 256, N = 256) that read both halves, so each SM pulls 32 KB per 128 depth
// bytes from L2 instead of 48 KB.  No copy is multicast: each CTA loads only what
// lands in its own shared memory; its completion bytes are counted on the
// leader's mbarrier.
constexpr int T2_STAGES = 6;
constexpr int T2_BN = 256;
enum { PAIR_PLAIN = 0, PAIR_CONV = 1, PAIR_SPLIT = 2 };
constexpr int SPLIT_FLAG_BYTES = 8192;                   // flags of the split last round, at the start of the workspace
constexpr int SPLIT_SLAB_INT4 = 2 * 8 * 32;              // one epilogue warp's partial sums: 2 chunks of 32 x 32 int32
constexpr size_t SPLIT_TILE_BYTES = (size_t)2 * 2 * EPI_WARPS * SPLIT_SLAB_INT4 * 16;   // both parts, both CTAs: 256 KB

template <int OUT_BITS>
struct Tc2Smem {
    alignas(1024) uint8_t act[T2_STAGES][TC_BP * TC_BK];
    alignas(1024) uint8_t wgt[T2_STAGES][128 * TC_BK];
    alignas(16) int thr[2][T2_BN * thr_slots(OUT_BITS)];
    alignas(8) uint64_t full[T2_STAGES];
    uint64_t empty[T2_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t thr_full[2];
    uint64_t thr_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

// Width (MMA N) of the channel tile that starts at channel ct: 256, or what is left of M rounded up
// to 64 (the two epilogue halves are whole 32-column chunks).
__device__ __forceinline__ int pair_tile_width(const TcParams &p, int ct) {
    const int left = p.M - ct;
    return left >= T2_BN ? T2_BN : ((left + 63) & ~63);
}

// One unit of work of a CTA pair: a whole tile, or (PAIR_SPLIT, last round) one half of a tile's depth.
struct PairUnit { int tile, kb_lo, kb_hi, part, j; };      // part < 0: whole tile; else j = index among the split tiles
template <int KIND>
__device__ __forceinline__ PairUnit pair_unit(const TcParams &p, int u, int num_tiles) {
    PairUnit r;
    r.tile = u; r.kb_lo = 0; r.kb_hi = p.num_kb; r.part = -1; r.j = 0;
    if (KIND == PAIR_SPLIT) {
        const int full = num_tiles - p.split_rem;
        if (u >= full) {
            r.j = (u - full) >> 1; r.part = (u - full) & 1;
            r.tile = full + r.j;
            r.kb_lo = r.part ? p.num_kb >> 1 : 0;
            r.kb_hi = r.part ? p.num_kb : p.num_kb >> 1;
        }
    }
    return r;
}

// Epilogue of a split unit.  The pair that ran depth part `part` of tile j finishes the 64-column
// groups g with (g & 1) == part and sends its partial sums of the other groups to the pair that ran
// the other part (the neighbouring pair, busy with the same tile at the same time).  Every epilogue
// warp covers two groups: it first writes the one it does not own to its slab in global memory and
// raises its flag (release), then waits (bounded) for the flag of the same warp of the partner pair,
// adds the partner's slab to the group it owns, counts thresholds and stores.  The reader clears the
// flag, so the flags are zero again when the kernel ends.
template <int OUT_MODE, int OUT_BITS>
__device__ __forceinline__ bool epilogue_tile_split(const TcParams &p, const int *thr_s, uint64_t *thr_full,
                                                    uint64_t *thr_empty, uint32_t thr_parity, uint64_t *tmem_full,
                                                    uint32_t full_parity, uint32_t t_acc, int p0, int c0,
                                                    const PairUnit &un, uint32_t rank, int warp, int lane,
                                                    volatile int *abort_flag) {
    constexpr int NT = thr_slots(OUT_BITS);
    const int quad = warp & 3, half = (warp - 2) >> 2, ew = warp - 2;
    if (OUT_MODE != OUT_RAW && !warp_wait(thr_full, thr_parity, lane, abort_flag)) return false;
    if (!warp_wait(tmem_full, full_parity, lane, abort_flag)) return false;
    tc_fence_after();
    const uint32_t t_row = t_acc + ((uint32_t)(quad * 32) << 16);
    const int n = p0 + quad * 32 + lane;
    const int own_c = half * 128 + un.part * 64, send_c = half * 128 + (un.part ^ 1) * 64;
    const size_t mine = (size_t)((un.j * 2 + un.part) * 2 + (int)rank) * EPI_WARPS + ew;
    const size_t theirs = (size_t)((un.j * 2 + (un.part ^ 1)) * 2 + (int)rank) * EPI_WARPS + ew;
    int acc[32];
    // ---- send (chunks wholly beyond M are neither sent nor awaited: both sides skip them alike)
    {
        int4 *slab = p.split_slabs + mine * SPLIT_SLAB_INT4;
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
            if (c0 + send_c + 32 * c >= p.M) break;
            tmem_ld32_issue(t_row + send_c + 32 * c, acc);
            tmem_ld_wait(acc);
#pragma unroll
            for (int v = 0; v < 8; ++v)
                slab[(c * 8 + v) * 32 + lane] = make_int4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
        }
        __syncwarp();
        // the warp's stores happen before lane 0's release (ordered by the __syncwarp above, made
        // visible GPU-wide by the release); a group wholly beyond M has no reader
        if (lane == 0 && c0 + send_c < p.M)
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.split_flags + mine), "r"(1u) : "memory");
    }
    // ---- receive, add, finish
    bool ok = true;
    if (c0 + own_c < p.M) {
        if (lane == 0) {
            const unsigned *flag = p.split_flags + theirs;
            const long long t0 = clock64();
            for (;;) {
                unsigned v;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
                if (v != 0u) break;
                if (*abort_flag) { ok = false; break; }
                if (clock64() - t0 > TC_WAIT_CYCLES) {
                    *abort_flag = 1;
                    atomicExch(&g_dev_status, (int)QNN_ERR_DEVICE_TIMEOUT);
                    ok = false;
                    break;
                }
                __nanosleep(100);
            }
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        if (!ok) return false;
        const int4 *slab = p.split_slabs + theirs * SPLIT_SLAB_INT4;
        // both chunks' partial sums are requested before the first is used (one L2 round trip, not two)
        int4 q[2][8];
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int v = 0; v < 8; ++v) q[c][v] = __ldcg(slab + (c * 8 + v) * 32 + lane);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            if (c0 + own_c + 32 * c >= p.M) break;
            tmem_ld32_issue(t_row + own_c + 32 * c, acc);
            tmem_ld_wait(acc);
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                acc[4 * v] += q[c][v].x; acc[4 * v + 1] += q[c][v].y; acc[4 * v + 2] += q[c][v].z; acc[4 * v + 3] += q[c][v].w;
            }
            epilogue_chunk<OUT_MODE, OUT_BITS>(p, thr_s + (own_c + 32 * c) * NT, acc, n, n < p.N, c0 + own_c + 32 * c);
        }
        __syncwarp();
        if (lane == 0) *(volatile unsigned *)(p.split_flags + theirs) = 0u;     // consumed: zero for the next launch
    }
    tc_fence_before();
    __syncwarp();
    if (OUT_MODE != OUT_RAW && lane == 0) mbar_arrive(thr_empty);
    return true;
}

// KIND PAIR_CONV: implicit convolution (see TcParams): each CTA of the pair fetches its 128 output
// pixels through the im2col tensor map, and the last channel tile is as wide as the channels left
// (the plain GEMM keeps 256-wide tiles and a loop body of four MMAs: the issuing thread is the one
// thread whose instruction count shows in the kernel's time).
// KIND PAIR_SPLIT: a plain GEMM whose last round of tiles would leave at least half of the pairs
// idle: each of those tiles is run by two neighbouring pairs, one per half of the depth, which
// exchange partial sums through the caller's workspace (epilogue_tile_split).  All CTAs of the
// grid are resident together (one per SM), and the partner works on the same tile at the same
// time, so the bounded wait normally lasts a few hundred cycles.
template <int OUT_MODE, int OUT_BITS, int KIND>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
qgemm_tc2_kernel(const __grid_constant__ CUtensorMap map_act, const __grid_constant__ CUtensorMap map_wgt,
                 const TcParams p) {
    constexpr bool CONV = KIND == PAIR_CONV;
    extern __shared__ uint8_t smem_raw[];
    using Smem = Tc2Smem<OUT_BITS>;
    // 1024-byte alignment by an offset into the array (not by rounding the pointer's integer
    // value), so that the compiler still knows these are shared-memory addresses
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    constexpr uint32_t TMEM_COLS = 2 * T2_BN;
    constexpr uint32_t PAIR_STAGE_BYTES = 2 * (TC_BP + 128) * TC_BK;   // both CTAs' copies of one stage

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    volatile int *abort_flag = &sm.abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < T2_STAGES; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.tmem_full[b], 1); mbar_init(&sm.tmem_empty[b], 2 * EPI_WARPS);
            mbar_init(&sm.thr_full[b], 1); mbar_init(&sm.thr_empty[b], EPI_WARPS);
        }
        sm.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(&sm.tmem_base, TMEM_COLS);
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    // set-up done (see the one-CTA kernel): dependents may be placed, and no global memory is
    // touched before the kernel ahead of this one has completed
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t tmem_base = sm.tmem_base;
    const int num_tiles = p.tiles_p * p.tiles_c;       // tiles of 256 pixels x 256 channels
    const int num_units = num_tiles + (KIND == PAIR_SPLIT ? p.split_rem : 0);

    if (warp == 0) {
        // ---------------------------------------- producer (one per CTA, own halves)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int u = pair; ok && u < num_units; u += num_pairs) {
                const PairUnit un = pair_unit<KIND>(p, u, num_tiles);
                const int tile = un.tile;
                const int p0 = (tile % p.tiles_p) * 256 + (int)rank * 128;
                const int ct = (tile / p.tiles_p) * T2_BN;
                // this CTA's half of the tile's channels (the copy always fetches 128 weight rows; a
                // narrower last tile uses the first half-width of them)
                const int c0 = ct + (int)rank * (CONV ? pair_tile_width(p, ct) >> 1 : 128);
                int cv_w = 0, cv_h = 0, cv_n = 0;          // CONV: base pixel of this CTA's first output pixel
                if (CONV) {
                    cv_n = p0 / p.cv_OHW;
                    const int r = p0 - cv_n * p.cv_OHW, oh = r / p.cv_OW;
                    cv_h = oh * p.cv_stride - p.cv_pad;
                    cv_w = (r - oh * p.cv_OW) * p.cv_stride - p.cv_pad;
                }
                int tap = 0, cc = 0, kh = 0, kw = 0;       // CONV: k-block = (filter tap, channel chunk)
                for (int kb = un.kb_lo; kb < un.kb_hi; ++kb, ++it) {
                    const int s = it % T2_STAGES;
                    const uint32_t ph = (it / T2_STAGES) & 1;
                    if (!(ok = mbar_wait(&sm.empty[s], ph ^ 1, abort_flag))) break;
                    if (rank == 0) mbar_arrive_expect_tx(&sm.full[s], PAIR_STAGE_BYTES);
                    const uint32_t leader_full = map_to_cta(smem_u32(&sm.full[s]), 0);
                    if (CONV) {
                        tma_load_im2col_pair(sm.act[s], &map_act, leader_full, cc * TC_BK, cv_w, cv_h, cv_n,
                                             (uint16_t)kw, (uint16_t)kh);
                        tma_load_2d_pair(sm.wgt[s], &map_wgt, leader_full, tap * p.cv_C + cc * TC_BK, c0);
                        if (++cc == p.cchunks) { cc = 0; ++tap; if (++kw == p.cv_KW) { kw = 0; ++kh; } }
                    } else {
                        tma_load_2d_pair(sm.act[s], &map_act, leader_full, kb * TC_BK, p0);
                        tma_load_2d_pair(sm.wgt[s], &map_wgt, leader_full, kb * TC_BK, c0);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------- MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            uint32_t tcount = 0;
            bool ok = true;
            // CONV: 32-byte slices of a tap's last channel chunk that hold real channels (4: all)
            const int tail_c = CONV ? p.cv_C - (p.cchunks - 1) * TC_BK : TC_BK;
            const int tail_kk = tail_c >= TC_BK ? TC_BK / 32 : (tail_c + 31) >> 5;
            // Everything that depends on the stage is carried incrementally (no division, no address
            // mapping in the loop): the fewer instructions this thread runs between MMAs, the less
            // often the tensor pipe waits for it.
            const uint64_t da0 = umma_smem_desc(smem_u32(sm.act[0])), db0 = umma_smem_desc(smem_u32(sm.wgt[0]));
            const uint32_t empty0 = map_to_cta(smem_u32(&sm.empty[0]), 0), empty1 = map_to_cta(smem_u32(&sm.empty[0]), 1);
            int s = 0;                                     // stage of the ring
            uint32_t ph = 0;                               // its phase
            for (int u = pair; ok && u < num_units; u += num_pairs, ++tcount) {
                const PairUnit un = pair_unit<KIND>(p, u, num_tiles);
                const int tile = un.tile;
                const int unit_kb = un.kb_hi - un.kb_lo;   // all k-blocks, or (a split tile) one half of them
                const uint32_t buf = tcount & 1, acc_ph = (tcount >> 1) & 1;
                if (!(ok = mbar_wait(&sm.tmem_empty[buf], acc_ph ^ 1, abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * T2_BN;
                // MMA N: 256, or (CONV) the width of a narrower last channel tile
                const uint32_t idesc = p.idesc | ((uint32_t)((CONV ? pair_tile_width(p, (tile / p.tiles_p) * T2_BN) : T2_BN) >> 3) << 17);
                int cc = 0;                                // CONV: channel chunk of the k-block
                for (int kb = 0; kb < unit_kb; ++kb) {
                    if (!(ok = mbar_wait(&sm.full[s], ph, abort_flag))) break;
                    tc_fence_after();
                    const uint64_t da = da0 + (uint64_t)(s * (TC_BP * TC_BK / 16));
                    const uint64_t db = db0 + (uint64_t)(s * (128 * TC_BK / 16));
                    if (CONV && tail_kk != TC_BK / 32 && cc == p.cchunks - 1) {
                        // the last channel chunk of a tap holds fewer than 128 real bytes: skip the all-zero MMAs
                        for (int kk = 0; kk < tail_kk; ++kk)
                            umma_i8_pair(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (kb | kk) != 0);
                    } else {
#pragma unroll
                        for (int kk = 0; kk < TC_BK / 32; ++kk)
                            umma_i8_pair(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (kb | kk) != 0);
                    }
                    if (CONV && ++cc == p.cchunks) cc = 0;
                    // free the stage in both CTAs
                    umma_commit_pair(empty0 + 8u * (uint32_t)s);
                    umma_commit_pair(empty1 + 8u * (uint32_t)s);
                    if (++s == T2_STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) {
                    umma_commit_pair(map_to_cta(smem_u32(&sm.tmem_full[buf]), 0));
                    umma_commit_pair(map_to_cta(smem_u32(&sm.tmem_full[buf]), 1));
                }
            }
        }
        __syncwarp();
    } else if (warp == STAGER_WARP) {
        // ------------------------------------ threshold stager (all 256 channels of the tile)
        if (OUT_MODE != OUT_RAW)
            stager_loop<OUT_BITS, T2_BN>(p, &sm.thr[0][0], sm.thr_full, sm.thr_empty, lane, abort_flag,
                                         [&](uint32_t i, int &c0, int &bn) {
                                             const long long u = pair + (long long)i * num_pairs;
                                             if (u >= num_units) return false;
                                             const int tile = pair_unit<KIND>(p, (int)u, num_tiles).tile;
                                             c0 = (tile / p.tiles_p) * T2_BN;
                                             bn = CONV ? pair_tile_width(p, c0) : T2_BN;
                                             return true;
                                         });
    } else {
        // ----------------------------- epilogue (each CTA: its 128 pixels, all 256 channels)
        uint32_t tcount = 0;
        for (int u = pair; u < num_units; u += num_pairs, ++tcount) {
            const PairUnit un = pair_unit<KIND>(p, u, num_tiles);
            const int tile = un.tile;
            const int p0 = (tile % p.tiles_p) * 256 + (int)rank * 128, c0 = (tile / p.tiles_p) * T2_BN;
            const uint32_t buf = tcount & 1, acc_ph = (tcount >> 1) & 1;
            if (KIND == PAIR_SPLIT && un.part >= 0) {
                if (!epilogue_tile_split<OUT_MODE, OUT_BITS>(p, sm.thr[buf], &sm.thr_full[buf], &sm.thr_empty[buf], acc_ph,
                                                             &sm.tmem_full[buf], acc_ph, tmem_base + buf * T2_BN, p0, c0, un,
                                                             rank, warp, lane, abort_flag))
                    break;
            } else if (!epilogue_tile<OUT_MODE, OUT_BITS>(p, sm.thr[buf], &sm.thr_full[buf], &sm.thr_empty[buf], acc_ph,
                                                          &sm.tmem_full[buf], acc_ph, tmem_base + buf * T2_BN,
                                                          CONV ? pair_tile_width(p, c0) : T2_BN, p0, c0, -1, TcExchange{}, warp,
                                                          lane, abort_flag))
                break;
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&sm.tmem_empty[buf]), 0));
        }
    }

    // the peer may still read this CTA's shared memory or signal its barriers
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
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

bool tc_make_tile_map(CUtensorMap *map, const void *base, int rows, int row_bytes, int ld, int box_rows) {
    return make_map(map, base, rows, row_bytes, ld, box_rows);
}

typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeIm2colFn encode_im2col_fn() {
    static EncodeIm2colFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeIm2colFn)p;
    }
    return fn;
}

// Channels-last byte map [B][H][W][pitch] seen through an im2col tensor map: a load yields 128
// pixels x 128 channel bytes; base pixels range over the padded map so that every filter tap
// (offset 0 .. K-1 from the base) of every output pixel is addressable, out of range = 0.
static bool make_im2col_map(CUtensorMap *map, const void *base, const qnn_conv_desc *d, int pitch) {
    EncodeIm2colFn fn = encode_im2col_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)d->C, (cuuint64_t)d->W, (cuuint64_t)d->H, (cuuint64_t)d->B};
    cuuint64_t strides[3] = {(cuuint64_t)pitch, (cuuint64_t)pitch * d->W, (cuuint64_t)pitch * d->W * d->H};
    int lower[2] = {-d->pad, -d->pad};
    int upper[2] = {d->pad - (d->KW - 1), d->pad - (d->KH - 1)};
    cuuint32_t estr[4] = {1, (cuuint32_t)d->stride, (cuuint32_t)d->stride, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, lower, upper,
              (cuuint32_t)TC_BK, (cuuint32_t)TC_BP, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Shared memory of a LOWER kernel besides its two staging buffers.
template <int BN, int STAGES, int OUT_BITS>
constexpr size_t tc_lower_base_smem() { return ((sizeof(TcSmem<BN, STAGES, OUT_BITS>) + 1023) & ~size_t(1023)) + 1024; }
constexpr size_t TC_SMEM_LIMIT = 227 * 1024;

template <int BN, int STAGES, int OUT_MODE, int OUT_BITS, int LOWER = 0>
static qnn_status launch_cfg(const CUtensorMap &ma, const CUtensorMap &mw, const TcParams &p, cudaStream_t s) {
    auto kern = qgemm_tc_kernel<BN, STAGES, OUT_MODE, OUT_BITS, LOWER>;
    size_t smem = sizeof(TcSmem<BN, STAGES, OUT_BITS>) + 1024;
    if (LOWER) {
        smem = tc_lower_base_smem<BN, STAGES, OUT_BITS>() + 2 * (size_t)p.lw_stage_bytes +
               (LOWER == 1 && p.num_kb > STAGES ? (size_t)(p.num_kb - STAGES) * BN * TC_BK : 0);
        if (smem > TC_SMEM_LIMIT) return QNN_ERR_UNSUPPORTED;
    }
    // per instantiation and device: the largest size configured so far
    static size_t attr_smem[QNN_MAX_DEVICES] = {0};
    const int dev = current_device();
    if (dev < 0) return QNN_ERR_CUDA;
    if (smem > attr_smem[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return QNN_ERR_CUDA;
        attr_smem[dev] = smem;
    }
    const int grid = p.units < sm_count() ? p.units : sm_count();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(LOWER ? TC_THREADS + LW_THREADS : TC_THREADS);
    cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    // Programmatic dependent launch: when the previous operation on the stream is a kernel that
    // has released its dependents, this kernel's CTAs may start on SMs as they fall idle and do
    // their set-up there; they touch no global memory before griddepcontrol.wait, which returns
    // once the previous kernel has completed.  Small grids too: a CTA of this kernel has an SM's
    // shared memory to itself, so early placement cannot crowd several onto one SM (the chain of
    // 13 small launches at batch 1: 73.8 -> 69.4 us).
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
    if (p.share) {
        // clusters of two CTAs: consecutive block indices share a tile of the last round
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 2; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, kern, ma, mw, p) != cudaSuccess) return QNN_ERR_CUDA;
    count_launch();
    return launch_status();
}

template <int OUT_MODE, int OUT_BITS, int KIND>
static qnn_status launch_pair_cfg(const CUtensorMap &ma, const CUtensorMap &mw, const TcParams &p, cudaStream_t s) {
    auto kern = qgemm_tc2_kernel<OUT_MODE, OUT_BITS, KIND>;
    const size_t smem = sizeof(Tc2Smem<OUT_BITS>) + 1024;
    static bool attr_done[QNN_MAX_DEVICES] = {false};       // per instantiation and device
    const int dev = current_device();
    if (dev < 0) return QNN_ERR_CUDA;
    if (!attr_done[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return QNN_ERR_CUDA;
        attr_done[dev] = true;
    }
    const int tiles = p.tiles_p * p.tiles_c;
    const int max_pairs = sm_count() / 2;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    int na = 0;
    if (2 * pairs >= sm_count() - 1) {     // a grid that fills the GPU: programmatic dependent launch (see launch_cfg)
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, kern, ma, mw, p) != cudaSuccess) return QNN_ERR_CUDA;
    count_launch();
    return launch_status();
}

#define QNN_TC_DISPATCH(CALL_RAW, CALL)                                                    \
    if (mode == OUT_RAW) return CALL_RAW;                                                  \
    switch (out_bits) {                                                                    \
        case 1: return mode == OUT_U8 ? CALL(OUT_U8, 1) : CALL(OUT_PLANES, 1);             \
        case 2: return mode == OUT_U8 ? CALL(OUT_U8, 2) : CALL(OUT_PLANES, 2);             \
        case 3: return mode == OUT_U8 ? CALL(OUT_U8, 3) : CALL(OUT_PLANES, 3);             \
        case 4: return mode == OUT_U8 ? CALL(OUT_U8, 4) : CALL(OUT_PLANES, 4);             \
    }                                                                                      \
    return QNN_ERR_UNSUPPORTED;

template <int BN, int STAGES, int LOWER = 0>
static qnn_status launch_out(int mode, int out_bits, const CUtensorMap &ma, const CUtensorMap &mw,
                             const TcParams &p, cudaStream_t s) {
#define QNN_C1(MODE_, BITS_) launch_cfg<BN, STAGES, MODE_, BITS_, LOWER>(ma, mw, p, s)
    QNN_TC_DISPATCH(QNN_C1(OUT_RAW, 0), QNN_C1)
#undef QNN_C1
}

static qnn_status launch_pair_out(int mode, int out_bits, const CUtensorMap &ma, const CUtensorMap &mw,
                                  const TcParams &p, cudaStream_t s) {
#define QNN_C2(MODE_, BITS_) (p.taps ? launch_pair_cfg<MODE_, BITS_, PAIR_CONV>(ma, mw, p, s)                      \
                                     : (p.split_rem ? launch_pair_cfg<MODE_, BITS_, PAIR_SPLIT>(ma, mw, p, s)     \
                                                    : launch_pair_cfg<MODE_, BITS_, PAIR_PLAIN>(ma, mw, p, s)))
    QNN_TC_DISPATCH(QNN_C2(OUT_RAW, 0), QNN_C2)
#undef QNN_C2
}

// Kernel choice.  QNN_TC_KERNEL=single|pair in the environment overrides it (tests, sweeps).
// The CTA-pair kernel (each SM pulls 32 KB instead of 48 KB per k-block, six stages instead of
// four) is the faster one wherever its 256 x 256 tiles fill the SM pairs for a round and a half or
// more and waste little of N: by 6 % on the 4096^3 sweep inside the packer + GEMM sequence, by
// 12-22 % at 4096 x 18944 x 512..4096 and 8192^3 (tensor pipe 88 % busy).  Smaller problems keep the
// one-CTA kernel, whose tiles of the last round are shared by CTA pairs that split the depth.
static bool choose_pair_kernel(const qnn_gemm_desc *d, int sms) {
    const char *force = getenv("QNN_TC_KERNEL");
    if (force && force[0] == 's') return false;
    if (force && force[0] == 'p') return true;
    const int pairs = sms / 2;
    const long long tiles2 = (long long)ceil_div(d->N, 256) * ceil_div(d->M, T2_BN);
    return d->M >= T2_BN && d->N >= 2048 && 2 * tiles2 >= 3ll * pairs;
}

// Tile plan of the one-CTA kernel: channel tile, grid, and whether the tiles of the last
// round are shared by the CTA pairs of two-CTA clusters.
struct TcPlan {
    int bn, tiles_p, tiles_c, grid, rem;
    bool share;
};

static bool tc_plan(const qnn_gemm_desc *d, int sms, int num_kb, TcPlan *pl) {
    const char *no_share = getenv("QNN_TC_NO_SHARE");
    const bool allowed = !(no_share && no_share[0] == '1');
    // Channel tile.  An MMA costs about the same for every N (measured: the 128 x 32-byte
    // activation operand bounds it), so a tile's main loop costs num_kb k-blocks whatever its
    // width; a narrower tile only shortens the epilogue of the last tile and adds rounds.  Pick the
    // width with the smallest estimated time: rounds x max(main loop, epilogue) + one exposed
    // epilogue, in cycles (about 640 per k-block, 2000 per 32-column chunk and epilogue warp).
    const int tiles_p = ceil_div(d->N, TC_BP);
    const int cand[3] = {256, 128, 32};
    double best_cost = 0.0;
    int bn = 0;
    const char *force_bn = getenv("QNN_TC_BN");               // "256" | "128" | "32": measurements only
    const int forced = force_bn ? atoi(force_bn) : 0;
    for (int ci = 0; ci < 3; ++ci) {
        const int b = cand[ci];
        if (forced && b != forced) continue;
        if (b > 32 && b / 2 >= round_up(d->M, 32)) continue;        // wider than the channels need
        const long long t = (long long)tiles_p * ceil_div(d->M, b);
        const double main_loop = 640.0 * num_kb, epi = 2000.0 * (b >= 64 ? b / 64 : 1);
        double cost;
        if (allowed && 2 * t <= sms && num_kb >= 4) {
            cost = 0.5 * main_loop + 1000.0 + epi;                   // every tile shared by a CTA pair
        } else {
            const long long full = t / sms, rem = t % sms;
            double rounds = (double)full;
            if (rem > 0) rounds += (allowed && full > 0 && 2 * rem <= sms && (sms % 2) == 0 && num_kb >= 2) ? 0.55 : 1.0;
            cost = rounds * (main_loop > epi ? main_loop : epi) + epi;
        }
        if (bn == 0 || cost < best_cost) { bn = b; best_cost = cost; }
    }
    pl->bn = bn; pl->tiles_p = tiles_p; pl->tiles_c = ceil_div(d->M, bn);
    const long long tiles = (long long)pl->tiles_p * pl->tiles_c;
    if (tiles > 0x3fffffff) return false;
    pl->grid = tiles < sms ? (int)tiles : sms;
    pl->rem = (int)(tiles % pl->grid);
    // sharing: a partial last round on at most half of an even number of SMs; the landing
    // zone is the weight ring (bn x 512 bytes of sums fit STAGES >= 4 stages of bn x 128 bytes)
    pl->share = allowed && pl->rem > 0 && 2 * pl->rem <= pl->grid && (pl->grid % 2) == 0 && num_kb >= 2;
    // Few tiles (at most half of the SMs): the kernel's time is the latency of one tile's serial
    // depth loop, so every tile is shared by a CTA pair and each CTA walks half of the depth.
    if (allowed && !pl->share && 2 * tiles <= sms && num_kb >= 4) {
        pl->share = true;
        pl->rem = (int)tiles;
        pl->grid = 2 * (int)tiles;
    }
    return true;
}

bool gemm_tc_uses_pair_kernel(const qnn_gemm_desc *d) { return choose_pair_kernel(d, sm_count()); }

// Split last round of the CTA-pair kernel: the number of tiles whose depth two pairs share (0: no
// split).  Applies when the tiles fill whole rounds of all pairs plus a last round that would keep
// at most half of the pairs busy, and the depth has at least two k-blocks.
static int pair_split_tiles(const qnn_gemm_desc *d, int sms) {
    if (!choose_pair_kernel(d, sms)) return 0;
    const long long tiles = (long long)ceil_div(d->N, 256) * ceil_div(d->M, T2_BN);
    const int pairs = sms / 2;
    if (pairs < 2 || tiles < pairs || ceil_div(d->K, TC_BK) < 2) return 0;
    const int rem = (int)(tiles % pairs);
    return (rem > 0 && 2 * rem <= pairs) ? rem : 0;
}

size_t gemm_tc_workspace_bytes(const qnn_gemm_desc *d) {
    const int rem = pair_split_tiles(d, sm_count());
    return rem ? (size_t)SPLIT_FLAG_BYTES + (size_t)rem * SPLIT_TILE_BYTES : 0;
}

// cv != nullptr: implicit convolution, A is the feature map (see TcParams); d is the lowered GEMM.
static qnn_status tc_launch(const qnn_gemm_desc *d, const qnn_conv_desc *cv, const void *W, const void *A,
                            const int32_t *thr, void *out, void *ws, size_t ws_bytes, cudaStream_t s) {
    const int ld = round_up(d->K, 16);
    const int sms = sm_count();
    const bool pair = choose_pair_kernel(d, sms);

    TcParams p;
    p.thr = thr; p.out = out; p.M = d->M; p.N = d->N; p.K = d->K;
    p.num_kb = ceil_div(d->K, TC_BK);
    p.ld_out = round_up(d->M, 16);
    p.kb_half = 0; p.share = 0;
    p.split_rem = 0; p.split_flags = nullptr; p.split_slabs = nullptr;
    p.taps = 0; p.cchunks = 1; p.cv_C = p.cv_KW = p.cv_OW = p.cv_OHW = p.cv_stride = 1; p.cv_pad = 0;
    if (cv) {
        p.taps = cv->KH * cv->KW; p.cchunks = ceil_div(cv->C, TC_BK);
        p.cv_C = cv->C; p.cv_KW = cv->KW; p.cv_stride = cv->stride; p.cv_pad = cv->pad;
        p.cv_OW = qnn_conv_out_w(cv); p.cv_OHW = qnn_conv_out_h(cv) * p.cv_OW;
        p.num_kb = p.taps * p.cchunks;
    }
    const double wmax = d->w_enc == QNN_ENC_BIPOLAR ? 1.0
                        : (d->w_enc == QNN_ENC_SIGNED ? double(1 << (d->w_bits - 1)) : double((1 << d->w_bits) - 1));
    const double amax = d->a_enc == QNN_ENC_BIPOLAR ? 1.0
                        : (d->a_enc == QNN_ENC_SIGNED ? double(1 << (d->a_bits - 1)) : double((1 << d->a_bits) - 1));
    p.fp_count = (double(d->K) * wmax * amax < double(FP_LIMIT)) ? 1 : 0;
    const uint32_t w_s8 = d->w_enc == QNN_ENC_UNSIGNED ? 0u : 1u;
    const uint32_t a_s8 = d->a_enc == QNN_ENC_UNSIGNED ? 0u : 1u;
    const uint32_t idesc_base = (2u << 4)      // accumulator format: s32
                                | (a_s8 << 7)  // MMA A operand = activations: 0 = u8, 1 = s8
                                | (w_s8 << 10);   // MMA B operand = weights; both K-major
    const int mode = !thr ? OUT_RAW : (d->out_fmt == QNN_FMT_INT8 ? OUT_U8 : OUT_PLANES);
    CUtensorMap ma, mw;

    if (pair) {
        if (cv) {
            const int pitch = cv->in_pitch ? cv->in_pitch : round_up(cv->C, 16);
            if (!make_im2col_map(&ma, A, cv, pitch)) return QNN_ERR_UNSUPPORTED;     // caller lowers explicitly
        } else if (!make_map(&ma, A, d->N, d->K, ld, TC_BP)) {
            return QNN_ERR_CUDA;
        }
        if (!make_map(&mw, W, d->M, d->K, ld, 128)) return QNN_ERR_CUDA;
        p.tiles_p = ceil_div(d->N, 256); p.tiles_c = ceil_div(d->M, T2_BN);
        p.units = p.full_units = p.tiles_p * p.tiles_c;
        p.idesc = idesc_base | ((uint32_t)(256 >> 4) << 24);          // the kernel adds the tile's N
        // a workspace from the caller lets the last, at most half-filled round be split between pairs
        const int rem = cv ? 0 : pair_split_tiles(d, sms);
        if (rem && ws && ws_bytes >= (size_t)SPLIT_FLAG_BYTES + (size_t)rem * SPLIT_TILE_BYTES &&
            (size_t)rem * 2 * 2 * EPI_WARPS * sizeof(unsigned) <= (size_t)SPLIT_FLAG_BYTES) {
            p.split_rem = rem;
            p.split_flags = reinterpret_cast<unsigned *>(ws);
            p.split_slabs = reinterpret_cast<int4 *>(reinterpret_cast<uint8_t *>(ws) + SPLIT_FLAG_BYTES);
        }
        return launch_pair_out(mode, d->out_bits, ma, mw, p, s);
    }
    TcPlan pl;
    if (!tc_plan(d, sms, p.num_kb, &pl)) return QNN_ERR_UNSUPPORTED;
    const int bn = pl.bn;
    p.tiles_p = pl.tiles_p; p.tiles_c = pl.tiles_c;
    const int tiles = pl.tiles_p * pl.tiles_c;
    p.units = p.full_units = tiles;
    if (pl.share) {                       // the last pl.rem tiles (possibly all) are shared by CTA pairs
        p.share = 1;
        p.full_units = tiles - pl.rem;
        p.units = p.full_units + 2 * pl.rem;
        p.kb_half = (p.num_kb + 1) / 2;
    }
    p.idesc = idesc_base | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BP >> 4) << 24);
    if (cv) {
        const int pitch = cv->in_pitch ? cv->in_pitch : round_up(cv->C, 16);
        if (!make_im2col_map(&ma, A, cv, pitch)) return QNN_ERR_UNSUPPORTED;     // caller lowers explicitly
    } else if (!make_map(&ma, A, d->N, d->K, ld, TC_BP)) {
        return QNN_ERR_CUDA;
    }
    if (!make_map(&mw, W, d->M, d->K, ld, bn)) return QNN_ERR_CUDA;
    switch (bn) {
        case 256: return launch_out<256, 4>(mode, d->out_bits, ma, mw, p, s);
        case 128: return launch_out<128, 6>(mode, d->out_bits, ma, mw, p, s);
        default:  return launch_out<32, 8>(mode, d->out_bits, ma, mw, p, s);
    }
}

qnn_status gemm_tc_launch(const qnn_gemm_desc *d, const void *W, const void *A, const int32_t *thr,
                          void *out, void *ws, size_t ws_bytes, cudaStream_t s) {
    return tc_launch(d, nullptr, W, A, thr, out, ws, ws_bytes, s);
}

// Convolution without a lowered matrix: the GEMM's loader reads the 8-bit channels-last map
// through an im2col tensor map (base pixels step by the stride).  UNSUPPORTED when the shape
// needs the explicit lowering (channel count or pixel pitch not a multiple of 16).
qnn_status gemm_tc_conv_launch(const qnn_conv_desc *cv, const qnn_gemm_desc *g, const void *W, const void *in,
                               const int32_t *thr, void *out, cudaStream_t s) {
    const int pitch = cv->in_pitch ? cv->in_pitch : round_up(cv->C, 16);
    if (cv->fmt != QNN_FMT_INT8 || (cv->C % 16) != 0 || (pitch % 16) != 0) return QNN_ERR_UNSUPPORTED;
    if (cv->KH > 255 || cv->KW > 255 || cv->stride > 8) return QNN_ERR_UNSUPPORTED;
    // A single round of tiles is bound by the latency of its serial depth loop.  When the channel
    // count is not a multiple of 128 that loop has more (partly empty) k-blocks here than over the
    // dense lowered matrix, so small problems keep the explicit lowering.
    TcPlan pl;
    if (!tc_plan(g, sm_count(), ceil_div(g->K, TC_BK), &pl)) return QNN_ERR_UNSUPPORTED;
    const long long tiles = (long long)pl.tiles_p * pl.tiles_c;
    const char *force = getenv("QNN_CONV_IMPLICIT");          // "1": skip this heuristic (tests)
    if (!(force && force[0] == '1') && tiles <= sm_count() &&
        cv->KH * cv->KW * ceil_div(cv->C, TC_BK) > ceil_div(g->K, TC_BK))
        return QNN_ERR_UNSUPPORTED;
    return tc_launch(g, cv, W, in, thr, out, nullptr, 0, s);
}

// Convolution of an 8-bit map with contiguous pixels, lowered inside the kernel (see TcParams).
// Mode 1: channel count not a multiple of 16 (the 3-channel first layer), no padding, at most 128
// output channels; weights in the run-per-filter-row layout of qnn_conv_lowered_k.  Mode 2: channel
// count a multiple of 16 but not of 128 (the tensor-map loader would spend a whole k-block on a
// partly filled channel chunk), any padding smaller than the filter, at least four rounds of tiles
// (measured on the 27 x 27 x 96 -> 256 layer: 43 vs 41 us at batch 64, 69 vs 72 at 128, 130 vs 146 at 256).  UNSUPPORTED:
// everything else, or staged image rows that do not fit shared memory -- the caller then takes
// another route.
constexpr int LW_BN = 128, LW_STAGES = 4;          // mode 1
constexpr int LW2_BN = 256, LW2_STAGES = 3;        // mode 2
qnn_status gemm_tc_lower_launch(const qnn_conv_desc *cv, const qnn_gemm_desc *g, const void *W, const void *in,
                                const int32_t *thr, void *out, cudaStream_t s) {
    const int pitch = cv->in_pitch ? cv->in_pitch : round_up(cv->C, 16);
    if (cv->fmt != QNN_FMT_INT8 || pitch != cv->C) return QNN_ERR_UNSUPPORTED;
    const int mode = (cv->C % 16) != 0 ? 1 : 2;
    const int run = cv->KW * cv->C, runp = round_up(run, 16);
    if (g->K != cv->KH * runp) return QNN_ERR_UNSUPPORTED;
    const int OH = qnn_conv_out_h(cv), OW = qnn_conv_out_w(cv);
    if ((long long)g->N * g->K >= (1ll << 40)) return QNN_ERR_UNSUPPORTED;
    const int bn = mode == 1 ? LW_BN : LW2_BN;
    const long long tiles = (long long)ceil_div(g->N, TC_BP) * ceil_div(g->M, bn);
    if (tiles > 0x3fffffff) return QNN_ERR_UNSUPPORTED;
    if (mode == 1) {
        // the whole weight matrix stays in shared memory: one channel tile
        if (cv->pad != 0 || g->M > LW_BN) return QNN_ERR_UNSUPPORTED;
        // The unaligned runs are not masked: image bytes, not zeros, sit opposite the pad columns
        // of the weight rows, which therefore have to be zero bytes.  A bipolar weight has no zero
        // (the packer writes -1 for a logical 0), so such layers take another route.
        if (g->w_enc == QNN_ENC_BIPOLAR && runp != run) return QNN_ERR_UNSUPPORTED;
    } else {
        const char *force = getenv("QNN_CONV_LOWER");            // "1": skip the heuristic (tests), "0": never
        if (force && force[0] == '0') return QNN_ERR_UNSUPPORTED;
        if (cv->pad >= cv->KH || cv->pad >= cv->KW) return QNN_ERR_UNSUPPORTED;
        // ... and not where the CTA-pair kernel takes the convolution through the tensor-map loader
        // (27 x 27 x 96 -> 256 at batch 256: 108 us there against 129 us here)
        if (!(force && force[0] == '1') &&
            ((cv->C % TC_BK) == 0 || tiles < 4 * sm_count() || choose_pair_kernel(g, sm_count())))
            return QNN_ERR_UNSUPPORTED;
    }

    TcParams p;
    p.thr = thr; p.out = out; p.M = g->M; p.N = g->N; p.K = g->K;
    p.num_kb = ceil_div(g->K, TC_BK);
    p.ld_out = round_up(g->M, 16);
    p.kb_half = 0; p.share = 0;
    p.taps = 0; p.cchunks = 1; p.cv_C = cv->C; p.cv_KW = cv->KW; p.cv_pad = cv->pad;
    p.cv_stride = cv->stride; p.cv_OW = OW; p.cv_OHW = OH * OW;
    p.lw_in = reinterpret_cast<const uint8_t *>(in);
    p.lw_total = (long long)cv->B * cv->H * cv->W * cv->C;
    p.lw_H = cv->H; p.lw_KH = cv->KH; p.lw_W = cv->W; p.lw_cpp = cv->C / 16;
    p.lw_rowbytes = cv->W * cv->C; p.lw_step = cv->stride * cv->C;
    p.lw_run = run; p.lw_vecs = runp / 16;
    // Most image rows a tile of TC_BP consecutive output pixels touches: KH rows for its first
    // output row, plus, per further output row, `stride` rows inside an image or the
    // H - (OH-1)*stride rows across an image boundary (an upper bound).
    const int moves = ceil_div(TC_BP - 1, OW);
    const int images = moves < ceil_div(TC_BP - 1, OH * OW) ? moves : ceil_div(TC_BP - 1, OH * OW);
    const int cross = cv->H - (OH - 1) * cv->stride > cv->stride ? cv->H - (OH - 1) * cv->stride : cv->stride;
    const long long rows = cv->KH + (long long)(moves - images) * cv->stride + (long long)images * cross;
    const long long stage = rows * p.lw_rowbytes + 16 + 48;          // rounding of the start, reads past a run
    if (stage > (long long)TC_SMEM_LIMIT) return QNN_ERR_UNSUPPORTED;
    p.lw_stage_bytes = (int)round_up((int)stage, 128);
    p.tiles_p = ceil_div(g->N, TC_BP); p.tiles_c = ceil_div(g->M, bn);
    p.units = p.full_units = (int)tiles;
    const double wmax = g->w_enc == QNN_ENC_BIPOLAR ? 1.0
                        : (g->w_enc == QNN_ENC_SIGNED ? double(1 << (g->w_bits - 1)) : double((1 << g->w_bits) - 1));
    const double amax = g->a_enc == QNN_ENC_BIPOLAR ? 1.0
                        : (g->a_enc == QNN_ENC_SIGNED ? double(1 << (g->a_bits - 1)) : double((1 << g->a_bits) - 1));
    p.fp_count = (double(g->K) * wmax * amax < double(FP_LIMIT)) ? 1 : 0;
    const uint32_t w_s8 = g->w_enc == QNN_ENC_UNSIGNED ? 0u : 1u;
    const uint32_t a_s8 = g->a_enc == QNN_ENC_UNSIGNED ? 0u : 1u;
    p.idesc = (2u << 4) | (a_s8 << 7) | (w_s8 << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BP >> 4) << 24);
    const int out_mode = !thr ? OUT_RAW : (g->out_fmt == QNN_FMT_INT8 ? OUT_U8 : OUT_PLANES);
    CUtensorMap mw;
    if (!make_map(&mw, W, g->M, g->K, round_up(g->K, 16), bn)) return QNN_ERR_CUDA;
    // shared memory is checked per instantiation (it depends on the number of thresholds)
    if (mode == 1) return launch_out<LW_BN, LW_STAGES, 1>(out_mode, g->out_bits, mw, mw, p, s);
    return launch_out<LW2_BN, LW2_STAGES, 2>(out_mode, g->out_bits, mw, mw, p, s);
}

#ifdef QNN_TC_TRACE
extern "C" int qnn_debug_read_trace(long long *host, int n) {
    return (int)cudaMemcpyFromSymbol(host, g_trace, sizeof(long long) * n);
}
extern "C" int qnn_debug_trace_cta(int cta) {
    return (int)cudaMemcpyToSymbol(g_trace_cta, &cta, sizeof(int));
}
#endif

int *device_status_word() {
    static int *cached[QNN_MAX_DEVICES] = {nullptr};
    const int dev = current_device();
    if (dev < 0) return nullptr;
    if (!cached[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_dev_status) != cudaSuccess) return nullptr;
        cached[dev] = reinterpret_cast<int *>(p);
    }
    return cached[dev];
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
