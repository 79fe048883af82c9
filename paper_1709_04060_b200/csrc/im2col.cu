// Interleaved lowering (Section 3.2): the feature map is channels-last, one
// bit position per plane, every pixel padded to whole words, so lowering moves
// whole words -- one im2col per activation bit plane, no masking or shifting.
// The same kernel lowers 8-bit-container maps in 16-byte units (channel count a
// multiple of 16); other channel counts (the 3-channel input image of the first
// layer) are lowered as one zero-padded run of bytes per filter row.
//
// One warp per output pixel: the pixel's coordinates are decoded once, lanes
// stream the lowered row (kh, kw, c order, c fastest) with coalesced stores.
#include "common.cuh"

namespace qnn {

struct FastDiv {          // n / d: by multiplication (exact for n, d < 65536), else magic == 0 and a plain division
    uint32_t d, magic;
};
static FastDiv make_fastdiv(int d, long long max_n = 0) {
    FastDiv f;
    f.d = (uint32_t)d;
    f.magic = (d >= 65536 || max_n >= 65536) ? 0u : (uint32_t)(((1ull << 32) + (uint64_t)d - 1) / (uint64_t)d);
    return f;
}
__device__ __forceinline__ uint32_t fdiv(uint32_t n, FastDiv f) {
    return f.d == 1 ? n : (f.magic ? __umulhi(n, f.magic) : n / f.d);
}

struct LowerParams {
    const void *in;
    void *out;
    int planes;                 // bit planes (1 for 8-bit containers)
    int B, H, W, OH, OW;
    int KH, KW, stride, pad;
    int cu;                     // units per pixel that are copied
    int pitch;                  // units between consecutive input pixels
    int row_units;              // units per lowered row that are written
    int row_copy;               // KH*KW*cu: units per lowered row that carry data
    long long npix;             // B*OH*OW
    FastDiv seg, cud, owd;
};

template <typename T>
__device__ __forceinline__ T zero_unit();
template <> __device__ __forceinline__ uint32_t zero_unit<uint32_t>() { return 0u; }
template <> __device__ __forceinline__ uint4 zero_unit<uint4>() { return make_uint4(0, 0, 0, 0); }

template <typename T>
__global__ void __launch_bounds__(256) lower_units_kernel(const LowerParams p) {
    pdl_enter();
    const int lane = threadIdx.x & 31;
    const long long warp0 = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const T *in = reinterpret_cast<const T *>(p.in);
    T *out = reinterpret_cast<T *>(p.out);
    const long long total = p.npix * p.planes;
    for (long long job = warp0; job < total; job += nwarps) {
        const int plane = (int)(job / p.npix);
        const long long pix = job - (long long)plane * p.npix;
        const int b = (int)(pix / (p.OH * p.OW));
        const uint32_t rem = (uint32_t)(pix - (long long)b * p.OH * p.OW);
        const int oh = (int)fdiv(rem, p.owd), ow = (int)(rem - oh * p.OW);
        const int ih0 = oh * p.stride - p.pad, iw0 = ow * p.stride - p.pad;
        const T *src = in + ((size_t)plane * p.B + b) * p.H * p.W * p.pitch;
        T *dst = out + (size_t)job * p.row_units;
        for (int w = lane; w < p.row_units; w += 32) {
            T v = zero_unit<T>();
            if (w < p.row_copy) {
                const int kh = (int)fdiv(w, p.seg), r = w - kh * (int)p.seg.d;
                const int kw = (int)fdiv(r, p.cud), c = r - kw * p.cu;
                const int ih = ih0 + kh, iw = iw0 + kw;
                if (ih >= 0 && ih < p.H && iw >= 0 && iw < p.W)
                    v = src[((size_t)ih * p.W + iw) * p.pitch + c];
            }
            dst[w] = v;
        }
    }
}

// Lowering of 8-bit maps whose channel count is not a multiple of 16 (the 3-channel input
// image of the first layer).  The lowered row keeps one run per filter row: the KW*C bytes that
// row contributes, zero padded to a multiple of 16, so every run starts on a 16-byte boundary
// of the output (the weight rows carry the same padding).  A CTA takes up to LR_PIX consecutive
// output pixels of one output row, stages the KH input-row segments they touch in shared memory
// (compact, C bytes per pixel, zeros outside the image), then one thread per (pixel, filter
// row) turns its run -- contiguous in the staged segment -- into 16-byte stores: an unaligned
// 16-byte read is five aligned words and four funnel shifts.
constexpr int LR_PIX = 64;

// Bytes of one staged input-row segment in shared memory: the segment may start up to three
// bytes into its first word (whole aligned words are staged).
__host__ __device__ inline int lr_seg_pitch(int span, int cu) { return (span * cu + 3 + 3) & ~3; }
__host__ __device__ inline int lr_head_bytes(int KH) { return (KH * 4 + 15) & ~15; }

__global__ void __launch_bounds__(256) lower_runs_kernel(const LowerParams p, int chunks, int span, int run,
                                                         int runp, FastDiv vecd) {
    extern __shared__ __align__(16) uint8_t lr_smem[];   // [KH] first-byte offsets, [KH][seg_pitch], slack
    pdl_enter();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint8_t *in = reinterpret_cast<const uint8_t *>(p.in);
    int *seg_off = reinterpret_cast<int *>(lr_smem);
    uint8_t *segs = lr_smem + lr_head_bytes(p.KH);
    uint32_t *seg_words = reinterpret_cast<uint32_t *>(segs);
    const int seg_bytes = span * p.cu;                   // bytes of one staged input-row segment
    const int seg_pitch = lr_seg_pitch(span, p.cu);
    const int vecs = runp >> 4;                          // 16-byte stores per run
    const long long jobs = (long long)p.B * p.OH * chunks;
    for (long long job = blockIdx.x; job < jobs; job += gridDim.x) {
        const int chunk = (int)(job % chunks);
        const long long t = job / chunks;
        const int oh = (int)(t % p.OH), b = (int)(t / p.OH);
        const int ow0 = chunk * LR_PIX;
        const int npx = min(LR_PIX, p.OW - ow0);
        const int ih0 = oh * p.stride - p.pad, iw0 = ow0 * p.stride - p.pad;
        __syncthreads();                                 // previous job's readers are done
        // stage: one warp per filter row, lanes along the segment
        for (int kh = warp; kh < p.KH; kh += 8) {
            const int ih = ih0 + kh;
            const bool row_ok = ih >= 0 && ih < p.H;
            if (p.pitch == p.cu) {
                // pixels are contiguous: the segment is bytes [off, off + seg_bytes) of the map.
                // Whole aligned words are copied (the segment then starts `a` bytes into its
                // first word); words that straddle the image row's ends are built from bytes.
                const long long off = (((long long)b * p.H + (row_ok ? ih : 0)) * p.W + iw0) * p.cu;
                const int a = row_ok ? (int)(off & 3) : 0;
                const int lo = row_ok ? max(0, -iw0) * p.cu : 0, hi = row_ok ? min(span, p.W - iw0) * p.cu : 0;
                const uint8_t *base = in + (off - a);
                uint32_t *dst = seg_words + kh * (seg_pitch >> 2);
                if (lane == 0) seg_off[kh] = a;
                for (int r = lane; r < (seg_pitch >> 2); r += 32) {
                    const int q0 = 4 * r - a;            // segment-relative index of the word's first byte
                    uint32_t w = 0;
                    if (q0 >= lo && q0 + 4 <= hi) {
                        w = *reinterpret_cast<const uint32_t *>(base + 4 * r);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (q0 + j >= lo && q0 + j < hi) w |= (uint32_t)base[4 * r + j] << (8 * j);
                    }
                    dst[r] = w;
                }
            } else {
                const uint8_t *row = in + (((size_t)b * p.H + (row_ok ? ih : 0)) * p.W) * p.pitch;
                uint8_t *dst = segs + kh * seg_pitch;
                if (lane == 0) seg_off[kh] = 0;
                for (int r = lane; r < seg_pitch; r += 32) {
                    const int px = (int)fdiv((uint32_t)r, p.cud), c = r - px * p.cu;
                    const int iw = iw0 + px;
                    dst[r] = (row_ok && r < seg_bytes && iw >= 0 && iw < p.W) ? row[(size_t)iw * p.pitch + c]
                                                                               : (uint8_t)0;
                }
            }
        }
        __syncthreads();
        // one 16-byte store per item; item = (pixel, filter row, 16-byte piece of the run), which is
        // also the order of the output, so a warp writes 512 consecutive bytes
        uint4 *out_row = reinterpret_cast<uint4 *>(p.out) +
                         (((size_t)b * p.OH + oh) * p.OW + ow0) * (size_t)(p.KH * vecs);
        const int items = npx * p.KH * vecs;
        for (int item = threadIdx.x; item < items; item += blockDim.x) {
            const int task = (int)fdiv((uint32_t)item, vecd), v = item - task * vecs;
            const int px = (int)fdiv((uint32_t)task, p.seg), kh = task - px * p.KH;    // p.seg divides by KH here
            const int src = kh * seg_pitch + seg_off[kh] + px * p.stride * p.cu + 16 * v;
            const int sh = (src & 3) * 8;
            const uint32_t *w = seg_words + (src >> 2);
            uint32_t x[5];
#pragma unroll
            for (int i = 0; i < 5; ++i) x[i] = w[i];
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                o[i] = __funnelshift_r(x[i], x[i + 1], sh);
                const int valid = run - (16 * v + 4 * i);              // bytes of this word inside the run
                if (valid <= 0) o[i] = 0;
                else if (valid < 4) o[i] &= (1u << (8 * valid)) - 1u;
            }
            out_row[item] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

qnn_status im2col_launch(const qnn_conv_desc *d, const void *in, void *lowered, cudaStream_t s) {
    LowerParams p;
    p.in = in; p.out = lowered;
    p.B = d->B; p.H = d->H; p.W = d->W;
    p.OH = qnn_conv_out_h(d); p.OW = qnn_conv_out_w(d);
    p.KH = d->KH; p.KW = d->KW; p.stride = d->stride; p.pad = d->pad;
    p.npix = (long long)d->B * p.OH * p.OW;
    p.owd = make_fastdiv(p.OW, (long long)p.OH * p.OW);      // large maps: plain division
    const int threads = 256;
    const long long max_blocks = (long long)sm_count() * 16;

    int mode;   // 0 words, 1 16-byte units, 2 padded runs of bytes
    int run = 0, runp = 0;
    if (d->fmt == QNN_FMT_BITPLANES) {
        mode = 0;
        p.planes = d->a_bits;
        p.cu = ceil_div(d->C, 32); p.pitch = p.cu;
        p.row_copy = d->KH * d->KW * p.cu; p.row_units = p.row_copy;
    } else {
        const int pitch = d->in_pitch ? d->in_pitch : round_up(d->C, 16);
        p.planes = 1;
        if (d->C % 16 == 0 && pitch % 16 == 0) {
            mode = 1;
            p.cu = d->C / 16; p.pitch = pitch / 16;
            p.row_copy = d->KH * d->KW * p.cu; p.row_units = p.row_copy;
        } else if (d->C % 16 == 0) {
            return QNN_ERR_ALIGNMENT;            // 16-byte channel groups need a 16-byte pixel pitch
        } else {
            mode = 2;
            p.cu = d->C; p.pitch = pitch;
            run = d->KW * d->C; runp = round_up(run, 16);
            p.row_copy = d->KH * runp; p.row_units = p.row_copy;
        }
    }
    if (p.row_units >= 65536 * 16 || d->KW * p.cu >= 65536) return QNN_ERR_UNSUPPORTED;
    p.cud = make_fastdiv(p.cu);

    if (mode == 2) {
        const int span = (LR_PIX - 1) * d->stride + d->KW;
        const size_t smem = (size_t)lr_head_bytes(d->KH) + (size_t)d->KH * lr_seg_pitch(span, p.cu) + 32;   // slack: reads run past a segment
        if (smem > 48 * 1024 || LR_PIX * d->KH * (runp >> 4) >= 65536) return QNN_ERR_UNSUPPORTED;
        p.seg = make_fastdiv(d->KH);
        const int chunks = ceil_div(p.OW, LR_PIX);
        long long nb = (long long)d->B * p.OH * chunks;
        if (nb > max_blocks) nb = max_blocks;
        lower_runs_kernel<<<(unsigned)nb, threads, smem, s>>>(p, chunks, span, run, runp, make_fastdiv(runp >> 4));
        count_launch();
        return launch_status();
    }
    if (p.row_units >= 65536) return QNN_ERR_UNSUPPORTED;
    p.seg = make_fastdiv(d->KW * p.cu);
    const long long jobs = p.npix * p.planes;
    long long blocks = (jobs * 32 + threads - 1) / threads;
    if (blocks > max_blocks) blocks = max_blocks;
    if (mode == 0) lower_units_kernel<uint32_t><<<(unsigned)blocks, threads, 0, s>>>(p);
    else lower_units_kernel<uint4><<<(unsigned)blocks, threads, 0, s>>>(p);
    count_launch();
    return launch_status();
}

}  // namespace qnn
