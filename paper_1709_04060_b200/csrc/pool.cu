// Integer max-pool on activation codes (Section 4.2 lists pooling among the
// cheap non-matrix layers; here it runs on the few-bit integer codes).
// INT8 maps: four channels per thread with a byte-wise unsigned max.
// Bit-plane maps: 32 channels per thread; the maximum of two bit-sliced numbers
// is selected with a mask built from the most significant plane downwards.
#include "common.cuh"

namespace qnn {

struct PoolParams {
    const void *in;
    void *out;
    int B, H, W, OH, OW, k, stride;
    int cu;                // units (4-byte words) per pixel
    int bits;
    long long plane_in, plane_out;   // words per bit plane (bit-plane format)
};

// 16 channels (one uint4) per thread; the padded channel count is a multiple of 16.
// KT > 0: window size known at compile time (all KT*KT loads of a thread are in flight together).
template <int KT>
__global__ void __launch_bounds__(256) maxpool_u8_kernel(const PoolParams p) {
    pdl_enter();
    const int k = KT > 0 ? KT : p.k;
    const int cu = p.cu >> 2;                                     // 16-byte units per pixel
    const long long total = (long long)p.B * p.OH * p.OW * cu;
    const uint4 *in = reinterpret_cast<const uint4 *>(p.in);
    uint4 *out = reinterpret_cast<uint4 *>(p.out);
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const unsigned u = (unsigned)(idx % cu);
        const unsigned t = (unsigned)(idx / cu);                  // output pixel (< 2^32)
        const unsigned ow = t % (unsigned)p.OW, t2 = t / (unsigned)p.OW;
        const unsigned oh = t2 % (unsigned)p.OH, b = t2 / (unsigned)p.OH;
        uint4 best = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < k; ++i) {
            const uint4 *row = in + (((size_t)b * p.H + oh * p.stride + i) * p.W + ow * p.stride) * cu + u;
#pragma unroll
            for (int j = 0; j < k; ++j) {
                const uint4 v = __ldg(row + (size_t)j * cu);
                best.x = __vmaxu4(best.x, v.x); best.y = __vmaxu4(best.y, v.y);
                best.z = __vmaxu4(best.z, v.z); best.w = __vmaxu4(best.w, v.w);
            }
        }
        out[idx] = best;
    }
}

template <int BITS>
__global__ void __launch_bounds__(256) maxpool_planes_kernel(const PoolParams p) {
    pdl_enter();
    const long long total = (long long)p.B * p.OH * p.OW * p.cu;
    const uint32_t *in = reinterpret_cast<const uint32_t *>(p.in);
    uint32_t *out = reinterpret_cast<uint32_t *>(p.out);
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % p.cu);
        long long t = idx / p.cu;
        const int ow = (int)(t % p.OW); t /= p.OW;
        const int oh = (int)(t % p.OH);
        const int b = (int)(t / p.OH);
        uint32_t best[BITS];
#pragma unroll
        for (int q = 0; q < BITS; ++q) best[q] = 0;
        for (int i = 0; i < p.k; ++i)
            for (int j = 0; j < p.k; ++j) {
                const size_t off = (((size_t)b * p.H + oh * p.stride + i) * p.W + ow * p.stride + j) * p.cu + c;
                uint32_t v[BITS];
#pragma unroll
                for (int q = 0; q < BITS; ++q) v[q] = in[(size_t)q * p.plane_in + off];
                uint32_t gt = 0, eq = 0xffffffffu;          // per channel: v > best, v == best so far
#pragma unroll
                for (int q = BITS - 1; q >= 0; --q) {
                    gt |= eq & v[q] & ~best[q];
                    eq &= ~(v[q] ^ best[q]);
                }
#pragma unroll
                for (int q = 0; q < BITS; ++q) best[q] = (gt & v[q]) | (~gt & best[q]);
            }
#pragma unroll
        for (int q = 0; q < BITS; ++q) out[(size_t)q * p.plane_out + idx] = best[q];
    }
}

qnn_status maxpool_launch(const qnn_pool_desc *d, const void *in, void *out, cudaStream_t s) {
    PoolParams p;
    p.in = in; p.out = out;
    p.B = d->B; p.H = d->H; p.W = d->W; p.k = d->k; p.stride = d->stride;
    p.OH = (d->H - d->k) / d->stride + 1;
    p.OW = (d->W - d->k) / d->stride + 1;
    p.bits = d->bits;
    if ((long long)d->B * p.OH * p.OW >= 0x7fffffffLL) return QNN_ERR_UNSUPPORTED;
    p.cu = d->fmt == QNN_FMT_INT8 ? round_up(d->C, 16) / 4 : ceil_div(d->C, 32);
    p.plane_in = (long long)d->B * d->H * d->W * p.cu;
    p.plane_out = (long long)d->B * p.OH * p.OW * p.cu;
    const int threads = 256;
    long long blocks = ((d->fmt == QNN_FMT_INT8 ? p.plane_out / 4 : p.plane_out) + threads - 1) / threads;
    const long long max_blocks = (long long)sm_count() * 16;
    if (blocks > max_blocks) blocks = max_blocks;
    if (d->fmt == QNN_FMT_INT8) {
        if (d->k == 3) maxpool_u8_kernel<3><<<(unsigned)blocks, threads, 0, s>>>(p);
        else if (d->k == 2) maxpool_u8_kernel<2><<<(unsigned)blocks, threads, 0, s>>>(p);
        else maxpool_u8_kernel<0><<<(unsigned)blocks, threads, 0, s>>>(p);
    } else {
        switch (d->bits) {
            case 1: maxpool_planes_kernel<1><<<(unsigned)blocks, threads, 0, s>>>(p); break;
            case 2: maxpool_planes_kernel<2><<<(unsigned)blocks, threads, 0, s>>>(p); break;
            case 3: maxpool_planes_kernel<3><<<(unsigned)blocks, threads, 0, s>>>(p); break;
            default: maxpool_planes_kernel<4><<<(unsigned)blocks, threads, 0, s>>>(p); break;
        }
    }
    count_launch();
    return launch_status();
}

}  // namespace qnn
