// Operand packer: logical bytes -> bit planes (Section 3.1: plane i = bit i of
// every element, packed along the depth) or zero-padded 8-bit containers
// (Section 3: operands cast to 8-bit integers); bit planes -> 8-bit containers (few-bit data
// crosses the host link packed and is widened on the device).  Also the threshold validator.
#include "common.cuh"

namespace qnn {

// Bits i, 8+i, 16+i, 24+i of x gathered into the low nibble.
__device__ __forceinline__ uint32_t gather_bit4(uint32_t x, int i) {
    return (((x >> i) & 0x01010101u) * 0x01020408u) >> 24;
}

// One thread per (row, depth word): reads up to 32 logical bytes, writes one
// word into each plane.
template <bool BIPOLAR>
__global__ void pack_planes_kernel(const uint8_t *__restrict__ logical, uint32_t *__restrict__ planes,
                                   int rows, int K, int kw, int bits, bool vec_ok) {
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (idx >= (long long)rows * kw) return;
    const int r = (int)(idx / kw);
    const int w = (int)(idx - (long long)r * kw);
    const int k0 = w * 32;
    const uint8_t *src = logical + (size_t)r * K + k0;
    uint32_t x[8];
    if (vec_ok && k0 + 32 <= K) {
        const uint4 lo = *reinterpret_cast<const uint4 *>(src);
        const uint4 hi = *reinterpret_cast<const uint4 *>(src + 16);
        x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w;
        x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint32_t v = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int k = k0 + q * 4 + b;
                if (k < K) v |= (uint32_t)src[q * 4 + b] << (8 * b);
            }
            x[q] = v;
        }
    }
    if (BIPOLAR) {
        // bit = (value > 0) per signed byte; zero pad bytes give bit 0
        uint32_t word = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t pos = __vcmpgts4(x[q], 0u) & 0x01010101u;
            word |= gather_bit4(pos, 0) << (4 * q);
        }
        planes[(size_t)r * kw + w] = word;
    } else {
        for (int i = 0; i < bits; ++i) {
            uint32_t word = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) word |= gather_bit4(x[q], i) << (4 * q);
            planes[((size_t)i * rows + r) * kw + w] = word;
        }
    }
}

// Per-byte conversion of four logical bytes to their 8-bit containers.
__device__ __forceinline__ uint32_t container4(uint32_t x, int bits, int enc) {
    if (enc == QNN_ENC_BIPOLAR) {
        const uint32_t gt = __vcmpgts4(x, 0u);                  // 0xFF where the byte is > 0
        return (gt & 0x01010101u) | ~gt;                        // +1 : -1
    }
    if (bits == 8) return x;
    const uint32_t low = x & (0x01010101u * ((1u << bits) - 1u));
    if (enc == QNN_ENC_UNSIGNED) return low;
    // sign extension inside every byte: the sign bit, moved up one place, times
    // 2^(8-bits) - 1 fills bits [bits, 8) and cannot carry into the next byte
    const uint32_t sign = low & (0x01010101u << (bits - 1));
    return low | ((sign << 1) * ((1u << (8 - bits)) - 1u));
}

// Bit planes -> 8-bit containers: one thread per 16 output bytes (16 consecutive depth indices,
// one half of a plane word).  Four bits of a plane become four bytes by one multiplication
// (bit b of the nibble lands in bit 0 of byte b); plane i adds them shifted by i.
__global__ void __launch_bounds__(256) planes_to_int8_kernel(const uint32_t *__restrict__ planes,
                                                             uint4 *__restrict__ packed, int rows, int K,
                                                             int kw, int chunks, int bits, int enc) {
    const long long total = (long long)rows * chunks;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(idx / chunks), c = (int)(idx - (long long)r * chunks);
        const int k0 = 16 * c, word = k0 >> 5, shift = k0 & 31;
        uint32_t o[4] = {0u, 0u, 0u, 0u};
        for (int i = 0; i < bits; ++i) {
            const uint32_t x = (planes[((size_t)i * rows + r) * kw + word] >> shift) & 0xFFFFu;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t spread = (((x >> (4 * q)) & 0xFu) * 0x00204081u) & 0x01010101u;
                // SIGNED: the top plane is the sign, which also fills the container's upper bits
                const uint32_t mul = (enc == QNN_ENC_SIGNED && i == bits - 1) ? ((0xFFu << i) & 0xFFu) : (1u << i);
                o[q] |= spread * mul;
            }
        }
        if (enc == QNN_ENC_BIPOLAR) {
            // bit 1 -> +1, bit 0 -> -1; pad bytes past K stay zero
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t v = 0xFFFFFFFFu ^ (o[q] * 0xFEu);
                const int left = K - (k0 + 4 * q);                 // elements of this word inside the row
                if (left < 4) v &= left <= 0 ? 0u : (0xFFFFFFFFu >> (8 * (4 - left)));
                o[q] = v;
            }
        }
        packed[idx] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// K a multiple of 16 (no padding): one thread per 16 bytes, 16-byte loads and stores.
__global__ void __launch_bounds__(256) pack_int8_vec_kernel(const uint4 *__restrict__ logical,
                                                            uint4 *__restrict__ packed, long long n16,
                                                            int bits, int enc) {
    pdl_trigger();        // a tensor-core kernel queued behind the packer may set up while it drains
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n16;
         i += (long long)gridDim.x * blockDim.x) {
        const uint4 v = logical[i];
        packed[i] = make_uint4(container4(v.x, bits, enc), container4(v.y, bits, enc),
                               container4(v.z, bits, enc), container4(v.w, bits, enc));
    }
}

// One thread per 16 output bytes of the [rows][ld] container matrix.
__global__ void pack_int8_kernel(const uint8_t *__restrict__ logical, uint8_t *__restrict__ packed,
                                 int rows, int K, int ld, int bits, int enc) {
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    const int chunks = ld / 16;
    if (idx >= (long long)rows * chunks) return;
    const int r = (int)(idx / chunks);
    const int c = (int)(idx - (long long)r * chunks);
    const uint8_t *src = logical + (size_t)r * K + c * 16;
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t v = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int k = c * 16 + q * 4 + b;
            uint32_t e = 0;
            if (k < K) {
                const uint32_t raw = src[q * 4 + b];
                if (enc == QNN_ENC_BIPOLAR) {
                    e = ((int8_t)raw > 0) ? 0x01u : 0xFFu;
                } else if (enc == QNN_ENC_SIGNED) {
                    const int sh = 32 - bits;
                    e = (uint32_t)(((int32_t)(raw << sh)) >> sh) & 0xFFu;
                } else {
                    e = raw & ((1u << bits) - 1u);
                }
            }
            v |= e << (8 * b);
        }
        o[q] = v;
    }
    *reinterpret_cast<uint4 *>(packed + (size_t)r * ld + c * 16) = make_uint4(o[0], o[1], o[2], o[3]);
}

// QNN_FMT_FIELDS: one thread per packed 32-bit word.  Byte j of 32-byte group g of a row holds,
// at bit position f*s, the field of element 32*S*g + 32*s + j (S = 8/f fields per byte).
__global__ void pack_fields_kernel(const uint8_t *__restrict__ logical, uint32_t *__restrict__ packed,
                                   int rows, int K, int ldw, int bits, int enc, int f) {
    const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (idx >= (long long)rows * ldw) return;
    const int r = (int)(idx / ldw);
    const int w = (int)(idx - (long long)r * ldw);
    const int S = 8 / f;
    const int g = w >> 3, j0 = (w & 7) * 4;
    const uint8_t *src = logical + (size_t)r * K;
    uint32_t word = 0;
    for (int b = 0; b < 4; ++b)
        for (int s = 0; s < S; ++s) {
            const long long k = (long long)32 * S * g + 32 * s + j0 + b;
            if (k >= K) continue;
            const int raw = (int8_t)src[k];
            uint32_t u;
            if (enc == QNN_ENC_BIPOLAR) u = raw > 0 ? 1u : 0u;
            else if (enc == QNN_ENC_SIGNED) {
                const int sh = 32 - bits;
                u = (uint32_t)(((int32_t)((uint32_t)raw << sh) >> sh) + (1 << (bits - 1)));   // value - minimum
            } else u = (uint32_t)raw & ((1u << bits) - 1u);
            word |= u << (8 * b + f * s);
        }
    packed[idx] = word;
}

qnn_status planes_to_int8_launch(const qnn_pack_desc *d, const void *planes, void *packed, cudaStream_t s) {
    const int threads = 256;
    const int kw = ceil_div(d->K, 32), chunks = round_up(d->K, 16) / 16;
    const long long total = (long long)d->rows * chunks;
    const long long want = (total + threads - 1) / threads, cap = (long long)sm_count() * 16;
    planes_to_int8_kernel<<<(unsigned)(want < cap ? want : cap), threads, 0, s>>>(
        (const uint32_t *)planes, (uint4 *)packed, d->rows, d->K, kw, chunks,
        d->enc == QNN_ENC_BIPOLAR ? 1 : d->bits, d->enc);
    count_launch();
    return launch_status();
}

qnn_status pack_launch(const qnn_pack_desc *d, const void *logical, void *packed, cudaStream_t s) {
    const int threads = 256;
    if (d->fmt == QNN_FMT_FIELDS) {
        const int f = d->bits == 1 ? 1 : (d->bits == 2 ? 2 : 4);
        const int ldw = 8 * ceil_div(d->K, 32 * (8 / f));           // words per packed row
        const long long total = (long long)d->rows * ldw;
        pack_fields_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, s>>>(
            (const uint8_t *)logical, (uint32_t *)packed, d->rows, d->K, ldw, d->bits, d->enc, f);
        count_launch();
        return launch_status();
    }
    if (d->fmt == QNN_FMT_BITPLANES) {
        const int kw = ceil_div(d->K, 32);
        const long long total = (long long)d->rows * kw;
        const unsigned blocks = (unsigned)((total + threads - 1) / threads);
        const bool vec_ok = (d->K % 16) == 0;
        if (d->enc == QNN_ENC_BIPOLAR)
            pack_planes_kernel<true><<<blocks, threads, 0, s>>>((const uint8_t *)logical, (uint32_t *)packed,
                                                               d->rows, d->K, kw, 1, vec_ok);
        else
            pack_planes_kernel<false><<<blocks, threads, 0, s>>>((const uint8_t *)logical, (uint32_t *)packed,
                                                                d->rows, d->K, kw, d->bits, vec_ok);
    } else {
        const int ld = round_up(d->K, 16);
        const long long total = (long long)d->rows * (ld / 16);
        if (d->K % 16 == 0) {
            const long long want = (total + threads - 1) / threads;
            const long long cap = (long long)sm_count() * 16;
            pack_int8_vec_kernel<<<(unsigned)(want < cap ? want : cap), threads, 0, s>>>(
                (const uint4 *)logical, (uint4 *)packed, total, d->bits, d->enc);
            count_launch();
            return launch_status();
        }
        const unsigned blocks = (unsigned)((total + threads - 1) / threads);
        pack_int8_kernel<<<blocks, threads, 0, s>>>((const uint8_t *)logical, (uint8_t *)packed,
                                                    d->rows, d->K, ld, d->bits, d->enc);
    }
    count_launch();
    return launch_status();
}

__global__ void validate_thresholds_kernel(const int32_t *__restrict__ thr, int M, int n_thr, int *n_bad) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= M) return;
    bool bad = false;
    for (int i = 1; i < n_thr; ++i) bad |= thr[(size_t)m * n_thr + i] < thr[(size_t)m * n_thr + i - 1];
    if (bad) atomicAdd(n_bad, 1);
}

// Counter for the validator; a file-scope device word so that no allocation is needed.
__device__ int g_bad_rows;

qnn_status validate_thresholds_launch(const int32_t *thr, int M, int n_thr, int *n_bad_host, cudaStream_t s) {
    int *dev_ptr = nullptr;
    if (cudaGetSymbolAddress((void **)&dev_ptr, g_bad_rows) != cudaSuccess) return QNN_ERR_CUDA;
    if (cudaMemsetAsync(dev_ptr, 0, sizeof(int), s) != cudaSuccess) return QNN_ERR_CUDA;
    validate_thresholds_kernel<<<ceil_div(M, 128), 128, 0, s>>>(thr, M, n_thr, dev_ptr);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return QNN_ERR_CUDA;
    if (cudaMemcpyAsync(n_bad_host, dev_ptr, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return QNN_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return QNN_ERR_CUDA;
    return QNN_OK;
}

}  // namespace qnn
