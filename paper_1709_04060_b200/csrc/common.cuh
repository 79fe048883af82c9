// Shared host-side helpers of the qnn C ABI implementation (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include <atomic>

#include "qnn.h"

namespace qnn {

// Host counter of kernels launched by this library (reported by benchmarks).
extern std::atomic<unsigned long long> g_launches;

inline void count_launch(int n = 1) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// Per-device host caches are arrays of this size; a device index beyond it is an error.
constexpr int QNN_MAX_DEVICES = 64;

// Index of the current device, or -1 (CUDA error, or an index the caches cannot hold).
inline int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= QNN_MAX_DEVICES) return -1;
    return dev;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }
inline int ceil_div(int x, int m) { return (x + m - 1) / m; }

inline bool valid_enc(int enc, int bits) {
    if (enc == QNN_ENC_BIPOLAR) return bits == 1;
    return enc == QNN_ENC_UNSIGNED || enc == QNN_ENC_SIGNED;
}

inline qnn_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? QNN_OK : QNN_ERR_CUDA;
}

// Programmatic dependent launch.  The tensor-core GEMM, when its grid fills the GPU, is launched
// so that its CTAs may be placed while the previous kernel of the stream drains (they wait in
// griddepcontrol.wait before touching global memory).  The other kernels only do their part as
// predecessors: pdl_trigger() tells the scheduler that a dependent may start placing CTAs (no
// effect unless the next kernel asked for it), pdl_wait() is a no-op for a normally launched
// kernel.  They are not launched that way themselves: early placement next to a draining kernel
// packs the CTAs of a small grid onto few SMs, which halved the bit-serial kernel's speed.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() {
    pdl_trigger();
    pdl_wait();
}
#endif

// Number of SMs of the current device (cached per device).
int sm_count();

// Path implementations (one translation unit each).
qnn_status pack_launch(const qnn_pack_desc *d, const void *logical, void *packed, cudaStream_t s);
qnn_status planes_to_int8_launch(const qnn_pack_desc *d, const void *planes, void *packed, cudaStream_t s);
qnn_status gemm_bitserial_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                                 const int32_t *thr, void *out, cudaStream_t s);
qnn_status gemm_bitserial_conv_launch(const qnn_conv_desc *cv, const qnn_gemm_desc *g, const void *W,
                                      const void *in, const int32_t *thr, void *out, cudaStream_t s);
bool gemv_i8_fits(const qnn_gemm_desc *d);
qnn_status gemv_i8_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                          const int32_t *thr, void *out, cudaStream_t s);
bool gemv_planes_fits(const qnn_gemm_desc *d);
qnn_status gemv_planes_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                              const int32_t *thr, void *out, cudaStream_t s);
bool gemv_fields_dp4a_fits(const qnn_gemm_desc *d);
qnn_status gemv_fields_dp4a_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                                   const int32_t *thr, void *out, cudaStream_t s);
bool gemv_fields_fits(const qnn_gemm_desc *d, bool has_thr);
qnn_status gemv_fields_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                              const int32_t *thr, void *out, cudaStream_t s);
qnn_status gemm_tc_launch(const qnn_gemm_desc *d, const void *W, const void *A,
                          const int32_t *thr, void *out, void *ws, size_t ws_bytes, cudaStream_t s);
size_t gemm_tc_workspace_bytes(const qnn_gemm_desc *d);   // optional scratch of the CTA-pair kernel (0: none)
bool gemm_tc_uses_pair_kernel(const qnn_gemm_desc *d);
qnn_status gemm_tc_conv_launch(const qnn_conv_desc *cv, const qnn_gemm_desc *g, const void *W, const void *in,
                               const int32_t *thr, void *out, cudaStream_t s);
qnn_status gemm_tc_lower_launch(const qnn_conv_desc *cv, const qnn_gemm_desc *g, const void *W, const void *in,
                                const int32_t *thr, void *out, cudaStream_t s);
qnn_status im2col_launch(const qnn_conv_desc *d, const void *in, void *lowered, cudaStream_t s);
qnn_status maxpool_launch(const qnn_pool_desc *d, const void *in, void *out, cudaStream_t s);
qnn_status validate_thresholds_launch(const int32_t *thr, int M, int n_thr, int *n_bad, cudaStream_t s);
qnn_status device_status_read(int *status);

}  // namespace qnn
