// Streamlining (Section 2.1 of the paper) as a host-side tool: the float operations that sit
// between a quantized matrix layer and its activation quantizer -- the previous quantizer's
// affine map moved past the integer product (2.1.2), alpha-scaling, batch normalisation --
// are absorbed into per-channel integer thresholds (2.1.3), which is all the fused GEMM
// epilogue needs.  No device code: this runs once per network, offline.
//
// For every channel the un-streamlined forward pass from an integer accumulator x is
//   z = a_prev * x + b_prev * row_sum,  z = alpha * z,  y = gamma * (z - mu) / sigma + beta,
//   code = #{ i : t_i <= y }                                   (T(x, t), Section 2.1.1)
// and threshold i becomes the smallest integer x in [acc_lo, acc_hi] whose code is at least
// i + 1.  Section 2.1.3's closed form ceil((t_i - b) / a) is the starting guess; it is then
// corrected against the forward pass itself, so that rounding in the closed form can never
// disagree with the float network at a tie.  A negative slope flips the inequality: the
// channel is flagged and its thresholds apply to the negated accumulator (the caller negates
// that weight row).  A zero slope gives a constant code, expressed with sentinels.
#include <math.h>
#include <limits.h>

#include "common.cuh"

namespace qnn {

static int forward_code(const qnn_channel_params &c, long long x, const double *t, int n) {
    double z = c.a_prev * (double)x + c.b_prev * (double)c.row_sum;
    z = c.alpha * z;
    const double y = c.gamma * (z - c.mu) / c.sigma + c.beta;
    int code = 0;
    for (int i = 0; i < n; ++i) code += (y >= t[i]) ? 1 : 0;
    return code;
}

}  // namespace qnn

using namespace qnn;

extern "C" qnn_status qnn_streamline(const qnn_channel_params *ch, int channels, const double *qthr, int n_thr,
                                     long long acc_lo, long long acc_hi, int32_t *thr_out, uint8_t *negate_out) {
    if (!ch || !qthr || !thr_out || !negate_out || channels <= 0 || n_thr <= 0 || n_thr > 15)
        return QNN_ERR_INVALID_ARG;
    if (acc_lo > acc_hi || acc_lo <= INT_MIN || acc_hi >= INT_MAX) return QNN_ERR_INVALID_ARG;
    for (int i = 1; i < n_thr; ++i)
        if (qthr[i] < qthr[i - 1]) return QNN_ERR_INVALID_ARG;
    for (int c = 0; c < channels; ++c) {
        const qnn_channel_params &p = ch[c];
        if (!(p.sigma != 0.0)) return QNN_ERR_INVALID_ARG;
        int32_t *out = thr_out + (size_t)c * n_thr;
        const double A = p.gamma * p.alpha * p.a_prev / p.sigma;                          // Section 2.1.2
        const double B = p.gamma * (p.alpha * p.b_prev * (double)p.row_sum - p.mu) / p.sigma + p.beta;
        if (A == 0.0) {
            const int code = forward_code(p, 0, qthr, n_thr);
            for (int i = 0; i < n_thr; ++i) out[i] = i < code ? INT_MIN : INT_MAX;
            negate_out[c] = 0;
            continue;
        }
        const bool neg = A < 0.0;
        negate_out[c] = neg ? 1 : 0;
        // code as a function of the (possibly negated) accumulator u; non-decreasing in u
        const long long lo = neg ? -acc_hi : acc_lo, hi = neg ? -acc_lo : acc_hi;
        auto code_at = [&](long long u) { return forward_code(p, neg ? -u : u, qthr, n_thr); };
        for (int i = 0; i < n_thr; ++i) {
            const int want = i + 1;
            if (code_at(hi) < want) { out[i] = INT_MAX; continue; }
            if (code_at(lo) >= want) { out[i] = INT_MIN; continue; }
            // closed form on the collapsed map |A| u + B >= t, then local correction
            double g = ceil((qthr[i] - B) / fabs(A));
            long long u = g < (double)lo ? lo : (g > (double)hi ? hi : (long long)g);
            int steps = 0;
            while (u > lo && code_at(u - 1) >= want && steps < 64) { --u; ++steps; }
            while (u < hi && code_at(u) < want && steps < 64) { ++u; ++steps; }
            if (steps >= 64 || code_at(u) < want || (u > lo && code_at(u - 1) >= want)) {
                long long a = lo, b = hi;                    // code(a) < want <= code(b)
                while (b - a > 1) {
                    const long long m = a + (b - a) / 2;
                    if (code_at(m) >= want) b = m; else a = m;
                }
                u = b;
            }
            out[i] = (int32_t)u;
        }
    }
    return QNN_OK;
}
