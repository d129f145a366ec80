// Host-side producers of logical BPDQ tensors (no CUDA): the data-free initialisation of the paper's quantizer and
// the truncated multi-precision view.
//
// bpdq_quantize_datafree follows Section 3.2 without calibration data: per (row, group) an asymmetric
// round-to-nearest quantizer to an unsigned 8-bit code Z (Eq. 5: Z = sum_i 2^i P_i), the K most significant planes
// B_i = P_{7-K+i}, and the coefficient fit of Eq. 6 with U_loc = I, i.e. ordinary least squares of the row's weights
// on [1, b_1, .., b_K], solved from the normal equations in binary64 with the paper's damping alpha added to the
// diagonal as alpha * trace / (K + 1).  bpdq_truncate_planes keeps the K2 most significant planes of a K-plane
// tensor and moves half of every dropped plane's coefficient into the offset.
#include <cmath>
#include <cstring>

#include <cuda_fp16.h>

#include "bpdq_internal.h"

using namespace bpdq;

namespace {

inline float half_bits_to_float(uint16_t b) {
    __half_raw r;
    r.x = b;
    return __half2float(__half(r));
}
inline uint16_t float_to_half_bits(float f) {
    const __half_raw r = static_cast<__half_raw>(__float2half_rn(f));
    return r.x;
}

// Solves the n x n system N c = rhs (n <= 5) by Gaussian elimination with partial pivoting; false if singular.
bool solve_small(double (&N)[5][5], double (&rhs)[5], int n, double (&c)[5]) {
    for (int col = 0; col < n; ++col) {
        int piv = col;
        for (int r = col + 1; r < n; ++r)
            if (std::fabs(N[r][col]) > std::fabs(N[piv][col])) piv = r;
        if (N[piv][col] == 0.0) return false;
        if (piv != col) {
            for (int k = 0; k < n; ++k) { const double t = N[col][k]; N[col][k] = N[piv][k]; N[piv][k] = t; }
            const double t = rhs[col]; rhs[col] = rhs[piv]; rhs[piv] = t;
        }
        for (int r = col + 1; r < n; ++r) {
            const double f = N[r][col] / N[col][col];
            for (int k = col; k < n; ++k) N[r][k] -= f * N[col][k];
            rhs[r] -= f * rhs[col];
        }
    }
    for (int r = n - 1; r >= 0; --r) {
        double s = rhs[r];
        for (int k = r + 1; k < n; ++k) s -= N[r][k] * c[k];
        c[r] = s / N[r][r];
    }
    return true;
}

}  // namespace

extern "C" int bpdq_quantize_datafree(const float* w, int out, int in, int K, int group, double alpha, uint8_t* bits,
                                      uint16_t* coef) {
    if (!w || !bits || !coef) return set_error(BPDQ_ERR_INVALID, "bpdq_quantize_datafree: null pointer");
    if (!shape_supported(out, in, K, group) || in % group)          // the fit works on whole groups
        return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_quantize_datafree: unsupported shape out=%d in=%d K=%d g=%d", out, in, K, group);
    if (!(alpha >= 0.0)) return set_error(BPDQ_ERR_INVALID, "bpdq_quantize_datafree: alpha must be >= 0");
    const int64_t ng = in / group;
    const int n = K + 1;
    for (int64_t r = 0; r < out; ++r) {
        for (int64_t G = 0; G < ng; ++G) {
            const float* wg = w + r * in + G * group;
            double lo = wg[0], hi = wg[0];
            for (int j = 1; j < group; ++j) {
                if (!(wg[j] == wg[j])) return set_error(BPDQ_ERR_INVALID, "bpdq_quantize_datafree: NaN weight at row %lld", (long long)r);
                lo = wg[j] < lo ? wg[j] : lo;
                hi = wg[j] > hi ? wg[j] : hi;
            }
            double scale = (hi - lo) / 255.0;
            if (!(scale > 0.0)) scale = 1.0;
            double N[5][5] = {}, rhs[5] = {}, c[5] = {};
            for (int j = 0; j < group; ++j) {
                double z = std::nearbyint(((double)wg[j] - lo) / scale);      // round to nearest, ties to even (default rounding mode)
                z = z < 0.0 ? 0.0 : (z > 255.0 ? 255.0 : z);
                const unsigned code = (unsigned)z;
                double row[5];
                row[0] = 1.0;
                for (int i = 1; i <= K; ++i) {
                    const unsigned b = (code >> (7 - K + i)) & 1u;            // B_i = P_{7-K+i}
                    bits[((int64_t)(i - 1) * out + r) * in + G * group + j] = (uint8_t)b;
                    row[i] = (double)b;
                }
                for (int a = 0; a < n; ++a) {
                    rhs[a] += row[a] * (double)wg[j];
                    for (int b = 0; b < n; ++b) N[a][b] += row[a] * row[b];
                }
            }
            double trace = 0.0;
            for (int a = 0; a < n; ++a) trace += N[a][a];
            for (int a = 0; a < n; ++a) N[a][a] += alpha * trace / n;
            if (!solve_small(N, rhs, n, c)) {
                // a plane constant within the group and no damping: fit the offset alone, the plane's coefficient is free (zero)
                for (int a = 0; a < n; ++a) c[a] = 0.0;
                double s = 0.0;
                for (int j = 0; j < group; ++j) s += wg[j];
                c[0] = s / group;
            }
            for (int i = 0; i <= K; ++i) coef[((int64_t)i * out + r) * ng + G] = float_to_half_bits((float)c[i]);
        }
    }
    return BPDQ_OK;
}

extern "C" int bpdq_truncate_planes(const uint8_t* bits, const uint16_t* coef, int out, int in, int K, int group, int K2,
                                    uint8_t* bits2, uint16_t* coef2) {
    if (!bits || !coef || !bits2 || !coef2) return set_error(BPDQ_ERR_INVALID, "bpdq_truncate_planes: null pointer");
    if (!shape_supported(out, in, K, group) || in % group || K2 < 1 || K2 > K)
        return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_truncate_planes: unsupported shape out=%d in=%d K=%d g=%d K2=%d", out, in, K, group, K2);
    const int drop = K - K2;
    const int64_t plane = (int64_t)out * in, ng = in / group, cplane = (int64_t)out * ng;
    std::memmove(bits2, bits + drop * plane, (size_t)(K2 * plane));
    for (int64_t e = 0; e < cplane; ++e) {
        volatile float c0 = half_bits_to_float(coef[e]);                      // binary32 steps in plane order, each rounded
        for (int i = 1; i <= drop; ++i) {
            const float half_ci = 0.5f * half_bits_to_float(coef[i * cplane + e]);
            c0 = c0 + half_ci;
        }
        coef2[e] = float_to_half_bits(c0);
    }
    for (int i = 1; i <= K2; ++i) std::memmove(coef2 + i * cplane, coef + (drop + i) * cplane, (size_t)cplane * sizeof(uint16_t));
    return BPDQ_OK;
}
