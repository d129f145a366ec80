// bpdq_gemv_simple: one-bit-at-a-time evaluation of y = x * W^T, kept as an on-device
// cross-check of the fast kernels and as the fallback for shapes they do not cover.
// One thread owns one output row and one token; it decodes each weight exactly as
// bpdq_dequant does (candidate table of Eq. 7, rounded to binary16) and accumulates
// x * w in binary32 in column order.  No shared memory, no scratch, no tuning.
#include "bpdq_internal.h"
#include "bpdq_decode.cuh"

#include <cuda_fp16.h>

namespace {

template <int K>
__global__ void __launch_bounds__(128)
gemv_simple_kernel(const uint8_t* __restrict__ blob, size_t planes_bytes, const __half* __restrict__ x,
                   __half* __restrict__ y, int out, int in, int group, const __half* __restrict__ bias) {
    constexpr int NC = 1 << K;
    const int r = blockIdx.x * 128 + threadIdx.x;
    const int m = blockIdx.y;
    if (r >= out) return;
    const uint8_t* cbase = blob + planes_bytes;
    const int nblocks = in / 128;
    const int nsub = group == 64 ? 2 : 1;
    const __half* xm = x + (size_t)m * in;
    float acc = 0.f;
    for (int b = 0; b < nblocks; ++b) {
        unsigned u[K][4];                            // logical words of this row's units
#pragma unroll
        for (int i = 0; i < K; ++i) {
            const uint4 v = bpdq::unrotate_unit(
                *reinterpret_cast<const uint4*>(blob + bpdq::plane_unit_offset(b, i, r, K, out)), r);
            u[i][0] = v.x; u[i][1] = v.y; u[i][2] = v.z; u[i][3] = v.w;
        }
        for (int sub = 0; sub < nsub; ++sub) {
            const int G = (b * 128 + sub * 64) / group;
            float c[K + 1];
#pragma unroll
            for (int i = 0; i <= K; ++i)
                c[i] = __half2float(*reinterpret_cast<const __half*>(cbase + bpdq::coef_offset(G, i, r, K, out)));
            float table[NC];
#pragma unroll
            for (int code = 0; code < NC; ++code) {
                float a = c[0];
#pragma unroll
                for (int i = 0; i < K; ++i)
                    if ((code >> i) & 1) a = __fadd_rn(a, c[i + 1]);
                table[code] = __half2float(__float2half_rn(a));
            }
            const int col_lo = (nsub == 2) ? sub * 64 : 0, col_hi = (nsub == 2) ? sub * 64 + 64 : 128;
            for (int col = col_lo; col < col_hi; ++col) {
                const int k = col >> 5, bit = 4 * (col & 7) + ((col >> 3) & 3);   // column = 32k + 8u + j  <->  bit 4j + u of word k
                unsigned code = 0;
#pragma unroll
                for (int i = 0; i < K; ++i) {
                    const unsigned word = k == 0 ? u[i][0] : k == 1 ? u[i][1] : k == 2 ? u[i][2] : u[i][3];
                    code |= ((word >> bit) & 1u) << i;
                }
                float wv = table[0];
#pragma unroll
                for (int kk = 1; kk < NC; ++kk) wv = (code == (unsigned)kk) ? table[kk] : wv;
                acc = fmaf(__half2float(xm[b * 128 + col]), wv, acc);
            }
        }
    }
    y[(size_t)m * out + r] = __float2half_rn(acc + (bias ? __half2float(bias[r]) : 0.f));
}

}  // namespace

namespace bpdq {

int launch_gemv_simple(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    const dim3 grid((h->out + 127) / 128, M), block(128);
    const __half* xp = static_cast<const __half*>(x);
    __half* yp = static_cast<__half*>(y);
    switch (h->K) {
        case 1: gemv_simple_kernel<1><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, xp, yp, h->out, h->in, h->group, static_cast<const __half*>(h->d_bias)); break;
        case 2: gemv_simple_kernel<2><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, xp, yp, h->out, h->in, h->group, static_cast<const __half*>(h->d_bias)); break;
        case 3: gemv_simple_kernel<3><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, xp, yp, h->out, h->in, h->group, static_cast<const __half*>(h->d_bias)); break;
        case 4: gemv_simple_kernel<4><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, xp, yp, h->out, h->in, h->group, static_cast<const __half*>(h->d_bias)); break;
        default: return set_error(BPDQ_ERR_UNSUPPORTED, "gemv_simple: K=%d", h->K);
    }
    h->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "gemv_simple launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

}  // namespace bpdq
