// Device-side generator of synthetic packed weights (bpdq_create with host_blob == NULL).
// Reproduces, bit for bit, the host generator of the synthetic workloads: a counter-based
// stream (splitmix64 output function) keyed by (seed, tensor id), drawn per LOGICAL element
// and written straight into the packed layout.  Only exact integer steps and individually
// rounded binary32 operations are used, so host and device agree exactly.
#include "bpdq_internal.h"

#include <cuda_fp16.h>

namespace {

constexpr unsigned long long kGolden = 0x9E3779B97F4A7C15ull;
constexpr int kTensorPlanes = 1, kTensorCoef = 2;

__host__ __device__ inline unsigned long long mix64(unsigned long long z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__host__ __device__ inline unsigned long long stream_key(unsigned long long seed, int tensor) {
    return mix64(seed ^ ((unsigned long long)tensor * kGolden));
}
__device__ inline unsigned long long draw64(unsigned long long key, unsigned long long counter) {
    return mix64(key + counter * kGolden);
}

__global__ void fill_planes_kernel(uint8_t* __restrict__ blob, unsigned long long key, int out, int in,
                                   int K) {
    const long long nblocks = in / 128;
    const long long total = nblocks * K * (long long)out;
    for (long long u = blockIdx.x * (long long)blockDim.x + threadIdx.x; u < total;
         u += (long long)gridDim.x * blockDim.x) {
        const long long r = u % out;
        const int i = (int)((u / out) % K);
        const long long b = u / ((long long)out * K);
        unsigned logical[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned long long q = ((unsigned long long)i * out + r) * (unsigned long long)(in / 32) + 4ull * b + k;
            const unsigned drawn = (unsigned)(draw64(key, q) >> 32);       // bit t = column 32k + t
            // layout word: bit 4j + u = column 32k + 8u + j, i.e. the bits of byte u spread one per nibble
            unsigned word = 0;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                unsigned x = (drawn >> (8 * u)) & 0xFFu;
                x = (x | (x << 12)) & 0x000F000Fu;
                x = (x | (x << 6)) & 0x03030303u;
                x = (x | (x << 3)) & 0x11111111u;
                word |= x << u;
            }
            logical[k] = word;
        }
        // physical byte p = logical byte (p + r) mod 16: rotate the 128-bit unit right by 8*(r mod 16) bits
        const int rot = (int)(r & 15);
        const int wrot = rot >> 2, brot = (rot & 3) * 8;
        unsigned phys[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned lo = logical[(k + wrot) & 3], hi = logical[(k + wrot + 1) & 3];
            phys[k] = __funnelshift_r(lo, hi, brot);
        }
        *reinterpret_cast<uint4*>(blob + bpdq::plane_unit_offset(b, i, r, K, out)) =
            make_uint4(phys[0], phys[1], phys[2], phys[3]);
    }
}

__global__ void fill_coefs_kernel(uint8_t* __restrict__ cbase, unsigned long long key, int out, int in,
                                  int K, int group) {
    const long long ngroups = (in + group - 1) / group;
    const long long total = ngroups * (K + 1) * (long long)out;
    // binary32 constants identical to the host generator's
    const float c0_scale = 0x1.47ae14p-6f * 0x1p-16f;
    const float lo12 = 0x1.47ae14p-8f, range12 = 0x1.70a3d8p-5f * 0x1p-24f;
    const float lo3 = 0x1.0624dep-9f, range3 = 0x1.26e978p-6f * 0x1p-24f;
    for (long long u = blockIdx.x * (long long)blockDim.x + threadIdx.x; u < total;
         u += (long long)gridDim.x * blockDim.x) {
        const long long r = u % out;
        const int i = (int)((u / out) % (K + 1));
        const long long G = u / ((long long)out * (K + 1));
        const unsigned long long e = ((unsigned long long)i * out + r) * (unsigned long long)ngroups + G;
        float v;
        if (i == 0) {
            long long total16 = 0;
            for (int part = 0; part < 3; ++part) {
                const unsigned long long w = draw64(key, 4ull * e + part);
                total16 += (long long)(w & 0xFFFF) + (long long)((w >> 16) & 0xFFFF) +
                           (long long)((w >> 32) & 0xFFFF) + (long long)((w >> 48) & 0xFFFF);
            }
            v = __fmul_rn((float)(total16 - 6 * 65535), c0_scale);
        } else {
            const float u24 = (float)(unsigned)(draw64(key, 4ull * e) >> 40);
            v = (i <= 2) ? __fadd_rn(__fmul_rn(u24, range12), lo12) : __fadd_rn(__fmul_rn(u24, range3), lo3);
        }
        const __half hv = __float2half_rn(v);
        *reinterpret_cast<__half*>(cbase + bpdq::coef_offset(G, i, r, K, out)) = hv;
    }
}

}  // namespace

namespace bpdq {

int launch_fill(bpdq_handle_s* h, uint64_t seed, cudaStream_t stream) {
    const int threads = 256;
    const int blocks = h->sm_count * 8;
    fill_planes_kernel<<<blocks, threads, 0, stream>>>(h->d_blob, stream_key(seed, kTensorPlanes), h->out,
                                                        h->in, h->K);
    fill_coefs_kernel<<<blocks, threads, 0, stream>>>(h->d_blob + h->planes_bytes,
                                                       stream_key(seed, kTensorCoef), h->out, h->in, h->K,
                                                       h->group);
    h->launches += 2;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "fill launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

}  // namespace bpdq
