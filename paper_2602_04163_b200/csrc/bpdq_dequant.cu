// bpdq_dequant: materialise W^ (Eq. 1) as binary16 [out][in].
//
// One warp owns 32 rows x one 128-column block.  Lane l reads its row's K plane units
// (consecutive rows are adjacent in the blob: one coalesced 512-byte request per plane), undoes the
// row's byte rotation, and builds the 2^K candidate values of its (row, group) (Eq. 7) with the
// decode rule's exact arithmetic: float(c0), then "+ float(ci)" in binary32 for the set bits in
// plane order, one rounding to binary16 -- kept as byte tables for the byte-permute decode that
// the tensor-core kernel uses too.  Units and tables are staged in shared memory; the warp then
// writes two rows per step, 16 lanes x 16 bytes each (eight consecutive columns: one bit per
// nibble of a logical word, turned into eight binary16 by eight byte-permutes), so every row
// segment leaves as one contiguous 256-byte store.  HBM-bound on the 2 bytes per weight it writes.
#include "bpdq_internal.h"
#include "bpdq_decode.cuh"

#include <cuda_fp16.h>

namespace {

constexpr int kWarpsPerCta = 8;

template <int K>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
dequant_kernel(const uint8_t* __restrict__ blob, size_t planes_bytes, __half* __restrict__ w, int out, int in,
               int group) {
    constexpr int NT = K == 4 ? 4 : 2;               // table words per half (low bytes, high bytes)
    __shared__ __align__(16) unsigned s_units[kWarpsPerCta][32][K][4];          // logical words, per row
    __shared__ __align__(16) unsigned s_tab[kWarpsPerCta][32][2][2 * NT];       // per row and 64-column half: lo[NT], hi[NT]

    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int nblocks = in / 128;
    const int nrb = (out + 31) / 32;
    const long long ntasks = (long long)nrb * nblocks;
    const int nsub = group == 64 ? 2 : 1;            // coefficient groups inside one 128-column block
    const uint8_t* cbase = blob + planes_bytes;

    for (long long task = (long long)blockIdx.x * kWarpsPerCta + wid; task < ntasks;
         task += (long long)gridDim.x * kWarpsPerCta) {
        const int rb = (int)(task % nrb);
        const int b = (int)(task / nrb);
        const int r = rb * 32 + lane;
        if (r < out) {
#pragma unroll
            for (int i = 0; i < K; ++i) {
                const uint4 u = *reinterpret_cast<const uint4*>(blob + bpdq::plane_unit_offset(b, i, r, K, out));
                *reinterpret_cast<uint4*>(&s_units[wid][lane][i][0]) = bpdq::unrotate_unit(u, r);   // staged in logical byte order
            }
            for (int sub = 0; sub < nsub; ++sub) {
                const int G = (b * 128 + sub * 64) / group;
                float c[K + 1];
#pragma unroll
                for (int i = 0; i <= K; ++i)
                    c[i] = __half2float(*reinterpret_cast<const __half*>(cbase + bpdq::coef_offset(G, i, r, K, out)));
                bpdq::ByteTables<K> t;
                bpdq::candidate_byte_tables<K>(c, t);
#pragma unroll
                for (int k = 0; k < NT; ++k) {
                    s_tab[wid][lane][sub][k] = t.lo[k];
                    s_tab[wid][lane][sub][NT + k] = t.hi[k];
                }
            }
        }
        __syncwarp();
        const int c8 = lane & 15;                    // eight-column chunk this lane writes: word c8 / 4, phase u = c8 % 4
        const int sub = (group == 64) ? (c8 >> 3) : 0;
#pragma unroll 4
        for (int it = 0; it < 16; ++it) {
            const int lr = it * 2 + (lane >> 4);     // local row
            const int rr = rb * 32 + lr;
            if (rr < out) {
                unsigned word[K];
#pragma unroll
                for (int i = 0; i < K; ++i) word[i] = s_units[wid][lr][i][c8 >> 2];
                bpdq::ByteTables<K> t;
#pragma unroll
                for (int k = 0; k < NT; ++k) {
                    t.lo[k] = s_tab[wid][lr][sub][k];
                    t.hi[k] = s_tab[wid][lr][sub][NT + k];
                }
                const uint4 v = bpdq::decode8<K>(bpdq::code_nibbles<K>(word, c8 & 3), t);
                *reinterpret_cast<uint4*>(w + (size_t)rr * in + (size_t)b * 128 + c8 * 8) = v;
            }
        }
        __syncwarp();
    }
}

}  // namespace

namespace bpdq {

int launch_dequant(bpdq_handle_s* h, void* w, cudaStream_t stream) {
    const long long ntasks = (long long)((h->out + 31) / 32) * (h->in / 128);
    long long ctas = (ntasks + kWarpsPerCta - 1) / kWarpsPerCta;
    const long long cap = (long long)h->sm_count * 8;
    if (ctas > cap) ctas = cap;
    const dim3 grid((unsigned)ctas), block(kWarpsPerCta * 32);
    __half* wp = static_cast<__half*>(w);
    switch (h->K) {
        case 1: dequant_kernel<1><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, wp, h->out, h->in, h->group); break;
        case 2: dequant_kernel<2><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, wp, h->out, h->in, h->group); break;
        case 3: dequant_kernel<3><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, wp, h->out, h->in, h->group); break;
        case 4: dequant_kernel<4><<<grid, block, 0, stream>>>(h->d_blob, h->planes_bytes, wp, h->out, h->in, h->group); break;
        default: return set_error(BPDQ_ERR_UNSUPPORTED, "dequant: K=%d", h->K);
    }
    h->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "dequant launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

}  // namespace bpdq
