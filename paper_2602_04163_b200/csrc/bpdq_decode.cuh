// Device helpers shared by the kernels that turn packed plane units back into columns.
// Layout of a 16-byte plane unit (see bpdq.h): physical byte p holds logical byte (p + r) mod 16;
// logical word k (logical bytes 4k..4k+3) covers columns 32k..32k+31 of the block and its bit
// 4*j + u is column 32k + 8u + j.
#pragma once
#include <cstdint>
#include <cuda_fp16.h>

namespace bpdq {

// Undo the byte rotation of row r: returns the unit's four logical words.
__device__ __forceinline__ uint4 unrotate_unit(const uint4 phys, const int r) {
    // logical byte L sits at physical byte (L - r) mod 16: rotate the 128-bit value LEFT by 8*(r mod 16) bits
    const int rot = r & 15;
    const int wrot = rot >> 2;
    const unsigned sh = (unsigned)(rot & 3) * 8u;
    // word rotation: logical word k takes physical words (k - wrot) and (k - wrot - 1)
    unsigned a0 = phys.x, a1 = phys.y, a2 = phys.z, a3 = phys.w;
    if (wrot & 1) { const unsigned t = a3; a3 = a2; a2 = a1; a1 = a0; a0 = t; }
    if (wrot & 2) { unsigned t = a0; a0 = a2; a2 = t; t = a1; a1 = a3; a3 = t; }
    // now a[k] = phys[(k - wrot) mod 4]; finish with a byte-granular funnel shift
    uint4 o;
    o.x = __funnelshift_l(a3, a0, sh);
    o.y = __funnelshift_l(a0, a1, sh);
    o.z = __funnelshift_l(a1, a2, sh);
    o.w = __funnelshift_l(a2, a3, sh);
    return o;
}

// Codes of the eight consecutive columns 8u..8u+7 of a 32-column word: nibble j of the result is
// sum_i bit_i(column 8u + j) << i, where w[i] is plane i's logical word.
template <int K>
__device__ __forceinline__ unsigned code_nibbles(const unsigned (&w)[K], const int u) {
    unsigned sel = (w[0] >> u) & 0x11111111u;
#pragma unroll
    for (int i = 1; i < K; ++i) sel |= ((w[i] >> u) & 0x11111111u) << i;
    return sel;
}

// The 2^K candidate values of one (row, group) (Eq. 7) with the decode rule's arithmetic: float(c0),
// then "+ float(ci)" in binary32 for the set bits in plane order, one rounding to binary16.
template <int K>
__device__ __forceinline__ void candidate_values(const float (&c)[K + 1], unsigned short (&v)[1 << K]) {
#pragma unroll
    for (int code = 0; code < (1 << K); ++code) {
        float acc = c[0];
#pragma unroll
        for (int i = 0; i < K; ++i)
            if ((code >> i) & 1) acc = __fadd_rn(acc, c[i + 1]);
        v[code] = __half_as_ushort(__float2half_rn(acc));
    }
}

// Byte tables for the byte-permute decode (K <= 3): lo[0] holds the low bytes of candidates 0..3,
// lo[1] of candidates 4..7 (zero when K < 3); hi[] the high bytes.
template <int K>
__device__ __forceinline__ void byte_tables(const unsigned short (&v)[1 << K], unsigned (&lo)[2], unsigned (&hi)[2]) {
    static_assert(K >= 1 && K <= 3, "byte-permute decode covers at most eight candidates");
    lo[0] = lo[1] = hi[0] = hi[1] = 0u;
#pragma unroll
    for (int e = 0; e < (1 << K); ++e) {
        lo[e >> 2] |= (unsigned)(v[e] & 0xFFu) << (8 * (e & 3));
        hi[e >> 2] |= (unsigned)(v[e] >> 8) << (8 * (e & 3));
    }
}

// Eight binary16 values (columns in order) from eight code nibbles.
__device__ __forceinline__ uint4 decode8(const unsigned sel, const unsigned (&lo)[2], const unsigned (&hi)[2]) {
    const unsigned sel_hi = sel >> 16;
    const unsigned l0 = __byte_perm(lo[0], lo[1], sel), h0 = __byte_perm(hi[0], hi[1], sel);
    const unsigned l1 = __byte_perm(lo[0], lo[1], sel_hi), h1 = __byte_perm(hi[0], hi[1], sel_hi);
    uint4 o;
    o.x = __byte_perm(l0, h0, 0x5140u);
    o.y = __byte_perm(l0, h0, 0x7362u);
    o.z = __byte_perm(l1, h1, 0x5140u);
    o.w = __byte_perm(l1, h1, 0x7362u);
    return o;
}

}  // namespace bpdq
