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

// Codes of all 32 columns of one logical word: sel[u] holds, in nibble j, the code of column 8u + j.
template <int K>
__device__ __forceinline__ void code_nibbles_word(const unsigned (&w)[K], unsigned (&sel)[4]) {
    if constexpr (K == 2) {
        // interleave the two planes once: e has plane 0 on even and plane 1 on odd bit positions
        // for the columns at even positions of the word, o the same for the odd positions
        const unsigned m = 0x55555555u;
        const unsigned e = (w[0] & m) | ((w[1] << 1) & ~m);
        const unsigned o = ((w[0] >> 1) & m) | (w[1] & ~m);
        sel[0] = e & 0x33333333u;
        sel[1] = o & 0x33333333u;
        sel[2] = (e >> 2) & 0x33333333u;
        sel[3] = (o >> 2) & 0x33333333u;
    } else {
#pragma unroll
        for (int u = 0; u < 4; ++u) sel[u] = code_nibbles<K>(w, u);
    }
}

// The 2^K candidate values of one (row, group) (Eq. 7) with the decode rule's arithmetic: float(c0),
// then "+ float(ci)" in binary32 for the set bits in plane order, one rounding to binary16.
// Returned as byte tables for the byte-permute decode (K <= 3): lo[0] holds the low bytes of
// candidates 0..3, lo[1] of candidates 4..7 (zero when K < 3); hi[] the high bytes.
template <int K>
__device__ __forceinline__ void candidate_byte_tables(const float (&c)[K + 1], unsigned (&lo)[2], unsigned (&hi)[2]) {
    static_assert(K >= 1 && K <= 3, "byte-permute decode covers at most eight candidates");
    float acc[1 << K];
#pragma unroll
    for (int code = 0; code < (1 << K); ++code) {
        float a = c[0];
#pragma unroll
        for (int i = 0; i < K; ++i)
            if ((code >> i) & 1) a = __fadd_rn(a, c[i + 1]);
        acc[code] = a;
    }
    unsigned pair[4] = {0u, 0u, 0u, 0u};             // candidates (2q, 2q+1) as two binary16 in one register
#pragma unroll
    for (int q = 0; q < (1 << K) / 2 || q < 1; ++q) {
        const __half2 h = __floats2half2_rn(acc[2 * q], (2 * q + 1) < (1 << K) ? acc[2 * q + 1] : 0.f);
        pair[q] = *reinterpret_cast<const unsigned*>(&h);
    }
    lo[0] = __byte_perm(pair[0], pair[1], 0x6420u);
    hi[0] = __byte_perm(pair[0], pair[1], 0x7531u);
    lo[1] = __byte_perm(pair[2], pair[3], 0x6420u);
    hi[1] = __byte_perm(pair[2], pair[3], 0x7531u);
}

// Eight binary16 values (columns in order) from eight code nibbles.
__device__ __forceinline__ uint4 decode8(const unsigned sel, const unsigned (&lo)[2], const unsigned (&hi)[2]) {
    const unsigned sel_hi = __umulhi(sel, 0x10000u);         // sel >> 16 on the multiplier instead of the shifter
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
