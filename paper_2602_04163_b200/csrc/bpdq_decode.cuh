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
    // Interleave planes 0 and 1 once: e has plane 0 on even and plane 1 on odd bit positions for the columns at
    // even positions of the word (u = 0, 2), o the same for the odd positions (u = 1, 3); two-bit codes then
    // come out with one mask.  Planes 2 and 3 are interleaved the same way and land two bits higher.
    const unsigned m5 = 0x55555555u, m3 = 0x33333333u;
    if constexpr (K == 1) {
#pragma unroll
        for (int u = 0; u < 4; ++u) sel[u] = code_nibbles<K>(w, u);
    } else {
        const unsigned e = (w[0] & m5) | ((w[1] << 1) & ~m5);
        const unsigned o = ((w[0] >> 1) & m5) | (w[1] & ~m5);
        if constexpr (K == 2) {
            sel[0] = e & m3;
            sel[1] = o & m3;
            sel[2] = (e >> 2) & m3;
            sel[3] = (o >> 2) & m3;
        } else if constexpr (K == 3) {
            const unsigned m4 = 0x44444444u;          // plane 2 goes to bit 2 of every nibble
            sel[0] = (e & m3) | ((w[2] << 2) & m4);
            sel[1] = (o & m3) | ((w[2] << 1) & m4);
            sel[2] = ((e >> 2) & m3) | (w[2] & m4);
            sel[3] = ((o >> 2) & m3) | ((w[2] >> 1) & m4);
        } else {
            const unsigned e2 = (w[2] & m5) | ((w[3] << 1) & ~m5);
            const unsigned o2 = ((w[2] >> 1) & m5) | (w[3] & ~m5);
            sel[0] = (e & m3) | ((e2 << 2) & ~m3);
            sel[1] = (o & m3) | ((o2 << 2) & ~m3);
            sel[2] = ((e >> 2) & m3) | (e2 & ~m3);
            sel[3] = ((o >> 2) & m3) | (o2 & ~m3);
        }
    }
}

// The 2^K candidate values of one (row, group) (Eq. 7) with the decode rule's arithmetic: float(c0),
// then "+ float(ci)" in binary32 for the set bits in plane order, one rounding to binary16.
// Returned as byte tables for the byte-permute decode: lo[t] holds the low bytes of candidates
// 4t..4t+3, hi[t] the high bytes (tables beyond 2^K candidates are zero); K = 4 uses all four.
template <int K> struct ByteTables { unsigned lo[K == 4 ? 4 : 2], hi[K == 4 ? 4 : 2]; };

template <int K>
__device__ __forceinline__ void candidate_byte_tables(const float (&c)[K + 1], ByteTables<K>& t) {
    static_assert(K >= 1 && K <= 4, "at most sixteen candidates");
    constexpr int NT = K == 4 ? 4 : 2;
    float acc[1 << K];
#pragma unroll
    for (int code = 0; code < (1 << K); ++code) {
        float a = c[0];
#pragma unroll
        for (int i = 0; i < K; ++i)
            if ((code >> i) & 1) a = __fadd_rn(a, c[i + 1]);
        acc[code] = a;
    }
    unsigned pair[2 * NT];                           // candidates (2q, 2q+1) as two binary16 in one register
#pragma unroll
    for (int q = 0; q < 2 * NT; ++q) {
        const __half2 h = __floats2half2_rn(2 * q < (1 << K) ? acc[(2 * q) & ((1 << K) - 1)] : 0.f,
                                            2 * q + 1 < (1 << K) ? acc[(2 * q + 1) & ((1 << K) - 1)] : 0.f);
        pair[q] = *reinterpret_cast<const unsigned*>(&h);
    }
#pragma unroll
    for (int k = 0; k < NT; ++k) {
        t.lo[k] = __byte_perm(pair[2 * k], pair[2 * k + 1], 0x6420u);
        t.hi[k] = __byte_perm(pair[2 * k], pair[2 * k + 1], 0x7531u);
    }
}

// prmt.b32 as the hardware defines it: byte n of the result is byte (selector nibble n) & 7 of {b, a} (a = bytes 0..3);
// a nibble with its top bit set would replicate that byte's sign instead.  Every selector used below keeps the top
// bit of its four low nibbles clear (codes are at most 7), so no masking instruction is needed in front of it;
// bits 16..31 of the selector are ignored.
__device__ __forceinline__ unsigned prmt_raw(unsigned a, unsigned b, unsigned sel) {
    unsigned d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Four binary16 values from the four code nibbles in the low half of `sel`.
template <int K>
__device__ __forceinline__ void decode4(const unsigned sel, const ByteTables<K>& t, unsigned& out01, unsigned& out23) {
    unsigned l, h;
    if constexpr (K == 4) {
        // a byte-permute selects among eight bytes: candidates 0..7 and 8..15 are looked up separately
        // (selector without its top bit) and the top bit of every code picks between the two results
        const unsigned s7 = sel & 0x7777u;
        unsigned m = (sel >> 3) & 0x1111u;                   // top bits at nibble positions 0, 4, 8, 12
        m = (m & 0x0011u) | ((m & 0x1100u) << 8);            // ... at 0, 4, 16, 20
        m = (m & 0x00010001u) | ((m & 0x00100010u) << 4);    // ... at 0, 8, 16, 24
        m *= 0xFFu;                                          // one full byte per code
        const unsigned la = prmt_raw(t.lo[0], t.lo[1], s7), lb = prmt_raw(t.lo[2], t.lo[3], s7);
        const unsigned ha = prmt_raw(t.hi[0], t.hi[1], s7), hb = prmt_raw(t.hi[2], t.hi[3], s7);
        l = (la & ~m) | (lb & m);
        h = (ha & ~m) | (hb & m);
    } else {
        l = prmt_raw(t.lo[0], t.lo[1], sel);
        h = prmt_raw(t.hi[0], t.hi[1], sel);
    }
    out01 = prmt_raw(l, h, 0x5140u);
    out23 = prmt_raw(l, h, 0x7362u);
}

// Eight binary16 values (columns in order) from eight code nibbles.
template <int K>
__device__ __forceinline__ uint4 decode8(const unsigned sel, const ByteTables<K>& t) {
    uint4 o;
    decode4<K>(sel, t, o.x, o.y);
    decode4<K>(__umulhi(sel, 0x10000u), t, o.z, o.w);        // sel >> 16 on the multiplier instead of the shifter
    return o;
}

}  // namespace bpdq
