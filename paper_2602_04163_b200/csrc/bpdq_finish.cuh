// What happens to a row sum between the binary32 accumulator and the binary16 output, shared by the kernels that
// complete rows from a workspace: an optional bias, and for a (gate, up) pair the gated unit silu(gate) * up.
#pragma once
#include <cuda_fp16.h>

namespace bpdq {

__device__ __forceinline__ float silu_f32(float v) { return v / (1.0f + expf(-v)); }

__device__ __forceinline__ float4 bias_quad(const __half* bias, int row) {
    const uint2 raw = *reinterpret_cast<const uint2*>(bias + row);       // row is a multiple of four: 8-byte aligned
    const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
    const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}

// a: the sums of rows row..row+3 (for a pair: the gate's), b: the up projection's when `pair`.  On return a holds
// what is rounded to binary16.
__device__ __forceinline__ void finish_quad(float4& a, const float4& b, const __half* bias_a, const __half* bias_b,
                                            bool pair, int row) {
    if (bias_a) {
        const float4 c = bias_quad(bias_a, row);
        a.x += c.x; a.y += c.y; a.z += c.z; a.w += c.w;
    }
    if (pair) {
        float4 u = b;
        if (bias_b) {
            const float4 c = bias_quad(bias_b, row);
            u.x += c.x; u.y += c.y; u.z += c.z; u.w += c.w;
        }
        a.x = silu_f32(a.x) * u.x; a.y = silu_f32(a.y) * u.y; a.z = silu_f32(a.z) * u.z; a.w = silu_f32(a.w) * u.w;
    }
}

}  // namespace bpdq
