// bpdq_gemv: batch-1 (M <= 2 per pass) evaluation of y = x * W^T straight from the packed planes.
//
// Method.  With Eq. 1 the dot product of a row with x regroups into the add-only form the paper
// points to for bit-plane hardware and for its look-up-table decode kernel:
//
//     y[r] = sum_G ( c0[r,G] * X_G  +  sum_i ci[r,G] * S_i[r,G] ),
//     X_G = sum of x over group G,    S_i[r,G] = sum of x_j over the set bits of plane i in G.
//
// S_i is read from look-up tables instead of being added bit by bit: for every 8 inputs that share
// a plane byte ("chunk") the 256 subset sums of x are precomputed in shared memory (binary32), so
// one plane BYTE costs one byte-permute (address), one shared-memory load and half a packed add.
//
// Work split.  A CTA owns a slice of 512 input columns (4 blocks of 128) and a range of 16-row
// groups; it builds the 64 chunk tables of its slice once (64 KB per token) and then streams
// planes.  A warp takes 16 rows x 4 blocks per task: lane (h, a) = (lane/16, lane%16) owns row a
// and the two blocks of parity h.  Its 16-byte plane units and binary16 coefficients come straight
// from global memory into registers (16 lanes x 16 bytes = 256 contiguous bytes per request), two
// tasks ahead, so that HBM latency is covered by loads in flight and shared memory
// carries nothing but the look-ups.  The blob stores, at byte p of row r, the 8-column chunk
// ("logical byte") (p + r) mod 16, and table entries are laid out as [entry][slot],
// slot = 16*block + chunk, so at every step the 32 lanes of a warp hit 32 different banks whatever
// the data: table loads are conflict-free by construction.  The tables start at a multiple of
// 64 KB in the shared window, so the byte-permute that splices the plane byte into bits 8..15 of
// the lane's slot address yields the final address.  Look-up results are accumulated two at a
// time with packed binary32 adds.
// Row sums are combined across slices with binary32 atomic adds into a small workspace
// [token][row] that lives in L2; per 128 rows an arrival counter tells the CTA that delivers the
// last contribution to round those rows to binary16, write y and zero the workspace again.
// Algorithmic HBM bytes per weight: K/8 + 2(K+1)/g.
#include "bpdq_internal.h"
#include "bpdq_partition.h"
#include "bpdq_finish.cuh"

#include <cuda_fp16.h>

namespace {

constexpr int kSliceBlocks = 4;                       // 128-column blocks per slice
constexpr int kSlots = 16 * kSliceBlocks;             // chunk tables per slice = slots per entry row
constexpr int kTableBytes = 256 * kSlots * 4;         // one token's tables: 64 KB
constexpr int kMaxMT = 2;                             // tokens per pass (64 KB of tables each)
constexpr int kChunkRgs = 8;                          // row groups (of 16 rows) per completion counter
constexpr int kMiscBytes = 4096;                      // xsum + completion list, at the start of shared memory
constexpr int kMaxDone = 512;                         // completed chunks handled per batch

// One linear of a launch.  A launch covers one or several linears (same K, same token count): their
// (slice, row group) task spaces are concatenated and every CTA takes a contiguous share of the whole.
struct GemvLinear {
    const uint8_t* blob;
    size_t planes_bytes, blob_bytes;
    const __half* x;          // [MT][in]
    __half* y;                // [MT][out]
    float* ws;                // [MT][out] binary32 row sums, zero between calls
    unsigned* counters;       // [ceil(out/16 / kChunkRgs)] arrival counters, zero between calls
    // completion: a finished chunk is converted from conv_a (this linear's sums) or, for a (gate, up) pair, from
    // conv_a = gate's and conv_b = up's sums as silu(a) * b; the pair shares gate's counters and both count into them
    float* conv_a;
    float* conv_b;            // null unless paired
    const __half* bias_a;     // null: none
    const __half* bias_b;
    int target_mul;           // 1, or 2 for a pair
    const int* perm;          // null: identity; else stored column j multiplies x[perm[j]]
    int out, in, group;
    int nblocks, nslices, nrg;
    int task_begin;           // first task of this linear in the concatenated task space
};
constexpr int kMaxBatch = BPDQ_BATCH_MAX;
constexpr int kMaxGrid = 192;                        // CTAs of a launch (one per SM)
// set-up and hand-over of one (slice, row range) segment, in tasks; measured optima for one / several linears per launch
constexpr int kSegmentCostSingle = 64, kSegmentCostBatch = 48;

struct GemvParams {
    GemvLinear lin[kMaxBatch];
    int n;                       // linears in this launch
    int* status;                 // device status word
    int t_begin[kMaxGrid + 1];   // CTA b takes the tasks [t_begin[b], t_begin[b+1]) of the concatenated space
    int dyn_smem;                // dynamic shared memory bytes of the launch
    int early_weights;           // the packed weights were complete before the preceding kernel of the stream started
};

// Registers of one task (16 rows x 4 blocks) of a lane: K plane units and K+1 coefficients for
// each of its two blocks.
template <int K, int NG>
struct Task {
    uint4 pl[2][K];
    unsigned short cf[2][K + 1];         // g >= 128: this row's coefficients of the block's group
    // g = 64 (NG = 2): two groups per block would double the registers a task in flight holds, so a lane pair shares
    // the loads: rows r (even lane) and r + 1 are adjacent in the blob, the even lane loads both rows' coefficients of
    // the block's first group as 32-bit words, the odd lane those of the second group, and they swap halves by shuffle
    // when the task is processed.
    unsigned cfp[2][NG == 2 ? K + 1 : 1];
};

__device__ __forceinline__ uint4 ldg_stream16(const uint8_t* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// Activations: the kernel before this one in the stream may have written them while this kernel was already
// resident, so they are read through the coherent path (L2), never the read-only one.  Volatile, so that the
// load stays behind griddepcontrol.wait and ahead of the weight requests issued after it.
__device__ __forceinline__ unsigned ldg_x4(const void* p) {
    unsigned v;
    asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned short ldg_x2(const void* p) {
    unsigned short v;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ldg_stream4(const uint8_t* p) {
    unsigned v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ unsigned short ldg_stream2(const uint8_t* p) {
    unsigned short v;
    asm volatile("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
// add into the workspace without a returned value: nothing for the warp to wait on
__device__ __forceinline__ void red_add(float* p, float v) {
    asm volatile("red.global.add.f32 [%0], %1;" :: "l"(p), "f"(v) : "memory");
}
// Table load.  Not volatile: its address is computed from plane bytes that were read after the
// barrier that published the tables, so it cannot move above that barrier, and the compiler may
// interleave the independent look-ups of a plane unit freely.
template <int IMM>
__device__ __forceinline__ float lds_table(unsigned addr) {
    float v;
    asm("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(IMM));
    return v;
}
// prmt.b32 in its generic form: selector nibble n picks byte n of {b, a} (a = bytes 0..3); with its top bit set
// the byte's sign is replicated instead
__device__ __forceinline__ unsigned prmt(unsigned a, unsigned b, unsigned sel) {
    unsigned d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ unsigned word_of(const uint4& v, int k) {
    return k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w;
}
// A pair of binary32 accumulators in one 64-bit register: (lo, hi) += (a, b) as one packed add.
__device__ __forceinline__ void add2(unsigned long long& acc, float a, float b) {
    asm("{\n\t.reg .b64 t;\n\tmov.b64 t, {%1, %2};\n\tadd.rn.f32x2 %0, %0, t;\n\t}" : "+l"(acc) : "f"(a), "f"(b));
}
// Two table look-ups and their packed add in one statement, so that the two loaded values are born as the
// register pair the packed add reads (separate loads would each need a move into the pair).
template <int IMM0, int IMM1>
__device__ __forceinline__ void lookup2_add(unsigned long long& acc, unsigned addr0, unsigned addr1) {
    asm("{\n\t.reg .f32 a, b;\n\t.reg .b64 t;\n\t"
        "ld.shared.f32 a, [%1+%3];\n\t"
        "ld.shared.f32 b, [%2+%4];\n\t"
        "mov.b64 t, {a, b};\n\t"
        "add.rn.f32x2 %0, %0, t;\n\t}"
        : "+l"(acc) : "r"(addr0), "r"(addr1), "n"(IMM0), "n"(IMM1));
}
// The same, and the two loaded values are handed back (g = 64 adds them to the first group's partial sums as well).
template <int IMM0, int IMM1>
__device__ __forceinline__ void lookup2v_add(unsigned long long& acc, unsigned addr0, unsigned addr1, float& a, float& b) {
    asm("{\n\t.reg .b64 t;\n\t"
        "ld.shared.f32 %1, [%3+%5];\n\t"
        "ld.shared.f32 %2, [%4+%6];\n\t"
        "mov.b64 t, {%1, %2};\n\t"
        "add.rn.f32x2 %0, %0, t;\n\t}"
        : "+l"(acc), "=&f"(a), "=&f"(b) : "r"(addr0), "r"(addr1), "n"(IMM0), "n"(IMM1));
}
__device__ __forceinline__ float2 unpack2(unsigned long long v) {
    float2 f;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(f.x), "=f"(f.y) : "l"(v));
    return f;
}

// EXT: the launch uses an input permutation, a bias or a (gate, up) pair somewhere.  The plain instantiation carries none of
// that code: the streaming loop sits at the 128-register cap, and the extra live values cost it spills (5 % of the
// headline, up to 50 % at g = 64) although they are only used outside the loop.
template <int K, int MT, int D, int W, bool G64, bool EXT>
__global__ void __launch_bounds__(W * 32, 1) gemv_lut_kernel(const __grid_constant__ GemvParams p) {
    constexpr int kThreads = W * 32;
    constexpr int NS = K * MT;                        // look-up streams per step: (plane, token) pairs
    constexpr int NP = (NS + 1) / 2;                  // packed accumulators
    constexpr int NG = G64 ? 2 : 1;                   // coefficient groups per block
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int h = lane >> 4, a = lane & 15;

    // Programmatic dependent launch: the next kernel of the stream may be scheduled as soon as this
    // one's CTAs leave their SMs; everything this kernel itself reads or writes that an earlier
    // kernel may have produced (x, y, the workspace) is touched only after griddepcontrol.wait below.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool dep_waited = false;

    // ---- shared memory map (addresses in the shared window) ----
    //   [smem0, +kMiscBytes)             xsum, completion list
    //   [lut0, lut0 + MT*64 KB)          tables, lut0 the next multiple of 64 KB
    const unsigned smem0 = (unsigned)__cvta_generic_to_shared(smem);
    const unsigned lut0 = (smem0 + kMiscBytes + 65535u) & ~65535u;
    if (lut0 + MT * kTableBytes > smem0 + (unsigned)p.dyn_smem) {       // tables do not fit
        if (tid == 0) atomicExch(p.status, BPDQ_ERR_UNSUPPORTED);
        return;                                                          // uniform: no barrier has been reached
    }
    float* xsum = reinterpret_cast<float*>(smem);                         // [MT][kSliceBlocks][2]: per 64-column half block
    int* done = reinterpret_cast<int*>(smem + 64);                        // [kMaxDone]
    int* ndone = done + kMaxDone;
    float* lut = reinterpret_cast<float*>(smem + (lut0 - smem0));         // [MT][256][kSlots]

    // The lane's table address at step s is lut0 + 256 * (plane byte) + slot(s), slot(s) = 4*((s + a) mod 16) + 64*h
    // (< 128).  lut0 is a multiple of 64 KB below 16 MB, so the address is four bytes: [slot][plane byte]
    // [lut0 >> 16][0], which one byte-permute assembles from the plane word and a register that holds
    // lut0 >> 16 in byte 0 and the slots of three consecutive steps in bytes 1..3 (the zero top byte is
    // the replicated sign of byte 0).
    unsigned slots[6];
#pragma unroll
    for (int j = 0; j < 6; ++j) {
        slots[j] = lut0 >> 16;
#pragma unroll
        for (int e = 0; e < 3; ++e) {
            const int s = 3 * j + e;
            if (s < 16) slots[j] |= (4u * ((s + a) & 15) + 64u * h) << (8 * (e + 1));
        }
    }
#pragma unroll
    for (int j = 0; j < 6; ++j) asm volatile("" : "+r"(slots[j]));   // opaque: kept in registers instead of being recomputed at every use
    // steps at which this lane's chunk (logical byte (s + a) mod 16) lies in the block's first 64 columns
    unsigned lo_steps = 0;
#pragma unroll
    for (int s = 0; s < 16; ++s) lo_steps |= (((s + a) & 15) < 8 ? 1u : 0u) << s;

    // contiguous share of the concatenated (linear, slice, row group) task space, cut by the host
    const int bid = blockIdx.x;
    int t = p.t_begin[bid];
    const int t_end = p.t_begin[bid + 1];
    int li = 0;                                       // linear that task t belongs to

    // rows of the chunks on the completion list: rounded to binary16, written to y, workspace zeroed again
    auto convert_done = [&](const GemvLinear& L) {
        const int nd = *ndone;
        if (nd > 0) {
            __threadfence();
            // items of four consecutive rows; a thread reads several before it writes, so that the
            // L2 round trips of a CTA that completes many chunks overlap
            constexpr int kQuads = kChunkRgs * 16 / 4, kAhead = 4;
            const int nitems = nd * MT * kQuads;
            for (int i0 = tid; i0 < nitems; i0 += kThreads * kAhead) {
                float4 v[kAhead], vb[kAhead];
                size_t at[kAhead];
                int row[kAhead];
                bool live[kAhead];
#pragma unroll
                for (int u = 0; u < kAhead; ++u) {
                    const int idx = i0 + u * kThreads;
                    live[u] = false;
                    if (idx < nitems) {
                        const int ckd = done[idx / (MT * kQuads)];
                        const int rem = idx % (MT * kQuads);
                        const int r = ckd * kChunkRgs * 16 + (rem % kQuads) * 4;
                        if (r < L.out) {                  // out is a multiple of 16: a quad is inside or outside as a whole
                            live[u] = true;
                            row[u] = r;
                            at[u] = (size_t)(rem / kQuads) * L.out + r;
                            v[u] = __ldcg(reinterpret_cast<const float4*>((EXT ? L.conv_a : L.ws) + at[u]));
                            if (EXT && L.conv_b) vb[u] = __ldcg(reinterpret_cast<const float4*>(L.conv_b + at[u]));
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < kAhead; ++u) {
                    if (live[u]) {
                        if (EXT) {
                            bpdq::finish_quad(v[u], vb[u], L.bias_a, L.bias_b, L.conv_b != nullptr, row[u]);
                            if (L.conv_b) __stcg(reinterpret_cast<float4*>(L.conv_b + at[u]), make_float4(0.f, 0.f, 0.f, 0.f));
                        }
                        const __half2 h01 = __floats2half2_rn(v[u].x, v[u].y), h23 = __floats2half2_rn(v[u].z, v[u].w);
                        uint2 o;
                        o.x = *reinterpret_cast<const unsigned*>(&h01);
                        o.y = *reinterpret_cast<const unsigned*>(&h23);
                        *reinterpret_cast<uint2*>(L.y + at[u]) = o;
                        __stcg(reinterpret_cast<float4*>((EXT ? L.conv_a : L.ws) + at[u]), make_float4(0.f, 0.f, 0.f, 0.f));
                    }
                }
            }
        }
    };
    // ---- hand-over of a finished segment ----
    // Row sums are accumulated across slices with binary32 atomic adds in `ws` (kept zero
    // between calls).  Row groups are counted in chunks of kChunkRgs; whoever delivers the last
    // contribution of a chunk converts its rows to binary16, writes y and zeroes `ws` again.
    // The caller has fenced the segment's atomic adds and passed a CTA barrier.
    auto hand_over = [&](const GemvLinear& L, const int rg_begin, const int rg_end) {
        const int ck_begin = rg_begin / kChunkRgs, ck_end = (rg_end + kChunkRgs - 1) / kChunkRgs;
        for (int ck0 = ck_begin; ck0 < ck_end; ck0 += kMaxDone) {
            if (tid == 0) *ndone = 0;
            __syncthreads();
            for (int ck = ck0 + tid; ck < min(ck_end, ck0 + kMaxDone); ck += kThreads) {
                const int lo = max(rg_begin, ck * kChunkRgs), hi = min(rg_end, (ck + 1) * kChunkRgs);
                const int size = min(L.nrg, (ck + 1) * kChunkRgs) - ck * kChunkRgs;
                const unsigned before = atomicAdd(&L.counters[ck], (unsigned)(hi - lo));
                if (before + (unsigned)(hi - lo) == (unsigned)(size * L.nslices * (EXT ? L.target_mul : 1))) {
                    L.counters[ck] = 0u;
                    done[atomicAdd(ndone, 1)] = ck;
                }
            }
            __syncthreads();
            convert_done(L);
            __syncthreads();
        }
    };
    int pend_li = -1, pend_begin = 0, pend_end = 0;   // finished segment whose hand-over is still due

    while (t < t_end) {
        while (li + 1 < p.n && t >= p.lin[li + 1].task_begin) ++li;
        const GemvLinear& L = p.lin[li];
        // byte offsets into the blob fit 32 bits (the launcher refuses larger blobs): addresses are the blob's
        // uniform base plus a 32-bit per-lane offset
        const unsigned plane_pitch = (unsigned)L.out * 16u;   // bytes between planes of one block
        const unsigned coef_pitch = (unsigned)L.out * 2u;     // bytes between coefficients of one group
        const int tl = t - L.task_begin;
        const int s = tl / L.nrg;
        const int rg_begin = tl - s * L.nrg;
        const int rg_end = min(L.nrg, rg_begin + (t_end - t));
        const int ntask = (rg_end - rg_begin - wid + W - 1) / W;          // tasks of this warp (may be <= 0)

        // per-lane source pointers of the first task; a task further on is W*16 rows further on
        unsigned psrc[2], csrc[2];
        bool valid[2];
        {
            const int r = (rg_begin + wid) * 16 + a;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int b = s * kSliceBlocks + 2 * q + h;
                valid[q] = b < L.nblocks;                                  // false past the end of a ragged last slice
                const int bb = valid[q] ? b : 0;
                psrc[q] = ((unsigned)bb * K * L.out + r) * 16u;
                const int G = (bb * 128) / L.group;
                csrc[q] = (unsigned)L.planes_bytes + ((unsigned)G * (K + 1) * L.out + r) * 2u;
            }
        }
        // one half of a task: the plane units and coefficients of the lane's block in block pair q
        auto load_half = [&](Task<K, NG>& tk, int n, int q) {
            if (valid[q]) {
                const unsigned ps = psrc[q] + (unsigned)n * (W * 256);
#pragma unroll
                for (int i = 0; i < K; ++i) tk.pl[q][i] = ldg_stream16(L.blob + (size_t)(ps + i * plane_pitch));
                const unsigned cs = csrc[q] + (unsigned)n * (W * 32);
                if constexpr (NG == 2) {          // the pair's even row, group a & 1 (rows are even-aligned: out is a multiple of 16)
                    const unsigned cp = cs - 2u * (a & 1) + (unsigned)(a & 1) * (K + 1) * coef_pitch;
#pragma unroll
                    for (int i = 0; i <= K; ++i) tk.cfp[q][i] = ldg_stream4(L.blob + (size_t)(cp + i * coef_pitch));
                } else {
#pragma unroll
                    for (int i = 0; i <= K; ++i) tk.cf[q][i] = ldg_stream2(L.blob + (size_t)(cs + i * coef_pitch));
                }
            } else {                              // contributes nothing: zero planes, zero coefficients
#pragma unroll
                for (int i = 0; i < K; ++i) tk.pl[q][i] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int i = 0; i <= K; ++i) {
                    if constexpr (NG == 2) tk.cfp[q][i] = 0u; else tk.cf[q][i] = 0;
                }
            }
        };
        auto load_task = [&](Task<K, NG>& tk, int n) {
#pragma unroll
            for (int q = 0; q < 2; ++q) load_half(tk, n, q);
        };

        // ---- this thread's inputs for the table build and the first tasks' weights ----
        // table items (slot, entry block): kSlots * 8 of them, IT per thread; item = tid + it * kThreads,
        // slot = item % 64 (chunk table), eh = item / 64 (entries eh*32 .. eh*32+31 share inputs 5..7).
        // slot = 16*block + logical byte L; L = 4k + q is byte q of 32-column word k, and bit
        // 4*jj + u of that byte is column 32k + 8u + 2q + jj: four pairs of adjacent inputs
        static_assert((kSlots * 8) % (W * 32) == 0, "whole table items per thread");
        constexpr int IT = kSlots * 8 / (W * 32);
        const int slot = tid & (kSlots - 1);          // kThreads is a multiple of 64: the same slot for all of a thread's items
        const int col = s * (kSliceBlocks * 128) + (slot >> 2) * 32 + (slot & 3) * 2;
        // Before the first wait on the preceding kernel only the weights may be requested (they
        // belong to the handle and were complete long ago); then x, which that kernel may have written.
        Task<K, NG> tk[D];
        const bool early = !dep_waited && p.early_weights != 0;
        if (early) {
#pragma unroll
            for (int d = 0; d < D; ++d)
                if (d < ntask) load_task(tk[d], d);
        }
        if (!dep_waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            dep_waited = true;
        }
        unsigned xraw[MT][4];
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int u = 0; u < 4; ++u)
                xraw[m][u] = col >= L.in ? 0u
                             : !(EXT && L.perm) ? ldg_x4(L.x + (size_t)m * L.in + col + 8 * u)
                                         : (unsigned)ldg_x2(L.x + (size_t)m * L.in + __ldg(L.perm + col + 8 * u)) |
                                               ((unsigned)ldg_x2(L.x + (size_t)m * L.in + __ldg(L.perm + col + 8 * u + 1)) << 16);
        if (!early) {
#pragma unroll
            for (int d = 0; d < D; ++d)
                if (d < ntask) load_task(tk[d], d);
        }

        // the previous segment is handed over while this segment's first loads are in flight
        if (pend_li >= 0) hand_over(p.lin[pend_li], pend_begin, pend_end);

        // ---- build the 64 chunk tables of this slice (per token) ----
#pragma unroll
        for (int it = 0; it < IT; ++it) {
            const int eh = (tid + it * kThreads) >> 6;
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                float xs[8];                          // xs[t]: the input that bit t of the plane byte selects
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&xraw[m][u]));
                    xs[u] = f.x; xs[4 + u] = f.y;
                }
                float lo[32];                         // subset sums of inputs 0..4
                lo[0] = 0.f;
#pragma unroll
                for (int k = 0; k < 5; ++k)
#pragma unroll
                    for (int j = 0; j < (1 << k); ++j) lo[(1 << k) + j] = lo[j] + xs[k];
                float base = 0.f;
                if (eh & 1) base += xs[5];
                if (eh & 2) base += xs[6];
                if (eh & 4) base += xs[7];
                float* dst = lut + m * (kTableBytes / 4) + (eh * 32) * kSlots + slot;
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[j * kSlots] = base + lo[j];
            }
        }
        __syncthreads();
        if (tid < MT * kSliceBlocks * 2) {            // sums of x over the two 64-column halves of every block
            const int m = tid / (kSliceBlocks * 2), hb = tid % (kSliceBlocks * 2);
            float acc = 0.f;
            for (int c = 0; c < 8; ++c) acc += lut[m * (kTableBytes / 4) + 255 * kSlots + hb * 8 + c];
            xsum[m * (kSliceBlocks * 2) + hb] = acc;
        }
        __syncthreads();

        // ---- stream the row groups of this slice ----
        // n_next >= 0: the task that takes this one's registers; each half is requested as soon as the half it
        // replaces has been used, so that nearly D tasks per warp are in flight rather than D - 1 (three planes
        // for two tokens keep the whole-task request: the other order costs that instantiation spills)
        constexpr bool kReloadHalves = !(K == 3 && MT == 2);
        auto process_task = [&](Task<K, NG>& tk, int n, int n_next) {
            float yacc[MT];
#pragma unroll
            for (int m = 0; m < MT; ++m) yacc[m] = 0.f;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                // stream sidx = i*MT + m; streams are added in pairs, and every pair keeps two
                // accumulators (even and odd steps) to shorten the add chains
                unsigned long long acc[NP][2];
#pragma unroll
                for (int j = 0; j < NP; ++j) acc[j][0] = acc[j][1] = 0ull;
                float held = 0.f;                     // odd stream count: the last stream pairs two steps
                unsigned held_addr = 0u;
                float Slo[NS];                        // g = 64: the part of every stream that falls into the block's first 64 columns
#pragma unroll
                for (int j = 0; j < NS; ++j) Slo[j] = 0.f;
#pragma unroll
                for (int st = 0; st < 16; ++st) {
                    // address = slot address with the plane byte in bits 8..15
                    unsigned addr[K];
#pragma unroll
                    for (int i = 0; i < K; ++i)
                        addr[i] = prmt(word_of(tk.pl[q][i], st >> 2), slots[st / 3], 0xC400u | ((st & 3) << 4) | (5 + st % 3));   // the selector is a constant once the step loop is unrolled
                    constexpr int QI = 128;               // the block pair and the token's table go into the immediate
                    if constexpr (G64) {
                        // pairs as below (two planes of one token, or the two tokens of a plane); the loaded values also go, on
                        // the steps of the block's first 64 columns, into the first group's partial sums
                        const bool lo = ((lo_steps >> st) & 1u) != 0u;
#pragma unroll
                        for (int j = 0; j < NS / 2; ++j) {
                            float va, vb;
                            if constexpr (MT == 2) {
                                if (q == 0) lookup2v_add<0, kTableBytes>(acc[j][st & 1], addr[j], addr[j], va, vb);
                                else lookup2v_add<QI, kTableBytes + QI>(acc[j][st & 1], addr[j], addr[j], va, vb);
                            } else {
                                if (q == 0) lookup2v_add<0, 0>(acc[j][st & 1], addr[2 * j], addr[2 * j + 1], va, vb);
                                else lookup2v_add<QI, QI>(acc[j][st & 1], addr[2 * j], addr[2 * j + 1], va, vb);
                            }
                            if (lo) { Slo[2 * j] += va; Slo[2 * j + 1] += vb; }
                        }
                        if (NS & 1) {                     // one token, odd K: the last plane pairs two consecutive steps
                            const float vl = q == 0 ? lds_table<0>(addr[K - 1]) : lds_table<QI>(addr[K - 1]);
                            if (lo) Slo[NS - 1] += vl;
                            if ((st & 1) == 0) held = vl;
                            else add2(acc[NP - 1][(st >> 1) & 1], held, vl);
                        }
                    } else if constexpr (MT == 2) {
                        // pair = the two tokens of one plane: one address, two tables
#pragma unroll
                        for (int i = 0; i < K; ++i) {
                            if (q == 0) lookup2_add<0, kTableBytes>(acc[i][st & 1], addr[i], addr[i]);
                            else lookup2_add<QI, kTableBytes + QI>(acc[i][st & 1], addr[i], addr[i]);
                        }
                    } else {
                        // one token: pair = two planes; an odd plane left over pairs two consecutive steps
#pragma unroll
                        for (int j = 0; j < K / 2; ++j) {
                            if (q == 0) lookup2_add<0, 0>(acc[j][st & 1], addr[2 * j], addr[2 * j + 1]);
                            else lookup2_add<QI, QI>(acc[j][st & 1], addr[2 * j], addr[2 * j + 1]);
                        }
                        if (K & 1) {
                            if ((st & 1) == 0) held_addr = addr[K - 1];
                            else if (q == 0) lookup2_add<0, 0>(acc[NP - 1][(st >> 1) & 1], held_addr, addr[K - 1]);
                            else lookup2_add<QI, QI>(acc[NP - 1][(st >> 1) & 1], held_addr, addr[K - 1]);
                        }
                    }
                }
                float S[NS];
#pragma unroll
                for (int j = 0; j < NS / 2; ++j) {
                    const float2 e = unpack2(acc[j][0]), o = unpack2(acc[j][1]);
                    S[2 * j] = e.x + o.x;
                    S[2 * j + 1] = e.y + o.y;
                }
                if (NS & 1) {
                    const float2 e = unpack2(acc[NP - 1][0]), o = unpack2(acc[NP - 1][1]);
                    S[NS - 1] = (e.x + e.y) + (o.x + o.y);
                }
                const int blk = 2 * q + h;
                if constexpr (G64) {
                    // swap with the pair's other lane: word = (even row, odd row) of one group; this lane's row is half a & 1
                    float cl[K + 1], ch[K + 1];       // this row's coefficients of the block's first and second group
#pragma unroll
                    for (int i = 0; i <= K; ++i) {
                        const unsigned mine = tk.cfp[q][i];
                        const unsigned other = __shfl_xor_sync(0xffffffffu, mine, 1);
                        const unsigned g0 = (a & 1) ? other : mine, g1 = (a & 1) ? mine : other;   // words of group 0 and group 1
                        cl[i] = __half2float(__ushort_as_half((unsigned short)((a & 1) ? (g0 >> 16) : (g0 & 0xffffu))));
                        ch[i] = __half2float(__ushort_as_half((unsigned short)((a & 1) ? (g1 >> 16) : (g1 & 0xffffu))));
                    }
                    const float c0l = cl[0], c0h = ch[0];
#pragma unroll
                    for (int m = 0; m < MT; ++m)
                        yacc[m] = fmaf(c0h, xsum[(m * kSliceBlocks + blk) * 2 + 1], fmaf(c0l, xsum[(m * kSliceBlocks + blk) * 2], yacc[m]));
#pragma unroll
                    for (int i = 0; i < K; ++i) {
                        const float cil = cl[i + 1];
                        const float cih = ch[i + 1];
#pragma unroll
                        for (int m = 0; m < MT; ++m)
                            yacc[m] = fmaf(cih, S[i * MT + m] - Slo[i * MT + m], fmaf(cil, Slo[i * MT + m], yacc[m]));
                    }
                } else {
                    const float c0 = __half2float(__ushort_as_half(tk.cf[q][0]));
#pragma unroll
                    for (int m = 0; m < MT; ++m)
                        yacc[m] = fmaf(c0, xsum[(m * kSliceBlocks + blk) * 2] + xsum[(m * kSliceBlocks + blk) * 2 + 1], yacc[m]);
#pragma unroll
                    for (int i = 0; i < K; ++i) {
                        const float ci = __half2float(__ushort_as_half(tk.cf[q][i + 1]));
#pragma unroll
                        for (int m = 0; m < MT; ++m) yacc[m] = fmaf(ci, S[i * MT + m], yacc[m]);
                    }
                }
                if (kReloadHalves && n_next >= 0) load_half(tk, n_next, q);
            }
            // the two half-warps hold the even-block and odd-block parts of the same 16 rows
#pragma unroll
            for (int m = 0; m < MT; ++m) yacc[m] += __shfl_xor_sync(0xffffffffu, yacc[m], 16);
            if (h == 0) {
                const int r = (rg_begin + wid + n * W) * 16 + a;
#pragma unroll
                for (int m = 0; m < MT; ++m) red_add(&L.ws[(size_t)m * L.out + r], yacc[m]);
            }
        };
        for (int n0 = 0; n0 < ntask; n0 += D) {
#pragma unroll
            for (int d = 0; d < D; ++d) {
                const int n = n0 + d;
                if (n < ntask) {                      // warp-uniform
                    if constexpr (kReloadHalves) {
                        process_task(tk[d], n, n + D < ntask ? n + D : -1);
                    } else {
                        process_task(tk[d], n, -1);
                        if (n + D < ntask) load_task(tk[d], n + D);
                    }
                }
            }
        }

        // ---- segment finished: its atomic adds are fenced, all warps are done with the tables ----
        __threadfence();
        __syncthreads();
        pend_li = li; pend_begin = rg_begin; pend_end = rg_end;
        t += rg_end - rg_begin;
    }
    if (pend_li >= 0) hand_over(p.lin[pend_li], pend_begin, pend_end);
}

template <int K, int MT, int D, int W, bool G64, bool EXT>
int launch_cfg(bpdq_handle_s* h, GemvParams p, cudaStream_t stream) {
    static bpdq::SmemOptin optin;
    const int smem = 65536 + MT * kTableBytes;        // tables start at the first 64 KB boundary of the shared window
    if (smem > h->smem_optin)
        return bpdq::set_error(BPDQ_ERR_UNSUPPORTED, "gemv: %d bytes of shared memory needed, device offers %d", smem, h->smem_optin);
    if (const int rc = bpdq::ensure_smem_optin(gemv_lut_kernel<K, MT, D, W, G64, EXT>, optin, h->device, smem, "gemv"); rc != BPDQ_OK) return rc;
    long long total = 0;
    for (int k = 0; k < p.n; ++k) {
        if ((unsigned long long)p.lin[k].blob_bytes >= (1ull << 32))
            return bpdq::set_error(BPDQ_ERR_UNSUPPORTED, "gemv: packed weights of 4 GB or more in one linear");
        p.lin[k].task_begin = (int)total;
        total += (long long)p.lin[k].nslices * p.lin[k].nrg;
        if (total >= (1ll << 31)) return bpdq::set_error(BPDQ_ERR_UNSUPPORTED, "gemv: task space too large");
    }
    // Cut the task space into one contiguous share per SM such that the most expensive share is as
    // cheap as possible, a segment (a CTA's visit to one slice of one linear: table set-up, drain,
    // hand-over) counting as kSegmentCost tasks.  Short slices (few output rows) would otherwise load
    // the CTAs that get them with many set-ups.  The cut itself is plain host code (bpdq_partition.h).
    int grid = h->sm_count < kMaxGrid ? h->sm_count : kMaxGrid;
    if ((long long)grid > total) grid = (int)total;
    const int kSegmentCost = p.n > 1 ? kSegmentCostBatch : kSegmentCostSingle;
    bpdq::LaunchPlan& plan = h->plan[0];
    static_assert(sizeof(plan.t_begin) == sizeof(p.t_begin), "one cached entry per CTA boundary");
    bool cached = plan.n == p.n && plan.cost == kSegmentCost && plan.grid == grid;
    for (int k = 0; cached && k < p.n; ++k) cached = plan.shape[k][0] == p.lin[k].nrg && plan.shape[k][1] == p.lin[k].nslices;
    if (cached) {
        for (int c = 0; c <= grid; ++c) p.t_begin[c] = plan.t_begin[c];
    } else {
        int nrg[kMaxBatch], nsl[kMaxBatch];
        for (int k = 0; k < p.n; ++k) { nrg[k] = p.lin[k].nrg; nsl[k] = p.lin[k].nslices; }
        bpdq::cut_task_space(nrg, nsl, p.n, grid, kSegmentCost, p.t_begin);
        plan.n = p.n; plan.cost = kSegmentCost; plan.grid = grid;
        for (int k = 0; k < p.n; ++k) { plan.shape[k][0] = p.lin[k].nrg; plan.shape[k][1] = p.lin[k].nslices; }
        for (int c = 0; c <= grid; ++c) plan.t_begin[c] = p.t_begin[c];
    }
    p.dyn_smem = smem;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(W * 32); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // lets this launch overlap the tail of the kernel before it
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_lut_kernel<K, MT, D, W, G64, EXT>, p);
    h->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemv launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

// Tasks kept in flight per lane: two (a third costs more in registers than it hides in latency: measured slower
// for every K); one where two tasks do not fit the register file (K = 4).
template <int K, int MT>
int launch_one(bpdq_handle_s* h, const GemvParams& p, cudaStream_t stream) {
    bool ext = false;
    for (int k = 0; k < p.n; ++k) ext = ext || p.lin[k].perm || p.lin[k].bias_a || p.lin[k].conv_b;
    constexpr int D = K <= 3 ? 2 : 1;
    if (p.lin[0].group == 64) return ext ? launch_cfg<K, MT, D, 16, true, true>(h, p, stream) : launch_cfg<K, MT, D, 16, true, false>(h, p, stream);
    return ext ? launch_cfg<K, MT, D, 16, false, true>(h, p, stream) : launch_cfg<K, MT, D, 16, false, false>(h, p, stream);
}

void fill_linear(GemvLinear& L, const bpdq_handle_s* h) {
    L.blob = h->d_blob;
    L.planes_bytes = h->planes_bytes;
    L.blob_bytes = h->blob_bytes;
    L.ws = h->d_ws;
    L.counters = h->d_counters;
    L.conv_a = h->d_ws; L.conv_b = nullptr;
    L.bias_a = static_cast<const __half*>(h->d_bias); L.bias_b = nullptr;
    L.target_mul = 1;
    L.perm = h->d_perm;
    L.out = h->out; L.in = h->in; L.group = h->group;
    L.nblocks = h->in / 128;
    L.nslices = (L.nblocks + kSliceBlocks - 1) / kSliceBlocks;
    L.nrg = h->out / 16;
    L.task_begin = 0;
}

// Passes of at most kMaxMT tokens over all linears of the batch.
template <int K>
int launch_k(bpdq_handle_s* const* hs, GemvParams p, const void* const* xs, void* const* ys, int M, cudaStream_t stream) {
    int m0 = 0;
    while (m0 < M) {
        int mt = M - m0;
        if (mt > kMaxMT) mt = kMaxMT;
        for (int k = 0; k < p.n; ++k) {
            p.lin[k].x = static_cast<const __half*>(xs[k]) + (size_t)m0 * hs[k]->in;
            p.lin[k].y = static_cast<__half*>(ys[p.lin[k].target_mul == 2 ? 0 : k]) + (size_t)m0 * hs[k]->out;   // a pair writes one output
        }
        const int rc = (mt == 1) ? launch_one<K, 1>(hs[0], p, stream) : launch_one<K, 2>(hs[0], p, stream);
        if (rc != BPDQ_OK) return rc;
        m0 += mt;
    }
    return BPDQ_OK;
}

}  // namespace

namespace bpdq {

// The kernel addresses the blob with 32-bit offsets: linears whose packed weights reach 4 GB go to the other kernels.
bool gemv_supported(int out, int in, int K, int group) {
    if (!(K >= 1 && K <= 4 && (group == 64 || group == 128 || group == 256))) return false;
    return (unsigned long long)planes_bytes(out, in, K) + coefs_bytes(out, in, K, group) < (1ull << 32);
}

// binary32 row sums: kMaxMT tokens for the look-up-table kernel; up to 64 tokens for the tensor-core kernel's split
// over the input dimension
size_t gemv_workspace_bytes(int out, int, int, int, int max_M, int) {
    const int tokens = max_M < kMaxMT ? kMaxMT : (max_M > 128 ? 128 : max_M);   // the tile kernel's split over the input dimension shares it, up to its largest token tile
    return (size_t)tokens * out * sizeof(float);
}

size_t gemv_counter_count(int out) { return ((size_t)out / 16 + kChunkRgs - 1) / kChunkRgs; }

int launch_gemv_batch(bpdq_handle_s* const* hs, const void* const* xs, void* const* ys, int n, int M, cudaStream_t stream, bool pair) {
    if (n < 1 || n > kMaxBatch) return set_error(BPDQ_ERR_INVALID, "gemv: %d linears in one launch (1..%d)", n, kMaxBatch);
    if (pair && (n != 2 || hs[0]->out != hs[1]->out)) return set_error(BPDQ_ERR_INVALID, "gemv: a (gate, up) pair is two linears with the same rows");
    GemvParams p;
    p.n = n;
    p.status = hs[0]->d_status;
    p.early_weights = 1;
    for (int k = 0; k < n; ++k) {
        if (hs[k]->K != hs[0]->K) return set_error(BPDQ_ERR_INVALID, "gemv: linears of one launch must share K");
        if ((hs[k]->group == 64) != (hs[0]->group == 64))
            return set_error(BPDQ_ERR_INVALID, "gemv: linears of one launch must all have group 64 or none of them");
        fill_linear(p.lin[k], hs[k]);
        if (hs[k]->caller_blob) p.early_weights = 0;
    }
    if (pair) {                                          // both count into gate's counters; whoever completes a chunk converts both sums
        for (int k = 0; k < 2; ++k) {
            GemvLinear& L = p.lin[k];
            L.counters = hs[0]->d_counters;
            L.conv_a = hs[0]->d_ws; L.conv_b = hs[1]->d_ws;
            L.bias_a = static_cast<const __half*>(hs[0]->d_bias); L.bias_b = static_cast<const __half*>(hs[1]->d_bias);
            L.target_mul = 2;
        }
    }
    switch (hs[0]->K) {
        case 1: return launch_k<1>(hs, p, xs, ys, M, stream);
        case 2: return launch_k<2>(hs, p, xs, ys, M, stream);
        case 3: return launch_k<3>(hs, p, xs, ys, M, stream);
        case 4: return launch_k<4>(hs, p, xs, ys, M, stream);
        default: return set_error(BPDQ_ERR_UNSUPPORTED, "gemv: K=%d", hs[0]->K);
    }
}

int launch_gemv(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    return launch_gemv_batch(&h, &x, &y, 1, M, stream);
}

}  // namespace bpdq

// ---------------------------------------------------------------------------------------------
// bpdq_linear_noalloc: the look-up-table kernel for callers that must not allocate.
// ---------------------------------------------------------------------------------------------
// The kernel's scratch (binary32 row sums, arrival counters, status word) lives in a file-scope
// device array instead of a handle.  In host code `g_noalloc_scratch` is only a stand-in for the
// symbol: its device address is fetched with cudaGetSymbolAddress, once per device, and that
// address is what the kernel receives.
namespace {

constexpr size_t kNoallocWsBytes = (size_t)kMaxMT * BPDQ_NOALLOC_MAX_OUT * sizeof(float);
constexpr size_t kNoallocCounterBytes = ((size_t)BPDQ_NOALLOC_MAX_OUT / 16 / kChunkRgs) * sizeof(unsigned);
constexpr size_t kNoallocBytes = kNoallocWsBytes + kNoallocCounterBytes + 256;   // + status word

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocBytes];

using bpdq::kMaxDevices;
struct NoallocDevice {
    bool ready;
    unsigned char* scratch;       // device address of g_noalloc_scratch on this device
    int sm_count, smem_optin;
    bpdq_handle_s view;           // what the launcher sees; owns nothing, keeps the last cut of the task space between calls
};
NoallocDevice g_noalloc_dev[kMaxDevices];

// Set-up of the current device: symbol address and the two device attributes the launcher needs.
int noalloc_setup(int dev) {
    NoallocDevice& d = g_noalloc_dev[dev];
    if (d.ready) return BPDQ_OK;
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "bpdq_linear_noalloc: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    int major = 0;
    if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess ||
        (e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess ||
        (e = cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
        return bpdq::set_error(BPDQ_ERR_CUDA, "bpdq_linear_noalloc: device attributes: %s", cudaGetErrorString(e));
    if (major != 10)
        return bpdq::set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_linear_noalloc: device is sm_%dx, this library is built for sm_100a only", major);
    d.scratch = static_cast<unsigned char*>(ptr);
    d.ready = true;
    return BPDQ_OK;
}

}  // namespace

extern "C" int bpdq_linear_noalloc(const void* blob_dev, int out, int in, int K, int group, const void* x_fp16_dev,
                                   void* y_fp16_dev, int M, void* stream) {
    using namespace bpdq;
    if (M < 0 || M > BPDQ_GEMV_MAX_M)
        return set_error(BPDQ_ERR_INVALID, "bpdq_linear_noalloc: M=%d outside [0, %d]", M, BPDQ_GEMV_MAX_M);
    if (!shape_supported(out, in, K, group) || !gemv_supported(out, in, K, group))
        return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_linear_noalloc: unsupported shape out=%d in=%d K=%d g=%d", out, in, K, group);
    if (out > BPDQ_NOALLOC_MAX_OUT)
        return set_error(BPDQ_ERR_INVALID, "bpdq_linear_noalloc: out=%d exceeds the static scratch limit of %d rows", out,
                         BPDQ_NOALLOC_MAX_OUT);
    if (M == 0) return BPDQ_OK;
    if (!blob_dev || !x_fp16_dev || !y_fp16_dev) return set_error(BPDQ_ERR_INVALID, "bpdq_linear_noalloc: null pointer");
    if ((reinterpret_cast<uintptr_t>(blob_dev) | reinterpret_cast<uintptr_t>(x_fp16_dev) | reinterpret_cast<uintptr_t>(y_fp16_dev)) & 15u)
        return set_error(BPDQ_ERR_INVALID, "bpdq_linear_noalloc: blob, x and y must be 16-byte aligned");
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_linear_noalloc: no CUDA device (%s)", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return set_error(BPDQ_ERR_UNSUPPORTED, "bpdq_linear_noalloc: device ordinal %d", dev);
    int rc = noalloc_setup(dev);
    if (rc != BPDQ_OK) return rc;
    NoallocDevice& d = g_noalloc_dev[dev];
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // The scratch keeps whatever the last call left; the kernel needs row sums and counters at zero.
    const size_t ws_used = (size_t)kMaxMT * out * sizeof(float);
    if ((e = cudaMemsetAsync(d.scratch, 0, ws_used, s)) != cudaSuccess ||
        (e = cudaMemsetAsync(d.scratch + kNoallocWsBytes, 0, kNoallocCounterBytes + 256, s)) != cudaSuccess)
        return set_error(BPDQ_ERR_CUDA, "bpdq_linear_noalloc: clearing the scratch: %s", cudaGetErrorString(e));

    bpdq_handle_s& h = d.view;                          // calls with the shape of the last one reuse its cut (launch_cfg compares shapes)
    h.out = out; h.in = in; h.K = K; h.group = group; h.max_M = BPDQ_GEMV_MAX_M; h.device = dev;
    h.sm_count = d.sm_count; h.smem_optin = d.smem_optin;
    h.d_blob = const_cast<uint8_t*>(static_cast<const uint8_t*>(blob_dev));
    h.caller_blob = 1;                                  // the caller may have produced it with the kernel just before this one
    h.planes_bytes = planes_bytes(out, in, K);
    h.blob_bytes = h.planes_bytes + coefs_bytes(out, in, K, group);
    h.d_ws = reinterpret_cast<float*>(d.scratch);
    h.ws_bytes = ws_used;
    h.d_counters = reinterpret_cast<unsigned*>(d.scratch + kNoallocWsBytes);
    h.n_counters = gemv_counter_count(out);
    h.d_status = reinterpret_cast<int*>(d.scratch + kNoallocWsBytes + kNoallocCounterBytes);
    return launch_gemv(&h, x_fp16_dev, y_fp16_dev, M, s);
}
