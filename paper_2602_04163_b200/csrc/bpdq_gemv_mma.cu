// bpdq_gemv_mma: y = x * W^T for a few tokens (3 <= M <= 32) with every packed weight read once.
//
// The look-up-table kernel pays one shared-memory look-up per plane byte AND token, so beyond a handful of
// tokens it re-reads the weights pass after pass; the tcgen05 tile kernel pays a full 128 x N x 16 instruction,
// a shared-memory round trip and two barrier hand-overs per stage however few token columns there are.  In
// between, the layer is still bound by HBM (the weights) and then by the integer work of the decode, so this
// kernel keeps the decoded weights in registers and feeds them straight to warp-level tensor-core instructions
// (mma.sync m16n8k16, binary16 operands, binary32 accumulators): no operand ever goes through shared memory,
// and no thread waits for another one inside the streaming loop.
//
//   D[token, row] (16 x 8) += A[token, k] (16 x 16, activations) * B[k, row] (16 x 8, decoded weights)
//
// Work split.  A warp task is 16 output rows x 512 input columns (a "slice" of four 128-column blocks): lane
// (g, t) = (lane / 4, lane % 4) owns the rows 8j + g (j = 0, 1) of block t.  The task's packed bytes -- 4 K runs of
// 512 bytes of plane units and a few 64-byte runs of binary16 coefficients -- arrive one task ahead in the warp's
// private landing area in shared memory as two boxes of tensor maps over the blob (two TMA copies per task whatever
// K is, completion on the warp's mbarrier; per-lane 16-byte asynchronous copies of the same bytes cost one
// shared-memory wavefront per lane and kept that pipe half busy).  Rows and blocks past the end of the linear are
// filled with zeros by the copy.  At the start of a task the lane moves its units into registers, undoes the byte rotation of
// its rows and builds the 2^K candidate values of every (row, group) with the decode rule's exact arithmetic
// (Eq. 7: float(c0), "+ float(ci)" in plane order, one rounding to binary16), as bpdq_dequant does.  Eight
// consecutive columns then cost one shift-and-mask per plane and eight byte-permutes, and come out as four
// registers of two binary16 each -- exactly the B fragments of two mma.sync instructions.  The k index of an
// instruction is ours to assign: lane t supplies four consecutive columns of ITS block, so one instruction
// contracts 4 blocks x 4 columns, and the activations are staged in shared memory in that order, already cut
// into A fragments (one 16-byte load per lane and instruction, shared by the two row groups of the task).
// Accumulators stay in registers while a warp walks along the columns of one row group and leave as binary32
// atomic adds into the handle's workspace [token][row]; arrival counters per 128 rows tell the CTA that
// delivers the last contribution to round those rows to binary16, write y and zero the workspace again
// (the look-up-table kernel's protocol, same workspace and counters).
//
// A CTA (16 warps) takes a contiguous share of the (column range, 32-row group) space of the launch's linears,
// cut on the host; a segment of it is a rectangle (up to four slices) x (row groups) whose 512-column tasks are
// dealt to the warps in row-major order, so a warp mostly continues along the columns of one row group.
// The arithmetic (rounded weights, binary16 x, binary32 accumulation) is that of the tcgen05 kernel.
#include "bpdq_internal.h"
#include "bpdq_decode.cuh"
#include "bpdq_partition.h"
#include "bpdq_tma.cuh"
#include "bpdq_finish.cuh"

#include <cuda_fp16.h>
#include <type_traits>


namespace {

constexpr int kSliceCols = 512;                       // four 128-column blocks, one per lane of a quad
constexpr int kChunkRows = 128;                       // rows per arrival counter (as in the look-up-table kernel)
constexpr int kXSliceBytes = 32 * 32 * 16;            // A fragments of one slice and 16 tokens: 32 instructions x 32 lanes x 16 bytes
constexpr int kMiscBytes = 4096;                      // completion list, abort flag, one mbarrier per warp
constexpr int kMaxDone = 512;
constexpr int kMaxBatch = BPDQ_BATCH_MAX;
constexpr int kMaxGrid = 192;
// Eight-row groups per task.  Two: with four, the units and tables of sixteen candidates per group (K = 4) do not fit the
// registers, and the other K ran 2 to 20 % slower (most with two token tiles).
constexpr int kRowGroups = 2;
constexpr int kSegmentCost = 2;                       // staging the activations of a segment, in (row group x column range) tasks

struct MmaLinear {
    const CUtensorMap* maps;  // device copies of the handle's two tensor maps: [0] plane units, [1] coefficients
    const __half* x;          // [M][in]
    __half* y;                // [M][out]
    float* ws;                // [M][out] binary32, zero between calls
    unsigned* counters;       // one per 128 rows, zero between calls
    // completion (as in the look-up-table kernel): a finished chunk is converted from conv_a, or for a (gate, up)
    // pair as silu(conv_a) * conv_b; the pair shares gate's counters and both count into them
    float* conv_a;
    float* conv_b;            // null unless paired
    const __half* bias_a;     // null: none
    const __half* bias_b;
    int target_mul;           // 1, or 2 for a pair
    int out, in, group;
    int gsh;                  // coefficient group of a half block: (2 b + half) >> gsh
    int nblocks, nslices;     // 128-column blocks, 512-column slices
    int ncr, nrg;             // column ranges (of `ns` slices), task rows (of 8 NJ output rows)
    int task_begin;
};

struct MmaParams {
    MmaLinear lin[kMaxBatch];
    int n, M;
    int ns;                      // slices per column range
    int* status;
    int t_begin[kMaxGrid + 1];
    int dyn_smem;
    int early_weights;
};

__device__ __forceinline__ uint4 lds128(unsigned addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// the A fragments are read-only between two CTA barriers: not volatile, so that the compiler may hoist and interleave them
__device__ __forceinline__ uint4 lds128_frag(unsigned addr) {
    uint4 v;
    asm("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ unsigned short lds16(unsigned addr) {
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
// coherent 16-byte load of activations (the kernel in front may have written them while this one was resident)
__device__ __forceinline__ uint4 ldg_x16(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void mma16816(float (&d)[4], const uint4& a, unsigned b0, unsigned b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

// A warp's landing area: the packed bytes of one task (8 NJ rows x 512 columns).
template <int K, bool G64, int NJ> struct Land {
    static constexpr int kGroups = G64 ? 2 : 1;                          // coefficient groups per block
    static constexpr int kPlaneBytes = NJ * 4 * K * 128;                 // lines (8-row group j, block, plane) of 8 rows x 16 bytes, 128-byte swizzle
    static constexpr int kCoefBytes = 4 * kGroups * (K + 1) * NJ * 16;   // at most (block, group, coefficient) x 8 NJ rows x 2 bytes
    static constexpr int kBytes = (kPlaneBytes + kCoefBytes + 1023) / 1024 * 1024;   // the swizzled plane box wants 1024-byte alignment
};

// K planes, MT token tiles of 16, NJ groups of eight rows per task, W warps per CTA
// EXT: the launch uses a bias or a (gate, up) pair somewhere (kept out of the plain instantiation, which sits at the register cap)
template <int K, int MT, bool G64, int NJ, int W, bool EXT>
__global__ void __launch_bounds__(W * 32, 1) gemv_mma_kernel(const __grid_constant__ MmaParams p) {
    using LD = Land<K, G64, NJ>;
    constexpr int NG = LD::kGroups;
    constexpr int kThreads = W * 32;
    constexpr int kTaskRows = 8 * NJ;
    constexpr int kChunkRgs = kChunkRows / kTaskRows;
    static_assert(W % 4 == 0 && NJ % 2 == 0, "warps come in fours, row groups in pairs");
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int g = lane >> 2, t = lane & 3;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool dep_waited = false;

    // shared memory: [misc][A fragments: MT x ns slices x 16 KB][landing areas: one per warp]
    const unsigned smem_raw = (unsigned)__cvta_generic_to_shared(smem);
    const unsigned smem0 = (smem_raw + 1023u) & ~1023u;                  // the swizzled TMA destinations want 1024-byte alignment
    int* done = reinterpret_cast<int*>(smem + (smem0 - smem_raw));
    int* ndone = done + kMaxDone;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ndone + 1);
    const unsigned bar = smem0 + 3072u + 8u * (unsigned)wid;             // this warp's "task has landed" barrier
    const unsigned xs0 = smem0 + kMiscBytes;
    const unsigned land0 = xs0 + (unsigned)(MT * p.ns) * kXSliceBytes + (unsigned)wid * LD::kBytes;
    if ((int)(smem0 - smem_raw) + kMiscBytes + MT * p.ns * kXSliceBytes + W * LD::kBytes > p.dyn_smem) {
        if (tid == 0) atomicExch(p.status, BPDQ_ERR_UNSUPPORTED);
        return;                                                          // uniform: no barrier has been reached
    }
    const int bid = blockIdx.x;
    int tsk = p.t_begin[bid];
    const int t_end = p.t_begin[bid + 1];
    int li = 0;

    if (tid == 0) {
        *abort_flag = 0;
        for (int w = 0; w < W; ++w) bpdq::tma::mbar_init(smem0 + 3072u + 8u * w, 1);
        bpdq::tma::fence_barrier_init();
    }
    __syncthreads();

    // ---- one task's packed bytes into this warp's landing area: two TMA copies, issued by lane 0 ----
    // planes map: 8-byte elements, (8 rows x 16 bytes) x (block, plane) x (8-row group); box = 128 bytes x 4 K x NJ with
    // the 128-byte swizzle, so that the 16-byte unit of row g in 128-byte line R = 4 K j + K t + i lands at chunk
    // g ^ (R mod 8): the four lanes of a quad (same g, blocks t = 0..3) then read four different bank groups
    // coefficient map: 8-byte elements, (1 per 4 rows) x (group, coefficient); box = 8 NJ rows x the slice's groups
    unsigned landed = 0;                                                  // tasks consumed by this warp: parity of the next wait
    auto issue_task = [&](const MmaLinear& L, const int rg, const int s) {
        if (lane == 0) {
            const int ngs = 8 >> L.gsh;                                   // coefficient groups per slice
            bpdq::tma::mbar_expect_tx(bar, (unsigned)(LD::kPlaneBytes + ngs * (K + 1) * kTaskRows * 2));
            bpdq::tma::tma_load_3d(land0, L.maps, 0, s * 4 * K, rg * NJ, bar);
            bpdq::tma::tma_load_2d(land0 + LD::kPlaneBytes, L.maps + 1, rg * (kTaskRows / 4), s * ngs * (K + 1), bar);
        }
    };

    // ---- hand-over of a finished segment (its atomic adds are fenced, the CTA has passed a barrier) ----
    auto hand_over = [&](const MmaLinear& L, const int rg_begin, const int rg_end, const int nsl) {
        const int ck_begin = rg_begin / kChunkRgs, ck_end = (rg_end + kChunkRgs - 1) / kChunkRgs;
        for (int ck0 = ck_begin; ck0 < ck_end; ck0 += kMaxDone) {
            if (tid == 0) *ndone = 0;
            __syncthreads();
            for (int ck = ck0 + tid; ck < min(ck_end, ck0 + kMaxDone); ck += kThreads) {
                const int lo = max(rg_begin, ck * kChunkRgs), hi = min(rg_end, (ck + 1) * kChunkRgs);
                const int size = min(L.nrg, (ck + 1) * kChunkRgs) - ck * kChunkRgs;
                const unsigned mine = (unsigned)((hi - lo) * nsl);
                const unsigned before = atomicAdd(&L.counters[ck], mine);
                if (before + mine == (unsigned)(size * L.nslices * (EXT ? L.target_mul : 1))) {
                    L.counters[ck] = 0u;
                    done[atomicAdd(ndone, 1)] = ck;
                }
            }
            __syncthreads();
            const int nd = *ndone;
            if (nd > 0) {
                __threadfence();
                constexpr int kQuads = kChunkRows / 4, kAhead = 4;
                const int nitems = nd * p.M * kQuads;
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
                            const int ckd = done[idx / (p.M * kQuads)];
                            const int rem = idx % (p.M * kQuads);
                            const int r = ckd * kChunkRows + (rem % kQuads) * 4;
                            if (r < L.out) {
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
            __syncthreads();
        }
    };
    int pend_li = -1, pend_begin = 0, pend_end = 0, pend_nsl = 0;

    while (tsk < t_end) {
        while (li + 1 < p.n && tsk >= p.lin[li + 1].task_begin) ++li;
        const MmaLinear& L = p.lin[li];
        const int tl = tsk - L.task_begin;
        const int cr = tl / L.nrg;
        const int rg_begin = tl - cr * L.nrg;
        const int rg_end = min(L.nrg, rg_begin + (t_end - tsk));
        const int s_begin = cr * p.ns;
        const int nsl = min(L.nslices, s_begin + p.ns) - s_begin;
        // The segment's 512-column tasks in (task row, slice) order, an equal run for every warp, counted in parts
        // of a task (the eight rows of one j): a run may begin and end inside a task, which both neighbours then fetch.
        // Warps that share a scheduler (w, w + 4, w + 8, ..) take neighbouring runs, so that they start a part of a
        // task apart and their set-up phases (landing, tables) do not coincide.
        const int nsub = (rg_end - rg_begin) * nsl;
        const int wperm = (wid & 3) * (W / 4) + (wid >> 2);
        const int a4 = (int)((long long)nsub * NJ * wperm / W), b4 = (int)((long long)nsub * NJ * (wperm + 1) / W);
        const int q_begin = a4 / NJ, q_end = a4 < b4 ? (b4 + NJ - 1) / NJ : q_begin;
        int rg = rg_begin + q_begin / nsl, sl = q_begin % nsl;      // this warp's first task; later ones follow by counting

        // the first task's weights may be requested before the kernel in front has finished (they are the handle's)
        const bool early = !dep_waited && p.early_weights != 0;
        if (early && q_begin < q_end) issue_task(L, rg, s_begin + sl);
        if (!dep_waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            dep_waited = true;
        }
        if (!early && q_begin < q_end) issue_task(L, rg, s_begin + sl);

        // ---- stage the segment's activations as A fragments ----
        // item = (token tile and slice msl, 8-column chunk q8, token m_lo, block bt): sixteen bytes of x become four
        // words, two per instruction (st = 2 q8, 2 q8 + 1); word (st, lane = 4 (m % 8) + bt, a = 2 (e / 2) + (m % 16) / 8)
        // holds the columns 4 st + 2 (e / 2) + {0, 1} of the block.  The low five bits of the item index are
        // (m bit 0, bt, m bit 3, m bit 1), which spreads a warp's stores over sixteen banks (two-way conflicts).
        {
            const int nitems = MT * nsl * 1024;
            const int rot = (bid & 7) * (nitems >> 3);               // CTAs that stage the same columns start at different places
            constexpr int kFly = 8;                                  // loads in flight per thread
            for (int it0 = tid; it0 < nitems; it0 += kThreads * kFly) {
                uint4 v[kFly];
                unsigned dst[kFly];
#pragma unroll
                for (int u = 0; u < kFly; ++u) {
                    const int itl = it0 + u * kThreads;
                    v[u] = make_uint4(0u, 0u, 0u, 0u);
                    dst[u] = 0u;
                    if (itl < nitems) {
                        const int it = itl + rot < nitems ? itl + rot : itl + rot - nitems;
                        const int m_lo = (it & 1) | (((it >> 4) & 1) << 1) | (((it >> 5) & 1) << 2) | (((it >> 3) & 1) << 3);
                        const int bt = (it >> 1) & 3;
                        const int q8 = (it >> 6) & 15, msl = it >> 10;
                        const int mt = (MT == 2 && msl >= nsl) ? 1 : 0, sl_ = msl - mt * nsl;
                        const int m = mt * 16 + m_lo;
                        const int col = (s_begin + sl_) * kSliceCols + bt * 128 + q8 * 8;
                        if (m < p.M && col < L.in) v[u] = ldg_x16(L.x + (size_t)m * L.in + col);
                        dst[u] = xs0 + (unsigned)((msl * 32 + 2 * q8) * 512 + (4 * (m_lo & 7) + bt) * 16 + (m_lo >> 3) * 4);
                    }
                }
#pragma unroll
                for (int u = 0; u < kFly; ++u) {
                    if (it0 + u * kThreads < nitems) {
                        asm volatile("st.shared.u32 [%0], %1;" ::"r"(dst[u]), "r"(v[u].x) : "memory");
                        asm volatile("st.shared.u32 [%0], %1;" ::"r"(dst[u] + 8u), "r"(v[u].y) : "memory");
                        asm volatile("st.shared.u32 [%0], %1;" ::"r"(dst[u] + 512u), "r"(v[u].z) : "memory");
                        asm volatile("st.shared.u32 [%0], %1;" ::"r"(dst[u] + 520u), "r"(v[u].w) : "memory");
                    }
                }
            }
        }
        // the previous segment is handed over while this segment's first weights are in flight
        if (pend_li >= 0) hand_over(p.lin[pend_li], pend_begin, pend_end, pend_nsl);
        __syncthreads();

        // ---- stream this warp's tasks ----
        float D[NJ][MT][4];
        int cur_rg = -1;
        auto flush = [&]() {
            // D[j][mt]: tokens 16 mt + g (+ 8), rows kTaskRows rg + 8 j + 2 t (+ 1)
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                const int r = cur_rg * kTaskRows + 8 * j + 2 * t;
                if (r < L.out) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const int m0 = mt * 16 + g;
                        if (m0 < p.M) atomicAdd(reinterpret_cast<float2*>(L.ws + (size_t)m0 * L.out + r), make_float2(D[j][mt][0], D[j][mt][1]));
                        if (m0 + 8 < p.M) atomicAdd(reinterpret_cast<float2*>(L.ws + (size_t)(m0 + 8) * L.out + r), make_float2(D[j][mt][2], D[j][mt][3]));
                    }
                }
            }
        };
        // candidate tables of (row group j, coefficient group gi of this lane's block), from the landing area
        auto tables_of = [&](const int j, const int gi, bpdq::ByteTables<K>& tab) {
            float c[K + 1];
#pragma unroll
            for (int i = 0; i <= K; ++i)
                c[i] = __half2float(__ushort_as_half(lds16(land0 + LD::kPlaneBytes +
                           (unsigned)(((((2 * t + gi) >> L.gsh) * (K + 1) + i) * kTaskRows + 8 * j + g) * 2))));
            bpdq::candidate_byte_tables<K>(c, tab);
        };
        auto unit_of = [&](const int rg_now, const int j, const int i, unsigned (&w)[4]) {
            const int R = j * 4 * K + t * K + i;                     // 128-byte line of the landing area; its chunks are swizzled
            const uint4 u = bpdq::unrotate_unit(lds128(land0 + (unsigned)(R * 128 + ((g ^ (R & 7)) << 4))), rg_now * kTaskRows + 8 * j + g);
            w[0] = u.x; w[1] = u.y; w[2] = u.z; w[3] = u.w;
        };
        // ---- a whole task: NJ row groups share every A fragment ----
        auto run_task = [&](const int rg_now, const int sl_now, const bool more) {
            bpdq::tma::mbar_wait(bar, landed & 1u, abort_flag, p.status);   // bounded; on expiry the status word says so and the result is void
            ++landed;
            unsigned pl[NJ][K][4];                                   // logical words of (row group j, plane i)
            bpdq::ByteTables<K> tab[NJ], tab2[G64 ? NJ : 1];         // tab2: the block's second coefficient group (g = 64)
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
#pragma unroll
                for (int i = 0; i < K; ++i) unit_of(rg_now, j, i, pl[j][i]);
                tables_of(j, 0, tab[j]);
                if (G64) tables_of(j, 1, tab2[G64 ? j : 0]);
            }
            __syncwarp();                                            // every lane has read the landing area: it may be refilled
            if (more) issue_task(L, rg, s_begin + sl);               // (rg, sl) already name the task after this one

            const unsigned xs = xs0 + (unsigned)sl_now * (32u * 512u) + (unsigned)lane * 16u;
#pragma unroll
            for (int k = 0; k < 4; ++k) {                            // 32-column words of the block
                unsigned sel[NJ][4];
#pragma unroll
                for (int j = 0; j < NJ; ++j) {
                    unsigned w[K];
#pragma unroll
                    for (int i = 0; i < K; ++i) w[i] = pl[j][i][k];
                    bpdq::code_nibbles_word<K>(w, sel[j]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    uint4 A[MT][2];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
                            A[mt][hh] = lds128_frag(xs + (unsigned)((mt * nsl * 32 + (k * 4 + u) * 2 + hh) * 512));
#pragma unroll
                    for (int jp = 0; jp < NJ; jp += 2) {             // two row groups at a time: their instructions alternate,
                        const uint4 v0 = bpdq::decode8<K>(sel[jp][u], (G64 && k >= 2) ? tab2[G64 ? jp : 0] : tab[jp]);          // so that no accumulator is used twice in a row
                        const uint4 v1 = bpdq::decode8<K>(sel[jp + 1][u], (G64 && k >= 2) ? tab2[G64 ? jp + 1 : 0] : tab[jp + 1]);
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            mma16816(D[jp][mt], A[mt][0], v0.x, v0.y);
                            mma16816(D[jp + 1][mt], A[mt][0], v1.x, v1.y);
                            mma16816(D[jp][mt], A[mt][1], v0.z, v0.w);
                            mma16816(D[jp + 1][mt], A[mt][1], v1.z, v1.w);
                        }
                    }
                }
            }
        };
        // ---- part of a task at the end of a run: the rows 8 j + g for j_lo <= j < j_hi, one j at a time (compact code:
        // a second copy of the loop above would not stay in the instruction cache); sums leave at once ----
        auto run_part = [&](const int rg_now, const int sl_now, const int j_lo, const int j_hi, const bool more) {
            bpdq::tma::mbar_wait(bar, landed & 1u, abort_flag, p.status);
            ++landed;
            const unsigned xs = xs0 + (unsigned)sl_now * (32u * 512u) + (unsigned)lane * 16u;
#pragma unroll 1
            for (int j = j_lo; j < j_hi; ++j) {
                unsigned pq[K][4];
#pragma unroll
                for (int i = 0; i < K; ++i) unit_of(rg_now, j, i, pq[i]);
                float Dq[MT][4];
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) Dq[mt][e] = 0.f;
                bpdq::ByteTables<K> tq;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (k == 0 || (G64 && k == 2)) tables_of(j, G64 ? k / 2 : 0, tq);
                    unsigned w[K], sq[4];
#pragma unroll
                    for (int i = 0; i < K; ++i) w[i] = pq[i][k];
                    bpdq::code_nibbles_word<K>(w, sq);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint4 v = bpdq::decode8<K>(sq[u], tq);
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            mma16816(Dq[mt], lds128_frag(xs + (unsigned)((mt * nsl * 32 + (k * 4 + u) * 2) * 512)), v.x, v.y);
                            mma16816(Dq[mt], lds128_frag(xs + (unsigned)((mt * nsl * 32 + (k * 4 + u) * 2 + 1) * 512)), v.z, v.w);
                        }
                    }
                }
                const int ro = rg_now * kTaskRows + 8 * j + 2 * t;
                if (ro < L.out) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const int m0 = mt * 16 + g;
                        if (m0 < p.M) atomicAdd(reinterpret_cast<float2*>(L.ws + (size_t)m0 * L.out + ro), make_float2(Dq[mt][0], Dq[mt][1]));
                        if (m0 + 8 < p.M) atomicAdd(reinterpret_cast<float2*>(L.ws + (size_t)(m0 + 8) * L.out + ro), make_float2(Dq[mt][2], Dq[mt][3]));
                    }
                }
            }
            __syncwarp();
            if (more) issue_task(L, rg, s_begin + sl);
        };
        for (int q = q_begin; q < q_end; ++q) {
            const int rg_now = rg, sl_now = sl;
            if (++sl == nsl) { sl = 0; ++rg; }                       // the task after this one
            const int j_lo = q == q_begin ? a4 - q_begin * NJ : 0, j_hi = q == q_end - 1 ? b4 - (q_end - 1) * NJ : NJ;
            if (j_lo == 0 && j_hi == NJ) {
                if (rg_now != cur_rg) {
                    if (cur_rg >= 0) flush();
                    cur_rg = rg_now;
#pragma unroll
                    for (int j = 0; j < NJ; ++j)
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int e = 0; e < 4; ++e) D[j][mt][e] = 0.f;
                }
                run_task(rg_now, sl_now, q + 1 < q_end);
            } else {
                run_part(rg_now, sl_now, j_lo, j_hi, q + 1 < q_end);
            }
        }
        if (cur_rg >= 0) flush();

        // ---- segment finished: its atomic adds are fenced, all warps are done with the A fragments ----
        __threadfence();
        __syncthreads();
        pend_li = li; pend_begin = rg_begin; pend_end = rg_end; pend_nsl = nsl;
        tsk += rg_end - rg_begin;
    }
    if (pend_li >= 0) hand_over(p.lin[pend_li], pend_begin, pend_end, pend_nsl);
}

template <int K, int MT, bool G64, int NJ, int W, bool EXT>
int launch_cfg(bpdq_handle_s* h, MmaParams p, cudaStream_t stream) {
    using LD = Land<K, G64, NJ>;
    static bpdq::SmemOptin optin;
    // as many slices per column range as fit beside the landing areas (longer ranges mean fewer atomic adds)
    int ns = 4;
    while (ns > 1 && 1024 + kMiscBytes + MT * ns * kXSliceBytes + W * LD::kBytes > h->smem_optin) ns >>= 1;
    const int smem = 1024 /*alignment slack*/ + kMiscBytes + MT * ns * kXSliceBytes + W * LD::kBytes;
    if (smem > h->smem_optin)
        return bpdq::set_error(BPDQ_ERR_UNSUPPORTED, "gemv_mma: %d bytes of shared memory needed, device offers %d", smem, h->smem_optin);
    if (const int rc = bpdq::ensure_smem_optin(gemv_mma_kernel<K, MT, G64, NJ, W, EXT>, optin, h->device, smem, "gemv_mma"); rc != BPDQ_OK) return rc;
    p.ns = ns;
    p.dyn_smem = smem;
    long long total = 0;
    int nrg[kMaxBatch], ncr[kMaxBatch];
    for (int k = 0; k < p.n; ++k) {
        MmaLinear& L = p.lin[k];
        L.nrg = (L.out + 8 * NJ - 1) / (8 * NJ);
        L.ncr = (L.nslices + ns - 1) / ns;
        L.task_begin = (int)total;
        total += (long long)L.ncr * L.nrg;
        if (total >= (1ll << 31)) return bpdq::set_error(BPDQ_ERR_UNSUPPORTED, "gemv_mma: task space too large");
        nrg[k] = L.nrg; ncr[k] = L.ncr;
    }
    int grid = h->sm_count < kMaxGrid ? h->sm_count : kMaxGrid;
    if ((long long)grid > total) grid = (int)total;
    bpdq::LaunchPlan& plan = h->plan[1];
    static_assert(sizeof(plan.t_begin) == sizeof(p.t_begin), "one cached entry per CTA boundary");
    const int key = (kSegmentCost * 8 + ns) * 8 + NJ;
    bool cached = plan.n == p.n && plan.cost == key && plan.grid == grid;
    for (int k = 0; cached && k < p.n; ++k) cached = plan.shape[k][0] == nrg[k] && plan.shape[k][1] == ncr[k];
    if (cached) {
        for (int c = 0; c <= grid; ++c) p.t_begin[c] = plan.t_begin[c];
    } else {
        bpdq::cut_task_space(nrg, ncr, p.n, grid, kSegmentCost * (4 / NJ), p.t_begin);
        plan.n = p.n; plan.cost = key; plan.grid = grid;
        for (int k = 0; k < p.n; ++k) { plan.shape[k][0] = nrg[k]; plan.shape[k][1] = ncr[k]; }
        for (int c = 0; c <= grid; ++c) plan.t_begin[c] = p.t_begin[c];
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(W * 32); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_mma_kernel<K, MT, G64, NJ, W, EXT>, p);
    h->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemv_mma launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

// Sixteen warps: eight warps with twice the registers, or 24 to 32 warps with fewer, ran within 5 % of this (the kernel is
// bound by the instruction pipes, not by latency).
template <int K>
int launch_k(bpdq_handle_s* h, const MmaParams& p, cudaStream_t stream) {
    const bool g64 = p.lin[0].group == 64;
    bool ext = false;
    for (int k = 0; k < p.n; ++k) ext = ext || p.lin[k].bias_a || p.lin[k].conv_b;
    constexpr int NJ = kRowGroups;
    if (p.M <= 16) {
        if (ext) return g64 ? launch_cfg<K, 1, true, NJ, 16, true>(h, p, stream) : launch_cfg<K, 1, false, NJ, 16, true>(h, p, stream);
        return g64 ? launch_cfg<K, 1, true, NJ, 16, false>(h, p, stream) : launch_cfg<K, 1, false, NJ, 16, false>(h, p, stream);
    }
    if (ext) return g64 ? launch_cfg<K, 2, true, NJ, 16, true>(h, p, stream) : launch_cfg<K, 2, false, NJ, 16, true>(h, p, stream);
    return g64 ? launch_cfg<K, 2, true, NJ, 16, false>(h, p, stream) : launch_cfg<K, 2, false, NJ, 16, false>(h, p, stream);
}

}  // namespace

namespace bpdq {

bool gemv_mma_supported(int out, int in, int K, int group) {
    if (!(K >= 1 && K <= 4 && (group == 64 || group == 128 || group == 256))) return false;
    return (long long)((out + 15) / 16) * ((in + kSliceCols - 1) / kSliceCols) < (1ll << 30);
}

// Tensor maps of a handle's blob for this kernel's two copies per task, encoded on the host and kept in device
// memory: plane units as (128 bytes = eight rows) x (block, plane) x (eight-row group), coefficients as rows (group,
// coefficient) of out x 2 bytes, both in 8-byte elements; boxes of one task (16 output rows x one 512-column
// slice).  Leaves d_few_maps null (and the kernel unavailable for this handle)
// when the driver has no encoder.
int few_prepare(bpdq_handle_s* h) {
    h->d_few_maps = nullptr;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return BPDQ_OK;
    const int K = h->K;
    const int ngs = 512 / h->group;
    alignas(64) CUtensorMap maps[2];
    constexpr int rows = 8 * kRowGroups;                                  // output rows of a task
    const cuuint32_t estr3[3] = {1, 1, 1};
    const cuuint64_t pd[3] = {16, (cuuint64_t)(h->in / 128) * K, (cuuint64_t)h->out / 8};
    const cuuint64_t ps[2] = {(cuuint64_t)h->out * 16, 128};
    const cuuint32_t pb[3] = {16, (cuuint32_t)(4 * K), (cuuint32_t)rows / 8};
    const cuuint64_t cd[2] = {(cuuint64_t)h->out / 4, (cuuint64_t)((h->in + h->group - 1) / h->group) * (K + 1)};
    const cuuint64_t cs[1] = {(cuuint64_t)h->out * 2};
    const cuuint32_t cb[2] = {(cuuint32_t)rows / 4, (cuuint32_t)(ngs * (K + 1))};
    const CUresult r1 = enc(&maps[0], CU_TENSOR_MAP_DATA_TYPE_UINT64, 3, h->d_blob, pd, ps, pb, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    const CUresult r2 = enc(&maps[1], CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, h->d_blob + h->planes_bytes, cd, cs, cb, estr3,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r1 != CUDA_SUCCESS || r2 != CUDA_SUCCESS)
        return set_error(BPDQ_ERR_CUDA, "bpdq_create: tensor map encode of the packed weights failed (CUresult %d, %d)", (int)r1, (int)r2);
    cudaError_t e = cudaMalloc(&h->d_few_maps, sizeof(maps));
    if (e != cudaSuccess) { h->d_few_maps = nullptr; return set_error(BPDQ_ERR_ALLOC, "bpdq_create: cudaMalloc failed (%s)", cudaGetErrorString(e)); }
    e = cudaMemcpy(h->d_few_maps, maps, sizeof(maps), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "bpdq_create: tensor map copy: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

int launch_gemv_mma_batch(bpdq_handle_s* const* hs, const void* const* xs, void* const* ys, int n, int M, cudaStream_t stream, bool pair) {
    if (n < 1 || n > kMaxBatch) return set_error(BPDQ_ERR_INVALID, "gemv_mma: %d linears in one launch (1..%d)", n, kMaxBatch);
    if (pair && (n != 2 || hs[0]->out != hs[1]->out)) return set_error(BPDQ_ERR_INVALID, "gemv_mma: a (gate, up) pair is two linears with the same rows");
    if (M < 1 || M > BPDQ_FEW_MAX_M) return set_error(BPDQ_ERR_INVALID, "gemv_mma: M=%d outside [1, %d]", M, BPDQ_FEW_MAX_M);
    MmaParams p;
    p.n = n; p.M = M;
    p.status = hs[0]->d_status;
    p.early_weights = 1;
    for (int k = 0; k < n; ++k) {
        const bpdq_handle_s* h = hs[k];
        if (h->K != hs[0]->K) return set_error(BPDQ_ERR_INVALID, "gemv_mma: linears of one launch must share K");
        if ((h->group == 64) != (hs[0]->group == 64))
            return set_error(BPDQ_ERR_INVALID, "gemv_mma: linears of one launch must all have group 64 or none of them");
        if (!h->d_few_maps)
            return set_error(BPDQ_ERR_UNSUPPORTED, "gemv_mma: linear %d has no tensor maps (the driver does not offer cuTensorMapEncodeTiled)", k);
        if ((size_t)M * h->out * sizeof(float) > h->ws_bytes)
            return set_error(BPDQ_ERR_INVALID, "gemv_mma: M=%d exceeds the workspace of linear %d (max_M=%d)", M, k, h->max_M);
        MmaLinear& L = p.lin[k];
        L.maps = static_cast<const CUtensorMap*>(h->d_few_maps);
        L.x = static_cast<const __half*>(xs[k]); L.y = static_cast<__half*>(ys[pair ? 0 : k]);
        L.ws = h->d_ws; L.counters = pair ? hs[0]->d_counters : h->d_counters;
        L.conv_a = pair ? hs[0]->d_ws : h->d_ws; L.conv_b = pair ? hs[1]->d_ws : nullptr;
        L.bias_a = static_cast<const __half*>(pair ? hs[0]->d_bias : h->d_bias);
        L.bias_b = pair ? static_cast<const __half*>(hs[1]->d_bias) : nullptr;
        L.target_mul = pair ? 2 : 1;
        L.out = h->out; L.in = h->in; L.group = h->group;
        L.gsh = h->group == 64 ? 0 : (h->group == 128 ? 1 : 2);
        L.nblocks = h->in / 128;
        L.nslices = (L.nblocks + 3) / 4;
        L.nrg = 0; L.ncr = 0; L.task_begin = 0;
        if (h->caller_blob) p.early_weights = 0;
    }
    switch (hs[0]->K) {
        case 1: return launch_k<1>(hs[0], p, stream);
        case 2: return launch_k<2>(hs[0], p, stream);
        case 3: return launch_k<3>(hs[0], p, stream);
        case 4: return launch_k<4>(hs[0], p, stream);
        default: return set_error(BPDQ_ERR_UNSUPPORTED, "gemv_mma: K=%d", hs[0]->K);
    }
}

int launch_gemv_mma(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    return launch_gemv_mma_batch(&h, &x, &y, 1, M, stream);
}

}  // namespace bpdq
