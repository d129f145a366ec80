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
// Work split.  A warp task is 32 output rows x 512 input columns (a "slice" of four 128-column blocks): lane
// (g, t) = (lane / 4, lane % 4) owns the rows 8j + g (j = 0..3) of block t.  Its K plane units per row come from
// global memory by 16-byte asynchronous copies into a private landing area in shared memory one task ahead
// (eight lanes x 16 bytes = 128 contiguous bytes per block, plane and row group), the binary16 coefficients of
// the task by a few more; at the start of a task the lane moves them into registers, undoes the byte rotation of
// its rows and builds the 2^K candidate values of every (row, group) with the decode rule's exact arithmetic
// (Eq. 7: float(c0), "+ float(ci)" in plane order, one rounding to binary16), as bpdq_dequant does.  Eight
// consecutive columns then cost one shift-and-mask per plane and eight byte-permutes, and come out as four
// registers of two binary16 each -- exactly the B fragments of two mma.sync instructions.  The k index of an
// instruction is ours to assign: lane t supplies four consecutive columns of ITS block, so one instruction
// contracts 4 blocks x 4 columns, and the activations are staged in shared memory in that order, already cut
// into A fragments (one 16-byte load per lane and instruction, shared by the four row groups of the task).
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

#include <cuda_fp16.h>

namespace {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kSliceCols = 512;                       // four 128-column blocks, one per lane of a quad
constexpr int kTaskRows = 32;
constexpr int kChunkRows = 128;                       // rows per arrival counter (as in the look-up-table kernel)
constexpr int kChunkRgs = kChunkRows / kTaskRows;
constexpr int kXSliceBytes = 32 * 32 * 16;            // A fragments of one slice and 16 tokens: 32 instructions x 32 lanes x 16 bytes
constexpr int kMiscBytes = 4096;                      // completion list
constexpr int kMaxDone = 512;
constexpr int kMaxBatch = BPDQ_BATCH_MAX;
constexpr int kMaxGrid = 192;
constexpr int kSegmentCost = 2;                       // staging the activations of a segment, in (row group x column range) tasks

struct MmaLinear {
    const uint8_t* blob;
    size_t planes_bytes;
    const __half* x;          // [M][in]
    __half* y;                // [M][out]
    float* ws;                // [M][out] binary32, zero between calls
    unsigned* counters;       // one per 128 rows, zero between calls
    int out, in, group;
    int nblocks, nslices;     // 128-column blocks, 512-column slices
    int ncr, nrg;             // column ranges (of `ns` slices), 32-row groups
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

__device__ __forceinline__ void cp_async16(unsigned dst, const void* src, unsigned src_bytes) {
    // src_bytes = 0 writes sixteen zero bytes (the source is not read)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
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
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

template <int K, bool G64> struct Land {
    static constexpr int kGroups = G64 ? 2 : 1;                          // coefficient groups per block
    static constexpr int kPlaneBytes = 4 * K * 512;                      // (row group j, plane i): 32 lanes x 16 bytes
    static constexpr int kCoefChunks = 4 * kGroups * (K + 1) * 4;        // 16-byte chunks: (block, group, coefficient) x 32 rows x 2 bytes
    static constexpr int kCoefBytes = kCoefChunks * 16;
    static constexpr int kBytes = kPlaneBytes + kCoefBytes;
};

template <int K, int MT, bool G64>
__global__ void __launch_bounds__(kThreads, 1) gemv_mma_kernel(const __grid_constant__ MmaParams p) {
    using LD = Land<K, G64>;
    constexpr int NG = LD::kGroups;
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int g = lane >> 2, t = lane & 3;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool dep_waited = false;

    // shared memory: [misc][A fragments: MT x ns slices x 16 KB][landing areas: one per warp]
    int* done = reinterpret_cast<int*>(smem);
    int* ndone = done + kMaxDone;
    const unsigned smem0 = (unsigned)__cvta_generic_to_shared(smem);
    const unsigned xs0 = smem0 + kMiscBytes;
    const unsigned land0 = xs0 + (unsigned)(MT * p.ns) * kXSliceBytes + (unsigned)wid * LD::kBytes;
    if (kMiscBytes + MT * p.ns * kXSliceBytes + kWarps * LD::kBytes > p.dyn_smem) {
        if (tid == 0) atomicExch(p.status, BPDQ_ERR_UNSUPPORTED);
        return;                                                          // uniform: no barrier has been reached
    }

    const int bid = blockIdx.x;
    int tsk = p.t_begin[bid];
    const int t_end = p.t_begin[bid + 1];
    int li = 0;

    // ---- asynchronous copies of one task's packed bytes into this warp's landing area ----
    auto issue_task = [&](const MmaLinear& L, const int rg, const int s) {
        const int R0 = rg * kTaskRows;
        const int b = s * 4 + t;
        const bool b_ok = b < L.nblocks;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int r = R0 + 8 * j + g;
            const bool ok = b_ok && r < L.out;
#pragma unroll
            for (int i = 0; i < K; ++i) {
                const uint8_t* src = L.blob + (ok ? bpdq::plane_unit_offset(b, i, r, K, L.out) : (size_t)0);
                cp_async16(land0 + (unsigned)(((j * K + i) * 32 + lane) * 16), src, ok ? 16u : 0u);
            }
        }
        const uint8_t* cbase = L.blob + L.planes_bytes;
        for (int c = lane; c < LD::kCoefChunks; c += 32) {
            const int q = c & 3;                                     // rows R0 + 8q .. + 7
            const int i = (c >> 2) % (K + 1);
            const int gi = ((c >> 2) / (K + 1)) % NG;
            const int bt = (c >> 2) / ((K + 1) * NG);
            const int bb = s * 4 + bt;
            const bool ok = bb < L.nblocks && R0 + 8 * q < L.out;        // out is a multiple of 16: eight rows are inside or outside together
            const int G = ok ? (bb * 128 + gi * 64) / L.group : 0;
            const uint8_t* src = cbase + (ok ? bpdq::coef_offset(G, i, R0 + 8 * q, K, L.out) : (size_t)0);
            cp_async16(land0 + LD::kPlaneBytes + (unsigned)c * 16u, src, ok ? 16u : 0u);
        }
        cp_async_commit();
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
                if (before + mine == (unsigned)(size * L.nslices)) {
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
                    float4 v[kAhead];
                    size_t at[kAhead];
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
                                at[u] = (size_t)(rem / kQuads) * L.out + r;
                                v[u] = __ldcg(reinterpret_cast<const float4*>(L.ws + at[u]));
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < kAhead; ++u) {
                        if (live[u]) {
                            const __half2 h01 = __floats2half2_rn(v[u].x, v[u].y), h23 = __floats2half2_rn(v[u].z, v[u].w);
                            uint2 o;
                            o.x = *reinterpret_cast<const unsigned*>(&h01);
                            o.y = *reinterpret_cast<const unsigned*>(&h23);
                            *reinterpret_cast<uint2*>(L.y + at[u]) = o;
                            __stcg(reinterpret_cast<float4*>(L.ws + at[u]), make_float4(0.f, 0.f, 0.f, 0.f));
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
        // the segment's 512-column tasks in (row group, slice) order, an equal run for every warp
        const int nsub = (rg_end - rg_begin) * nsl;
        const int q_begin = (int)((long long)nsub * wid / kWarps), q_end = (int)((long long)nsub * (wid + 1) / kWarps);

        // the first task's weights may be requested before the kernel in front has finished (they are the handle's)
        const bool early = !dep_waited && p.early_weights != 0;
        if (early && q_begin < q_end) issue_task(L, rg_begin + q_begin / nsl, s_begin + q_begin % nsl);
        if (!dep_waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            dep_waited = true;
        }
        if (!early && q_begin < q_end) issue_task(L, rg_begin + q_begin / nsl, s_begin + q_begin % nsl);

        // ---- stage the segment's activations as A fragments ----
        // item = (token m, slice sl, block bt, 8-column chunk q8): sixteen bytes of x become four words, two per
        // instruction (st = 2 q8, 2 q8 + 1); word (st, lane = 4 (m % 8) + bt, a = 2 (e / 2) + (m % 16) / 8) holds the
        // columns 4 st + 2 (e / 2) + {0, 1} of the block.  The low five bits of the item index are (m bit 0, bt,
        // m bit 3, m bit 1), which spreads a warp's stores over sixteen banks (two-way conflicts).
        {
            const int nitems = MT * 16 * nsl * 64;
            for (int it0 = tid; it0 < nitems; it0 += kThreads * 4) {
                uint4 v[4];
                unsigned dst[4];
                bool live[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int it = it0 + u * kThreads;
                    live[u] = it < nitems;
                    v[u] = make_uint4(0u, 0u, 0u, 0u);
                    dst[u] = 0u;
                    if (live[u]) {
                        const int m_lo = (it & 1) | (((it >> 4) & 1) << 1) | (((it >> 5) & 1) << 2) | (((it >> 3) & 1) << 3);
                        const int bt = (it >> 1) & 3;
                        int rest = it >> 6;
                        const int q8 = rest & 15; rest >>= 4;
                        const int sl = rest % nsl;
                        const int mt = rest / nsl;
                        const int m = mt * 16 + m_lo;
                        const int col = (s_begin + sl) * kSliceCols + bt * 128 + q8 * 8;
                        if (m < p.M && col < L.in) v[u] = ldg_x16(L.x + (size_t)m * L.in + col);
                        const int ln = 4 * (m_lo & 7) + bt;
                        dst[u] = xs0 + (unsigned)(((mt * nsl + sl) * 32 + 2 * q8) * 512 + ln * 16 + (m_lo >> 3) * 4);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (live[u]) {
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
        float D[4][MT][4];
        int cur_rg = -1;
        auto flush = [&]() {
            // D[j][mt]: tokens 16 mt + g (+ 8), rows 32 rg + 8 j + 2 t (+ 1)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
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
        for (int q = q_begin; q < q_end; ++q) {
            const int rg = rg_begin + q / nsl, sl = q % nsl;
            if (rg != cur_rg) {
                if (cur_rg >= 0) flush();
                cur_rg = rg;
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) D[j][mt][e] = 0.f;
            }
            // the task's packed bytes: landing area -> registers
            cp_async_wait_all();
            __syncwarp();                                            // the coefficient chunks were copied by other lanes
            unsigned pl[4][K][4];                                    // logical words of (row group j, plane i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = rg * kTaskRows + 8 * j + g;
#pragma unroll
                for (int i = 0; i < K; ++i) {
                    const uint4 u = bpdq::unrotate_unit(lds128(land0 + (unsigned)(((j * K + i) * 32 + lane) * 16)), r);
                    pl[j][i][0] = u.x; pl[j][i][1] = u.y; pl[j][i][2] = u.z; pl[j][i][3] = u.w;
                }
            }
            unsigned short cb[4][NG][K + 1];
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int gi = 0; gi < NG; ++gi)
#pragma unroll
                    for (int i = 0; i <= K; ++i)
                        cb[j][gi][i] = lds16(land0 + LD::kPlaneBytes + (unsigned)((((t * NG + gi) * (K + 1) + i) * 32 + 8 * j + g) * 2));
            __syncwarp();                                            // every lane has read the landing area: it may be refilled
            if (q + 1 < q_end) issue_task(L, rg_begin + (q + 1) / nsl, s_begin + (q + 1) % nsl);

            const unsigned xs = xs0 + (unsigned)sl * (32u * 512u) + (unsigned)lane * 16u;
            bpdq::ByteTables<K> tab[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {                            // 32-column words of the block
                if (k == 0 || (G64 && k == 2)) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float c[K + 1];
#pragma unroll
                        for (int i = 0; i <= K; ++i) c[i] = __half2float(__ushort_as_half(cb[j][G64 ? k / 2 : 0][i]));
                        bpdq::candidate_byte_tables<K>(c, tab[j]);
                    }
                }
                unsigned sel[4][4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
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
                    for (int j = 0; j < 4; ++j) {
                        const uint4 v = bpdq::decode8<K>(sel[j][u], tab[j]);
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            mma16816(D[j][mt], A[mt][0], v.x, v.y);
                            mma16816(D[j][mt], A[mt][1], v.z, v.w);
                        }
                    }
                }
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

template <int K, int MT, bool G64>
int launch_cfg(bpdq_handle_s* h, MmaParams p, cudaStream_t stream) {
    using LD = Land<K, G64>;
    static bpdq::SmemOptin optin;
    // as many slices per column range as fit beside the landing areas (longer ranges mean fewer atomic adds)
    int ns = 4;
    while (ns > 1 && kMiscBytes + MT * ns * kXSliceBytes + kWarps * LD::kBytes > h->smem_optin) ns >>= 1;
    const int smem = kMiscBytes + MT * ns * kXSliceBytes + kWarps * LD::kBytes;
    if (smem > h->smem_optin)
        return bpdq::set_error(BPDQ_ERR_UNSUPPORTED, "gemv_mma: %d bytes of shared memory needed, device offers %d", smem, h->smem_optin);
    if (const int rc = bpdq::ensure_smem_optin(gemv_mma_kernel<K, MT, G64>, optin, h->device, smem, "gemv_mma"); rc != BPDQ_OK) return rc;
    p.ns = ns;
    p.dyn_smem = smem;
    long long total = 0;
    int nrg[kMaxBatch], ncr[kMaxBatch];
    for (int k = 0; k < p.n; ++k) {
        MmaLinear& L = p.lin[k];
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
    bool cached = plan.n == p.n && plan.cost == kSegmentCost * 8 + ns && plan.grid == grid;
    for (int k = 0; cached && k < p.n; ++k) cached = plan.shape[k][0] == nrg[k] && plan.shape[k][1] == ncr[k];
    if (cached) {
        for (int c = 0; c <= grid; ++c) p.t_begin[c] = plan.t_begin[c];
    } else {
        bpdq::cut_task_space(nrg, ncr, p.n, grid, kSegmentCost, p.t_begin);
        plan.n = p.n; plan.cost = kSegmentCost * 8 + ns; plan.grid = grid;
        for (int k = 0; k < p.n; ++k) { plan.shape[k][0] = nrg[k]; plan.shape[k][1] = ncr[k]; }
        for (int c = 0; c <= grid; ++c) plan.t_begin[c] = p.t_begin[c];
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_mma_kernel<K, MT, G64>, p);
    h->launches += 1;
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemv_mma launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

template <int K>
int launch_k(bpdq_handle_s* h, const MmaParams& p, cudaStream_t stream) {
    const bool g64 = p.lin[0].group == 64;
    if (p.M <= 16) return g64 ? launch_cfg<K, 1, true>(h, p, stream) : launch_cfg<K, 1, false>(h, p, stream);
    return g64 ? launch_cfg<K, 2, true>(h, p, stream) : launch_cfg<K, 2, false>(h, p, stream);
}

}  // namespace

namespace bpdq {

bool gemv_mma_supported(int out, int in, int K, int group) {
    if (!(K >= 1 && K <= 4 && (group == 64 || group == 128 || group == 256))) return false;
    return (long long)((out + kTaskRows - 1) / kTaskRows) * ((in + kSliceCols - 1) / kSliceCols) < (1ll << 30);
}

int launch_gemv_mma_batch(bpdq_handle_s* const* hs, const void* const* xs, void* const* ys, int n, int M, cudaStream_t stream) {
    if (n < 1 || n > kMaxBatch) return set_error(BPDQ_ERR_INVALID, "gemv_mma: %d linears in one launch (1..%d)", n, kMaxBatch);
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
        if ((size_t)M * h->out * sizeof(float) > h->ws_bytes)
            return set_error(BPDQ_ERR_INVALID, "gemv_mma: M=%d exceeds the workspace of linear %d (max_M=%d)", M, k, h->max_M);
        MmaLinear& L = p.lin[k];
        L.blob = h->d_blob; L.planes_bytes = h->planes_bytes;
        L.x = static_cast<const __half*>(xs[k]); L.y = static_cast<__half*>(ys[k]);
        L.ws = h->d_ws; L.counters = h->d_counters;
        L.out = h->out; L.in = h->in; L.group = h->group;
        L.nblocks = h->in / 128;
        L.nslices = (L.nblocks + 3) / 4;
        L.nrg = (h->out + kTaskRows - 1) / kTaskRows;
        L.ncr = 0; L.task_begin = 0;
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
