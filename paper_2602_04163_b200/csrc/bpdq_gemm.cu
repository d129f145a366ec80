// bpdq_gemm: prefill evaluation of y = x * W^T on the tensor cores (tcgen05, accumulators in TMEM).
//
// The contraction is dense once W^ (Eq. 1) exists as binary16, so the kernel rebuilds W^ tile by
// tile in shared memory and feeds it to tcgen05.mma:
//
//   D[r, t] (128 output rows x BN tokens, binary32 in TMEM) += A[r, k] * B[t, k]
//   A = W^ tile, 128 rows x 64 columns per stage, decoded on the fly (operand from shared memory)
//   B = x tile, BN tokens x 64 columns per stage, brought in by TMA (x is [M][in]: K-major as is)
//
// Both operand tiles use the canonical K-major layout with 128-byte swizzle: a row is 128 bytes
// (64 binary16), rows are 128 bytes apart, eight rows form a 1024-byte swizzle atom, and the
// 16-byte chunk c of row r is stored at chunk position c ^ (r mod 8).  TMA writes that layout by
// itself; the decode threads reproduce it by hand.
//
// Roles (320 threads; the tile kernel has a second MMA-issuing warp, 352): warp 0 is the producer (one lane: TMA
// loads of x and of the packed weights); warp 1 allocates TMEM and issues the MMAs (one lane); eight warps decode in two groups of four
// warps, thread = output row, group 0 taking the even 128-column blocks (two stages each) and
// group 1 the odd ones (one warp per scheduler could not hide its own instruction latencies).
// The packed planes and coefficients come through the pipeline as well, so that no decode thread
// ever waits on global memory: in the tile kernel a block's K plane segments (128 rows x 16 bytes)
// are one box of a tensor map over the blob's planes and its coefficient segments (128 rows x
// 2 bytes) one box of a map over the coefficients -- two copies per block whatever K is (the TMA
// unit takes about 55 ns per copy however small, and 2K+1 bulk copies per block made the kernel
// slower with every plane); the persistent kernel issues bulk copies per segment.
// A decode thread reads its row's units and coefficients from the stage, builds the 2^K
// candidate values of the group (Eq. 7, the decode rule's exact arithmetic) as two byte tables,
// and then eight columns cost one shift-and-mask per plane to form eight
// code nibbles and eight byte-permutes to select and interleave the binary16 bytes, then one
// 16-byte shared-memory store.  The same eight warps run the epilogue, each group on one half of
// the token columns: tcgen05.ld gives a thread its output row for 16 tokens at a time; adjacent
// threads hold adjacent output indices, so a warp writes 64 contiguous bytes of y per token.
//
// Three kernels share this scheme: gemm_kernel (one output tile per CTA; token tiles of 16..128, two CTAs per SM
// and a split over the input dimension when tokens are few), gemm_persistent_kernel (129..256 tokens: token tile 256,
// one CTA per SM walks over tiles, two TMEM accumulators, separate epilogue warps; described at its definition) and
// gemm_wide_kernel (more than 256 tokens: token tile 512, two issuing warps; bpdq_gemm_wide.cuh).
//
// Pipeline of the tile kernel: three rings, each with full / empty mbarriers -- packed blocks (full_p by the
// copies' bytes, empty_p by one arrival per decode warp once the block is in registers), x tiles (full_b by
// the TMA's bytes, empty_b by tcgen05.commit) and A tiles (full_a by one arrival per decode warp after a proxy
// fence, empty_a by tcgen05.commit of the MMAs that read the slot); the persistent kernel keeps one ring with
// four barriers per stage (full_b, full_p, full_a of 128 arrivals, empty).  Both have one
// acc_full barrier for the epilogue.  Every wait is bounded: on expiry the thread records
// BPDQ_ERR_TIMEOUT in the handle's status word, raises a CTA-wide abort flag that lets all other
// waits fall through, and the CTA still runs to its common exit where TMEM is freed.
#include "bpdq_internal.h"
#include "bpdq_decode.cuh"
#include "bpdq_tma.cuh"

#include <cuda.h>
#include <cuda_fp16.h>

namespace {

constexpr int BM = 128;                 // output rows per CTA (MMA M)
constexpr int BK = 64;                  // columns per stage: one 128-byte swizzle row of binary16
constexpr int kDecodeGroups = 2;
constexpr int kDecodeThreads = 128;               // per group: one thread per output row
constexpr int kThreads = 64 + kDecodeGroups * kDecodeThreads;
constexpr int kTileThreads = 96 + kDecodeGroups * kDecodeThreads;   // tile kernel: producer warp, two MMA-issuing warps, eight decode warps
constexpr int kATileBytes = BM * BK * 2;                       // 16 KB

template <int K, int BN> struct Cfg {
    static constexpr int kBTileBytes = BN * BK * 2;
    static constexpr int kPlaneBytes = K * BM * 16;             // K segments of 128 rows x 16 bytes
    static constexpr int kCoefBytes = (K + 1) * BM * 2;         // K+1 segments of 128 rows x 2 bytes
    static constexpr int kPackedBytes = (kPlaneBytes + kCoefBytes + 1023) / 1024 * 1024;
    static constexpr int kStageBytes = kATileBytes + kBTileBytes + kPackedBytes;
    // Few tokens (BN <= 64): the kernel is bound by the decode threads, not by the MMAs, so two CTAs share an SM
    // (half the shared memory each) and a 72B-shaped projection's row tiles run in one wave.
    static constexpr int kCtasPerSm = BN <= 64 ? 2 : 1;
    static constexpr int kSmemBudget = kCtasPerSm == 2 ? 110 * 1024 : 222 * 1024;
    static constexpr int kStages = kSmemBudget / kStageBytes > 8 ? 8 : kSmemBudget / kStageBytes;
    static constexpr int kTmemCols = BN < 32 ? 32 : BN;        // power of two >= 32
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;
};

struct GemmParams {
    const uint8_t* blob;
    size_t planes_bytes;
    __half* y;                // [M][out]
    int* status;
    int out, in, group, M;
    // split over the input dimension (few tokens, fewer row tiles than SMs): gridDim.z CTAs share an output tile,
    // each takes kb_per stages, adds its partial tile into `ws` and the last to arrive writes y
    int kb_per;               // stages per CTA (even: a 128-column block is never cut)
    float* ws;                // [M][out] binary32, zero between calls (only used when gridDim.z > 1)
    unsigned* counters;       // one arrival counter per 128-row tile, zero between calls
    const __half* bias;       // binary16 [out] added before the rounding, or null
};

// ---- PTX wrappers (mbarrier and TMA ones live in bpdq_tma.cuh) ------------------------------
using namespace bpdq::tma;
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(unsigned dst_smem, unsigned cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, unsigned cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_f16(unsigned d_tmem, uint64_t adesc, uint64_t bdesc, unsigned idesc, unsigned accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(unsigned taddr, unsigned (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile with 128-byte swizzle whose rows are 128
// bytes apart: start address / 16 in bits 0..13, leading byte offset (unused by swizzled K-major
// layouts) 1 in bits 16..29, stride byte offset 1024 / 16 (distance between 8-row groups) in
// bits 32..45, descriptor version 1 in bits 46..47, layout type 2 (128-byte swizzle) in bits 61..63.
__device__ __forceinline__ uint64_t smem_desc_sw128(unsigned addr) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor of kind::f16: D binary32 (bits 4..5 = 1), A and B binary16 (0), both
// K-major (bits 15, 16 = 0), N / 8 in bits 17..22, M / 16 in bits 24..28.
__host__ __device__ constexpr unsigned instr_desc_f16(int m, int n) {
    return (1u << 4) | ((unsigned)(n >> 3) << 17) | ((unsigned)(m >> 4) << 24);
}

// Ring depths of the tile kernel.  Its three operand streams have very different sizes per 64-column stage -- 16 KB of
// decoded weights (A), BN x 128 bytes of activations (B), about 2.5 KB of packed planes and coefficients -- and very
// different latencies (A is produced on the SM, B comes from L2, the packed bytes from HBM), so each has its own
// ring: a few A slots, more B slots, and packed 128-column blocks several stages ahead.
template <int K, int BN> struct TileCfg {
    static constexpr int kBTileBytes = BN * BK * 2;
    static constexpr int kPlaneBytes = K * BM * 16;             // K segments of 128 rows x 16 bytes
    static constexpr int kCoefBytes = (K + 1) * BM * 2;         // K+1 segments of 128 rows x 2 bytes: one coefficient group
    static constexpr int kBlockBytes = (kPlaneBytes + 2 * kCoefBytes + 1023) / 1024 * 1024;   // a block's planes and up to two groups (g = 64)
    static constexpr int kCtasPerSm = 2;                        // bound by the decode threads, so two CTAs share an SM (128 tokens: with two x slots)
    static constexpr int kSmemBudget = 111 * 1024;
    // One thread issues a tcgen05.mma every 160 clocks or so whatever its shape, while the pipe could take one of these
    // few-column MMAs every 40 to 50 clocks: up to 64 tokens two warps issue, stage `it` going to issuer it % 2, each into
    // an accumulator of its own (added up in the epilogue).  A parity wait is only safe on consecutive phases, so every
    // barrier must always be waited on by the same thread or group: the ring lengths are multiples of the issuer count
    // and of the number of decode groups (each group then owns two A slots and every other packed slot).  With one
    // issuer the A ring may have three slots although the groups then share them: a group that waits for the release of
    // use u of a slot (stage it) has, for the stage it stored before (it - 1 or it - 3), already waited for an MMA no
    // earlier than it - 6, the one that ended use u - 2; MMAs complete in order, so the wait is on the next phase.
    static constexpr int kIssuers = BN <= 64 ? 2 : 1;
    static constexpr int kSA = kIssuers == 2 ? 4 : 3;
    static constexpr int kSB = BN <= 16 ? 8 : (BN <= 32 ? (K <= 3 ? 6 : 4) : 2);
    static constexpr int kRest = kSmemBudget - kSA * kATileBytes - kSB * kBTileBytes - 2048;
    static constexpr int kSP = (kRest / kBlockBytes > 8 ? 8 : kRest / kBlockBytes) / kDecodeGroups * kDecodeGroups;
    static_assert(kSP >= 2, "at least two packed blocks in flight");
    static_assert(kSA % kIssuers == 0 && kSB % kIssuers == 0, "all uses of a slot go to one issuer");
    static constexpr int kAccCols = kIssuers * BN;
    static constexpr int kTmemCols = kAccCols <= 32 ? 32 : (kAccCols <= 64 ? 64 : (kAccCols <= 128 ? 128 : 256));   // power of two >= 32
    static constexpr int kSmemBytes = kSA * kATileBytes + kSB * kBTileBytes + kSP * kBlockBytes + 1024 /*alignment slack*/ + 1024 /*barriers*/;
};

template <int K, int BN>
__global__ void __launch_bounds__(kTileThreads, TileCfg<K, BN>::kCtasPerSm)
gemm_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap planes_map,
            const __grid_constant__ CUtensorMap coefs_map, const GemmParams p) {
    using C = TileCfg<K, BN>;
    constexpr int SA = C::kSA, SB = C::kSB, SP = C::kSP, NI = C::kIssuers;
    extern __shared__ unsigned char smem_raw[];
    const unsigned base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
    const unsigned a_base = base;                                  // SA x 16 KB
    const unsigned b_base = a_base + SA * kATileBytes;             // SB x BN*128 bytes
    const unsigned p_base = b_base + SB * C::kBTileBytes;          // SP x (planes, coefficients) of a 128-column block
    const unsigned bar_base = p_base + SP * C::kBlockBytes;
    auto full_a = [&](int s) { return bar_base + 8u * s; };
    auto empty_a = [&](int s) { return bar_base + 8u * (SA + s); };
    auto full_b = [&](int s) { return bar_base + 8u * (2 * SA + s); };
    auto empty_b = [&](int s) { return bar_base + 8u * (2 * SA + SB + s); };
    auto full_p = [&](int s) { return bar_base + 8u * (2 * SA + 2 * SB + s); };
    auto empty_p = [&](int s) { return bar_base + 8u * (2 * SA + 2 * SB + SP + s); };
    constexpr int kBars = 2 * SA + 2 * SB + 2 * SP;
    const unsigned acc_full = bar_base + 8u * kBars;
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(smem + (bar_base - base) + 8 * (kBars + 1));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row0 = blockIdx.x * BM;          // first output row of this CTA
    const int tok0 = blockIdx.y * BN;          // first token of this CTA
    const int kb0 = blockIdx.z * p.kb_per;           // this CTA's stages: [kb0, kb1) of the in / 64 stages of the row
    const int kb1 = min(p.in / BK, kb0 + p.kb_per);
    const int nst = kb1 - kb0;                       // even: whole 128-column blocks
    const int b0 = kb0 / 2, nblk = nst / 2;
    const int ng = p.group == 64 ? 2 : 1;            // coefficient groups per block

    if (tid == 0) {
        for (int s = 0; s < SA; ++s) { mbar_init(full_a(s), kDecodeThreads / 32); mbar_init(empty_a(s), 1); }   // one arrival per decode warp
        for (int s = 0; s < SB; ++s) { mbar_init(full_b(s), 1); mbar_init(empty_b(s), 1); }
        for (int s = 0; s < SP; ++s) { mbar_init(full_p(s), 1); mbar_init(empty_p(s), kDecodeThreads / 32); }
        mbar_init(acc_full, NI);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = *tmem_slot;

    if (warp == 0) {
        // ---------------- producer: packed blocks (bulk copies) and x tiles (TMA), each as its ring has room ----------------
        if (lane == 0) {
            // A block's K plane segments (128 rows x 16 bytes each) are one box of the planes' tensor map, its one or two
            // coefficient groups one box of the coefficients' map: two copies per block, whatever K is.  Rows past a
            // ragged last tile are filled with zeros (and count as received bytes).
            int pb = 0, xb = 0;                          // next packed block, next x stage
            unsigned idle = 0;
            unsigned long long idle_since = 0;
            while (pb < nblk || xb < nst) {
                bool moved = false;
                if (pb < nblk && mbar_try_wait(empty_p(pb % SP), ((unsigned)(pb / SP) & 1u) ^ 1u)) {
                    const int sp = pb % SP, b = b0 + pb;
                    mbar_expect_tx(full_p(sp), (unsigned)(C::kPlaneBytes + ng * C::kCoefBytes));
                    const unsigned pdst = p_base + sp * C::kBlockBytes;
                    tma_load_2d(pdst, &planes_map, row0 * 2, b * K, full_p(sp));                 // 8-byte elements: 2 per row
                    tma_load_2d(pdst + C::kPlaneBytes, &coefs_map, row0 / 4, ((b * 128) / p.group) * (K + 1), full_p(sp));
                    ++pb;
                    moved = true;
                }
                if (xb < nst && mbar_try_wait(empty_b(xb % SB), ((unsigned)(xb / SB) & 1u) ^ 1u)) {
                    const int sb = xb % SB;
                    mbar_expect_tx(full_b(sb), C::kBTileBytes);
                    tma_load_2d(b_base + sb * C::kBTileBytes, &x_map, (kb0 + xb) * BK, tok0, full_b(sb));
                    ++xb;
                    moved = true;
                }
                if (moved) {
                    idle = 0;
                } else if (++idle == 1) {
                    idle_since = global_ns();
                } else if ((idle & 63u) == 63u) {
                    if (*abort_flag) break;
                    if (global_ns() - idle_since > kWaitNanos) {   // neither ring has freed a slot for too long
                        *abort_flag = 1;
                        atomicExch(p.status, BPDQ_ERR_TIMEOUT);
                        break;
                    }
                }
            }
        }
    } else if (warp <= 2) {
        // ---------------- MMA issuers: warp 1 + j takes the stages it % NI == j, into accumulator j ----------------
        if (lane == 0 && warp <= NI) {
            constexpr unsigned idesc = instr_desc_f16(BM, BN);
            const int j = warp - 1;
            for (int it = j; it < nst; it += NI) {
                const int sa = it % SA, sb = it % SB;
                if (!mbar_wait(full_a(sa), (unsigned)(it / SA) & 1u, abort_flag, p.status) ||
                    !mbar_wait(full_b(sb), (unsigned)(it / SB) & 1u, abort_flag, p.status))
                    break;
                tc_fence_after();
                const uint64_t adesc = smem_desc_sw128(a_base + sa * kATileBytes);
                const uint64_t bdesc = smem_desc_sw128(b_base + sb * C::kBTileBytes);
#pragma unroll
                for (int k4 = 0; k4 < BK / 16; ++k4)     // 16 columns = 32 bytes further along the swizzled row
                    umma_f16(tmem_d + (unsigned)(j * BN), adesc + 2u * k4, bdesc + 2u * k4, idesc, (it >= NI || k4 != 0) ? 1u : 0u);
                umma_commit(empty_a(sa));                // each frees its slot once these MMAs have read it
                umma_commit(empty_b(sb));
            }
            umma_commit(acc_full);                       // arrives when every MMA of this issuer has completed
        }
    } else {
        // ---------------- decode warps (thread = output row), then epilogue ----------------
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
        const int grp = (warp - 3) >> 2;                 // decode group: takes every other 128-column block
        const int rl = quad * 32 + lane;                 // row inside the tile
        const int r = row0 + rl;
        const bool row_ok = r < p.out;                   // rows past a ragged last tile decode stale bytes; nothing of theirs is stored
        unsigned a_off[8];                               // swizzled byte offset of each 16-byte chunk of this thread's row
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) a_off[ch] = (unsigned)rl * 128u + (((unsigned)ch ^ (unsigned)(rl & 7)) << 4);
        bool ok = true;
        for (int bi = grp; bi < nblk && ok; bi += kDecodeGroups) {
            const int sp = bi % SP;
            if (!mbar_wait(full_p(sp), (unsigned)(bi / SP) & 1u, abort_flag, p.status)) { ok = false; break; }
            const unsigned psrc = p_base + sp * C::kBlockBytes;
            unsigned cur[K][4];                          // logical words of this row's plane units
#pragma unroll
            for (int i = 0; i < K; ++i) {
                uint4 raw;
                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(raw.x), "=r"(raw.y), "=r"(raw.z), "=r"(raw.w)
                             : "r"(psrc + i * (BM * 16) + rl * 16));
                const uint4 u = bpdq::unrotate_unit(raw, r);
                cur[i][0] = u.x; cur[i][1] = u.y; cur[i][2] = u.z; cur[i][3] = u.w;
            }
            unsigned short cbits[2][K + 1];              // coefficients of the block's one or two groups
#pragma unroll
            for (int gg = 0; gg < 2; ++gg)
#pragma unroll
                for (int i = 0; i <= K; ++i) {
                    cbits[gg][i] = 0;
                    if (gg < ng)
                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(cbits[gg][i])
                                     : "r"(psrc + C::kPlaneBytes + gg * C::kCoefBytes + i * (BM * 2) + rl * 2));
                }
            __syncwarp();                                // every lane's loads have returned (their results were used above)
            if (lane == 0) mbar_arrive(empty_p(sp));     // the block's packed bytes are in registers: its slot may be refilled
            bpdq::ByteTables<K> tab;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int it = 2 * bi + half;
                const int sa = it % SA;
                if (half == 0 || ng == 2) {              // candidate tables of the coefficient group that starts here
                    float c[K + 1];
#pragma unroll
                    for (int i = 0; i <= K; ++i) c[i] = __half2float(__ushort_as_half(cbits[ng == 2 ? half : 0][i]));
                    bpdq::candidate_byte_tables<K>(c, tab);
                }
                // decode the stage's 64 columns into registers first (eight independent chains the compiler can interleave,
                // and nothing of it waits for the slot), then wait for the slot and store
                uint4 v8[8];
#pragma unroll
                for (int wd = 0; wd < 2; ++wd) {         // two 32-column words per 64-column stage
                    unsigned w[K], sel[4];
#pragma unroll
                    for (int i = 0; i < K; ++i) w[i] = cur[i][2 * half + wd];
                    bpdq::code_nibbles_word<K>(w, sel);
#pragma unroll
                    for (int u = 0; u < 4; ++u) v8[4 * wd + u] = bpdq::decode8<K>(sel[u], tab);
                }
                if (!mbar_wait(empty_a(sa), ((unsigned)(it / SA) & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
                const unsigned dst = a_base + sa * kATileBytes;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + a_off[ch]),
                                 "r"(v8[ch].x), "r"(v8[ch].y), "r"(v8[ch].z), "r"(v8[ch].w) : "memory");
                fence_proxy_async();                     // make the generic-proxy stores visible to the MMA's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(full_a(sa));  // one arrival per warp, after all its lanes' stores and fences
            }
        }
        // ---------------- epilogue: each decode group takes half of the token columns (all of them when there are only 16) ----------------
        constexpr int kColsPerGroup = BN >= 32 ? BN / 2 : BN;
        if (ok && (BN >= 32 || grp == 0) && mbar_wait(acc_full, 0u, abort_flag, p.status)) {
            tc_fence_after();
            const unsigned taddr = tmem_d + ((unsigned)(quad * 32) << 16);
#pragma unroll 1
            for (int c0 = grp * kColsPerGroup; c0 < (grp + 1) * kColsPerGroup; c0 += 16) {
                if (tok0 + c0 >= p.M) break;             // warp-uniform
                float acc[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] = 0.f;
#pragma unroll
                for (int a = 0; a < NI; ++a) {           // the issuers' accumulators, in a fixed order (every issuer has a stage: nst >= 2)
                    unsigned v[16];
                    tmem_ld16(taddr + (unsigned)(a * BN + c0), v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) acc[j] += __uint_as_float(v[j]);
                }
                if (row_ok) {
                    const float br = (p.bias && gridDim.z == 1) ? __half2float(p.bias[r]) : 0.f;   // a shared tile gets it when it is completed
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int t = tok0 + c0 + j;
                        if (t < p.M) {
                            if (gridDim.z > 1) atomicAdd(p.ws + (size_t)t * p.out + r, acc[j]);
                            else p.y[(size_t)t * p.out + r] = __float2half_rn(acc[j] + br);
                        }
                    }
                }
            }
        }
    }
    if (gridDim.z > 1) __threadfence();              // this thread's partial sums are out before the tile's counter moves
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, C::kTmemCols);
    }
    if (gridDim.z > 1) {
        // the last of the CTAs that share this output tile rounds it to binary16, writes y and zeroes the workspace
        int* last = reinterpret_cast<int*>(const_cast<int*>(abort_flag)) + 1;
        if (tid == 0) {
            const unsigned before = atomicAdd(p.counters + blockIdx.x, 1u);
            *last = before == gridDim.z - 1;
            if (*last) p.counters[blockIdx.x] = 0u;
        }
        __syncthreads();
        if (*last) {
            __threadfence();
            const int ntok = min(BN, p.M - tok0);
            for (int idx = tid; idx < ntok * BM; idx += kTileThreads) {
                const int t = tok0 + idx / BM, r = row0 + idx % BM;
                if (r < p.out) {
                    float* src = p.ws + (size_t)t * p.out + r;
                    p.y[(size_t)t * p.out + r] = __float2half_rn(__ldcg(src) + (p.bias ? __half2float(p.bias[r]) : 0.f));
                    __stcg(src, 0.f);
                }
            }
        }
    }
}

// ---- persistent variant for many tokens (token tile 256) -------------------------------------------------
// One CTA per SM walks over output tiles (row tile fastest, so that the CTAs running together share one
// 256-token slab of x in L2).  TMEM holds two 128 x 256 accumulators: while four epilogue warps drain one, the
// MMA warp fills the other, and the producer and decode warps run straight on into the next tile's stages.
// Roles (448 threads): warp 0 producer, warp 1 MMA, warps 2..9 decode (two groups, as above), warps 10..13
// epilogue.  Barriers: the four per-stage barriers of the kernel above, used over one stage sequence that
// continues across tiles, plus acc_full[2] (tcgen05.commit after a tile's last MMA) and acc_empty[2]
// (128 epilogue threads after they have read the accumulator).
constexpr int kPersistThreads = 64 + kDecodeGroups * kDecodeThreads + 128;
constexpr int kPersistBN = 256;

template <int K>
__global__ void __launch_bounds__(kPersistThreads, 1)
gemm_persistent_kernel(const __grid_constant__ CUtensorMap x_map, const GemmParams p) {
    constexpr int BN = kPersistBN;
    using C = Cfg<K, BN>;
    constexpr int S = C::kStages;
    extern __shared__ unsigned char smem_raw[];
    const unsigned base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
    const unsigned a_base = base;
    const unsigned b_base = base + S * kATileBytes;
    const unsigned p_base = b_base + S * C::kBTileBytes;
    const unsigned bar_base = p_base + S * C::kPackedBytes;
    auto full_b = [&](int s) { return bar_base + 8u * s; };
    auto full_a = [&](int s) { return bar_base + 8u * (S + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * S + s); };
    auto full_p = [&](int s) { return bar_base + 8u * (3 * S + s); };
    auto acc_full = [&](int b) { return bar_base + 8u * (4 * S + b); };
    auto acc_empty = [&](int b) { return bar_base + 8u * (4 * S + 2 + b); };
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(smem + (bar_base - base) + 8 * (4 * S + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nkb = p.in / BK;
    const int nrt = (p.out + BM - 1) / BM;            // row tiles
    const int ntt = (p.M + BN - 1) / BN;              // token tiles
    const int ntiles = nrt * ntt;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_b(s), 1);
            mbar_init(full_a(s), kDecodeThreads);
            mbar_init(empty(s), 1);
            mbar_init(full_p(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full(b), 1);
            mbar_init(acc_empty(b), 128);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_d = *tmem_slot;

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint8_t* cbase = p.blob + p.planes_bytes;
            int it = 0;                                  // stage sequence number, continues across tiles
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int row0 = (tile % nrt) * BM, tok0 = (tile / nrt) * BN;
                const int nrows = min(BM, p.out - row0);
                const unsigned seg_p = (unsigned)nrows * 16u, seg_c = (unsigned)nrows * 2u;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % S;
                    const unsigned ph = (unsigned)(it / S) & 1u;
                    if (!mbar_wait(empty(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    const bool first_half = (kb & 1) == 0;
                    mbar_expect_tx(full_p(s), (first_half ? (unsigned)K * seg_p : 0u) + (unsigned)(K + 1) * seg_c);
                    const unsigned pdst = p_base + s * C::kPackedBytes;
                    const int b = kb >> 1, G = (kb * BK) / p.group;
                    if (first_half) {
#pragma unroll
                        for (int i = 0; i < K; ++i)
                            bulk_load(pdst + i * (BM * 16), p.blob + (((size_t)b * K + i) * p.out + row0) * 16, seg_p, full_p(s));
                    }
#pragma unroll
                    for (int i = 0; i <= K; ++i)
                        bulk_load(pdst + C::kPlaneBytes + i * (BM * 2), cbase + (((size_t)G * (K + 1) + i) * p.out + row0) * 2, seg_c, full_p(s));
                    mbar_expect_tx(full_b(s), C::kBTileBytes);
                    tma_load_2d(b_base + s * C::kBTileBytes, &x_map, kb * BK, tok0, full_b(s));
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr unsigned idesc = instr_desc_f16(BM, BN);
            int it = 0, j = 0;                           // stage sequence number; tiles done by this CTA
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++j) {
                const int buf = j & 1;
                // the epilogue must have drained this accumulator (two tiles ago)
                if (!mbar_wait(acc_empty(buf), ((unsigned)(j >> 1) & 1u) ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                const unsigned d = tmem_d + (unsigned)(buf * BN);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % S;
                    const unsigned ph = (unsigned)(it / S) & 1u;
                    ok = mbar_wait(full_a(s), ph, abort_flag, p.status) && mbar_wait(full_b(s), ph, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(a_base + s * kATileBytes);
                    const uint64_t bdesc = smem_desc_sw128(b_base + s * C::kBTileBytes);
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4)
                        umma_f16(d, adesc + 2u * k4, bdesc + 2u * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
                    umma_commit(empty(s));
                }
                if (ok) umma_commit(acc_full(buf));
            }
        }
    } else if (warp < 2 + 4 * kDecodeGroups) {
        // ---------------- decode warps (thread = output row) ----------------
        const int quad = warp & 3;
        const int grp = (warp - 2) >> 2;
        const int rl = quad * 32 + lane;
        unsigned a_off[8];
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) a_off[ch] = (unsigned)rl * 128u + (((unsigned)ch ^ (unsigned)(rl & 7)) << 4);
        const int nblocks = nkb / 2;
        int it0 = 0;                                     // stage sequence number of the current tile's first stage
        bool ok = true;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, it0 += nkb) {
            const int r = (tile % nrt) * BM + rl;        // rows past a ragged last tile decode stale bytes; nothing of theirs is stored
            // A group keeps to every other block of the stage sequence ACROSS tiles (with an odd number of blocks per
            // tile its parity inside the tile flips): its waits then follow the sequence two stages at a time and
            // never run a whole ring ahead of a barrier's phase, which a parity wait could not tell from "ready".
            static_assert(kDecodeGroups == 2, "two groups alternate blocks");
            for (int b = grp ^ ((it0 >> 1) & 1); b < nblocks && ok; b += kDecodeGroups) {
                unsigned cur[K][4];
                bpdq::ByteTables<K> tab;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int it = it0 + 2 * b + half;
                    const int s = it % S;
                    const unsigned ph = (unsigned)(it / S) & 1u;
                    if (!mbar_wait(full_p(s), ph, abort_flag, p.status)) { ok = false; break; }
                    const unsigned psrc = p_base + s * C::kPackedBytes;
                    if (half == 0) {
#pragma unroll
                        for (int i = 0; i < K; ++i) {
                            uint4 raw;
                            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(raw.x), "=r"(raw.y), "=r"(raw.z), "=r"(raw.w)
                                         : "r"(psrc + i * (BM * 16) + rl * 16));
                            const uint4 u = bpdq::unrotate_unit(raw, r);
                            cur[i][0] = u.x; cur[i][1] = u.y; cur[i][2] = u.z; cur[i][3] = u.w;
                        }
                    }
                    if (half == 0 || p.group == 64) {
                        float c[K + 1];
#pragma unroll
                        for (int i = 0; i <= K; ++i) {
                            unsigned short hbits;
                            asm volatile("ld.shared.u16 %0, [%1];" : "=h"(hbits) : "r"(psrc + C::kPlaneBytes + i * (BM * 2) + rl * 2));
                            c[i] = __half2float(__ushort_as_half(hbits));
                        }
                        bpdq::candidate_byte_tables<K>(c, tab);
                    }
                    const unsigned dst = a_base + s * kATileBytes;
#pragma unroll
                    for (int wd = 0; wd < 2; ++wd) {
                        unsigned w[K], sel[4];
#pragma unroll
                        for (int i = 0; i < K; ++i) w[i] = cur[i][2 * half + wd];
                        bpdq::code_nibbles_word<K>(w, sel);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const uint4 v8 = bpdq::decode8<K>(sel[u], tab);
                            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + a_off[4 * wd + u]),
                                         "r"(v8.x), "r"(v8.y), "r"(v8.z), "r"(v8.w) : "memory");
                        }
                    }
                    fence_proxy_async();
                    mbar_arrive(full_a(s));
                }
            }
        }
    } else {
        // ---------------- epilogue warps: drain one accumulator while the other is being filled ----------------
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
        const int rl = quad * 32 + lane;
        int j = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_full(buf), (unsigned)(j >> 1) & 1u, abort_flag, p.status)) break;
            tc_fence_after();
            const int row0 = (tile % nrt) * BM, tok0 = (tile / nrt) * BN;
            const int r = row0 + rl;
            const bool row_ok = r < p.out;
            const unsigned taddr = tmem_d + ((unsigned)(quad * 32) << 16) + (unsigned)(buf * BN);
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 16) {
                if (tok0 + c0 >= p.M) break;             // warp-uniform
                unsigned v[16];
                tmem_ld16(taddr + (unsigned)c0, v);
                tmem_ld_wait();
                if (row_ok) {
                    const float br = p.bias ? __half2float(p.bias[r]) : 0.f;
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj) {
                        const int t = tok0 + c0 + jj;
                        if (t < p.M) p.y[(size_t)t * p.out + r] = __float2half_rn(__uint_as_float(v[jj]) + br);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty(buf));                 // 128 arrivals: the accumulator may be overwritten
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, 512);
    }
}

#include "bpdq_gemm_wide.cuh"

// ---- host side ------------------------------------------------------------------------------
using bpdq::EncodeTiledFn;
using bpdq::encode_tiled_fn;

// Tensor maps of the blob's planes and coefficients (one box = the K plane segments resp. the coefficient groups of a
// 128-row x 128-column block), encoded at a handle's first tensor-core launch.
template <int K>
int ensure_packed_maps(bpdq_handle_s* h, EncodeTiledFn enc) {
    if (h->gemm_maps_ready) return BPDQ_OK;
    const cuuint32_t estr[2] = {1, 1};
        // planes: rows (block, plane) of out x 16 bytes; coefficients: rows (group, coefficient) of out x 2 bytes; both
    // as 8-byte elements, so that 128 output rows are 256 resp. 32 elements (a box dimension holds at most 256)
    const int ng = h->group == 64 ? 2 : 1;
    const cuuint64_t pd[2] = {(cuuint64_t)h->out * 2, (cuuint64_t)(h->in / 128) * K};
    const cuuint64_t ps[1] = {(cuuint64_t)h->out * 16};
    const cuuint32_t pb[2] = {(cuuint32_t)BM * 2, (cuuint32_t)K};
    const cuuint64_t cd[2] = {(cuuint64_t)h->out / 4, (cuuint64_t)((h->in + h->group - 1) / h->group) * (K + 1)};
    const cuuint64_t cs[1] = {(cuuint64_t)h->out * 2};
    const cuuint32_t cb[2] = {(cuuint32_t)BM / 4, (cuuint32_t)(ng * (K + 1))};
    CUresult r1 = enc(reinterpret_cast<CUtensorMap*>(h->gemm_maps[0]), CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, h->d_blob, pd, ps, pb, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    CUresult r2 = enc(reinterpret_cast<CUtensorMap*>(h->gemm_maps[1]), CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, h->d_blob + h->planes_bytes, cd, cs, cb,
                      estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r1 != CUDA_SUCCESS || r2 != CUDA_SUCCESS)
        return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: tensor map encode of the packed weights failed (CUresult %d, %d)", (int)r1, (int)r2);
    h->gemm_maps_ready = 1;
    return BPDQ_OK;
}

template <int K, int BN>
int launch_tile(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    using C = TileCfg<K, BN>;
    static bpdq::SmemOptin optin;
    if (const int rc = bpdq::ensure_smem_optin(gemm_kernel<K, BN>, optin, h->device, C::kSmemBytes, "gemm"); rc != BPDQ_OK) return rc;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: cuTensorMapEncodeTiled is not available from this driver");
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)h->in, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)h->in * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BN};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: tensor map encode failed (CUresult %d)", (int)cr);
    if (const int rc = ensure_packed_maps<K>(h, enc); rc != BPDQ_OK) return rc;
    GemmParams p;
    p.blob = h->d_blob; p.planes_bytes = h->planes_bytes; p.y = static_cast<__half*>(y); p.status = h->d_status;
    p.out = h->out; p.in = h->in; p.group = h->group; p.M = M;
    p.ws = h->d_ws; p.counters = h->d_counters; p.bias = static_cast<const __half*>(h->d_bias);
    dim3 grid((h->out + BM - 1) / BM, (M + BN - 1) / BN);
    const int nkb = h->in / BK;
    p.kb_per = nkb;
    if (grid.y == 1 && (size_t)M * h->out * sizeof(float) <= h->ws_bytes) {
        // fewer output tiles than CTA slots: split the input dimension so that every SM gets work
        const int slots = h->sm_count * C::kCtasPerSm;
        int splits = slots / (int)grid.x;
        constexpr int kMaxSplits = BN <= 32 ? 8 : 4;   // every split adds BN x 128 atomic adds per tile: fewer with many tokens
        if (splits > kMaxSplits) splits = kMaxSplits;
        if (splits > nkb / 16) splits = nkb / 16;     // at least 16 stages (1024 columns) per CTA
        if (splits > 1) {
            p.kb_per = ((nkb + splits - 1) / splits + 1) / 2 * 2;
            grid.z = (nkb + p.kb_per - 1) / p.kb_per;
        }
    }
    gemm_kernel<K, BN><<<grid, kTileThreads, C::kSmemBytes, stream>>>(map, *reinterpret_cast<const CUtensorMap*>(h->gemm_maps[0]),
                                                                   *reinterpret_cast<const CUtensorMap*>(h->gemm_maps[1]), p);
    h->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

template <int K>
int launch_persistent(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    using C = Cfg<K, kPersistBN>;
    static bpdq::SmemOptin optin;
    if (const int rc = bpdq::ensure_smem_optin(gemm_persistent_kernel<K>, optin, h->device, C::kSmemBytes, "gemm"); rc != BPDQ_OK) return rc;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: cuTensorMapEncodeTiled is not available from this driver");
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)h->in, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)h->in * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)kPersistBN};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: tensor map encode failed (CUresult %d)", (int)cr);
    GemmParams p;
    p.blob = h->d_blob; p.planes_bytes = h->planes_bytes; p.y = static_cast<__half*>(y); p.status = h->d_status;
    p.out = h->out; p.in = h->in; p.group = h->group; p.M = M;
    p.ws = h->d_ws; p.counters = h->d_counters; p.kb_per = h->in / BK; p.bias = static_cast<const __half*>(h->d_bias);
    const long long ntiles = (long long)((h->out + BM - 1) / BM) * ((M + kPersistBN - 1) / kPersistBN);
    const int grid = ntiles < h->sm_count ? (int)ntiles : h->sm_count;
    gemm_persistent_kernel<K><<<grid, kPersistThreads, C::kSmemBytes, stream>>>(map, p);
    h->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

template <int K>
int launch_wide(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    using C = WideCfg<K>;
    static bpdq::SmemOptin optin;
    if (const int rc = bpdq::ensure_smem_optin(gemm_wide_kernel<K>, optin, h->device, C::kSmemBytes, "gemm"); rc != BPDQ_OK) return rc;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: cuTensorMapEncodeTiled is not available from this driver");
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)h->in, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)h->in * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kWideBK, 256};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), dims, strides, box, estr,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: tensor map encode failed (CUresult %d)", (int)cr);
    if (const int rc = ensure_packed_maps<K>(h, enc); rc != BPDQ_OK) return rc;
    GemmParams p;
    p.blob = h->d_blob; p.planes_bytes = h->planes_bytes; p.y = static_cast<__half*>(y); p.status = h->d_status;
    p.out = h->out; p.in = h->in; p.group = h->group; p.M = M;
    p.ws = h->d_ws; p.counters = h->d_counters; p.kb_per = h->in / kWideBK; p.bias = static_cast<const __half*>(h->d_bias);
    const long long ntiles = (long long)((h->out + BM - 1) / BM) * ((M + kWideBN - 1) / kWideBN);
    const int grid = ntiles < h->sm_count ? (int)ntiles : h->sm_count;
    gemm_wide_kernel<K><<<grid, kWideThreads, C::kSmemBytes, stream>>>(map, *reinterpret_cast<const CUtensorMap*>(h->gemm_maps[0]),
                                                                      *reinterpret_cast<const CUtensorMap*>(h->gemm_maps[1]), p);
    h->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

template <int K>
int launch_k(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    if (M <= 16) return launch_tile<K, 16>(h, x, y, M, stream);
    if (M <= 32) return launch_tile<K, 32>(h, x, y, M, stream);
    if (M <= 64) return launch_tile<K, 64>(h, x, y, M, stream);
    if (M <= 128) return launch_tile<K, 128>(h, x, y, M, stream);
    if (M <= 256) return launch_persistent<K>(h, x, y, M, stream);
    return launch_wide<K>(h, x, y, M, stream);       // 512-token tiles: measured faster than the 256-token kernel from 257 tokens on
}

// Diagnostic: the library's bounded wait on a barrier that nothing arrives at.  It must give up after its limit, record
// BPDQ_ERR_TIMEOUT in the status word and let the kernel end normally.
__global__ void wait_limit_probe_kernel(int* status) {
    __shared__ alignas(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait_ns(smem_u32(&bar), 0u, &abort_flag, status, 50000000ull);   // 50 ms here; the kernels allow two seconds
    __syncthreads();
}

}  // namespace

namespace bpdq {

int launch_wait_limit_probe(bpdq_handle_s* h, cudaStream_t stream) {
    wait_limit_probe_kernel<<<1, 32, 0, stream>>>(h->d_status);
    h->launches += 1;
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_error(BPDQ_ERR_CUDA, "probe launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

bool gemm_supported(int, int, int K, int group) {
    return K >= 1 && K <= 4 && (group == 64 || group == 128 || group == 256);
}

int launch_gemm(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    switch (h->K) {
        case 1: return launch_k<1>(h, x, y, M, stream);
        case 2: return launch_k<2>(h, x, y, M, stream);
        case 3: return launch_k<3>(h, x, y, M, stream);
        case 4: return launch_k<4>(h, x, y, M, stream);
        default: return set_error(BPDQ_ERR_UNSUPPORTED, "gemm: K=%d", h->K);
    }
}

}  // namespace bpdq
