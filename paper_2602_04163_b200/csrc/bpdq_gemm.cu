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
// Roles (320 threads): warp 0 issues the TMA loads of x; warp 1 allocates TMEM and issues the
// MMAs (one lane); warps 2..9 decode in two groups of four warps, thread = output row, group 0
// taking the even 64-column stages and group 1 the odd ones (one warp per scheduler could not
// hide its own instruction latencies).  A decode thread keeps its row's plane
// units (K x 16 bytes per 128 columns, direct coalesced global loads, prefetched one block
// ahead) and the 2^K candidate values of the current group (Eq. 7, the decode rule's exact
// arithmetic) as two byte tables; eight columns cost one shift-and-mask per plane to form eight
// code nibbles and eight byte-permutes to select and interleave the binary16 bytes, then one
// 16-byte shared-memory store.  The same eight warps run the epilogue, each group on one half of
// the token columns: tcgen05.ld gives a thread its output row for 16 tokens at a time; adjacent
// threads hold adjacent output indices, so a warp writes 64 contiguous bytes of y per token.
//
// Pipeline: per stage three mbarriers -- full_b (TMA bytes landed), full_a (128 decode threads
// arrived after a proxy fence), empty (tcgen05.commit of the MMAs that read the stage) -- and one
// acc_full barrier for the epilogue.  Every wait is bounded: on expiry the thread records
// BPDQ_ERR_TIMEOUT in the handle's status word, raises a CTA-wide abort flag that lets all other
// waits fall through, and the CTA still runs to its common exit where TMEM is freed.
#include "bpdq_internal.h"
#include "bpdq_decode.cuh"

#include <cuda.h>
#include <cuda_fp16.h>

namespace {

constexpr int BM = 128;                 // output rows per CTA (MMA M)
constexpr int BK = 64;                  // columns per stage: one 128-byte swizzle row of binary16
constexpr int kDecodeGroups = 2;
constexpr int kDecodeThreads = 128;               // per group: one thread per output row
constexpr int kThreads = 64 + kDecodeGroups * kDecodeThreads;
constexpr int kATileBytes = BM * BK * 2;                       // 16 KB
constexpr unsigned kWaitLimit = 1u << 24;                      // polls of try_wait before a wait gives up

template <int BN> struct Cfg {
    static constexpr int kBTileBytes = BN * BK * 2;
    static constexpr int kStageBytes = kATileBytes + kBTileBytes;
    static constexpr int kStages = (200 * 1024) / kStageBytes > 8 ? 8 : (200 * 1024) / kStageBytes;
    static constexpr int kTmemCols = BN < 32 ? 32 : BN;        // power of two >= 32
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

struct GemmParams {
    const uint8_t* blob;
    size_t planes_bytes;
    __half* y;                // [M][out]
    int* status;
    int out, in, group, M;
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the CTA has been aborted or the limit ran out (and aborts it).
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag, int* status) {
    for (unsigned n = 0; n < kWaitLimit; ++n) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((n & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicExch(status, BPDQ_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap* map, int c0, int c1, unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
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

template <int K, int BN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap x_map, const GemmParams p) {
    using C = Cfg<BN>;
    constexpr int S = C::kStages;
    extern __shared__ unsigned char smem_raw[];
    const unsigned base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
    const unsigned a_base = base;                                  // S x 16 KB
    const unsigned b_base = base + S * kATileBytes;                // S x BN*128 bytes
    const unsigned bar_base = b_base + S * C::kBTileBytes;
    auto full_b = [&](int s) { return bar_base + 8u * s; };
    auto full_a = [&](int s) { return bar_base + 8u * (S + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * S + s); };
    const unsigned acc_full = bar_base + 8u * (3 * S);
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(smem + (bar_base - base) + 8 * (3 * S + 1));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row0 = blockIdx.x * BM;          // first output row of this CTA
    const int tok0 = blockIdx.y * BN;          // first token of this CTA
    const int nkb = p.in / BK;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_b(s), 1);
            mbar_init(full_a(s), kDecodeThreads);
            mbar_init(empty(s), 1);
        }
        mbar_init(acc_full, 1);
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
        // ---------------- TMA producer: x tiles ----------------
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % S;
                const unsigned ph = (unsigned)(kb / S) & 1u;
                if (!mbar_wait(empty(s), ph ^ 1u, abort_flag, p.status)) break;
                mbar_expect_tx(full_b(s), C::kBTileBytes);
                tma_load_2d(b_base + s * C::kBTileBytes, &x_map, kb * BK, tok0, full_b(s));
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr unsigned idesc = instr_desc_f16(BM, BN);
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % S;
                const unsigned ph = (unsigned)(kb / S) & 1u;
                ok = mbar_wait(full_a(s), ph, abort_flag, p.status) && mbar_wait(full_b(s), ph, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after();
                const uint64_t adesc = smem_desc_sw128(a_base + s * kATileBytes);
                const uint64_t bdesc = smem_desc_sw128(b_base + s * C::kBTileBytes);
#pragma unroll
                for (int k4 = 0; k4 < BK / 16; ++k4)     // 16 columns = 32 bytes further along the swizzled row
                    umma_f16(tmem_d, adesc + 2u * k4, bdesc + 2u * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
                umma_commit(empty(s));                   // frees the stage once these MMAs have read it
            }
            umma_commit(acc_full);                       // arrives when every MMA above has completed
        }
    } else {
        // ---------------- decode warps (thread = output row), then epilogue ----------------
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
        const int grp = (warp - 2) >> 2;                 // decode group: takes the stages with kb % 2 == grp
        const int rl = quad * 32 + lane;                 // row inside the tile
        const int r = row0 + rl;
        const bool row_ok = r < p.out;
        const int rr = row_ok ? r : p.out - 1;           // clamp loads of a ragged last tile (results are not stored)
        const uint8_t* cbase = p.blob + p.planes_bytes;
        const int nblocks = p.in / 128;
        const int ngroups = p.in / p.group;
        const int gstep = p.group >= 128 ? 1 : 2;        // coefficient groups between two visits of this thread
        const size_t plane_pitch = (size_t)p.out * 16;
        const size_t coef_pitch = (size_t)p.out * 2;

        uint4 unext[K];
        unsigned short cnext[K + 1];
        {
            const uint8_t* src = p.blob + (size_t)rr * 16;
#pragma unroll
            for (int i = 0; i < K; ++i) unext[i] = __ldg(reinterpret_cast<const uint4*>(src + i * plane_pitch));
            const int G0 = (grp * BK) / p.group;
            const uint8_t* cs = cbase + ((size_t)G0 * (K + 1) * p.out + rr) * 2;
#pragma unroll
            for (int i = 0; i <= K; ++i) cnext[i] = __ldg(reinterpret_cast<const unsigned short*>(cs + i * coef_pitch));
        }
        unsigned lo[2] = {0, 0}, hi[2] = {0, 0};
        int cur_group = -1;
        const unsigned a_row = (unsigned)rl * 128u;
        const unsigned sw = (unsigned)(rl & 7);
        bool ok = true;
        for (int b = 0; b < nblocks && ok; ++b) {
            unsigned cur[K][2];                          // the two logical words of this thread's half of the block
#pragma unroll
            for (int i = 0; i < K; ++i) {
                const uint4 u = bpdq::unrotate_unit(unext[i], rr);
                cur[i][0] = grp ? u.z : u.x;
                cur[i][1] = grp ? u.w : u.y;
            }
            if (b + 1 < nblocks) {
                const uint8_t* src = p.blob + ((size_t)(b + 1) * K * p.out + rr) * 16;
#pragma unroll
                for (int i = 0; i < K; ++i) unext[i] = __ldg(reinterpret_cast<const uint4*>(src + i * plane_pitch));
            }
            const int kb = 2 * b + grp;
            const int G = (kb * BK) / p.group;
            if (G != cur_group) {                        // a new coefficient group: rebuild the candidate tables
                cur_group = G;
                float c[K + 1];
#pragma unroll
                for (int i = 0; i <= K; ++i) c[i] = __half2float(__ushort_as_half(cnext[i]));
                unsigned short v[1 << K];
                bpdq::candidate_values<K>(c, v);
                bpdq::byte_tables<K>(v, lo, hi);
                if (G + gstep < ngroups) {
                    const uint8_t* cs = cbase + ((size_t)(G + gstep) * (K + 1) * p.out + rr) * 2;
#pragma unroll
                    for (int i = 0; i <= K; ++i) cnext[i] = __ldg(reinterpret_cast<const unsigned short*>(cs + i * coef_pitch));
                }
            }
            const int s = kb % S;
            const unsigned ph = (unsigned)(kb / S) & 1u;
            if (!mbar_wait(empty(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
            const unsigned dst = a_base + s * kATileBytes + a_row;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {             // eight 8-column chunks of this 64-column stage
                unsigned w[K];
#pragma unroll
                for (int i = 0; i < K; ++i) w[i] = cur[i][ch >> 2];
                const uint4 v8 = bpdq::decode8(bpdq::code_nibbles<K>(w, ch & 3), lo, hi);
                asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (((unsigned)ch ^ sw) << 4)),
                             "r"(v8.x), "r"(v8.y), "r"(v8.z), "r"(v8.w) : "memory");
            }
            fence_proxy_async();                         // make the generic-proxy stores visible to the MMA's reads
            mbar_arrive(full_a(s));
        }
        // ---------------- epilogue ----------------
        if (ok && mbar_wait(acc_full, 0u, abort_flag, p.status)) {
            tc_fence_after();
            const unsigned taddr = tmem_d + ((unsigned)(quad * 32) << 16);
#pragma unroll 1
            for (int c0 = grp * (BN / 2); c0 < (grp + 1) * (BN / 2); c0 += 16) {
                if (tok0 + c0 >= p.M) break;             // warp-uniform
                unsigned v[16];
                tmem_ld16(taddr + (unsigned)c0, v);
                tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int t = tok0 + c0 + j;
                        if (t < p.M) p.y[(size_t)t * p.out + r] = __float2half_rn(__uint_as_float(v[j]));
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, C::kTmemCols);
    }
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

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

template <int K, int BN>
int launch_tile(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    using C = Cfg<BN>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<K, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
        if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm: shared memory opt-in: %s", cudaGetErrorString(e));
        configured = true;
    }
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
    GemmParams p;
    p.blob = h->d_blob; p.planes_bytes = h->planes_bytes; p.y = static_cast<__half*>(y); p.status = h->d_status;
    p.out = h->out; p.in = h->in; p.group = h->group; p.M = M;
    const dim3 grid((h->out + BM - 1) / BM, (M + BN - 1) / BN);
    gemm_kernel<K, BN><<<grid, kThreads, C::kSmemBytes, stream>>>(map, p);
    h->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return bpdq::set_error(BPDQ_ERR_CUDA, "gemm launch: %s", cudaGetErrorString(e));
    return BPDQ_OK;
}

template <int K>
int launch_k(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    if (M <= 32) return launch_tile<K, 32>(h, x, y, M, stream);
    if (M <= 64) return launch_tile<K, 64>(h, x, y, M, stream);
    if (M <= 128) return launch_tile<K, 128>(h, x, y, M, stream);
    return launch_tile<K, 256>(h, x, y, M, stream);
}

}  // namespace

namespace bpdq {

bool gemm_supported(int, int, int K, int group) {
    return K >= 1 && K <= 3 && (group == 64 || group == 128 || group == 256);
}

int launch_gemm(bpdq_handle_s* h, const void* x, void* y, int M, cudaStream_t stream) {
    switch (h->K) {
        case 1: return launch_k<1>(h, x, y, M, stream);
        case 2: return launch_k<2>(h, x, y, M, stream);
        case 3: return launch_k<3>(h, x, y, M, stream);
        default: return set_error(BPDQ_ERR_UNSUPPORTED, "gemm: K=%d", h->K);
    }
}

}  // namespace bpdq
