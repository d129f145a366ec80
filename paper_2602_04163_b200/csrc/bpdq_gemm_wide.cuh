// Included by bpdq_gemm.cu (inside its unnamed namespace, after the PTX wrappers): the prefill kernel for many tokens.
//
// gemm_wide_kernel: one decoded weight stage feeds TWO 256-token halves of a 512-token tile.  The persistent
// 256-token kernel decodes every weight once per 256 tokens and one thread issues all of its MMAs; measured, a
// single thread gets a tcgen05.mma out every 155-167 clocks whatever its shape while a 128 x 256 x 16 one occupies
// the pipe for 128, and the decode's energy is what the 1 kW cap charges (every further plane costs 8-20 %).  Here
// two warps issue, each into a 128 x 256 accumulator of its own (the two halves of TMEM's 512 columns) from the
// same A stage and its own x half, so the decode work and the A-tile traffic per FLOP are halved and the issue cap
// is lifted.  TMEM is full with one tile, so the epilogue no longer overlaps the next tile's MMAs (about 3 % of a
// 72B-shaped tile's time); producer and decode warps run ahead into the next tile's stages meanwhile.
//
// Stages are 32 columns (64-byte swizzle rows): 8 KB of decoded weights and 2 x 16 KB of activations per stage, five
// stages; packed 128-column blocks (two tensor-map boxes each, as in the tile kernel) in a ring of two, one slot
// per decode group.  Roles (480 threads): warp 0 producer, warps 1-2 MMA issuers (half 0, half 1), warps 3-10
// decode (two groups of four warps, thread = output row, alternating 128-column blocks of the stage sequence, which
// continues across tiles), warps 11-14 epilogue.  Barriers per stage: full_b (bytes of both x halves), full_a (one
// arrival per warp of the owning decode group), empty (one tcgen05.commit per issuer); per packed slot: full_p,
// empty_p; acc_full (one commit per issuer), acc_empty (one arrival per epilogue warp).  All waits are bounded.
constexpr int kWideBK = 32;                                   // columns per stage: one 64-byte swizzle row of binary16
constexpr int kWideBN = 512;                                  // tokens per tile: two halves of 256
constexpr int kWideThreads = 32 * (3 + 4 * kDecodeGroups + 4);
constexpr int kWideATile = BM * kWideBK * 2;                  // 8 KB
constexpr int kWideBHalf = 256 * kWideBK * 2;                 // 16 KB
constexpr int kWideStage = kWideATile + 2 * kWideBHalf;       // 40 KB
constexpr int kWideStages = 5;
constexpr int kWideSP = 2;                                    // packed blocks in flight: one slot per decode group

template <int K> struct WideCfg {
    static constexpr int kPlaneBytes = K * BM * 16;
    static constexpr int kCoefBytes = (K + 1) * BM * 2;
    static constexpr int kBlockBytes = (kPlaneBytes + 2 * kCoefBytes + 1023) / 1024 * 1024;
    static constexpr int kSmemBytes = kWideStages * kWideStage + kWideSP * kBlockBytes + 1024 /*alignment slack*/ + 1024 /*barriers*/;
    static_assert(kSmemBytes <= 232448, "fits the opt-in shared memory of a CTA");
};

// Shared-memory matrix descriptor of a K-major tile with 64-byte swizzle whose rows are 64 bytes apart: start address
// / 16, leading byte offset (unused by swizzled K-major layouts) 1, stride byte offset 512 / 16 (distance between
// 8-row groups), descriptor version 1, layout type 4 (64-byte swizzle) in bits 61..63.
__device__ __forceinline__ uint64_t smem_desc_sw64(unsigned addr) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(512 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)4 << 61);
}

template <int K>
__global__ void __launch_bounds__(kWideThreads, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap planes_map,
                 const __grid_constant__ CUtensorMap coefs_map, const GemmParams p) {
    using C = WideCfg<K>;
    constexpr int S = kWideStages, SP = kWideSP;
    extern __shared__ unsigned char smem_raw[];
    const unsigned base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
    const unsigned st_base = base;                                 // S x (A tile, x half 0, x half 1)
    const unsigned p_base = st_base + S * kWideStage;              // SP x packed block
    const unsigned bar_base = p_base + SP * C::kBlockBytes;
    auto full_b = [&](int s) { return bar_base + 8u * s; };
    auto full_a = [&](int s) { return bar_base + 8u * (S + s); };
    auto empty = [&](int s) { return bar_base + 8u * (2 * S + s); };
    auto full_p = [&](int s) { return bar_base + 8u * (3 * S + s); };
    auto empty_p = [&](int s) { return bar_base + 8u * (3 * S + SP + s); };
    const unsigned acc_full = bar_base + 8u * (3 * S + 2 * SP), acc_empty = acc_full + 8u;
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(smem + (bar_base - base) + 8 * (3 * S + 2 * SP + 2));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int nkb = p.in / kWideBK;                  // stages per tile
    const int nblk = p.in / 128;                     // packed blocks per tile (four stages each)
    const int nrt = (p.out + BM - 1) / BM;
    const int ntt = (p.M + kWideBN - 1) / kWideBN;
    const int ntiles = nrt * ntt;
    const int ng = p.group == 64 ? 2 : 1;

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_b(s), 1);
            mbar_init(full_a(s), kDecodeThreads / 32);
            mbar_init(empty(s), 2);
        }
        for (int s = 0; s < SP; ++s) { mbar_init(full_p(s), 1); mbar_init(empty_p(s), kDecodeThreads / 32); }
        mbar_init(acc_full, 2);
        mbar_init(acc_empty, 4);
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
        // ---------------- producer: packed blocks and both x halves of every stage ----------------
        if (lane == 0) {
            int it = 0, bseq = 0;                        // stage and block sequence numbers, continuing across tiles
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int row0 = (tile % nrt) * BM, tok0 = (tile / nrt) * kWideBN;
                for (int b = 0; b < nblk && ok; ++b, ++bseq) {
                    const int sp = bseq % SP;
                    if (!mbar_wait(empty_p(sp), ((unsigned)(bseq / SP) & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    mbar_expect_tx(full_p(sp), (unsigned)(C::kPlaneBytes + ng * C::kCoefBytes));
                    const unsigned pdst = p_base + sp * C::kBlockBytes;
                    tma_load_2d(pdst, &planes_map, row0 * 2, b * K, full_p(sp));
                    tma_load_2d(pdst + C::kPlaneBytes, &coefs_map, row0 / 4, ((b * 128) / p.group) * (K + 1), full_p(sp));
                    for (int q = 0; q < 4; ++q, ++it) {
                        const int s = it % S;
                        if (!mbar_wait(empty(s), ((unsigned)(it / S) & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
                        mbar_expect_tx(full_b(s), 2u * kWideBHalf);
                        const unsigned bdst = st_base + s * kWideStage + kWideATile;
                        tma_load_2d(bdst, &x_map, (b * 4 + q) * kWideBK, tok0, full_b(s));
                        tma_load_2d(bdst + kWideBHalf, &x_map, (b * 4 + q) * kWideBK, tok0 + 256, full_b(s));
                    }
                }
            }
        }
    } else if (warp <= 2) {
        // ---------------- MMA issuers: warp 1 + h multiplies every stage with x half h into accumulator h ----------------
        if (lane == 0) {
            constexpr unsigned idesc = instr_desc_f16(BM, 256);
            const int h = warp - 1;
            const unsigned d = tmem_d + (unsigned)(h * 256);
            int it = 0, j = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++j) {
                // the epilogue must have drained the accumulators of the tile before
                if (!mbar_wait(acc_empty, ((unsigned)j & 1u) ^ 1u, abort_flag, p.status)) break;
                tc_fence_after();
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % S;
                    const unsigned ph = (unsigned)(it / S) & 1u;
                    ok = mbar_wait(full_a(s), ph, abort_flag, p.status) && mbar_wait(full_b(s), ph, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const unsigned a_addr = st_base + s * kWideStage;
                    const uint64_t adesc = smem_desc_sw64(a_addr);
                    const uint64_t bdesc = smem_desc_sw64(a_addr + kWideATile + h * kWideBHalf);
#pragma unroll
                    for (int k2 = 0; k2 < kWideBK / 16; ++k2)    // 16 columns = 32 bytes further along the swizzled row
                        umma_f16(d, adesc + 2u * k2, bdesc + 2u * k2, idesc, (kb | k2) != 0 ? 1u : 0u);
                    umma_commit(empty(s));
                }
                if (ok) umma_commit(acc_full);
            }
        }
    } else if (warp < 3 + 4 * kDecodeGroups) {
        // ---------------- decode warps (thread = output row) ----------------
        const int grp = (warp - 3) >> 2;                 // takes every other block of the block sequence
        const int rl = ((warp - 3) & 3) * 32 + lane;     // row inside the tile
        unsigned a_off[4];                               // swizzled byte offset of each 16-byte chunk of this thread's 64-byte row
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) a_off[ch] = (unsigned)rl * 64u + (((unsigned)ch ^ (unsigned)((rl >> 1) & 3)) << 4);
        const int my_tiles = blockIdx.x < ntiles ? (ntiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
        const long long nbseq = (long long)my_tiles * nblk;
        bool ok = true;
        for (long long bseq = grp; bseq < nbseq && ok; bseq += kDecodeGroups) {
            const int tj = (int)(bseq / nblk);                                   // this CTA's tj-th tile
            const int tile = blockIdx.x + tj * gridDim.x;
            const int r = (tile % nrt) * BM + rl;        // rows past a ragged last tile decode the copy's zero fill; nothing of theirs is stored
            const int sp = (int)(bseq % SP);
            if (!mbar_wait(full_p(sp), (unsigned)(bseq / SP) & 1u, abort_flag, p.status)) { ok = false; break; }
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
            for (int q = 0; q < 4; ++q) {                // the block's four 32-column stages
                const long long it = bseq * 4 + q;
                const int s = (int)(it % S);
                if (q == 0 || (ng == 2 && q == 2)) {     // candidate tables of the coefficient group that starts here
                    float c[K + 1];
#pragma unroll
                    for (int i = 0; i <= K; ++i) c[i] = __half2float(__ushort_as_half(cbits[ng == 2 ? q / 2 : 0][i]));
                    bpdq::candidate_byte_tables<K>(c, tab);
                }
                unsigned w[K], sel[4];
#pragma unroll
                for (int i = 0; i < K; ++i) w[i] = cur[i][q];
                bpdq::code_nibbles_word<K>(w, sel);
                uint4 v8[4];                             // decode first (nothing of it waits for the slot), then wait and store
#pragma unroll
                for (int u = 0; u < 4; ++u) v8[u] = bpdq::decode8<K>(sel[u], tab);
                if (!mbar_wait(empty(s), ((unsigned)(it / S) & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
                const unsigned dst = st_base + s * kWideStage;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch)
                    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + a_off[ch]),
                                 "r"(v8[ch].x), "r"(v8[ch].y), "r"(v8[ch].z), "r"(v8[ch].w) : "memory");
                fence_proxy_async();                     // make the generic-proxy stores visible to the MMA's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(full_a(s));   // one arrival per warp, after all its lanes' stores and fences
            }
        }
    } else {
        // ---------------- epilogue warps: drain both accumulators of a tile ----------------
        const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
        const int rl = quad * 32 + lane;
        int j = 0;
        for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++j) {
            if (!mbar_wait(acc_full, (unsigned)j & 1u, abort_flag, p.status)) break;
            tc_fence_after();
            const int row0 = (tile % nrt) * BM, tok0 = (tile / nrt) * kWideBN;
            const int r = row0 + rl;
            const bool row_ok = r < p.out;
            const float br = (p.bias && row_ok) ? __half2float(p.bias[r]) : 0.f;
            const unsigned taddr = tmem_d + ((unsigned)(quad * 32) << 16);
#pragma unroll 1
            for (int c0 = 0; c0 < kWideBN; c0 += 16) {
                if (tok0 + c0 >= p.M) break;             // warp-uniform
                unsigned v[16];
                tmem_ld16(taddr + (unsigned)c0, v);
                tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj) {
                        const int t = tok0 + c0 + jj;
                        if (t < p.M) p.y[(size_t)t * p.out + r] = __float2half_rn(__uint_as_float(v[jj]) + br);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty);       // one arrival per epilogue warp: the accumulators may be overwritten
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_d, 512);
    }
}
