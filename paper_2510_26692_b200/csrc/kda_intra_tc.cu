// bf16 tensor-core path of the chunkwise KDA forward: the intra-chunk stage (paper Section 3.1,
// "UT transform"; Appendix C up to the sequential loop).  Persistent CTAs of 256 threads, two per SM, each
// walking over (chunk, head) tiles with the next tile's inputs prefetched.
//
//   a1   G = cumulative sum of log alpha over the chunk's tokens (fp32, registers + one exchange
//        through shared memory)
//        gated operands, all bf16:  Kg = K exp(G - G_m),  Qg = scale Q exp(G - G_m),
//        Ki = K exp(G_m - G)   (G_m = G_C / 2 per channel, the middle of the chunk's log-decay range,
//        so that neither factor of exp(G_i - G_j) = exp(G_i - G_m) exp(G_m - G_j) leaves the
//        bf16/fp32 range; exponents are clamped to +-80).  The same three images serve the inter-chunk stage, which restores the
//        true scales exp(G_m), exp(G_C - G_m) in fp32 on its side
//   a2/a5  one tcgen05 MMA group  [Kg ; Qg] (128 x 128)  x  Ki^T (128 x 64)  ->  TMEM:
//        rows 0-63  = raw key Gram matrix, rows 64-127 = raw query-key matrix
//        L = Diag(beta) StrictTril(rows 0-63) (fp32, shared memory);  Aqk = Tril(rows 64-127)
//   a3   T = (I + L)^-1 by blocked forward substitution: the four 16x16 diagonal blocks are
//        inverted column by column in fp32 registers, then X = T_II L_IM for the six sub-diagonal
//        blocks and  T_IJ = - sum_M X_IM T_MJ  in three dependency stages, as warp-level 16x16 products
//        (mma.sync, tf32 inputs, fp32 accumulation; T is rounded to bf16 afterwards anyway)
//   a4   Mm = T Diag(beta) (bf16);  second MMA group  [Mm ; Mm] (128 x 64) x [Kg | V] (64 x 256) -> TMEM
//        (the rows are held twice so that all 128 TMEM lanes, i.e. all eight warps, share the read-out);
//        W' = Mm Kg (= W / exp(G_m) column-wise),  U = Mm V.  Kg and V are used as MN-major B operands in
//        the token-major layout they already have in shared memory.
// Outputs go to the scratch tile of kda_tiles.cuh as ready-made operand images of the inter-chunk
// kernel.  Tail chunks: rows past the sequence end behave as identity steps (log alpha = 0,
// beta = 0, k = q = v = 0).
#include <cuda.h>

#include <type_traits>

#include "kda_common.cuh"
#include "kda_ptx.cuh"
#include "kda_tiles.cuh"

namespace kda {
namespace {

constexpr uint64_t kWaitLimitNs = 1000000000ull;
constexpr int LDT = 68;                                   // padded fp32 row of the 64x64 matrices

// shared-memory map (bytes from a 1024-aligned base)
constexpr uint32_t S_KQ = 0;          // [2 K-halves][128 rows][64] bf16: rows 0-63 Kg, 64-127 Qg
constexpr uint32_t S_KQ_HALF = 16384;
constexpr uint32_t S_KI = 32768;      // [2 K-halves][64][64] bf16
constexpr uint32_t S_KI_HALF = 8192;
constexpr uint32_t S_V = 49152;       // [2 column blocks][64 tokens][64] bf16 (token-major)
constexpr uint32_t S_V_BLOCK = 8192;
constexpr uint32_t S_M = 65536;       // 8 KiB: Aqk staging; start of the 32 KiB output staging area
constexpr uint32_t S_A = 73728;       // fp32 [64][LDT]: L, later X in its sub-diagonal blocks
constexpr uint32_t S_T = S_A + 64 * LDT * 4;   // fp32 [64][LDT]: T
// staging of outputs for bulk stores (aliases buffers that are dead at the time):
constexpr uint32_t S_TOT = S_M + 32768;        // scan exchange [8..16][128] fp32, <= 8 KiB
constexpr uint32_t S_AQ = S_M;                 // Aqk image [64][64] bf16 (after the first MMA group)
constexpr uint32_t S_MM = S_KI;                // [128][64] bf16: T Diag(beta) twice (rows 64-127 repeat rows 0-63)
constexpr uint32_t S_W = S_M;                  // W image [2 halves][64][64] bf16 (after the second group)
constexpr uint32_t S_U = S_M + 16384;          // U: four [64][32] bf16 blocks
constexpr uint32_t S_BETA = S_T + 64 * LDT * 4;
constexpr uint32_t S_BAR = S_BETA + 256;        // mma barrier, tma barrier, TMEM slot
constexpr uint32_t S_TOTAL = S_BAR + 64;
constexpr int kNT = 256;                 // threads per CTA, two CTAs per SM
constexpr int kNW = kNT / 32;            // warps
constexpr int kRPT = kC / kNW;           // token rows per thread in the gating phase
constexpr int kBulkThread = kNT / 2;     // lane 0 of a middle warp issues every bulk copy; thread 0 the MMAs
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kClamp2 = 80.f * 1.4426950408889634f;   // the +-80 clamp in the log2 domain
constexpr uint32_t kIntraTcSmem = S_TOTAL + 1024;
static_assert(S_TOT + 16 * 128 * 4 <= S_BETA, "staging + scan exchange fit below the small arrays");
constexpr uint32_t kTmemCols = 256;

// loads that the compiler may not sink below their issue point (register prefetch of the next tile)
__device__ __forceinline__ void ld_nc_f4(const float* p, float& a, float& b, float& c, float& d) {
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(a), "=f"(b), "=f"(c), "=f"(d)
                 : "l"(p));
}
// 16x16 block products of the forward substitution on the legacy warp-level tensor path
// (mma.sync m16n8k8, tf32 inputs rounded to nearest, fp32 accumulation): acc += A * B with A, B
// 16x16 fp32 blocks in shared memory (row stride `ld` floats).
__device__ __forceinline__ uint32_t to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void block16_mma(float (&acc)[2][4], const float* pa, const float* pb,
                                            int ld, int lane) {
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
        const uint32_t a0 = to_tf32(pa[g * ld + ks * 8 + t4]);
        const uint32_t a1 = to_tf32(pa[(g + 8) * ld + ks * 8 + t4]);
        const uint32_t a2 = to_tf32(pa[g * ld + ks * 8 + t4 + 4]);
        const uint32_t a3 = to_tf32(pa[(g + 8) * ld + ks * 8 + t4 + 4]);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const uint32_t b0 = to_tf32(pb[(ks * 8 + t4) * ld + nt * 8 + g]);
            const uint32_t b1 = to_tf32(pb[(ks * 8 + t4 + 4) * ld + nt * 8 + g]);
            asm volatile(
                "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
                "{%8,%9}, {%0,%1,%2,%3};"
                : "+f"(acc[nt][0]), "+f"(acc[nt][1]), "+f"(acc[nt][2]), "+f"(acc[nt][3])
                : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
        }
    }
}
__device__ __forceinline__ void block16_load(float (&acc)[2][4], const float* pc, int ld, int lane) {
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        const float2 lo = *reinterpret_cast<const float2*>(pc + g * ld + nt * 8 + 2 * t4);
        const float2 hi = *reinterpret_cast<const float2*>(pc + (g + 8) * ld + nt * 8 + 2 * t4);
        acc[nt][0] = lo.x; acc[nt][1] = lo.y; acc[nt][2] = hi.x; acc[nt][3] = hi.y;
    }
}
__device__ __forceinline__ void block16_store(float* pc, const float (&acc)[2][4], float sign, int ld,
                                              int lane) {
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        *reinterpret_cast<float2*>(pc + g * ld + nt * 8 + 2 * t4) =
            make_float2(sign * acc[nt][0], sign * acc[nt][1]);
        *reinterpret_cast<float2*>(pc + (g + 8) * ld + nt * 8 + 2 * t4) =
            make_float2(sign * acc[nt][2], sign * acc[nt][3]);
    }
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&p);
}
// kHasQ = false: state-only call (no output requested): the query half of the work is compiled out.
template <bool kHasQ>
__global__ void __launch_bounds__(kNT, 2)
kda_intra_tc(ChunkArgs a, char* __restrict__ tiles, WsHeader* hdr,
             const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_q,
             const __grid_constant__ CUtensorMap tm_v, int clear_status)
{
    constexpr bool has_q = kHasQ;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* sA = reinterpret_cast<float*>(smem + S_A);
    float* sT = reinterpret_cast<float*>(smem + S_T);
    float* sTot = reinterpret_cast<float*>(smem + S_TOT);   // [16][128] during the scan
    float* sBeta = reinterpret_cast<float*>(smem + S_BETA);
    uint64_t* mma_bar = reinterpret_cast<uint64_t*>(smem + S_BAR);
    uint64_t* tma_bar = mma_bar + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mma_bar + 2);
    volatile uint32_t* abort_word = tmem_slot + 1;   // set by the first thread whose bounded wait runs out

    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;

    ptx::grid_dep_launch();   // the inter-chunk kernel may set itself up while this one drains
    if (clear_status && blockIdx.x == 0 && t == 0) {
        hdr->status = 0;      // (an equal-length call has no prologue kernel to do this)
        hdr->where = 0;
        hdr->flags = 0;
    }
    if (t == 0) {
        ptx::mbar_init(mma_bar, 1);
        ptx::mbar_init(tma_bar, 1);
        *abort_word = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_k);
        ptx::prefetch_tmap(&tm_q);
        ptx::prefetch_tmap(&tm_v);
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }

    // Persistent CTA: tiles cur, cur + gridDim.x, ...  (tile = chunk-in-pass * H + head).  The
    // inputs of the next tile are requested as soon as the buffers of the current one are free:
    // k, q and v by 2-D tiled TMA loads straight into the swizzled operand images (k and q are then
    // gated in place), log alpha into registers (thread (w, c4) owns rows 8w..8w+7 and channels
    // 4c4..4c4+3), beta by small asynchronous copies.
    const int c4 = lane, d0 = c4 * 4, i0 = warp * kRPT;
    const uint32_t ntiles = (uint32_t)((a.g1 - a.g0) * a.H);
    float G[kRPT][4];
    auto locate = [&](uint32_t tl, ChunkLoc& Lo, int& ho) {
        const uint32_t gl = tl / (uint32_t)a.H;
        ho = (int)(tl - gl * (uint32_t)a.H);
        Lo = locate_chunk(a, a.g0 + gl);
    };
    // log alpha -> registers (may be issued while the second MMA group still runs)
    auto prefetch_regs = [&](const ChunkLoc& Lo, int ho) {
        const float* gp = a.log_alpha + ((size_t)Lo.tok0 * a.H + ho) * kD + d0;
#pragma unroll
        for (int r = 0; r < kRPT; ++r) {
            const int i = i0 + r;
            if (i < Lo.len) {
                ld_nc_f4(gp + (size_t)i * a.H * kD, G[r][0], G[r][1], G[r][2], G[r][3]);
            } else {
                G[r][0] = G[r][1] = G[r][2] = G[r][3] = 0.f;
            }
        }
    };
    // k, q, v, beta -> shared memory (only once the second MMA group has finished reading Kg and V)
    auto prefetch_bufs = [&](const ChunkLoc& Lo, int ho) {
        if (t == kBulkThread) {
            ptx::mbar_expect_tx(tma_bar, (has_q ? 3 : 2) * 16384);
            const int x = ho * kD, y = (int)Lo.tok0;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                ptx::tma_load_2d(smem + S_KQ + hf * S_KQ_HALF, &tm_k, x + hf * 64, y, tma_bar);
                if (has_q)
                    ptx::tma_load_2d(smem + S_KQ + hf * S_KQ_HALF + 8192, &tm_q, x + hf * 64, y, tma_bar);
                ptx::tma_load_2d(smem + S_V + hf * S_V_BLOCK, &tm_v, x + hf * 64, y, tma_bar);
            }
        }
        if (t < kC) {
            const bool ok = t < Lo.len;
            ptx::cp_async4(sBeta + t, a.beta + (Lo.tok0 + (ok ? t : 0)) * a.H + ho, ok ? 4u : 0u);
        }
        ptx::cp_async_commit();
    };

    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    bool timed_out = false, load_pending = false, out_of_range = false;
    uint32_t tma_parity = 0;

    uint32_t cur = blockIdx.x;
    ChunkLoc L;
    int h = 0;
    if (cur < ntiles) {
        locate(cur, L, h);
        prefetch_regs(L, h);
        prefetch_bufs(L, h);
        load_pending = true;
    }
    for (; cur < ntiles; cur += gridDim.x) {
    char* tile = tiles + (size_t)cur * tc::TILE_BYTES;
    const uint32_t nxt = cur + gridDim.x;
    ChunkLoc Ln = L;
    int hn = h;

    // ---- a1: cumulative log-decay, in the log2 domain (exponentials below are bare ex2) -------
#pragma unroll
    for (int e = 0; e < 4; ++e) G[0][e] *= kLog2e;
#pragma unroll
    for (int r = 1; r < kRPT; ++r)
#pragma unroll
        for (int e = 0; e < 4; ++e) G[r][e] = fmaf(G[r][e], kLog2e, G[r - 1][e]);
    *reinterpret_cast<float4*>(sTot + warp * kD + d0) = make_float4(G[kRPT - 1][0], G[kRPT - 1][1], G[kRPT - 1][2], G[kRPT - 1][3]);
    ptx::cp_async_wait_all();             // beta
    __syncthreads();
    // a wait of the previous tile ran out: stop here (uniform: the flag was set before the barrier);
    // the copies in flight are drained after the loop
    if (*abort_word) break;
    float base[4] = {0.f, 0.f, 0.f, 0.f}, gref[4] = {0.f, 0.f, 0.f, 0.f}, glast[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int r2 = 0; r2 < kNW; ++r2) {
        const float4 x4 = *reinterpret_cast<const float4*>(sTot + r2 * kD + d0);
        const float x[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (r2 < warp) base[e] += x[e];
            glast[e] += x[e];
        }
    }
    // reference of the decay factorisation: half the chunk's total log-decay, per channel, so that
    // |G_i - G_ref| <= |G_C| / 2 for every row whatever the distribution of the decay over the chunk
#pragma unroll
    for (int e = 0; e < 4; ++e) gref[e] = 0.5f * glast[e];

    // ---- gated operands ---------------------------------------------------------------------------------
    // the true scales exp(G_m), exp(G_C - G_m) and gamma^C go to the tile as fp32 vectors; the
    // inter-chunk kernel applies them to the state in fp32
    if (warp == 0) {
        *reinterpret_cast<float4*>(tile + tc::OFF_GV + d0 * 4) =
            make_float4(ex2(glast[0]), ex2(glast[1]), ex2(glast[2]), ex2(glast[3]));
        *reinterpret_cast<float4*>(tile + tc::OFF_GV + 512 + d0 * 4) =
            make_float4(ex2(gref[0]), ex2(gref[1]), ex2(gref[2]), ex2(gref[3]));
        *reinterpret_cast<float4*>(tile + tc::OFF_GV + 1024 + d0 * 4) =
            make_float4(ex2(glast[0] - gref[0]), ex2(glast[1] - gref[1]), ex2(glast[2] - gref[2]),
                        ex2(glast[3] - gref[3]));
        // a channel that decays by more than e^-160 inside this chunk leaves the range of the
        // two-factor form (the clamp below keeps everything finite): flag the call at the end
        if (fminf(fminf(glast[0], glast[1]), fminf(glast[2], glast[3])) < -2.f * kClamp2) out_of_range = true;
    }
    if (!ptx::mbar_wait(tma_bar, tma_parity, kWaitLimitNs)) { timed_out = true; *abort_word = 1; }   // k, q, v have landed
    tma_parity ^= 1;
    load_pending = false;
    if (L.len < kC) {   // short last chunk: rows past the end hold the next sequence's v; zero them
        for (int idx = t; idx < (kC - L.len) * 16; idx += kNT) {
            const int j = L.len + (idx >> 4), c16 = idx & 15;
            *reinterpret_cast<uint4*>(smem + S_V + (c16 >> 3) * S_V_BLOCK + j * 128 +
                                      (((c16 & 7) ^ (j & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    const int hf = c4 >> 4;                       // K-half (channels 0-63 / 64-127)
    // (state-only calls produce no output: the query half is skipped altogether; the choice is made
    // outside the loop so that each version stays branch-free)
    auto gate_rows = [&](auto with_q) {
        constexpr bool kQ = decltype(with_q)::value;
#pragma unroll
        for (int r = 0; r < kRPT; ++r) {
            const int i = i0 + r;
            const uint32_t off = (uint32_t)(i * 128 + ((((c4 >> 1) & 7) ^ (i & 7)) << 4) + (c4 & 1) * 8);
            uint8_t* pk = smem + S_KQ + hf * S_KQ_HALF + off;
            uint2 k2 = *reinterpret_cast<const uint2*>(pk);
            uint2 q2 = make_uint2(0u, 0u);
            if (kQ) q2 = *reinterpret_cast<const uint2*>(pk + 8192);
            if (i >= L.len) k2 = q2 = make_uint2(0u, 0u);
            const float kf[4] = {__uint_as_float(k2.x << 16), __uint_as_float(k2.x & 0xffff0000u),
                                 __uint_as_float(k2.y << 16), __uint_as_float(k2.y & 0xffff0000u)};
            const float qf[4] = {__uint_as_float(q2.x << 16), __uint_as_float(q2.x & 0xffff0000u),
                                 __uint_as_float(q2.y << 16), __uint_as_float(q2.y & 0xffff0000u)};
            float okg[4], oqg[4], oki[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float x = fminf(fmaxf(G[r][e] + base[e] - gref[e], -kClamp2), kClamp2);
                const float e1 = ex2(x);                     // exp(G - G_m)
                const float e2 = ex2(-x);                    // exp(G_m - G)
                okg[e] = kf[e] * e1;
                oqg[e] = a.scale * qf[e] * e1;
                oki[e] = kf[e] * e2;
            }
            *reinterpret_cast<uint2*>(pk) = make_uint2(pack_bf16(okg[0], okg[1]), pack_bf16(okg[2], okg[3]));
            if (kQ)
                *reinterpret_cast<uint2*>(pk + 8192) =
                    make_uint2(pack_bf16(oqg[0], oqg[1]), pack_bf16(oqg[2], oqg[3]));
            *reinterpret_cast<uint2*>(smem + S_KI + hf * S_KI_HALF + off) =
                make_uint2(pack_bf16(oki[0], oki[1]), pack_bf16(oki[2], oki[3]));
        }
    };
    gate_rows(std::integral_constant<bool, kHasQ>{});

    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();

    // ---- a2 + a5: [Kg ; Qg] Ki^T ------------------------------------------------------------------------
    if (t == kBulkThread) {
        // phase-1 outputs leave through the TMA engine while the MMA runs
        // Q' (rows 64-127 of both K-halves of the operand image) and K' are tile contents as they are
        if (has_q) {
            ptx::bulk_s2g(tile + tc::OFF_QW + 8192, smem + S_KQ + 8192, 8192);
            ptx::bulk_s2g(tile + tc::OFF_QW + tc::QW_HALF + 8192, smem + S_KQ + S_KQ_HALF + 8192, 8192);
        }
        ptx::bulk_s2g(tile + tc::OFF_KI, smem + S_KI, 16384);
        ptx::bulk_commit();
    }
    if (t == 0) {
        const uint32_t idesc = ptx::umma_idesc_bf16(128, 64);
        const uint32_t a0 = ptx::smem_u32(smem + S_KQ), b0 = ptx::smem_u32(smem + S_KI);
#pragma unroll
        for (int k = 0; k < 8; ++k)
            ptx::umma_bf16(tmem_base, ptx::umma_desc_sw128(a0 + (k >> 2) * S_KQ_HALF + (k & 3) * 32),
                           ptx::umma_desc_sw128(b0 + (k >> 2) * S_KI_HALF + (k & 3) * 32), idesc, k > 0);
        ptx::umma_commit(mma_bar);
    }
    if (nxt < ntiles) {   // the next tile's log alpha: a whole tile ahead (its registers are free since the gating loop)
        locate(nxt, Ln, hn);
        prefetch_regs(Ln, hn);
    }
    if (!ptx::mbar_wait(mma_bar, 0, kWaitLimitNs)) { timed_out = true; *abort_word = 1; }
    // the previous tile's W/U staging (and this tile's Q', K' stores) have been read out by now; the
    // staging area is written next (L, Aqk)
    if (t == kBulkThread) ptx::bulk_wait_read0();
    __syncthreads();
    ptx::tc_fence_after();
    {
        constexpr int NCA = 32;   // accumulator columns per warp
        const int q4 = warp & 3, c0 = (warp >> 2) * NCA;
        const int R = q4 * 32 + lane;
        uint32_t r[NCA];
        ptx::tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q4 * 32) << 16) + c0, r);
        ptx::tmem_ld_wait();
        if (R < 64) {
            const int i = R;
            const float bi = sBeta[i];
#pragma unroll
            for (int j4 = 0; j4 < NCA; j4 += 4) {
                float x[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int j = c0 + j4 + e;
                    x[e] = (j < i) ? bi * __uint_as_float(r[j4 + e]) : 0.f;
                }
                *reinterpret_cast<float4*>(sA + i * LDT + c0 + j4) = make_float4(x[0], x[1], x[2], x[3]);
            }
        } else if (has_q) {
            const int i = R - 64;
#pragma unroll
            for (int j8 = 0; j8 < NCA; j8 += 8) {
                float x[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int j = c0 + j8 + e;
                    x[e] = (j <= i) ? __uint_as_float(r[j8 + e]) : 0.f;
                }
                *reinterpret_cast<uint4*>(smem + S_AQ + ptx::sw128_off(i, c0 + j8)) =
                    make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]),
                               pack_bf16(x[6], x[7]));
            }
        }
    }
    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    if (t == kBulkThread && has_q) {
        ptx::bulk_s2g(tile + tc::OFF_AQ, smem + S_AQ, 8192);
        ptx::bulk_commit();
    }

    // ---- a3: T = (I + L)^-1, blocked forward substitution -------------------------------------------
    if (t < 64) {   // diagonal 16x16 blocks: one column per thread, rows unrolled in registers
        const int I = t >> 4, c = t & 15;
        const float* Lb = sA + (I * 16) * LDT + I * 16;
        float x[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            float s = (r == c) ? 1.f : 0.f;
#pragma unroll
            for (int m = 0; m < r; ++m) s -= Lb[r * LDT + m] * x[m];
            x[r] = s;
        }
#pragma unroll
        for (int r = 0; r < 16; ++r) sT[(I * 16 + r) * LDT + I * 16 + c] = x[r];
    }
    __syncthreads();
    // X_IM = T_II L_IM for the six sub-diagonal blocks (one warp each, in place), then
    // T_IJ = - sum_{M=J..I-1} X_IM T_MJ in three dependency stages; the terms of a sum that do not
    // depend on blocks still being computed are taken early (kept, un-negated, in the block's place).
    //   stage A: T10, T21, T32 final;  P20 = X20 T00,  P31 = X31 T11,  P30 = X30 T00
    //            (each uses only the X block its own warp has just formed)
    //   stage B: T20 = -(P20 + X21 T10),  T31 = -(P31 + X32 T21),  P30 += X31 T10
    //   stage C: T30 = -(P30 + X32 T20)
    auto blk = [&](float* base, int I, int J) { return base + (I * 16) * LDT + J * 16; };
    if (warp < 6) {
        const int I = warp < 1 ? 1 : (warp < 3 ? 2 : 3);
        const int M = warp < 1 ? 0 : (warp < 3 ? warp - 1 : warp - 3);
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        block16_mma(acc, blk(sT, I, I), blk(sA, I, M), LDT, lane);
        __syncwarp();   // every lane has read its part of L_IM before anyone overwrites it
        block16_store(blk(sA, I, M), acc, 1.f, LDT, lane);
        __syncwarp();
        float acc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        block16_mma(acc2, blk(sA, I, M), blk(sT, M, M), LDT, lane);
        block16_store(blk(sT, I, M), acc2, (I - M == 1) ? -1.f : 1.f, LDT, lane);
    }
    __syncthreads();
    if (warp < 3) {
        // warp 0: T20 (M = 1), warp 1: T31 (M = 2), warp 2: P30 += X31 T10
        const int I = warp == 0 ? 2 : 3, J = warp == 1 ? 1 : 0, M = warp == 1 ? 2 : 1;
        float acc[2][4];
        block16_load(acc, blk(sT, I, J), LDT, lane);
        block16_mma(acc, blk(sA, I, M), blk(sT, M, J), LDT, lane);
        block16_store(blk(sT, I, J), acc, warp < 2 ? -1.f : 1.f, LDT, lane);
    }
    __syncthreads();
    if (warp == 0) {
        float acc[2][4];
        block16_load(acc, blk(sT, 3, 0), LDT, lane);
        block16_mma(acc, blk(sA, 3, 2), blk(sT, 2, 0), LDT, lane);
        block16_store(blk(sT, 3, 0), acc, -1.f, LDT, lane);
    }
    __syncthreads();

    // ---- a4: Mm = T Diag(beta) as the A operand; [W | U] = Mm [Kg | V] ---------------------------------
    {
        constexpr int NCM = 16;   // columns per thread
        const int i = t / (kNT / 64), jq = t % (kNT / 64);
        const int j0 = jq * NCM;
        float x[NCM];
        if ((j0 >> 4) > (i >> 4)) {
#pragma unroll
            for (int e = 0; e < NCM; ++e) x[e] = 0.f;
        } else {
#pragma unroll
            for (int e4 = 0; e4 < NCM; e4 += 4) {
                const float4 tv = *reinterpret_cast<const float4*>(sT + i * LDT + j0 + e4);
                const float4 bv = *reinterpret_cast<const float4*>(sBeta + j0 + e4);
                x[e4] = tv.x * bv.x; x[e4 + 1] = tv.y * bv.y; x[e4 + 2] = tv.z * bv.z; x[e4 + 3] = tv.w * bv.w;
            }
        }
#pragma unroll
        for (int c8 = 0; c8 < NCM / 8; ++c8) {
            const uint4 pk = make_uint4(pack_bf16(x[c8 * 8], x[c8 * 8 + 1]), pack_bf16(x[c8 * 8 + 2], x[c8 * 8 + 3]),
                                        pack_bf16(x[c8 * 8 + 4], x[c8 * 8 + 5]), pack_bf16(x[c8 * 8 + 6], x[c8 * 8 + 7]));
            uint8_t* dst = smem + S_MM + i * 128 + ((((j0 >> 3) + c8) ^ (i & 7)) << 4);
            *reinterpret_cast<uint4*>(dst) = pk;
            *reinterpret_cast<uint4*>(dst + 8192) = pk;   // rows 64-127 repeat rows 0-63
        }
    }
    if (t == kBulkThread) ptx::bulk_wait_read0();   // K' (overwritten by the Mm image) and the Aqk staging (reused by the W/U epilogue) have been read out
    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    if (t == 0) {
        ptx::tc_fence_after();
        const uint32_t idesc = ptx::umma_idesc_bf16(128, 128) | ptx::kIdescBMajorMN;
        const uint32_t m0 = ptx::smem_u32(smem + S_MM);
        const uint32_t kg0 = ptx::smem_u32(smem + S_KQ), v0 = ptx::smem_u32(smem + S_V);
#pragma unroll
        for (int k = 0; k < 4; ++k)
            ptx::umma_bf16(tmem_base, ptx::umma_desc_sw128(m0 + k * 32),
                           ptx::umma_desc_sw128_mn(kg0 + k * 2048, S_KQ_HALF), idesc, k > 0);
#pragma unroll
        for (int k = 0; k < 4; ++k)
            ptx::umma_bf16(tmem_base + 128, ptx::umma_desc_sw128(m0 + k * 32),
                           ptx::umma_desc_sw128_mn(v0 + k * 2048, S_V_BLOCK), idesc, k > 0);
        ptx::umma_commit(mma_bar);
    }
    if (!ptx::mbar_wait(mma_bar, 1, kWaitLimitNs)) { timed_out = true; *abort_word = 1; }
    if (nxt < ntiles) {
        prefetch_bufs(Ln, hn);
        load_pending = true;
    }
    ptx::tc_fence_after();
    {   // The A operand held every row twice, so TMEM lanes 0-63 and 64-127 both carry rows 0-63:
        // each warp converts rows 32 (q4 & 1) + lane of one NCE-column block of [W | U].
        constexpr int NCE = 64;   // columns per warp
        const int q4 = warp & 3, cbk = (warp >> 2) * 2 + (q4 >> 1);
        const int col0 = cbk * NCE;            // first column inside [W | U]
        const int i = (q4 & 1) * 32 + lane;
        uint32_t r[NCE];
        const uint32_t ta = tmem_base + ((uint32_t)(q4 * 32) << 16) + col0;
#pragma unroll
        for (int b = 0; b < NCE / 32; ++b)
            ptx::tmem_ld_32x32b_x32(ta + b * 32, reinterpret_cast<uint32_t(&)[32]>(r[b * 32]));
        ptx::tmem_ld_wait();
        if (col0 < 128) {   // W' = Mm Kg: K-half col0 / 64 of the [W' ; Q'] image
            uint8_t* dst = smem + S_W + (col0 >> 6) * 8192;
#pragma unroll
            for (int j8 = 0; j8 < NCE; j8 += 8)
                *reinterpret_cast<uint4*>(dst + ptx::sw128_off(i, (col0 & 63) + j8)) =
                    make_uint4(pack_bf16(__uint_as_float(r[j8]), __uint_as_float(r[j8 + 1])),
                               pack_bf16(__uint_as_float(r[j8 + 2]), __uint_as_float(r[j8 + 3])),
                               pack_bf16(__uint_as_float(r[j8 + 4]), __uint_as_float(r[j8 + 5])),
                               pack_bf16(__uint_as_float(r[j8 + 6]), __uint_as_float(r[j8 + 7])));
        } else {            // U: 32-column blocks (col0 - 128) / 32 ...
#pragma unroll
            for (int j8 = 0; j8 < NCE; j8 += 8) {
                const int cu = col0 - 128 + j8;
                *reinterpret_cast<uint4*>(smem + S_U + (cu >> 5) * tc::U_BLOCK + tc::u_off(i, (cu & 31) >> 3)) =
                    make_uint4(pack_bf16(__uint_as_float(r[j8]), __uint_as_float(r[j8 + 1])),
                               pack_bf16(__uint_as_float(r[j8 + 2]), __uint_as_float(r[j8 + 3])),
                               pack_bf16(__uint_as_float(r[j8 + 4]), __uint_as_float(r[j8 + 5])),
                               pack_bf16(__uint_as_float(r[j8 + 6]), __uint_as_float(r[j8 + 7])));
            }
        }
    }
    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    if (t == kBulkThread) {
        ptx::bulk_s2g(tile + tc::OFF_QW, smem + S_W, 8192);
        ptx::bulk_s2g(tile + tc::OFF_QW + tc::QW_HALF, smem + S_W + 8192, 8192);
        ptx::bulk_s2g(tile + tc::OFF_U, smem + S_U, 16384);
        ptx::bulk_commit();   // read-out completion is awaited before the staging area is reused
    }
    L = Ln;
    h = hn;
    }   // tile loop

    if (timed_out && atomicCAS(&hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) hdr->where = 10;
    if (out_of_range) atomicOr(&hdr->flags, 1);
    if (load_pending && t == 0) ptx::mbar_wait(tma_bar, tma_parity, kWaitLimitNs);   // a requested tile must land before the CTA ends
    if (t == kBulkThread) ptx::bulk_wait_read0();   // shared memory must outlive the reads of every bulk store
    ptx::cp_async_wait_all();
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

namespace {
// cuTensorMapEncodeTiled through the runtime's driver entry-point query (no link dependency on
// libcuda, so the library still loads on a machine without a driver)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}
// [total_tokens, H*128] bf16 matrix, boxes of 64 tokens x 64 channels, 128-byte swizzle
kda_status_t make_tmap(CUtensorMap* tm, const void* base, int64_t total_tokens, int H)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return fail(KDA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const cuuint64_t dims[2] = {(cuuint64_t)H * kD, (cuuint64_t)total_tokens};
    const cuuint64_t strides[1] = {(cuuint64_t)H * kD * 2};
    const cuuint32_t box[2] = {64, 64};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(KDA_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return KDA_OK;
}
}  // namespace

kda_status_t launch_intra_tc(const ChunkArgs& a, void* tiles, WsHeader* hdr, bool clear_status,
                             cudaStream_t st)
{
    int n_sm = 0;
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (!lk.st->attr_done[1]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kIntraTcSmem));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kIntraTcSmem));
            lk.st->attr_done[1] = true;
        }
        if (lk.st->n_sm == 0) {
            int dev = 0;
            KDA_CUDA_TRY(cudaGetDevice(&dev));
            KDA_CUDA_TRY(cudaDeviceGetAttribute(&lk.st->n_sm, cudaDevAttrMultiProcessorCount, dev));
        }
        n_sm = lk.st->n_sm;
    }
    const int64_t n_tiles = (a.g1 - a.g0) * a.H;
    if (n_tiles <= 0) return KDA_OK;
    if (n_tiles > 0x7fffffff || a.total_tokens > 0x7fffffff)
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: more than 2^31 tokens or tiles in one pass");
    CUtensorMap tm_k, tm_q, tm_v;
    kda_status_t rc = make_tmap(&tm_k, a.k, a.total_tokens, a.H);
    if (rc == KDA_OK) rc = make_tmap(&tm_v, a.v, a.total_tokens, a.H);
    if (rc == KDA_OK) rc = make_tmap(&tm_q, a.q ? a.q : a.k, a.total_tokens, a.H);
    if (rc != KDA_OK) return rc;
    const int64_t resident = 2 * (int64_t)n_sm;   // two CTAs per SM
    const unsigned grid = (unsigned)(n_tiles < resident ? n_tiles : resident);
    ProfScope ps(PROF_INTRA, st);
    if (a.q && a.o)
        kda_intra_tc<true><<<grid, kNT, kIntraTcSmem, st>>>(a, (char*)tiles, hdr, tm_k, tm_q, tm_v, clear_status ? 1 : 0);
    else
        kda_intra_tc<false><<<grid, kNT, kIntraTcSmem, st>>>(a, (char*)tiles, hdr, tm_k, tm_q, tm_v, clear_status ? 1 : 0);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

}  // namespace kda
