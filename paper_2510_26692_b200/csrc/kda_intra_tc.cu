// bf16 tensor-core path of the chunkwise KDA forward: the intra-chunk stage (paper Section 3.1,
// "UT transform"; Appendix C up to the sequential loop).  Persistent CTAs of 256 threads, two per SM, each
// walking over (chunk, head) tiles with the next tile's inputs prefetched.
//
//   a1   G = cumulative sum of log alpha over the chunk's tokens (fp32, registers + one exchange
//        through shared memory)
//        gated operands, all bf16:  Kg = K exp(G - G_m),  Qg = scale Q exp(G - G_m),
//        Ki = K exp(G_m - G)   (m = row 31, the middle of the chunk, so that neither factor of
//        exp(G_i - G_j) = exp(G_i - G_m) exp(G_m - G_j) leaves the bf16/fp32 range; exponents are
//        clamped to +-80),
//        and for the inter-chunk stage  scale Q exp(G)  and  (K exp(G_C - G))^T
//   a2/a5  one tcgen05 MMA group  [Kg ; Qg] (128 x 128)  x  Ki^T (128 x 64)  ->  TMEM:
//        rows 0-63  = raw key Gram matrix, rows 64-127 = raw query-key matrix
//        L = Diag(beta) StrictTril(rows 0-63) (fp32, shared memory);  Aqk = Tril(rows 64-127)
//   a3   T = (I + L)^-1 by blocked forward substitution in fp32: the four 16x16 diagonal blocks are
//        inverted column by column in registers, then X = T_II L_IM for the six sub-diagonal blocks
//        and three block levels  T_IJ = - sum_M X_IM T_MJ
//   a4   Mm = T Diag(beta) (bf16);  second MMA group  Mm (64 x 64) x [Kg | V] (64 x 256) -> TMEM;
//        W = (Mm Kg) exp(G_m) column-wise,  U = Mm V.  Kg and V are used as MN-major B operands in
//        the token-major layout they already have in shared memory.
// Outputs go to the scratch tile of kda_tiles.cuh as ready-made operand images of the inter-chunk
// kernel.  Tail chunks: rows past the sequence end behave as identity steps (log alpha = 0,
// beta = 0, k = q = v = 0).
#include "kda_common.cuh"
#include "kda_ptx.cuh"
#include "kda_tiles.cuh"

namespace kda {
namespace {

constexpr uint64_t kWaitLimitNs = 1000000000ull;
constexpr int LDT = 68;                                   // padded fp32 row of the 64x64 matrices
constexpr float kExpClamp = 80.f;

// shared-memory map (bytes from a 1024-aligned base)
constexpr uint32_t S_KQ = 0;          // [2 K-halves][128 rows][64] bf16: rows 0-63 Kg, 64-127 Qg
constexpr uint32_t S_KQ_HALF = 16384;
constexpr uint32_t S_KI = 32768;      // [2 K-halves][64][64] bf16
constexpr uint32_t S_KI_HALF = 8192;
constexpr uint32_t S_V = 49152;       // [2 column blocks][64 tokens][64] bf16 (token-major)
constexpr uint32_t S_V_BLOCK = 8192;
constexpr uint32_t S_M = 65536;       // [64][64] bf16: T Diag(beta)
constexpr uint32_t S_A = 73728;       // fp32 [64][LDT]: L, later X in its sub-diagonal blocks
constexpr uint32_t S_T = S_A + 64 * LDT * 4;   // fp32 [64][LDT]: T
// staging of outputs for bulk stores (aliases buffers that are dead at the time):
constexpr uint32_t S_QG = S_M;                 // scale Q exp(G): [2 halves][64][64] bf16, 16 KiB   (phase 1)
constexpr uint32_t S_KT = S_M + 16384;         // (K exp(G_C - G))^T: [128][64] bf16, 16 KiB        (phase 1)
constexpr uint32_t S_TOT = S_M + 32768;        // scan exchange [16][128] fp32, 8 KiB
constexpr uint32_t S_AQ = S_KI;                // Aqk image [64][64] bf16 (after the first MMA group)
constexpr uint32_t S_W = S_M;                  // W image [2 halves][64][64] bf16 (after the second group)
constexpr uint32_t S_U = S_M + 16384;          // U [4 blocks][64][32] bf16
constexpr uint32_t S_BETA = S_T + 64 * LDT * 4;
constexpr uint32_t S_CG = S_BETA + 256;        // exp(G_m) per channel (undoes the Kg reference)
constexpr uint32_t S_BAR = S_CG + 512;
constexpr uint32_t S_TOTAL = S_BAR + 64;
constexpr uint32_t kIntraTcSmem = S_TOTAL + 1024;
static_assert(S_TOT + 16 * 128 * 4 <= S_BETA, "staging + scan exchange fit below the small arrays");
constexpr uint32_t kTmemCols = 256;

// loads that the compiler may not sink below their issue point (register prefetch of the next tile)
__device__ __forceinline__ void ld_nc_f4(const float* p, float& a, float& b, float& c, float& d) {
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(a), "=f"(b), "=f"(c), "=f"(d)
                 : "l"(p));
}
__device__ __forceinline__ uint4 ld_nc_u4(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ void unpack8(const uint4& r, float (&f)[8]) {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&r);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        float2 x = __bfloat1622float2(p[e]);
        f[2 * e] = x.x;
        f[2 * e + 1] = x.y;
    }
}

__global__ void __launch_bounds__(256, 2)
kda_intra_tc(ChunkArgs a, char* __restrict__ tiles, WsHeader* hdr)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* sA = reinterpret_cast<float*>(smem + S_A);
    float* sT = reinterpret_cast<float*>(smem + S_T);
    float* sTot = reinterpret_cast<float*>(smem + S_TOT);   // [16][128] during the scan
    float* sBeta = reinterpret_cast<float*>(smem + S_BETA);
    float* sCG = reinterpret_cast<float*>(smem + S_CG);
    uint64_t* mma_bar = reinterpret_cast<uint64_t*>(smem + S_BAR);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mma_bar + 1);

    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(a.q);
    const __nv_bfloat16* kp = reinterpret_cast<const __nv_bfloat16*>(a.k);
    const __nv_bfloat16* vp = reinterpret_cast<const __nv_bfloat16*>(a.v);

    KDA_PHASE_DECL;
    if (t == 0) {
        ptx::mbar_init(mma_bar, 1);
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }

    // Persistent CTA: tiles cur, cur + gridDim.x, ...  (tile = chunk-in-pass * H + head).  The
    // inputs of the next tile are requested while the current one is being processed: log alpha,
    // k and q into registers (thread (rg, dc) owns rows 4rg..4rg+3, channels 8dc..8dc+7), v and
    // beta by asynchronous copies into shared memory.
    const int dc = t & 15, rg = t >> 4;
    const int d0 = dc * 8, i0 = rg * 4;
    const int64_t ntiles = (a.g1 - a.g0) * a.H;
    float G[4][8];
    auto locate = [&](int64_t tl, ChunkLoc& Lo, int& ho) {
        const int64_t gl = tl / a.H;
        ho = (int)(tl - gl * a.H);
        Lo = locate_chunk(a, a.g0 + gl);
    };
    const int half = dc >> 3, cc = dc & 7;
    auto issue_prefetch = [&](const ChunkLoc& Lo, int ho) {
        // log alpha -> registers; k, q -> their slots of the [Kg ; Qg] operand image (each thread
        // copies exactly the 16-byte chunks it will later read and overwrite in place); v -> its
        // token-major image; beta.  Rows past the sequence end are zero-filled.
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int i = i0 + r;
            const bool ok = i < Lo.len;
            const size_t off = ((Lo.tok0 + (ok ? i : 0)) * a.H + ho) * kD + d0;
            if (ok) {
                ld_nc_f4(a.log_alpha + off, G[r][0], G[r][1], G[r][2], G[r][3]);
                ld_nc_f4(a.log_alpha + off + 4, G[r][4], G[r][5], G[r][6], G[r][7]);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) G[r][e] = 0.f;
            }
            const uint32_t sw = (uint32_t)((cc ^ (i & 7)) << 4);
            ptx::cp_async16(smem + S_KQ + half * S_KQ_HALF + i * 128 + sw, kp + off, ok ? 16u : 0u);
            ptx::cp_async16(smem + S_KQ + half * S_KQ_HALF + (64 + i) * 128 + sw, qp ? qp + off : kp + off,
                            (ok && qp) ? 16u : 0u);
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            const int j = (t >> 4) + 16 * m, c16 = t & 15;
            const bool ok = j < Lo.len;
            const __nv_bfloat16* src = vp + ((Lo.tok0 + (ok ? j : 0)) * a.H + ho) * kD + c16 * 8;
            ptx::cp_async16(smem + S_V + (c16 >> 3) * S_V_BLOCK + j * 128 + (((c16 & 7) ^ (j & 7)) << 4),
                            src, ok ? 16u : 0u);
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
    bool timed_out = false;

    int64_t cur = blockIdx.x;
    ChunkLoc L;
    int h = 0;
    if (cur < ntiles) {
        locate(cur, L, h);
        issue_prefetch(L, h);
    }
    for (; cur < ntiles; cur += gridDim.x) {
    char* tile = tiles + (size_t)cur * tc::TILE_BYTES;
    const int64_t nxt = cur + gridDim.x;
    ChunkLoc Ln = L;
    int hn = h;

    // ---- a1: cumulative log-decay ---------------------------------------------------------------------
#pragma unroll
    for (int r = 1; r < 4; ++r)
#pragma unroll
        for (int e = 0; e < 8; ++e) G[r][e] += G[r - 1][e];
    *reinterpret_cast<float4*>(sTot + rg * kD + d0) = make_float4(G[3][0], G[3][1], G[3][2], G[3][3]);
    *reinterpret_cast<float4*>(sTot + rg * kD + d0 + 4) = make_float4(G[3][4], G[3][5], G[3][6], G[3][7]);
    __syncthreads();
    KDA_PHASE(hdr, 0);   // loads arrived + local scan
    float base[8], gref[8], glast[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) base[e] = gref[e] = glast[e] = 0.f;
#pragma unroll
    for (int r2 = 0; r2 < 16; ++r2) {
        const float4 x0 = *reinterpret_cast<const float4*>(sTot + r2 * kD + d0);
        const float4 x1 = *reinterpret_cast<const float4*>(sTot + r2 * kD + d0 + 4);
        const float x[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            if (r2 < rg) base[e] += x[e];
            if (r2 < 8) gref[e] += x[e];
            glast[e] += x[e];
        }
    }

    // ---- gated operands ---------------------------------------------------------------------------------
    // exp(G) = exp(G - G_m) exp(G_m) and exp(G_C - G) = exp(G_m - G) exp(G_C - G_m) reuse the two
    // exponentials of the intra-chunk operands unless a channel decays by more than e^-80 on one
    // side of the middle row, in which case they are evaluated directly (no underflow of the factor)
    float cg[8], ct[8];
    bool harsh = false;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        cg[e] = __expf(gref[e]);               // exp(G_m)
        ct[e] = __expf(glast[e] - gref[e]);    // exp(G_C - G_m)
        harsh = harsh || (gref[e] < -kExpClamp) || (glast[e] - gref[e] < -kExpClamp);
    }
    if (rg == 0) {
        float gc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) gc[e] = __expf(glast[e]);
        *reinterpret_cast<float4*>(tile + tc::OFF_GC + d0 * 4) = make_float4(gc[0], gc[1], gc[2], gc[3]);
        *reinterpret_cast<float4*>(tile + tc::OFF_GC + d0 * 4 + 16) = make_float4(gc[4], gc[5], gc[6], gc[7]);
        *reinterpret_cast<float4*>(sCG + d0) = make_float4(cg[0], cg[1], cg[2], cg[3]);
        *reinterpret_cast<float4*>(sCG + d0 + 4) = make_float4(cg[4], cg[5], cg[6], cg[7]);
    }
    KDA_PHASE(hdr, 10);  // prefix + per-channel factors
    ptx::cp_async_wait_all();   // this thread's k, q chunks (and its share of v, beta) have landed
    KDA_PHASE(hdr, 11);  // cp.async wait
    float kt[4][8];   // K exp(G_C - G) for the transposed store
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int i = i0 + r;
        float kf[8], qf[8];
        const uint32_t sw = (uint32_t)((cc ^ (i & 7)) << 4);
        unpack8(*reinterpret_cast<const uint4*>(smem + S_KQ + half * S_KQ_HALF + i * 128 + sw), kf);
        unpack8(*reinterpret_cast<const uint4*>(smem + S_KQ + half * S_KQ_HALF + (64 + i) * 128 + sw), qf);
        float okg[8], oqg[8], oki[8], oqt[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float gg = G[r][e] + base[e];
            const float x = fminf(fmaxf(gg - gref[e], -kExpClamp), kExpClamp);
            const float e1 = __expf(x);                  // exp(G - G_m)
            const float e2 = __expf(-x);                 // exp(G_m - G)
            const float qs = a.scale * qf[e];
            okg[e] = kf[e] * e1;
            oqg[e] = qs * e1;
            oki[e] = kf[e] * e2;
            if (!harsh) {
                oqt[e] = oqg[e] * cg[e];
                kt[r][e] = oki[e] * ct[e];
            } else {
                oqt[e] = qs * __expf(gg);
                kt[r][e] = kf[e] * __expf(glast[e] - gg);
            }
        }
        *reinterpret_cast<uint4*>(smem + S_KQ + half * S_KQ_HALF + i * 128 + sw) =
            make_uint4(pack_bf16(okg[0], okg[1]), pack_bf16(okg[2], okg[3]), pack_bf16(okg[4], okg[5]),
                       pack_bf16(okg[6], okg[7]));
        *reinterpret_cast<uint4*>(smem + S_KQ + half * S_KQ_HALF + (64 + i) * 128 + sw) =
            make_uint4(pack_bf16(oqg[0], oqg[1]), pack_bf16(oqg[2], oqg[3]), pack_bf16(oqg[4], oqg[5]),
                       pack_bf16(oqg[6], oqg[7]));
        *reinterpret_cast<uint4*>(smem + S_KI + half * S_KI_HALF + i * 128 + sw) =
            make_uint4(pack_bf16(oki[0], oki[1]), pack_bf16(oki[2], oki[3]), pack_bf16(oki[4], oki[5]),
                       pack_bf16(oki[6], oki[7]));
        *reinterpret_cast<uint4*>(smem + S_QG + half * 8192 + i * 128 + sw) =
            make_uint4(pack_bf16(oqt[0], oqt[1]), pack_bf16(oqt[2], oqt[3]), pack_bf16(oqt[4], oqt[5]),
                       pack_bf16(oqt[6], oqt[7]));
    }
    // (K exp(G_C - G))^T: row = channel, 4 consecutive tokens per 8-byte store
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        uint2 p;
        p.x = pack_bf16(kt[0][e], kt[1][e]);
        p.y = pack_bf16(kt[2][e], kt[3][e]);
        *reinterpret_cast<uint2*>(smem + S_KT + ptx::sw128_off(d0 + e, i0)) = p;
    }

    KDA_PHASE(hdr, 12);  // element loop + stores (thread 0)
    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    KDA_PHASE(hdr, 1);   // gated operands
    ptx::tc_fence_after();

    // ---- a2 + a5: [Kg ; Qg] Ki^T ------------------------------------------------------------------------
    if (t == 0) {
        // phase-1 outputs leave through the TMA engine while the MMA runs
        ptx::bulk_s2g(tile + tc::OFF_QW, smem + S_QG, 8192);
        ptx::bulk_s2g(tile + tc::OFF_QW + tc::QW_HALF, smem + S_QG + 8192, 8192);
        ptx::bulk_s2g(tile + tc::OFF_KT, smem + S_KT, 16384);
        ptx::bulk_commit();
        const uint32_t idesc = ptx::umma_idesc_bf16(128, 64);
        const uint32_t a0 = ptx::smem_u32(smem + S_KQ), b0 = ptx::smem_u32(smem + S_KI);
#pragma unroll
        for (int k = 0; k < 8; ++k)
            ptx::umma_bf16(tmem_base, ptx::umma_desc_sw128(a0 + (k >> 2) * S_KQ_HALF + (k & 3) * 32),
                           ptx::umma_desc_sw128(b0 + (k >> 2) * S_KI_HALF + (k & 3) * 32), idesc, k > 0);
        ptx::umma_commit(mma_bar);
    }
    if (!ptx::mbar_wait(mma_bar, 0, kWaitLimitNs)) timed_out = true;
    if (t == 0) ptx::bulk_wait_read0();   // staging buffers are about to be reused
    __syncthreads();
    KDA_PHASE(hdr, 2);   // first MMA group
    ptx::tc_fence_after();
    {
        const int q4 = warp & 3, ch = warp >> 2;
        const int R = q4 * 32 + lane;
        uint32_t r[32];
        ptx::tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q4 * 32) << 16) + ch * 32, r);
        ptx::tmem_ld_wait();
        if (R < 64) {
            const int i = R;
            const float bi = sBeta[i];
#pragma unroll
            for (int j4 = 0; j4 < 32; j4 += 4) {
                float x[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int j = ch * 32 + j4 + e;
                    x[e] = (j < i) ? bi * __uint_as_float(r[j4 + e]) : 0.f;
                }
                *reinterpret_cast<float4*>(sA + i * LDT + ch * 32 + j4) = make_float4(x[0], x[1], x[2], x[3]);
            }
        } else {
            const int i = R - 64;
#pragma unroll
            for (int j8 = 0; j8 < 32; j8 += 8) {
                float x[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int j = ch * 32 + j8 + e;
                    x[e] = (j <= i) ? __uint_as_float(r[j8 + e]) : 0.f;
                }
                *reinterpret_cast<uint4*>(smem + S_AQ + ptx::sw128_off(i, ch * 32 + j8)) =
                    make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]),
                               pack_bf16(x[6], x[7]));
            }
        }
    }
    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    if (t == 0) {
        ptx::bulk_s2g(tile + tc::OFF_AQ, smem + S_AQ, 8192);
        ptx::bulk_commit();
    }
    KDA_PHASE(hdr, 3);   // TMEM -> L, Aqk

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
    KDA_PHASE(hdr, 4);   // diagonal blocks
    {   // X_IM = T_II L_IM for the six sub-diagonal blocks (1x4 outputs per work item)
        float xo[2][4];
        int nitem = 0;
        for (int item = t; item < 6 * 64; item += 256, ++nitem) {
            const int blk = item >> 6, r = (item >> 2) & 15, cg = (item & 3) * 4;
            const int I = blk < 1 ? 1 : (blk < 3 ? 2 : 3);
            const int M = blk < 1 ? 0 : (blk < 3 ? blk - 1 : blk - 3);
            const float* Tii = sT + (I * 16 + r) * LDT + I * 16;
            const float* Lim = sA + (I * 16) * LDT + M * 16 + cg;
            float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
#pragma unroll
            for (int m = 0; m < 16; ++m) {
                const float tv = Tii[m];
                const float4 lv = *reinterpret_cast<const float4*>(Lim + m * LDT);
                o0 += tv * lv.x; o1 += tv * lv.y; o2 += tv * lv.z; o3 += tv * lv.w;
            }
            xo[nitem][0] = o0; xo[nitem][1] = o1; xo[nitem][2] = o2; xo[nitem][3] = o3;
        }
        __syncthreads();
        nitem = 0;
        for (int item = t; item < 6 * 64; item += 256, ++nitem) {
            const int blk = item >> 6, r = (item >> 2) & 15, cg = (item & 3) * 4;
            const int I = blk < 1 ? 1 : (blk < 3 ? 2 : 3);
            const int M = blk < 1 ? 0 : (blk < 3 ? blk - 1 : blk - 3);
            *reinterpret_cast<float4*>(sA + (I * 16 + r) * LDT + M * 16 + cg) =
                make_float4(xo[nitem][0], xo[nitem][1], xo[nitem][2], xo[nitem][3]);
        }
    }
    __syncthreads();
    KDA_PHASE(hdr, 5);   // X
#pragma unroll
    for (int lvl = 1; lvl <= 3; ++lvl) {   // T_IJ = - sum_{M=J..I-1} X_IM T_MJ,  J = I - lvl
        const int nblk = 4 - lvl;
        if (t < nblk * 64) {
            const int I = lvl + (t >> 6), J = I - lvl, r = (t >> 2) & 15, cg = (t & 3) * 4;
            float o0 = 0.f, o1 = 0.f, o2 = 0.f, o3 = 0.f;
            for (int M = J; M < I; ++M) {
                const float* Xim = sA + (I * 16 + r) * LDT + M * 16;
                const float* Tmj = sT + (M * 16) * LDT + J * 16 + cg;
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    const float xv = Xim[m];
                    const float4 tv = *reinterpret_cast<const float4*>(Tmj + m * LDT);
                    o0 -= xv * tv.x; o1 -= xv * tv.y; o2 -= xv * tv.z; o3 -= xv * tv.w;
                }
            }
            *reinterpret_cast<float4*>(sT + (I * 16 + r) * LDT + J * 16 + cg) = make_float4(o0, o1, o2, o3);
        }
        __syncthreads();
    }

    KDA_PHASE(hdr, 6);   // block levels
    // ---- a4: Mm = T Diag(beta) as the A operand; [W | U] = Mm [Kg | V] ---------------------------------
    {
        const int i = t >> 2, jq = t & 3;
        float x[16];
        if (jq > (i >> 4)) {
#pragma unroll
            for (int e = 0; e < 16; ++e) x[e] = 0.f;
        } else {
#pragma unroll
            for (int e4 = 0; e4 < 16; e4 += 4) {
                const float4 tv = *reinterpret_cast<const float4*>(sT + i * LDT + jq * 16 + e4);
                const float4 bv = *reinterpret_cast<const float4*>(sBeta + jq * 16 + e4);
                x[e4] = tv.x * bv.x; x[e4 + 1] = tv.y * bv.y; x[e4 + 2] = tv.z * bv.z; x[e4 + 3] = tv.w * bv.w;
            }
        }
#pragma unroll
        for (int c8 = 0; c8 < 2; ++c8)
            *reinterpret_cast<uint4*>(smem + S_M + i * 128 + ((((jq * 2 + c8) ^ (i & 7))) << 4)) =
                make_uint4(pack_bf16(x[c8 * 8], x[c8 * 8 + 1]), pack_bf16(x[c8 * 8 + 2], x[c8 * 8 + 3]),
                           pack_bf16(x[c8 * 8 + 4], x[c8 * 8 + 5]), pack_bf16(x[c8 * 8 + 6], x[c8 * 8 + 7]));
    }
    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    KDA_PHASE(hdr, 7);   // Mm
    if (t == 0) {
        ptx::tc_fence_after();
        const uint32_t idesc = ptx::umma_idesc_bf16(64, 128) | ptx::kIdescBMajorMN;
        const uint32_t m0 = ptx::smem_u32(smem + S_M);
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
    if (!ptx::mbar_wait(mma_bar, 1, kWaitLimitNs)) timed_out = true;
    if (nxt < ntiles) {   // every input buffer is free again: request the next tile
        locate(nxt, Ln, hn);
        issue_prefetch(Ln, hn);
    }
    KDA_PHASE(hdr, 8);   // second MMA group
    ptx::tc_fence_after();
    {   // M = 64 accumulator: row i sits in TMEM lane 32 (i / 16) + i % 16
        const int q4 = warp & 3, part = warp >> 2;   // part 0: W (columns 0-127), part 1: U
        const int i = q4 * 16 + (lane & 15);
        const bool valid = lane < 16;
#pragma unroll
        for (int blk = 0; blk < 4; ++blk) {
            uint32_t r[32];
            ptx::tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q4 * 32) << 16) + part * 128 + blk * 32, r);
            ptx::tmem_ld_wait();
            if (valid) {
                if (part == 0) {
                    uint8_t* dst = smem + S_W + (blk >> 1) * 8192;
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8) {
                        float x[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            x[e] = __uint_as_float(r[j8 + e]) * sCG[blk * 32 + j8 + e];
                        *reinterpret_cast<uint4*>(dst + ptx::sw128_off(i, (blk & 1) * 32 + j8)) =
                            make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]),
                                       pack_bf16(x[6], x[7]));
                    }
                } else {
                    uint8_t* dst = smem + S_U + blk * tc::U_BLOCK + i * 64;
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8)
                        *reinterpret_cast<uint4*>(dst + j8 * 2) =
                            make_uint4(pack_bf16(__uint_as_float(r[j8]), __uint_as_float(r[j8 + 1])),
                                       pack_bf16(__uint_as_float(r[j8 + 2]), __uint_as_float(r[j8 + 3])),
                                       pack_bf16(__uint_as_float(r[j8 + 4]), __uint_as_float(r[j8 + 5])),
                                       pack_bf16(__uint_as_float(r[j8 + 6]), __uint_as_float(r[j8 + 7])));
                }
            }
        }
    }
    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    if (t == 0) {
        ptx::bulk_s2g(tile + tc::OFF_QW + 8192, smem + S_W, 8192);
        ptx::bulk_s2g(tile + tc::OFF_QW + tc::QW_HALF + 8192, smem + S_W + 8192, 8192);
        ptx::bulk_s2g(tile + tc::OFF_U, smem + S_U, 16384);
        ptx::bulk_commit();
        ptx::bulk_wait_read0();   // shared memory must outlive the reads of every bulk store
    }
    KDA_PHASE(hdr, 9);   // W, U epilogue
    L = Ln;
    h = hn;
    }   // tile loop

    if (timed_out && atomicCAS(&hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) hdr->where = 10;
    ptx::cp_async_wait_all();
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

kda_status_t launch_intra_tc(const ChunkArgs& a, void* tiles, WsHeader* hdr, cudaStream_t st)
{
    static bool attr_done = false;
    if (!attr_done) {
        KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)kIntraTcSmem));
        attr_done = true;
    }
    const int64_t n_tiles = (a.g1 - a.g0) * a.H;
    if (n_tiles <= 0) return KDA_OK;
    static int n_sm = 0;
    if (n_sm == 0) {
        int dev = 0;
        KDA_CUDA_TRY(cudaGetDevice(&dev));
        KDA_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    }
    const int64_t resident = 2 * (int64_t)n_sm;   // two CTAs per SM
    const unsigned grid = (unsigned)(n_tiles < resident ? n_tiles : resident);
    ProfScope ps(PROF_INTRA, st);
    kda_intra_tc<<<grid, 256, kIntraTcSmem, st>>>(a, (char*)tiles, hdr);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

}  // namespace kda
