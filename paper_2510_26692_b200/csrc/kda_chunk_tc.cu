// bf16 tensor-core path of the chunkwise KDA forward: the inter-chunk stage (paper Section 3.1,
// state hand-over and output equations; Appendix C's sequential loop over chunks).
//
// One CTA owns one (sequence, head, NS-column slice of dv) -- the columns of the state are
// independent under  S <- Diag(gamma^C) S + Kt^T (U - W S) -- and walks the sequence's chunks in
// order.  Per chunk:
//   MMA1  D1[128 x NS]  = [Gamma.Q ; W] (128 x 128, bf16)  x  S (128 x NS, bf16 copy of the state)
//         rows 0-63 of D1 = (Gamma.Q) S  (inter-chunk output term), rows 64-127 = W S
//   a6    V_new = U - W S            TMEM -> registers, rounded to bf16 into shared memory
//   MMA2  D1[0:64] += Aqk V_new      (a7, intra-chunk output term; rows 64-127 of the operand are 0)
//         D3[128 x NS] = Kt^T V_new  (a8, Kt = (gamma^C/Gamma).K)
//   a8    S <- gamma^C . S + D3      fp32 master copy of the state lives in registers (thread = dk
//                                    row), refreshed bf16 copy goes back to shared memory
//   a7    O rows 0-63 of D1 -> bf16 -> global
// Operands arrive as ready-made 128-byte-swizzled K-major images through 1-D bulk copies (TMA
// engine) into a two-stage ring, completion on mbarriers; MMAs are tcgen05.mma (cta_group::1,
// kind::f16) issued by one thread, accumulators in TMEM, read back with tcgen05.ld.
// Every wait is bounded: on a timeout the CTA records KDA_ERR_TIMEOUT in the workspace header,
// drains its copies, frees its TMEM and returns.
#include <cstdlib>

#include "kda_common.cuh"
#include "kda_ptx.cuh"
#include "kda_tiles.cuh"

namespace kda {

kda_status_t launch_intra_fma_tc(const ChunkArgs& a, void* tiles, cudaStream_t st);
kda_status_t launch_intra_tc(const ChunkArgs& a, void* tiles, WsHeader* hdr, cudaStream_t st);

namespace {

constexpr uint64_t kWaitLimitNs = 1000000000ull;   // 1 s per wait

template <int NS> struct InterCfg {
    static constexpr uint32_t kQW = 0;
    static constexpr uint32_t kKT = 32768;
    static constexpr uint32_t kAQ = 49152;                 // 16 KiB: rows 64-127 stay zero
    static constexpr uint32_t kU = 65536;
    static constexpr uint32_t kUBytes = 64 * NS * 2;
    static constexpr uint32_t kGC = kU + kUBytes;
    static constexpr uint32_t kStage = (kGC + 512 + 1023) / 1024 * 1024;
    static constexpr uint32_t kSbf = 2 * kStage;            // [2 K-halves][NS][64] bf16
    static constexpr uint32_t kSbfHalf = NS * 128;
    static constexpr uint32_t kVn = kSbf + 2 * kSbfHalf;    // [NS][64] bf16
    static constexpr uint32_t kBars = kVn + NS * 128;
    static constexpr uint32_t kTotal = kBars + 64;
    static constexpr uint32_t kSmem = kTotal + 1024;        // slack for manual 1024-byte alignment
    static constexpr uint32_t kTxBytes = 32768 + 16384 + 8192 + kUBytes + 512;
    static constexpr uint32_t kTmemCols = (2 * NS <= 32) ? 32 : (2 * NS <= 64) ? 64
                                          : (2 * NS <= 128) ? 128 : 256;
};

template <int NS>
__global__ void __launch_bounds__(128, 1)
kda_inter_tc(ChunkArgs a, const char* __restrict__ tiles, int n_begin, WsHeader* hdr)
{
    using Cfg = InterCfg<NS>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + Cfg::kBars);        // [2]
    uint64_t* mma_bar = full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(full + 3);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int slice = blockIdx.x, h = blockIdx.y, n = n_begin + blockIdx.z;
    const int col0 = slice * NS;
    __nv_bfloat16* op = reinterpret_cast<__nv_bfloat16*>(a.o);

    int64_t cb, ce, tok_begin, tok_end;
    if (a.cu_seqlens) {
        cb = a.chunk_cu[n]; ce = a.chunk_cu[n + 1];
        tok_begin = a.cu_seqlens[n]; tok_end = a.cu_seqlens[n + 1];
    } else {
        cb = (int64_t)n * a.chunks_per_seq; ce = cb + a.chunks_per_seq;
        tok_begin = (int64_t)n * a.seq_len; tok_end = tok_begin + a.seq_len;
    }
    const int64_t seq_c0 = cb;
    if (cb < a.g0) cb = a.g0;
    if (ce > a.g1) ce = a.g1;
    const int nchunks = ce > cb ? (int)(ce - cb) : 0;

    KDA_PHASE_DECL;
    if (tid == 0) {
        ptx::mbar_init(&full[0], 1);
        ptx::mbar_init(&full[1], 1);
        ptx::mbar_init(mma_bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, Cfg::kTmemCols);
        ptx::tmem_relinquish();
    }
    // rows 64-127 of the Aqk operand are zero in both stages
    for (int idx = tid; idx < 2 * 512; idx += 128) {
        const int s = idx >> 9, w = idx & 511;
        *reinterpret_cast<uint4*>(smem + s * Cfg::kStage + Cfg::kAQ + 8192 + w * 16) =
            make_uint4(0u, 0u, 0u, 0u);
    }

    // state: fp32 master in registers (thread = dk row), bf16 copy as the B operand of MMA1
    float S[NS];
    const size_t sbase = ((size_t)n * a.H + h) * (size_t)(kD * kD) + (size_t)tid * kD + col0;
#pragma unroll
    for (int j = 0; j < NS; j += 4) {
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (a.S_in) x = *reinterpret_cast<const float4*>(a.S_in + sbase + j);
        S[j] = x.x; S[j + 1] = x.y; S[j + 2] = x.z; S[j + 3] = x.w;
    }
    uint8_t* sbf = smem + Cfg::kSbf + (tid >> 6) * Cfg::kSbfHalf;
    const uint32_t kcol = tid & 63;
#pragma unroll
    for (int j = 0; j < NS; ++j)
        *reinterpret_cast<__nv_bfloat16*>(sbf + ptx::sw128_off(j, kcol)) = __float2bfloat16_rn(S[j]);

    ptx::fence_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
    const uint32_t d1 = tmem_base, d3 = tmem_base + NS;
    const uint32_t idesc = ptx::umma_idesc_bf16(128, NS);

    auto issue_loads = [&](int s, int it) {
        const char* tile = tiles + ((size_t)(cb + it - a.g0) * a.H + h) * tc::TILE_BYTES;
        uint8_t* sb = smem + s * Cfg::kStage;
        ptx::mbar_expect_tx(&full[s], Cfg::kTxBytes);
        ptx::bulk_g2s(sb + Cfg::kQW, tile + tc::OFF_QW, 32768, &full[s]);
        ptx::bulk_g2s(sb + Cfg::kKT, tile + tc::OFF_KT, 16384, &full[s]);
        ptx::bulk_g2s(sb + Cfg::kAQ, tile + tc::OFF_AQ, 8192, &full[s]);
        ptx::bulk_g2s(sb + Cfg::kU, tile + tc::OFF_U + (size_t)(col0 / 32) * tc::U_BLOCK,
                      Cfg::kUBytes, &full[s]);
        ptx::bulk_g2s(sb + Cfg::kGC, tile + tc::OFF_GC, 512, &full[s]);
    };
    auto wait = [&](uint64_t* bar, uint32_t parity, int where) {
        if (*abort_flag) return;
        if (!ptx::mbar_wait(bar, parity, kWaitLimitNs)) {
            *abort_flag = 1;
            if (atomicCAS(&hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) hdr->where = where;
        }
    };

    KDA_PHASE(hdr, 16);  // set-up
    int loads_issued = 0;
    if (tid == 0 && nchunks > 0) { issue_loads(0, 0); loads_issued = 1; }
    uint32_t mma_phase = 0;
    int it = 0;
    for (; it < nchunks; ++it) {
        const int s = it & 1;
        uint8_t* sb = smem + s * Cfg::kStage;
        if (tid == 0 && it + 1 < nchunks) { issue_loads(s ^ 1, it + 1); loads_issued = it + 2; }
        wait(&full[s], (uint32_t)(it >> 1) & 1u, 1);
        KDA_PHASE(hdr, 17);  // operand wait

        if (tid == 0) {   // MMA1: D1 = [Gamma.Q ; W] S
            ptx::tc_fence_after();
            const uint32_t a0 = ptx::smem_u32(sb + Cfg::kQW), b0 = ptx::smem_u32(smem + Cfg::kSbf);
#pragma unroll
            for (int k = 0; k < 8; ++k)
                ptx::umma_bf16(d1,
                               ptx::umma_desc_sw128(a0 + (k >> 2) * tc::QW_HALF + (k & 3) * 32),
                               ptx::umma_desc_sw128(b0 + (k >> 2) * Cfg::kSbfHalf + (k & 3) * 32),
                               idesc, k > 0);
            ptx::umma_commit(mma_bar);
        }
        wait(mma_bar, mma_phase, 2);
        KDA_PHASE(hdr, 18);  // MMA1
        mma_phase ^= 1;
        ptx::tc_fence_after();

        if (warp >= 2) {   // a6: V_new = U - W S  (token row = tid - 64)
            const int i = tid - 64;
            uint8_t* vn = smem + Cfg::kVn;
#pragma unroll
            for (int blk = 0; blk < NS / 32; ++blk) {
                uint32_t r[32];
                ptx::tmem_ld_32x32b_x32(tmem_lane + blk * 32, r);
                // this token's 32 values of U (one 64-byte row of the column block)
                const uint4* up = reinterpret_cast<const uint4*>(sb + Cfg::kU + blk * tc::U_BLOCK + i * 64);
                uint4 uq[4] = {up[0], up[1], up[2], up[3]};
                const __nv_bfloat16* U = reinterpret_cast<const __nv_bfloat16*>(uq);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int nn = blk * 32 + j;
                    const float x = __bfloat162float(U[j]) - __uint_as_float(r[j]);
                    *reinterpret_cast<__nv_bfloat16*>(vn + ptx::sw128_off(nn, i)) =
                        __float2bfloat16_rn(x);
                }
            }
        }
        ptx::fence_async_smem();
        ptx::tc_fence_before();
        __syncthreads();
        KDA_PHASE(hdr, 19);  // V_new

        if (tid == 0) {   // MMA2: D1 += [Aqk ; 0] V_new,  D3 = Kt^T V_new
            ptx::tc_fence_after();
            const uint32_t aq = ptx::smem_u32(sb + Cfg::kAQ), kt = ptx::smem_u32(sb + Cfg::kKT);
            const uint32_t b0 = ptx::smem_u32(smem + Cfg::kVn);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                ptx::umma_bf16(d1, ptx::umma_desc_sw128(aq + k * 32), ptx::umma_desc_sw128(b0 + k * 32),
                               idesc, 1);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                ptx::umma_bf16(d3, ptx::umma_desc_sw128(kt + k * 32), ptx::umma_desc_sw128(b0 + k * 32),
                               idesc, k > 0);
            ptx::umma_commit(mma_bar);
        }
        wait(mma_bar, mma_phase, 3);
        KDA_PHASE(hdr, 20);  // MMA2
        mma_phase ^= 1;
        ptx::tc_fence_after();

        {   // a8: S <- gamma^C . S + Kt^T V_new ; refresh the bf16 operand copy
            const float gc = reinterpret_cast<const float*>(sb + Cfg::kGC)[tid];
#pragma unroll
            for (int blk = 0; blk < NS / 32; ++blk) {
                uint32_t r[32];
                ptx::tmem_ld_32x32b_x32(tmem_lane + NS + blk * 32, r);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int nn = blk * 32 + j;
                    S[nn] = gc * S[nn] + __uint_as_float(r[j]);
                    *reinterpret_cast<__nv_bfloat16*>(sbf + ptx::sw128_off(nn, kcol)) =
                        __float2bfloat16_rn(S[nn]);
                }
            }
        }
        if (warp < 2 && op) {   // a7: O = (Gamma.Q) S + Aqk V_new  (token row = tid)
            const int64_t tok0 = tok_begin + (cb + it - seq_c0) * kC;
            const int len = (tok_end - tok0) < kC ? (int)(tok_end - tok0) : kC;
            __nv_bfloat16* orow = op + ((tok0 + tid) * a.H + h) * kD + col0;
#pragma unroll
            for (int blk = 0; blk < NS / 32; ++blk) {
                uint32_t r[32];
                ptx::tmem_ld_32x32b_x32(tmem_lane + blk * 32, r);
                ptx::tmem_ld_wait();
                if (tid < len) {
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        uint4 pk;
                        __nv_bfloat162 p0 = __floats2bfloat162_rn(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
                        __nv_bfloat162 p1 = __floats2bfloat162_rn(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                        __nv_bfloat162 p2 = __floats2bfloat162_rn(__uint_as_float(r[j + 4]), __uint_as_float(r[j + 5]));
                        __nv_bfloat162 p3 = __floats2bfloat162_rn(__uint_as_float(r[j + 6]), __uint_as_float(r[j + 7]));
                        pk.x = *reinterpret_cast<uint32_t*>(&p0);
                        pk.y = *reinterpret_cast<uint32_t*>(&p1);
                        pk.z = *reinterpret_cast<uint32_t*>(&p2);
                        pk.w = *reinterpret_cast<uint32_t*>(&p3);
                        *reinterpret_cast<uint4*>(orow + blk * 32 + j) = pk;
                    }
                }
            }
        }
        ptx::fence_async_smem();
        ptx::tc_fence_before();
        if (__syncthreads_or((int)*abort_flag)) break;
        KDA_PHASE(hdr, 21);  // state update + output
    }

    const bool aborted = *abort_flag != 0;
    if (aborted && tid == 0) {
        // drain the bulk copies this CTA still has in flight before its shared memory goes away
        for (int j = it; j < loads_issued; ++j)
            ptx::mbar_wait(&full[j & 1], (uint32_t)(j >> 1) & 1u, kWaitLimitNs);
    }
    if (!aborted) {
        float* so = a.S_out + sbase;
#pragma unroll
        for (int j = 0; j < NS; j += 4)
            *reinterpret_cast<float4*>(so + j) = make_float4(S[j], S[j + 1], S[j + 2], S[j + 3]);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

template <int NS>
kda_status_t launch_inter_tc_t(const ChunkArgs& a, const char* tiles, int n_begin, int n_count,
                               WsHeader* hdr, cudaStream_t st)
{
    using Cfg = InterCfg<NS>;
    static bool attr_done = false;
    if (!attr_done) {
        KDA_CUDA_TRY(cudaFuncSetAttribute(kda_inter_tc<NS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)Cfg::kSmem));
        attr_done = true;
    }
    dim3 grid(kD / NS, (unsigned)a.H, (unsigned)n_count);
    ProfScope ps(PROF_INTER, st);
    kda_inter_tc<NS><<<grid, 128, Cfg::kSmem, st>>>(a, tiles, n_begin, hdr);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

}  // namespace

size_t tc_tile_bytes() { return tc::TILE_BYTES; }

kda_status_t launch_chunk_tc(const ChunkArgs& a, void* tiles, int n_begin, int n_count,
                             WsHeader* hdr, cudaStream_t st)
{
    static const bool fma_intra = getenv("KDA_INTRA_FMA") != nullptr;   // debugging aid
    kda_status_t rc = fma_intra ? launch_intra_fma_tc(a, tiles, st) : launch_intra_tc(a, tiles, hdr, st);
    if (rc != KDA_OK) return rc;
    if (n_count <= 0) return KDA_OK;
    return launch_inter_tc_t<32>(a, (const char*)tiles, n_begin, n_count, hdr, st);
}

}  // namespace kda
