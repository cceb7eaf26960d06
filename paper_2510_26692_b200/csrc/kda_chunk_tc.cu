// bf16 tensor-core path of the chunkwise KDA forward: the inter-chunk stage (paper Section 3.1,
// state hand-over and output equations; Appendix C's sequential loop over chunks).
//
// One CTA owns one (sequence, head, 32-column slice of dv) -- the columns of the state are
// independent under  S <- Diag(gamma^C) S + Kt^T (U - W S) -- and walks the sequence's chunks in
// order.  Per chunk:
//   MMA1  D1[128 x 32]  = [W' ; Q'] (128 x 128, bf16)  x  bf16(exp(G_m) . S) (128 x 32)
//         (the tile holds W, Gamma.Q and K relative to the chunk's middle row m; the true scales
//         exp(G_m), exp(G_C - G_m) are applied to the state here, in fp32)
//         rows 0-63 of D1 = W S, rows 64-127 = (Gamma.Q) S  (inter-chunk output term)
//   a6    V_new = U - W S            TMEM -> registers, rounded to bf16 into shared memory
//   MMA2  D1[64:128] += Aqk V_new    (a7, intra-chunk output term)
//         D3[128 x 32] = K'^T V_new  (a8; (gamma^C/Gamma).K = exp(G_C - G_m) . K')
//   a8    S <- gamma^C . S + exp(G_C - G_m) . D3      fp32 master copy of the state lives in registers (thread = dk
//                                    row), refreshed bf16 copy goes back to shared memory
//   MMA1 of the next chunk is issued (D1 is double-buffered), and while it runs:
//   a7    O = rows 64-127 of D1 -> bf16 -> global
// Operands arrive as ready-made 128-byte-swizzled K-major images through 1-D bulk copies (TMA
// engine) into a three-stage ring, completion on mbarriers; the two operands this kernel produces
// itself (state copy, V_new) are written one 64-byte row per thread and consumed as MN-major B
// operands.  MMAs are tcgen05.mma (cta_group::1, kind::f16) issued by one thread, accumulators in
// TMEM, read back with tcgen05.ld.
// Every wait is bounded: on a timeout the CTA records KDA_ERR_TIMEOUT in the workspace header,
// drains its copies, frees its TMEM and returns.
#include <cstring>

#include "kda_common.cuh"
#include "kda_ptx.cuh"
#include "kda_tiles.cuh"

namespace kda {

kda_status_t launch_intra_tc(const ChunkArgs& a, void* tiles, WsHeader* hdr, bool clear_status,
                             cudaStream_t st);

namespace {

constexpr int kNCtrl = 2;                          // MMA-issuing threads (one per control warp)

template <int NS> struct InterCfg {
    static_assert(NS == 32 || NS == 64, "state columns per CTA: one or two 32-column blocks");
    static constexpr int kStages = 3;
    static constexpr uint32_t kQW = 0;                      // [2 K-halves][128][64]: rows 0-63 W, 64-127 Gamma.Q
    static constexpr uint32_t kKT = 32768;                  // K': [2 dk-halves][64 tokens][64], MN-major A operand
    static constexpr uint32_t kAQ = 49152;                  // [64][64]; used as rows 64-127 of a 128-row operand
    static constexpr uint32_t kGC = 57344;                  // gamma^C | exp(G_m) | exp(G_C - G_m), 128 fp32 each
    static constexpr uint32_t kMainBytes = tc::OFF_U;       // the images and the three vectors are contiguous in a tile
    static constexpr uint32_t kU = tc::OFF_U;               // [64 tokens][NS] block of U
    static constexpr uint32_t kUBytes = (NS / 32) * tc::U_BLOCK;
    static constexpr uint32_t kStage = (kU + kUBytes + 1023) / 1024 * 1024;
    static constexpr uint32_t kSbf = kStages * kStage;      // B operand of MMA1, MN-major: [128 dk rows][128 B]
    static constexpr uint32_t kVn = kSbf + 128 * 128;       // B operand of MMA2, MN-major: [64 token rows][128 B]
    static constexpr uint32_t kBars = kVn + 64 * 128;
    static constexpr uint32_t kSsq = kBars + 256;           // output stage: [2][slices][64] fp32 row sums of squares
    static constexpr uint32_t kWgt = kSsq + 2 * (128 / NS) * 64 * 4;   // output stage: this slice's NS RMSNorm weights
    static constexpr uint32_t kGate = (kWgt + NS * 4 + 127) / 128 * 128;   // output stage: four [32 rows][NS] bf16 gate blocks
    static constexpr uint32_t kTotal = kGate + (NS == 32 ? 4 * 32 * NS * 2 : 0);   // (the output stage runs with 32-column slices only)
    static constexpr uint32_t kSmem = kTotal + 1024;        // slack for manual 1024-byte alignment
    static constexpr uint32_t kTxBytes = kMainBytes + kUBytes;
    static constexpr uint32_t kTmemCols = 3 * kNCtrl * NS <= 256 ? 256 : 512;   // 2 kNCtrl x D1 + kNCtrl x D3, NS columns each
    static_assert(3 * kNCtrl * NS <= 512 && kSmem <= 232448, "fits TMEM and the shared memory of one SM");
};

// sum of the kNCtrl partial accumulators (NS columns each, side by side in TMEM) of one matrix
template <int NS>
__device__ __forceinline__ void tmem_ld_sum(uint32_t taddr, float (&acc)[NS]) {
#pragma unroll
    for (int blk = 0; blk < NS / 32; ++blk) {
        uint32_t r[32], r2[32];
        ptx::tmem_ld_32x32b_x32(taddr + blk * 32, r);
        ptx::tmem_ld_32x32b_x32(taddr + NS + blk * 32, r2);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[blk * 32 + j] = __uint_as_float(r[j]) + __uint_as_float(r2[j]);
    }
}
// 1 / x by the special-function unit alone (no rounding fix-up, no branches: 32 of them interleave)
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&p);
}

// Writes NS fp32 values as one bf16 row (NS / 8 16-byte chunks) of an MN-major operand image with
// 128-byte rows and 128-byte swizzle.
template <int NS>
__device__ __forceinline__ void store_row(uint8_t* img, int row, const float (&x)[NS]) {
#pragma unroll
    for (int c = 0; c < NS / 8; ++c)
        *reinterpret_cast<uint4*>(img + row * 128 + ((c ^ (row & 7)) << 4)) =
            make_uint4(pack2(x[8 * c], x[8 * c + 1]), pack2(x[8 * c + 2], x[8 * c + 3]),
                       pack2(x[8 * c + 4], x[8 * c + 5]), pack2(x[8 * c + 6], x[8 * c + 7]));
}

// Thread roles: warps 0-3 compute (TMEM lane quadrant = warp index; thread = token row for
// V_new / O, thread = dk row for the state), warps 4 and 5 are control warps whose lane 0 issues
// the MMAs (and, in warp 4, the bulk copies).  The roles meet only on mbarriers, so issue
// latencies never sit on the compute warps' path and the output conversion overlaps the next
// chunk's first MMA.
//
// kEpi (launched as clusters of the kD / NS slice CTAs of one (sequence, head)): the output stage of
// the layer wrap runs on the output rows before they are stored.  The mean square of a row spans
// the slices, so every CTA writes its share of the row's sum of squares into the shared memory of
// all CTAs of the cluster and arrives on their barriers; two buffers used alternately suffice,
// because nobody can send chunk g + 2 before everybody has finished reading chunk g.
template <int NS, bool kEpi>
__global__ void __launch_bounds__(kEpi ? 384 : 128 + 32 * kNCtrl, 1)
kda_inter_tc(ChunkArgs a, const char* __restrict__ tiles, int n_begin, WsHeader* hdr,
             const __grid_constant__ CUtensorMap tm_g)
{
    using Cfg = InterCfg<NS>;
    constexpr int NSL = kD / NS;   // slices = CTAs of a cluster
    constexpr int NSTG = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + Cfg::kBars);        // [NSTG] operands landed
    uint64_t* mma1_bar = full + NSTG;      // MMA1 of a chunk complete
    uint64_t* mma2_bar = mma1_bar + 1;     // MMA2 of a chunk complete
    // out_bar is waited on by warps that the rest of the pipeline could, in principle, overtake by a
    // whole chunk; two barriers used alternately keep a parity wait from ever being lapped
    uint64_t* out_bar = mma2_bar + 1;      // [2] the output accumulator of a chunk is complete
    uint64_t* sbf_ready = out_bar + 2;     // 4 warp arrivals: bf16 state copy written (and stage reads done)
    uint64_t* vn_ready = sbf_ready + 1;    // 2 warp arrivals: V_new written
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(vn_ready + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint64_t* ssq_bar = vn_ready + 2;      // [2] the sums of squares of every slice's 64 rows have landed
    uint64_t* o_done = ssq_bar + 2;        // [2] (kEpi) the output warps have read a chunk's accumulator
    uint64_t* gate_bar = o_done + 2;       // [4] (kEpi) an output warp's block of gate pre-activations has landed
    float* ssq = reinterpret_cast<float*>(smem + Cfg::kSsq);
    float* s_wgt = reinterpret_cast<float*>(smem + Cfg::kWgt);
    uint8_t* sbf = smem + Cfg::kSbf;
    uint8_t* vn = smem + Cfg::kVn;

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

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < NSTG; ++s) ptx::mbar_init(&full[s], 1);
        ptx::mbar_init(mma1_bar, kNCtrl);   // one commit from each control thread
        ptx::mbar_init(mma2_bar, kNCtrl);
        ptx::mbar_init(&out_bar[0], 1);
        ptx::mbar_init(&out_bar[1], 1);
        ptx::mbar_init(sbf_ready, 4);    // one arrival per compute warp (after a warp-level sync)
        ptx::mbar_init(vn_ready, 2);
        ptx::mbar_init(&ssq_bar[0], 1);
        ptx::mbar_init(&ssq_bar[1], 1);
        ptx::mbar_init(&o_done[0], 2);
        ptx::mbar_init(&o_done[1], 2);
#pragma unroll
        for (int w4 = 0; w4 < 4; ++w4) ptx::mbar_init(&gate_bar[w4], 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, Cfg::kTmemCols);
        ptx::tmem_relinquish();
    }
    if (kEpi && tid < NS) s_wgt[tid] = a.rms_weight[slice * NS + tid];
    ptx::tc_fence_before();
    __syncthreads();
    if (kEpi) ptx::cluster_sync_all();   // every CTA's barriers exist before anybody arrives on them
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t d3 = 2 * kNCtrl * NS;   // TMEM columns: D1 {parity 0,1} x {part} first, then the D3 parts

    auto wait = [&](uint64_t* bar, uint32_t parity, int where) {
        if (*abort_flag) return;
        if (!ptx::mbar_wait(bar, parity, a.wait_limit_ns)) {
            *abort_flag = 1;
            if (atomicCAS(&hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) hdr->where = where;
        }
    };

    // a7: O = (Gamma.Q) S + Aqk V_new for token row i of chunk `it` (a thread of TMEM lanes 64-127);
    // kEpi: followed by the output stage of the layer wrap
    auto output_row = [&](int it, int i, uint32_t tmem_lane, const uint4 (&gq)[NS / 8]) {
        const uint32_t d1 = (uint32_t)(it & 1) * kNCtrl * NS;
        const int64_t tok0 = tok_begin + (cb + it - seq_c0) * kC;
        const int len = (tok_end - tok0) < kC ? (int)(tok_end - tok0) : kC;
        __nv_bfloat16* orow = op + ((tok0 + i) * a.H + h) * kD + col0;
        wait(&out_bar[it & 1], (uint32_t)(it >> 1) & 1u, 6);
        ptx::tc_fence_after();
        float ov[NS];
        tmem_ld_sum<NS>(tmem_lane + d1, ov);
        ptx::tc_fence_before();
        if (kEpi) {
            // the accumulator may be written again; this slice's share of the row's sum of squares
            // goes to every CTA of the cluster
            __syncwarp();
            if ((tid & 31) == 0) ptx::mbar_arrive(&o_done[it & 1]);
            const int b = it & 1;
            const uint32_t rank = ptx::cluster_ctarank();
            float part = 0.f;
#pragma unroll
            for (int j = 0; j < NS; ++j) part = fmaf(ov[j], ov[j], part);
            // (asynchronous stores that report their bytes to the receiver's barrier: nothing to fence)
            const uint32_t slot = ptx::smem_u32(ssq + (b * NSL + (int)rank) * kC + i);
            const uint32_t bar = ptx::smem_u32(&ssq_bar[b]);
#pragma unroll
            for (int r = 0; r < NSL; ++r)
                ptx::st_async_cluster_f32(ptx::map_to_cta(slot, (uint32_t)r), part, ptx::map_to_cta(bar, (uint32_t)r));
            // one thread per CTA and chunk arms the own barrier: the 64 rows of every slice, 4 bytes each
            if (i == 0) ptx::mbar_expect_tx(&ssq_bar[b], NSL * kC * 4);
            if (!*abort_flag && !ptx::mbar_wait_cluster(&ssq_bar[b], (uint32_t)(it >> 1) & 1u, a.wait_limit_ns)) {
                *abort_flag = 1;
                if (atomicCAS(&hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) hdr->where = 9;
            }
            float tot = 0.f;
#pragma unroll
            for (int r = 0; r < NSL; ++r) tot += ssq[(b * NSL + r) * kC + i];
            const float rstd = rsqrtf(tot * (1.f / kD) + a.rms_eps);
            const __nv_bfloat16* G = reinterpret_cast<const __nv_bfloat16*>(gq);
#pragma unroll
            for (int j = 0; j < NS; ++j)
                ov[j] = ov[j] * (rstd * s_wgt[j]) * rcp_approx(1.f + __expf(-__bfloat162float(G[j])));
        }
        if (i < len) {
#pragma unroll
            for (int j = 0; j < NS; j += 8)
                *reinterpret_cast<uint4*>(orow + j) =
                    make_uint4(pack2(ov[j], ov[j + 1]), pack2(ov[j + 2], ov[j + 3]),
                               pack2(ov[j + 4], ov[j + 5]), pack2(ov[j + 6], ov[j + 7]));
        }
    };

    if (warp >= 6) {
        // ================= output warps (kEpi launches only) =================
        // Warps 6, 7 take the even chunks, warps 10, 11 the odd ones (TMEM lanes 64-127 belong to warps
        // with index 2 or 3 modulo 4), so each has two steps of the chain for one chunk's rows.  Each
        // fetches its own 32 rows of gate pre-activations one chunk ahead with a 2-D tiled TMA load.
        if (kEpi && op && (warp & 3) >= 2) {
            const int lane = tid & 31, q2 = (warp & 3) - 2, set = warp >= 10 ? 1 : 0;
            const uint32_t tmem_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
            uint8_t* gbuf = smem + Cfg::kGate + (set * 2 + q2) * (32 * NS * 2);
            uint64_t* gbar = &gate_bar[set * 2 + q2];
            auto request_gate = [&](int it) {
                const int64_t tok0 = tok_begin + (cb + it - seq_c0) * kC;
                ptx::mbar_expect_tx(gbar, 32 * NS * 2);
                ptx::tma_load_2d(gbuf, &tm_g, h * kD + col0, (int)(tok0 + q2 * 32), gbar);
            };
            if (lane == 0 && set < nchunks) request_gate(set);
            uint32_t k = 0;
            for (int it = set; it < nchunks; it += 2, ++k) {
                uint4 gq[NS / 8];
                wait(gbar, k & 1u, 11);
#pragma unroll
                for (int c = 0; c < NS / 8; ++c) gq[c] = *reinterpret_cast<const uint4*>(gbuf + lane * (NS * 2) + c * 16);
                __syncwarp();
                if (lane == 0 && it + 2 < nchunks) {
                    ptx::fence_async_smem();   // the rows were read before the next block lands over them
                    request_gate(it + 2);
                }
                output_row(it, q2 * 32 + lane, tmem_lane, gq);
            }
        }
    } else if (warp >= 4) {
        // ================= control warps: lane 0 of each issues MMAs =================
        // Issuing one tcgen05.mma costs the issuing thread several tens of cycles whatever the tile
        // size, and both products on the sequential chain are tiny, so each is split along its
        // summation index between the control threads, into one accumulator each; the accumulators
        // are added when they are read back.  Warp 4's thread also issues the bulk copies and the
        // output product.
        const int half = warp - 4;
        if ((tid & 31) == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16(128, NS) | ptx::kIdescBMajorMN;
            const uint32_t sbf_a = ptx::smem_u32(sbf), vn_a = ptx::smem_u32(vn);
            auto issue_loads = [&](int it) {
                const int s = it % NSTG;
                const char* tile = tiles + ((size_t)(cb + it - a.g0) * a.H + h) * tc::TILE_BYTES;
                uint8_t* sb = smem + s * Cfg::kStage;
                ptx::mbar_expect_tx(&full[s], Cfg::kTxBytes);
                ptx::bulk_g2s(sb + Cfg::kQW, tile + tc::OFF_QW, Cfg::kMainBytes, &full[s]);
                ptx::bulk_g2s(sb + Cfg::kU, tile + tc::OFF_U + (size_t)(col0 / 32) * tc::U_BLOCK,
                              Cfg::kUBytes, &full[s]);
            };
            int loads_issued = 0;
            if (half == 0) {
                // the tiles come from the intra-chunk kernel launched just before this one; everything
                // above (barriers, TMEM, reading the state) may overlap that kernel's tail
                ptx::grid_dep_wait();
                for (; loads_issued < NSTG && loads_issued < nchunks; ++loads_issued) issue_loads(loads_issued);
            }
            for (int it = 0; it < nchunks; ++it) {
                const int s = it % NSTG;
                const uint32_t sb = ptx::smem_u32(smem + s * Cfg::kStage);
                // accumulators of this chunk: D1 (two parities x two halves), D3 (two halves)
                const uint32_t d1 = tmem_base + (uint32_t)((it & 1) * kNCtrl + half) * NS;
                // MMA1(it): D1 = [W ; Gamma.Q] S, this thread's half of the sum over dk
                wait(&full[s], (uint32_t)(it / NSTG) & 1u, 1);
                wait(sbf_ready, (uint32_t)it & 1u, 4);
                // (kEpi: the output rows are read by warps of their own, which may lag: this chunk's
                // accumulator is the one of chunk it - 2)
                if (kEpi && op && it >= 2) wait(&o_done[it & 1], (uint32_t)((it >> 1) - 1) & 1u, 10);
                ptx::tc_fence_after();
#pragma unroll
                for (int k = 0; k < 8 / kNCtrl; ++k) {
                    const int kk = half * (8 / kNCtrl) + k;   // 16-wide step of the sum over dk
                    ptx::umma_bf16(d1, ptx::umma_desc_sw128(sb + Cfg::kQW + (kk >> 2) * tc::QW_HALF + (kk & 3) * 32),
                                   ptx::umma_desc_sw128_mn(sbf_a + kk * 2048, 8192), idesc, k > 0);
                }
                ptx::umma_commit(mma1_bar);
                // the stage of the previous chunk is free now (its readers arrived on sbf_ready)
                if (half == 0 && it > 0 && loads_issued < nchunks) { issue_loads(loads_issued); ++loads_issued; }
                // MMA2(it): D3 = K'^T V_new (K' token-major = MN-major A operand), this thread's half of the
                // sum over the chunk's tokens.
                // The state product sits on the sequential chain: it is issued and committed first.
                wait(vn_ready, (uint32_t)it & 1u, 5);
                ptx::tc_fence_after();
#pragma unroll
                for (int k = 0; k < 4 / kNCtrl; ++k) {
                    const int kk = half * (4 / kNCtrl) + k;   // 16-wide step of the sum over tokens
                    ptx::umma_bf16(tmem_base + d3 + half * NS,
                                   ptx::umma_desc_sw128_mn(sb + Cfg::kKT + kk * 2048, tc::KI_HALF),
                                   ptx::umma_desc_sw128_mn(vn_a + kk * 2048, 8192), idesc | ptx::kIdescAMajorMN,
                                   k > 0);
                }
                ptx::umma_commit(mma2_bar);
                if (half == 0 && op) {
                    // D1[64:128] += Aqk V_new.  The 128-row A operand starts 64 rows before Aqk: those
                    // rows (the tail of the Kt image) only touch accumulator rows 0-63, which are dead
                    // once V_new has been taken.
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        ptx::umma_bf16(d1, ptx::umma_desc_sw128(sb + Cfg::kAQ - 8192 + k * 32),
                                       ptx::umma_desc_sw128_mn(vn_a + k * 2048, 8192), idesc, 1);
                    ptx::umma_commit(&out_bar[it & 1]);
                }
            }
            if (half == 0) {
                if (nchunks > 0 && op) wait(&out_bar[(nchunks - 1) & 1], (uint32_t)((nchunks - 1) >> 1) & 1u, 7);   // last output product done
                if (*abort_flag) {
                    // drain the bulk copies still in flight before the shared memory goes away
                    for (int j = (loads_issued > NSTG ? loads_issued - NSTG : 0); j < loads_issued; ++j)
                        ptx::mbar_wait(&full[j % NSTG], (uint32_t)(j / NSTG) & 1u, a.wait_limit_ns);
                }
            }
        }
    } else {
        // ================= compute warps =================
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(warp * 32) << 16);
        // one barrier arrival per warp: every lane has fenced its own writes, the warp-level sync
        // orders them before lane 0's (releasing) arrive -- 32x fewer serialised arrivals per hop
        auto warp_arrive = [&](uint64_t* bar) {
            __syncwarp();
            if ((tid & 31) == 0) ptx::mbar_arrive(bar);
        };
        // state: fp32 master in registers (thread = dk row), bf16 copy as the B operand of MMA1
        float S[NS];
        const size_t sbase = ((size_t)n * a.H + h) * (size_t)(kD * kD) + (size_t)tid * kD + col0;
#pragma unroll
        for (int j = 0; j < NS; j += 4) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (a.S_in) x = *reinterpret_cast<const float4*>(a.S_in + sbase + j);
            S[j] = x.x; S[j + 1] = x.y; S[j + 2] = x.z; S[j + 3] = x.w;
        }
        // the operand copy carries the next chunk's reference scale: bf16(exp(G_m) . S)
        auto ref_scale_of = [&](int it_next) {   // exp(G_m) of a chunk (0 past the last one)
            if (it_next >= nchunks) return 0.f;
            const int sn = it_next % NSTG;
            wait(&full[sn], (uint32_t)(it_next / NSTG) & 1u, 8);
            return reinterpret_cast<const float*>(smem + sn * Cfg::kStage + Cfg::kGC + 512)[tid];
        };
        auto store_scaled = [&](float cgn) {
            float z[NS];
#pragma unroll
            for (int j = 0; j < NS; ++j) z[j] = cgn * S[j];
            store_row<NS>(sbf, tid, z);
        };
        store_scaled(ref_scale_of(0));
        ptx::fence_async_smem();
        warp_arrive(sbf_ready);

        for (int it = 0; it < nchunks; ++it) {
            const int s = it % NSTG;
            const uint8_t* sb = smem + s * Cfg::kStage;
            const uint32_t d1 = (uint32_t)(it & 1) * kNCtrl * NS;   // first of this chunk's D1 parts
            const uint32_t par = (uint32_t)it & 1u;
            wait(&full[s], (uint32_t)(it / NSTG) & 1u, 1);   // U and gamma^C are read with plain loads
            if (warp < 2) {   // a6: V_new = U - W S  (token row = tid)
                uint4 uq[NS / 8];   // this token's NS values of U
#pragma unroll
                for (int c = 0; c < NS / 8; ++c)
                    uq[c] = *reinterpret_cast<const uint4*>(sb + Cfg::kU + (c >> 2) * tc::U_BLOCK + tc::u_off(tid, c & 3));
                const __nv_bfloat16* U = reinterpret_cast<const __nv_bfloat16*>(uq);
                wait(mma1_bar, par, 2);
                ptx::tc_fence_after();
                float x[NS];
                tmem_ld_sum<NS>(tmem_lane + d1, x);
#pragma unroll
                for (int j = 0; j < NS; ++j) x[j] = __bfloat162float(U[j]) - x[j];
                store_row<NS>(vn, tid, x);
                ptx::fence_async_smem();
                ptx::tc_fence_before();
                warp_arrive(vn_ready);
            }
            const float gc = reinterpret_cast<const float*>(sb + Cfg::kGC)[tid];          // gamma^C
            const float ct = reinterpret_cast<const float*>(sb + Cfg::kGC + 1024)[tid];   // exp(G_C - G_m)
            const float cgn = ref_scale_of(it + 1);   // fetched off the chain, before the wait below
            // S_new = gc . S + ct . D3; the part that does not need D3 is formed before the wait.  (The
            // scales are applied one after the other: ct . D3 is of ordinary size although ct can be
            // e^-80 and D3 e^+80, whereas a pre-multiplied cgn * ct would underflow.)
#pragma unroll
            for (int j = 0; j < NS; ++j) S[j] *= gc;
            wait(mma2_bar, par, 3);
            ptx::tc_fence_after();
            {   // a8: S <- gamma^C . S + exp(G_C - G_m) . (K'^T V_new) ; refresh the bf16 operand copy
                float ds[NS];
                tmem_ld_sum<NS>(tmem_lane + d3, ds);
#pragma unroll
                for (int j = 0; j < NS; ++j) S[j] = fmaf(ct, ds[j], S[j]);
                store_scaled(cgn);   // next chunk's operand copy: bf16(exp(G_m') . S_new)
                ptx::fence_async_smem();
                ptx::tc_fence_before();
                warp_arrive(sbf_ready);
            }
            if (!kEpi && warp >= 2 && op) {
                const uint4 no_gate[NS / 8] = {};
                output_row(it, tid - 64, tmem_lane, no_gate);
            }
        }
        if (*abort_flag == 0) {
            float* so = a.S_out + sbase;
#pragma unroll
            for (int j = 0; j < NS; j += 4)
                *reinterpret_cast<float4*>(so + j) = make_float4(S[j], S[j + 1], S[j + 2], S[j + 3]);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (kEpi) ptx::cluster_sync_all();   // no CTA leaves while another may still write into its shared memory
    if (warp == 0) ptx::tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

// ---- all 128 state columns in one CTA (throughput form, for calls with more chains than SMs) ------------
// Sixteen compute warps (TMEM lane quadrant = warp & 3, 32-column group = warp >> 2) share one set of
// operand images and one MMA per product with N = 128: per SM and step this moves four times the
// columns of the 32-column form.  Two control threads issue the products (one the first product, the
// other the state product and the output product); a loader thread requests every piece of a tile as
// early as its buffer frees up: the [W' ; Q'] image (free once the first product has completed), the
// K' / Aqk / U part (free once the last product of its chunk has completed and U has been read) and the
// three gate vectors, each with its own ring and its own empty / full barriers.
struct WideCfg {
    static constexpr uint32_t kA = 0;                        // [2] x [W' ; Q'] images, 32 KB each
    static constexpr uint32_t kABytes = 32768;
    static constexpr uint32_t kB = 2 * kABytes;              // [2] x (K' 16 KB | Aqk 8 KB | U 16 KB)
    static constexpr uint32_t kBBytes = 40960;
    static constexpr uint32_t kBU = 24576;                   // U inside a B part
    static constexpr uint32_t kG = kB + 2 * kBBytes;         // [3] x (gamma^C | exp(G_m) | exp(G_C - G_m))
    static constexpr uint32_t kSbf = (kG + 3 * tc::GV_BYTES + 1023) / 1024 * 1024;   // B operand of MMA1: [2 column halves][128 dk rows][128 B]
    static constexpr uint32_t kSbfHalf = 128 * 128;
    static constexpr uint32_t kVn = kSbf + 2 * kSbfHalf;     // B operand of MMA2: [2 column halves][64 token rows][128 B]
    static constexpr uint32_t kVnHalf = 64 * 128;
    static constexpr uint32_t kBars = kVn + 2 * kVnHalf;
    static constexpr uint32_t kTotal = kBars + 256;
    static constexpr uint32_t kSmem = kTotal + 1024;
    static constexpr int kThreads = 16 * 32 + 96;            // + two control warps and the loader warp
    static_assert(kSmem <= 232448, "fits the shared memory of one SM");
    static_assert(tc::OFF_AQ == tc::OFF_KI + 16384 && tc::OFF_GV == tc::OFF_AQ + 8192, "K' and Aqk are contiguous in a tile");
};

__device__ __forceinline__ void store_row32_at(uint8_t* img, int row, int c0, const float (&x)[32]) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
        *reinterpret_cast<uint4*>(img + row * 128 + (((c0 + c) ^ (row & 7)) << 4)) =
            make_uint4(pack2(x[8 * c], x[8 * c + 1]), pack2(x[8 * c + 2], x[8 * c + 3]),
                       pack2(x[8 * c + 4], x[8 * c + 5]), pack2(x[8 * c + 6], x[8 * c + 7]));
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&acc)[32]) {
    uint32_t r[32];
    ptx::tmem_ld_32x32b_x32(taddr, r);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 32; ++j) acc[j] = __uint_as_float(r[j]);
}

__global__ void __launch_bounds__(WideCfg::kThreads, 1)
kda_inter_tc_wide(ChunkArgs a, const char* __restrict__ tiles, int n_begin, WsHeader* hdr)
{
    using Cfg = WideCfg;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* fullA = reinterpret_cast<uint64_t*>(smem + Cfg::kBars);   // [2]
    uint64_t* fullB = fullA + 2;           // [2]
    uint64_t* fullG = fullB + 2;           // [3]
    uint64_t* emptyA = fullG + 3;          // [2] the first product of the chunk has completed
    uint64_t* emptyB = emptyA + 2;         // [2] the last product of the chunk has completed and U has been read
    uint64_t* emptyG = emptyB + 2;         // [3] all compute warps have read the vectors
    uint64_t* mma1_bar = emptyG + 3;
    uint64_t* mma2_bar = mma1_bar + 1;
    uint64_t* out_bar = mma2_bar + 1;      // [2]
    uint64_t* sbf_ready = out_bar + 2;     // 16 warp arrivals
    uint64_t* vn_ready = sbf_ready + 1;    // 8 warp arrivals
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(vn_ready + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint8_t* sbf = smem + Cfg::kSbf;
    uint8_t* vn = smem + Cfg::kVn;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, n = n_begin + blockIdx.z;
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

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&fullA[s], 1);
            ptx::mbar_init(&fullB[s], 1);
            ptx::mbar_init(&emptyA[s], 1);                // commit of the first control thread
            ptx::mbar_init(&emptyB[s], 1 + 8);            // commit of the second + the eight warps that read U
            ptx::mbar_init(&out_bar[s], 1);
        }
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            ptx::mbar_init(&fullG[s], 1);
            ptx::mbar_init(&emptyG[s], 16);
        }
        ptx::mbar_init(mma1_bar, 1);
        ptx::mbar_init(mma2_bar, 1);
        ptx::mbar_init(sbf_ready, 16);
        ptx::mbar_init(vn_ready, 8);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t d3 = 256;   // TMEM columns: D1 {parity 0, 1} at 0 and 128, D3 at 256

    auto wait = [&](uint64_t* bar, uint32_t parity, int where) {
        if (*abort_flag) return;
        if (!ptx::mbar_wait(bar, parity, a.wait_limit_ns)) {
            *abort_flag = 1;
            if (atomicCAS(&hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) hdr->where = where;
        }
    };
    const uint32_t idesc = ptx::umma_idesc_bf16(128, 128) | ptx::kIdescBMajorMN;
    const uint32_t sbf_a = ptx::smem_u32(sbf), vn_a = ptx::smem_u32(vn);

    if (warp == 18) {
        // ---- loader ----
        if (lane == 0) {
            ptx::grid_dep_wait();   // the tiles come from the intra-chunk kernel launched just before
            int nA = 0, nB = 0, nG = 0;
            for (int p = 0; p < nchunks && !*abort_flag; ++p) {
                const char* tile = tiles + ((size_t)(cb + p - a.g0) * a.H + h) * tc::TILE_BYTES;
                const int s2 = p & 1, s3 = p % 3;
                if (p >= 3) wait(&emptyG[s3], (uint32_t)(p / 3 - 1) & 1u, 31);
                if (*abort_flag) break;
                ptx::mbar_expect_tx(&fullG[s3], tc::GV_BYTES);
                ptx::bulk_g2s(smem + Cfg::kG + s3 * tc::GV_BYTES, tile + tc::OFF_GV, tc::GV_BYTES, &fullG[s3]);
                ++nG;
                if (p >= 2) wait(&emptyA[s2], (uint32_t)(p / 2 - 1) & 1u, 32);
                if (*abort_flag) break;
                ptx::mbar_expect_tx(&fullA[s2], Cfg::kABytes);
                ptx::bulk_g2s(smem + Cfg::kA + s2 * Cfg::kABytes, tile + tc::OFF_QW, Cfg::kABytes, &fullA[s2]);
                ++nA;
                if (p >= 2) wait(&emptyB[s2], (uint32_t)(p / 2 - 1) & 1u, 33);
                if (*abort_flag) break;
                uint8_t* sbB = smem + Cfg::kB + s2 * Cfg::kBBytes;
                ptx::mbar_expect_tx(&fullB[s2], Cfg::kBBytes);
                ptx::bulk_g2s(sbB, tile + tc::OFF_KI, 24576, &fullB[s2]);
                ptx::bulk_g2s(sbB + Cfg::kBU, tile + tc::OFF_U, 16384, &fullB[s2]);
                ++nB;
            }
            if (*abort_flag) {   // drain the copies still in flight before the shared memory goes away
                for (int j = (nG > 3 ? nG - 3 : 0); j < nG; ++j) ptx::mbar_wait(&fullG[j % 3], (uint32_t)(j / 3) & 1u, a.wait_limit_ns / 8);
                for (int j = (nA > 2 ? nA - 2 : 0); j < nA; ++j) ptx::mbar_wait(&fullA[j & 1], (uint32_t)(j >> 1) & 1u, a.wait_limit_ns / 8);
                for (int j = (nB > 2 ? nB - 2 : 0); j < nB; ++j) ptx::mbar_wait(&fullB[j & 1], (uint32_t)(j >> 1) & 1u, a.wait_limit_ns / 8);
            }
        }
    } else if (warp == 16) {
        // ---- control thread A: the first product ----
        if (lane == 0) {
            for (int it = 0; it < nchunks; ++it) {
                const int s = it & 1;
                const uint32_t sa = ptx::smem_u32(smem + Cfg::kA + s * Cfg::kABytes);
                const uint32_t d1 = tmem_base + (uint32_t)(it & 1) * 128;
                wait(&fullA[s], (uint32_t)(it >> 1) & 1u, 1);
                wait(sbf_ready, (uint32_t)it & 1u, 4);
                ptx::tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    ptx::umma_bf16(d1, ptx::umma_desc_sw128(sa + (kk >> 2) * tc::QW_HALF + (kk & 3) * 32),
                                   ptx::umma_desc_sw128_mn(sbf_a + kk * 2048, Cfg::kSbfHalf), idesc, kk > 0);
                ptx::umma_commit(mma1_bar);
                ptx::umma_commit(&emptyA[s]);
            }
            if (nchunks > 0) wait(&emptyA[(nchunks - 1) & 1], (uint32_t)((nchunks - 1) >> 1) & 1u, 7);
        }
    } else if (warp == 17) {
        // ---- control thread B: the state product and the output product ----
        if (lane == 0) {
            for (int it = 0; it < nchunks; ++it) {
                const int s = it & 1;
                const uint32_t sbB = ptx::smem_u32(smem + Cfg::kB + s * Cfg::kBBytes);
                const uint32_t d1 = tmem_base + (uint32_t)(it & 1) * 128;
                wait(&fullB[s], (uint32_t)(it >> 1) & 1u, 2);
                wait(vn_ready, (uint32_t)it & 1u, 5);
                ptx::tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    ptx::umma_bf16(tmem_base + d3, ptx::umma_desc_sw128_mn(sbB + kk * 2048, tc::KI_HALF),
                                   ptx::umma_desc_sw128_mn(vn_a + kk * 2048, Cfg::kVnHalf),
                                   idesc | ptx::kIdescAMajorMN, kk > 0);
                ptx::umma_commit(mma2_bar);
                if (op) {
                    // D1[64:128] += Aqk V_new (the 128-row A operand starts 64 rows before Aqk, in the
                    // second half of the K' image; those rows only touch accumulator rows 0-63, dead
                    // once V_new has been taken)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ptx::umma_bf16(d1, ptx::umma_desc_sw128(sbB + 8192 + kk * 32),
                                       ptx::umma_desc_sw128_mn(vn_a + kk * 2048, Cfg::kVnHalf), idesc, 1);
                    ptx::umma_commit(&out_bar[it & 1]);
                }
                ptx::umma_commit(&emptyB[s]);
            }
            // every product of this thread has completed before the TMEM goes away
            if (nchunks > 0) wait(&emptyB[(nchunks - 1) & 1], (uint32_t)((nchunks - 1) >> 1) & 1u, 8);
        }
    } else if (warp < 16) {
        // ---- compute warps ----
        const int quad = warp & 3, ch = warp >> 2;
        const int row = quad * 32 + lane;                  // token row for V_new / O, dk row for the state
        const int half = ch >> 1, c0 = (ch & 1) * 4;       // column half of the operand images, first 16-byte chunk
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)ch * 32;
        auto warp_arrive = [&](uint64_t* bar) {
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar);
        };
        float S[32];
        const size_t sbase = ((size_t)n * a.H + h) * (size_t)(kD * kD) + (size_t)row * kD + ch * 32;
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (a.S_in) x = *reinterpret_cast<const float4*>(a.S_in + sbase + j);
            S[j] = x.x; S[j + 1] = x.y; S[j + 2] = x.z; S[j + 3] = x.w;
        }
        auto ref_scale_of = [&](int g) {   // exp(G_m) of chunk g (0 past the last one)
            if (g >= nchunks) return 0.f;
            wait(&fullG[g % 3], (uint32_t)(g / 3) & 1u, 9);
            return reinterpret_cast<const float*>(smem + Cfg::kG + (g % 3) * tc::GV_BYTES + 512)[row];
        };
        auto store_scaled = [&](float cgn) {
            float z[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) z[j] = cgn * S[j];
            store_row32_at(sbf + half * Cfg::kSbfHalf, row, c0, z);
        };
        store_scaled(ref_scale_of(0));
        ptx::fence_async_smem();
        warp_arrive(sbf_ready);

        for (int it = 0; it < nchunks; ++it) {
            const int s = it & 1;
            const uint8_t* sbB = smem + Cfg::kB + s * Cfg::kBBytes;
            const uint32_t d1 = (uint32_t)(it & 1) * 128;
            const uint32_t par = (uint32_t)it & 1u;
            if (quad < 2) {   // V_new = U - W S  (token row = row)
                wait(&fullB[s], (uint32_t)(it >> 1) & 1u, 1);
                uint4 uq[4];
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    uq[c] = *reinterpret_cast<const uint4*>(sbB + Cfg::kBU + ch * tc::U_BLOCK + tc::u_off(row, c));
                warp_arrive(&emptyB[s]);
                const __nv_bfloat16* U = reinterpret_cast<const __nv_bfloat16*>(uq);
                wait(mma1_bar, par, 2);
                ptx::tc_fence_after();
                float x[32];
                tmem_ld32(tmem_lane + d1, x);
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = __bfloat162float(U[j]) - x[j];
                store_row32_at(vn + half * Cfg::kVnHalf, row, c0, x);
                ptx::fence_async_smem();
                ptx::tc_fence_before();
                warp_arrive(vn_ready);
            }
            wait(&fullG[it % 3], (uint32_t)(it / 3) & 1u, 10);
            const float* gv = reinterpret_cast<const float*>(smem + Cfg::kG + (it % 3) * tc::GV_BYTES);
            const float gc = gv[row];          // gamma^C
            const float ct = gv[256 + row];    // exp(G_C - G_m)
            const float cgn = ref_scale_of(it + 1);   // fetched off the chain, before the wait below
            warp_arrive(&emptyG[it % 3]);
#pragma unroll
            for (int j = 0; j < 32; ++j) S[j] *= gc;
            wait(mma2_bar, par, 3);
            ptx::tc_fence_after();
            {
                float ds[32];
                tmem_ld32(tmem_lane + d3, ds);
#pragma unroll
                for (int j = 0; j < 32; ++j) S[j] = fmaf(ct, ds[j], S[j]);
                store_scaled(cgn);   // next chunk's operand copy: bf16(exp(G_m') . S_new)
                ptx::fence_async_smem();
                ptx::tc_fence_before();
                warp_arrive(sbf_ready);
            }
            if (quad >= 2 && op) {   // O = (Gamma.Q) S + Aqk V_new  (token row = row - 64)
                const int i = row - 64;
                const int64_t tok0 = tok_begin + (cb + it - seq_c0) * kC;
                const int len = (tok_end - tok0) < kC ? (int)(tok_end - tok0) : kC;
                __nv_bfloat16* orow = op + ((tok0 + i) * a.H + h) * kD + ch * 32;
                wait(&out_bar[it & 1], (uint32_t)(it >> 1) & 1u, 6);
                ptx::tc_fence_after();
                float ov[32];
                tmem_ld32(tmem_lane + d1, ov);
                if (i < len) {
#pragma unroll
                    for (int j = 0; j < 32; j += 8)
                        *reinterpret_cast<uint4*>(orow + j) =
                            make_uint4(pack2(ov[j], ov[j + 1]), pack2(ov[j + 2], ov[j + 3]),
                                       pack2(ov[j + 4], ov[j + 5]), pack2(ov[j + 6], ov[j + 7]));
                }
                ptx::tc_fence_before();
            }
        }
        if (*abort_flag == 0) {
            float* so = a.S_out + sbase;
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(so + j) = make_float4(S[j], S[j + 1], S[j + 2], S[j + 3]);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem_base, 512);
}

template <int NS>
kda_status_t launch_inter_tc_t(const ChunkArgs& a, const char* tiles, int n_begin, int n_count,
                               WsHeader* hdr, bool after_intra, cudaStream_t st)
{
    using Cfg = InterCfg<NS>;
    const bool want_epi = NS == 32 && a.out_gate != nullptr && a.o != nullptr;
    if (a.out_gate != nullptr && a.o != nullptr && !want_epi)
        return fail(KDA_ERR_UNSUPPORTED, "the fused output stage runs with 32-column slices only");
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        const int slot = NS == 32 ? 2 : 3;
        if (!lk.st->attr_done[slot]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_inter_tc<NS, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)Cfg::kSmem));
            if (NS == 32)
                KDA_CUDA_TRY(cudaFuncSetAttribute(kda_inter_tc<32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                  (int)InterCfg<32>::kSmem));
            lk.st->attr_done[slot] = true;
        }
    }
    CUtensorMap tm_g;
    memset(&tm_g, 0, sizeof(tm_g));
    if (want_epi) {
        if (a.total_tokens > 0x7fffffff)
            return fail(KDA_ERR_UNSUPPORTED, "kda_layer_fwd: more than 2^31 tokens in one call");
        kda_status_t rc = make_plain_tmap(&tm_g, a.out_gate, a.total_tokens, a.H, NS, 32);
        if (rc != KDA_OK) return rc;
    }
    ProfScope ps(PROF_INTER, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kD / NS, (unsigned)a.H, (unsigned)n_count);
    cfg.blockDim = dim3(128 + 32 * kNCtrl);
    cfg.dynamicSmemBytes = Cfg::kSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    // only overlap with this library's own intra-chunk kernel, never with a caller's kernel that may
    // still be producing S0
    if (after_intra) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    if (want_epi) {
        // the slice CTAs of one (sequence, head) form a cluster (the caller has checked that enough
        // of them fit the device at once: inter_can_fuse_epilogue)
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = kD / NS;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        cfg.numAttrs = na + 1;
        cfg.blockDim = dim3(384);   // warps 6, 7, 10, 11: the output rows
        KDA_CUDA_TRY(cudaLaunchKernelEx(&cfg, kda_inter_tc<32, true>, a, tiles, n_begin, hdr, tm_g));
        count_launch();
        return KDA_OK;
    }
    KDA_CUDA_TRY(cudaLaunchKernelEx(&cfg, kda_inter_tc<NS, false>, a, tiles, n_begin, hdr, tm_g));
    count_launch();
    return KDA_OK;
}

kda_status_t launch_inter_tc_wide(const ChunkArgs& a, const char* tiles, int n_begin, int n_count, WsHeader* hdr,
                                  bool after_intra, cudaStream_t st)
{
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (!lk.st->attr_done[9]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_inter_tc_wide, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)WideCfg::kSmem));
            lk.st->attr_done[9] = true;
        }
    }
    ProfScope ps(PROF_INTER, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, (unsigned)a.H, (unsigned)n_count);
    cfg.blockDim = dim3(WideCfg::kThreads);
    cfg.dynamicSmemBytes = WideCfg::kSmem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_intra ? 1 : 0;
    KDA_CUDA_TRY(cudaLaunchKernelEx(&cfg, kda_inter_tc_wide, a, tiles, n_begin, hdr));
    count_launch();
    return KDA_OK;
}

}  // namespace

// Self-test of the bounded-wait path: one CTA waits on an mbarrier that nothing ever arrives on,
// with a short limit, and must come back with KDA_ERR_TIMEOUT in the status word.
__global__ void kda_wait_selftest_kernel(WsHeader* hdr, uint64_t limit_ns)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (!ptx::mbar_wait(&bar, 0, limit_ns)) {
        if (atomicCAS(&hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) hdr->where = 99;
    }
}

kda_status_t launch_wait_selftest(WsHeader* hdr, uint64_t limit_ns, cudaStream_t st)
{
    kda_wait_selftest_kernel<<<1, 32, 0, st>>>(hdr, limit_ns);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

namespace {
// resident clusters of the four slice CTAs of kda_inter_tc<32, true> on the current device
int query_max_clusters()
{
    using Cfg = InterCfg<32>;
    if (cudaFuncSetAttribute(kda_inter_tc<32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Cfg::kSmem) != cudaSuccess)
        return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kD / 32, 1, 1);
    cfg.blockDim = dim3(384);
    cfg.dynamicSmemBytes = Cfg::kSmem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kD / 32;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kda_inter_tc<32, true>, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}
}  // namespace

// Whether the output stage of the layer wrap can run inside the inter-chunk kernel for a call with
// `groups` (sequence, head) pairs: its slice CTAs then form clusters, and a GPC holds fewer clusters
// than its SM count suggests; if the device cannot keep as many (sequence, head) pairs in flight as
// without clusters, or the call is large enough for wider slices, the stage runs as a separate pass
// instead.  The device's answer is asked once and kept in its slot of the per-device table.
bool inter_can_fuse_epilogue(int64_t groups)
{
    DeviceLock lk;
    if (!lk.st) return false;
    if (lk.st->n_sm == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&lk.st->n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return false;
    }
    const int n_sm = lk.st->n_sm;
    if (groups * 4 > 2 * (int64_t)n_sm) return false;   // the launcher picks wider slices there
    if (lk.st->max_clusters < 0) lk.st->max_clusters = query_max_clusters();
    const int64_t plain = n_sm / (kD / 32);   // groups of slice CTAs that a launch without clusters holds
    return lk.st->max_clusters >= (groups < plain ? groups : plain);
}

size_t tc_tile_bytes() { return tc::TILE_BYTES; }

kda_status_t launch_chunk_tc(const ChunkArgs& a, void* tiles, int n_begin, int n_count,
                             WsHeader* hdr, bool clear_status, cudaStream_t st)
{
    kda_status_t rc = launch_intra_tc(a, tiles, hdr, clear_status, st);
    if (rc != KDA_OK) return rc;
    if (n_count <= 0) return KDA_OK;
    // 32 state columns per CTA give the most CTAs (the chains are latency-bound); once there are
    // more chains than the GPU can hold at one CTA per SM, 64 columns per CTA do twice the work per
    // MMA issue and halve the operand traffic from L2.
    int n_sm = 0;
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (lk.st->n_sm == 0) {
            int dev = 0;
            KDA_CUDA_TRY(cudaGetDevice(&dev));
            KDA_CUDA_TRY(cudaDeviceGetAttribute(&lk.st->n_sm, cudaDevAttrMultiProcessorCount, dev));
        }
        n_sm = lk.st->n_sm;
    }
    if (n_count > 65535)
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: more than 65535 sequences in one two-kernel pass "
                    "(use kda_set_chunk_path(2) or fewer sequences per call)");
    // more chains than SMs: the throughput form (all 128 columns per CTA); not with the fused output
    // stage.  Decided on the whole call, not on the pass, so that every pass of a call sums in the
    // same order.
    if ((int64_t)a.n_seqs * a.H > (int64_t)n_sm && a.out_gate == nullptr)
        return launch_inter_tc_wide(a, (const char*)tiles, n_begin, n_count, hdr, a.g1 > a.g0, st);
    if ((int64_t)n_count * a.H * 4 > 2 * (int64_t)n_sm)
        return launch_inter_tc_t<64>(a, (const char*)tiles, n_begin, n_count, hdr, a.g1 > a.g0, st);
    return launch_inter_tc_t<32>(a, (const char*)tiles, n_begin, n_count, hdr, a.g1 > a.g0, st);
}

}  // namespace kda
