// bf16 tensor-core path of the chunkwise KDA forward (paper Section 3.1; Appendix C), as ONE
// persistent cooperative kernel with one CTA of 512 threads per SM.  Every CTA runs warp-specialised
// roles that meet only on mbarriers, named barriers and a few flag words in global memory:
//
//   intra-chunk engine (8 warps; every CTA has one in warps 0-7, CTAs without a chain role a second
//   one in warps 8-15): everything of a (chunk, head) tile that does not depend on the state --
//     a1   G = cumulative sum of log alpha over the chunk's tokens (fp32, log2 domain)
//          gated operands, bf16:  Kg = K exp(G - G_m),  Qg = scale Q exp(G - G_m),  Ki = K exp(G_m - G)
//          with G_m = G_C / 2 per channel (the middle of the chunk's log-decay range), so that
//          exp(G_i - G_j) = exp(G_i - G_m) exp(G_m - G_j) is formed from two factors of bounded range
//     a2/a5  one tcgen05 MMA group  [Kg ; Qg] (128 x 128)  x  Ki^T (128 x 64)  ->  TMEM:
//          L = Diag(beta) StrictTril(rows 0-63) (fp32),  Aqk = Tril(rows 64-127) (bf16)
//     a3   T = (I + L)^-1 by blocked forward substitution: 16x16 diagonal blocks column by column in
//          fp32 registers, sub-diagonal blocks as warp-level 16x16 products (mma.sync, tf32 inputs)
//     a4   Mm = T Diag(beta) (bf16);  second MMA group  [Mm ; Mm] x [Kg | V]  ->  W' = Mm Kg, U = Mm V
//   The tile (operand images of kda_tiles.cuh) goes to a small ring in global memory that stays in
//   L2: R tiles per running (sequence, head).
//
//   inter-chunk chain (CTAs 0 .. 4 Q - 1; warps 8-11 compute, 12-13 issue MMAs, 14 loads): one
//   32-column slice of the state of one (sequence, head), walked over the chunks in order --
//     MMA1  D1 = [W' ; Q'] x bf16(exp(G_m) . S)         rows 0-63 = W S, rows 64-127 = (Gamma.Q) S
//     a6    V_new = U - W S                              TMEM -> registers -> bf16 -> shared memory
//     MMA2  D3 = K'^T V_new ;  D1[64:128] += Aqk V_new   (a8, a7)
//     a8    S <- gamma^C . S + exp(G_C - G_m) . D3       fp32 master copy in registers
//     a7    O = D1[64:128] -> bf16 -> global
//   Tiles arrive by 1-D bulk copies (TMA engine) in three pieces with their own rings (gate vectors
//   3 deep, [W';Q'] 2 deep, K'/Aqk/U 2 deep) so that each piece is requested as early as its buffer
//   frees up.
//
// Every wait (mbarrier, flag word) is bounded by a wall-clock limit; when one runs out the role
// records KDA_ERR_TIMEOUT in the workspace header, marks the call as aborted so that every other
// waiter of the call returns at once, drains its own copies and leaves; TMEM is freed at the end.
// Tail chunks: rows past the sequence end behave as identity steps (log alpha = 0, beta = 0,
// k = q = v = 0).
#include <cuda.h>

#include <type_traits>

#include "kda_common.cuh"
#include "kda_ptx.cuh"
#include "kda_tiles.cuh"

namespace kda {
namespace {

constexpr int kThreads = 512;
constexpr int kEngThreads = 256;
constexpr int LDT = 68;                                   // padded fp32 row of the 64x64 matrix
constexpr int LDD = 16;                                   // padded fp32 row of a 16x16 diagonal block
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kClamp2 = 80.f * 1.4426950408889634f;     // the +-80 clamp in the log2 domain

// Optional role timing (compile with -DKDA_FUSED_TIMING): one thread per role accumulates the
// nanoseconds spent between marks and adds them to the header's spare words at the end.
#ifdef KDA_FUSED_TIMING
#define KT_DECL(n) uint64_t kt_last_ = ptx::globaltimer_ns(); uint32_t kt_acc_[n] = {0}
#define KT_MARK(cond, slot) do { if (cond) { const uint64_t now_ = ptx::globaltimer_ns(); kt_acc_[slot] += (uint32_t)(now_ - kt_last_); kt_last_ = now_; } } while (0)
#define KT_FLUSH(cond, hdr, base, n) do { if (cond) { for (int s_ = 0; s_ < n; ++s_) atomicAdd(&(hdr)->pad[(base) + s_], (int)(kt_acc_[s_] >> 4)); } } while (0)
#else
#define KT_DECL(n) do {} while (0)
#define KT_MARK(cond, slot) do {} while (0)
#define KT_FLUSH(cond, hdr, base, n) do {} while (0)
#endif

// ---- shared-memory map of one engine (bytes from a 1024-aligned base) ------------------------------
constexpr uint32_t E_KQ = 0;            // [2 K-halves][128 rows][64] bf16: rows 0-63 Kg, 64-127 Qg
constexpr uint32_t E_KQ_HALF = 16384;
constexpr uint32_t E_AQ = E_KQ + 8192;  // Aqk image [64][64] bf16: over rows 64-127 of the first K-half (Q' has left by then)
constexpr uint32_t E_KI = 32768;        // Ki [2 K-halves][64][64] bf16; then Mm [128][64]; then the W' staging
constexpr uint32_t E_KI_HALF = 8192;
constexpr uint32_t E_V = 49152;         // V [2 column blocks][64 tokens][64] bf16 (token-major)
constexpr uint32_t E_V_BLOCK = 8192;
constexpr uint32_t E_A = 65536;         // fp32 [64][LDT]: L, X below the diagonal, T above it (transposed block
                                        // positions); then the U staging (four [64][32] bf16 blocks)
constexpr uint32_t E_TD = E_A + 64 * LDT * 4;     // fp32 4 x [16][LDD]: diagonal blocks of T; scan exchange [8][128] before
constexpr uint32_t E_TD_BYTES = 4096;
constexpr uint32_t E_BETA = E_TD + E_TD_BYTES;    // 64 fp32
constexpr uint32_t E_DESC = E_BETA + 256;         // two tile descriptors
constexpr uint32_t E_BAR = E_DESC + 128;          // 8-byte words: mma barrier, K barrier, abort word, Q barrier,
                                                  // (first engine) TMEM slot, V barrier
constexpr uint32_t E_KS = (E_BAR + 64 + 1023) / 1024 * 1024;   // raw k of the NEXT tile [2 K-halves][64][64] bf16
constexpr uint32_t E_NORM = E_KS + 16384;         // layer mode: 1 / |k_i|, 1 / |q_i| (64 fp32 each)
constexpr uint32_t E_BYTES = E_NORM + 1024;
static_assert(E_TD_BYTES >= 8 * 128 * 4 && E_TD_BYTES >= 4 * 16 * LDD * 4, "scan exchange and diagonal blocks fit");

// ---- shared-memory map of a chain CTA (bytes from the 1024-aligned base) -----------------------------
constexpr int NS = 64;                             // state columns per chain CTA
constexpr int kSlices = kD / NS;                   // chain CTAs per (sequence, head)
constexpr int kStagesAB = 2, kStagesG = 3;
constexpr uint32_t C_QW = 0;                       // [2 K-halves][128][64]: rows 0-63 W', 64-127 Q'
constexpr uint32_t C_KT = 32768;                   // K': [2 dk-halves][64 tokens][64], MN-major A operand
constexpr uint32_t C_AQ = 49152;                   // Aqk [64][64]; used as rows 64-127 of a 128-row operand
constexpr uint32_t C_U = 57344;                    // two [64 tokens][32] blocks of U
constexpr uint32_t C_UBYTES = (NS / 32) * tc::U_BLOCK;
constexpr uint32_t C_STAGE = C_U + C_UBYTES;
constexpr uint32_t C_SBF = kStagesAB * C_STAGE;    // B operand of MMA1, MN-major: [128 dk rows][128 B] = bf16(exp(G_m) . S)
constexpr uint32_t C_VN = C_SBF + 128 * 128;       // B operand of MMA2, MN-major: [64 token rows][128 B] = V_new
constexpr uint32_t C_GV = C_VN + 64 * 128;         // [3] x (gamma^C | exp(G_m) | exp(G_C - G_m))
constexpr uint32_t C_BAR = C_GV + kStagesG * tc::GV_BYTES;
constexpr uint32_t C_BYTES = C_BAR + 256;
constexpr uint32_t kSmemBytes = 2 * E_BYTES > C_BYTES ? 2 * E_BYTES : C_BYTES;
static_assert(C_STAGE % 1024 == 0 && E_BYTES % 1024 == 0, "operand images stay 1024-byte aligned");
static_assert(kSmemBytes <= 232448, "fits the shared memory of one SM");
constexpr uint32_t kTmemCols = 512;                // two engines of 256 columns, or one chain of 384

// loads that the compiler may not sink below their issue point (register prefetch of the next tile)
__device__ __forceinline__ void ld_nc_f4(const float* p, float& a, float& b, float& c, float& d) {
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(a), "=f"(b), "=f"(c), "=f"(d)
                 : "l"(p));
}
__device__ __forceinline__ uint32_t to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
// 16x16 block products of the forward substitution on the warp-level tensor path (mma.sync
// m16n8k8, tf32 inputs rounded to nearest, fp32 accumulation): acc += A * B with A, B 16x16 fp32
// blocks in shared memory (row strides lda, ldb floats).
__device__ __forceinline__ void block16_mma(float (&acc)[2][4], const float* pa, int lda, const float* pb,
                                            int ldb, int lane) {
    const int g = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
        const uint32_t a0 = to_tf32(pa[g * lda + ks * 8 + t4]);
        const uint32_t a1 = to_tf32(pa[(g + 8) * lda + ks * 8 + t4]);
        const uint32_t a2 = to_tf32(pa[g * lda + ks * 8 + t4 + 4]);
        const uint32_t a3 = to_tf32(pa[(g + 8) * lda + ks * 8 + t4 + 4]);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const uint32_t b0 = to_tf32(pb[(ks * 8 + t4) * ldb + nt * 8 + g]);
            const uint32_t b1 = to_tf32(pb[(ks * 8 + t4 + 4) * ldb + nt * 8 + g]);
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

// ---- job / round geometry (the same formulas on the producing and the consuming side) --------------
struct RoundInfo {
    uint32_t base;   // production index of (chunk 0, slot 0) of the round
    int Qr;          // jobs in the round
};
__device__ __forceinline__ RoundInfo round_info(const FusedArgs& f, int r) {
    RoundInfo R;
    R.base = f.round_base ? f.round_base[r] : (uint32_t)r * (uint32_t)f.a.chunks_per_seq * (uint32_t)f.Q;
    const int left = f.J - r * f.Q;
    R.Qr = left < f.Q ? left : f.Q;
    return R;
}
struct JobInfo {
    int n, h, nch;
    int64_t tok_begin, tok_end;
};
__device__ __forceinline__ JobInfo job_info(const FusedArgs& f, int j) {
    JobInfo I;
    I.n = j / f.a.H;
    I.h = j - I.n * f.a.H;
    if (f.a.cu_seqlens) {
        I.tok_begin = f.a.cu_seqlens[I.n];
        I.tok_end = f.a.cu_seqlens[I.n + 1];
    } else {
        I.tok_begin = (int64_t)I.n * f.a.seq_len;
        I.tok_end = I.tok_begin + f.a.seq_len;
    }
    I.nch = (int)((I.tok_end - I.tok_begin + kC - 1) / kC);
    return I;
}
__device__ __forceinline__ unsigned long long tag(uint32_t epoch, uint32_t x) {
    return ((unsigned long long)epoch << 32) | x;
}
__device__ __forceinline__ bool call_aborted(const FusedArgs& f) {
    return *reinterpret_cast<volatile unsigned int*>(&f.hdr->abort_epoch) == f.epoch;
}
__device__ __forceinline__ void report_timeout(const FusedArgs& f, int where) {
    if (atomicCAS(&f.hdr->status, 0, (int)KDA_ERR_TIMEOUT) == 0) f.hdr->where = where;
    *reinterpret_cast<volatile unsigned int*>(&f.hdr->abort_epoch) = f.epoch;
    __threadfence();
}

// One (chunk, head) tile as the engine's scheduler thread hands it to the other 255 threads.
struct TileDesc {
    long long tok0;                  // first token of the chunk
    char* tile;                      // ring position
    unsigned long long* ready;       // its flag word
    unsigned long long ready_val;
    const unsigned long long* consumed;   // the four progress words of the slot's chain roles
    int h;
    int len;                         // valid tokens, 1..64; 0 = no more tiles for this engine
    uint32_t need;                   // the ring position is free once every progress word has reached this
    int pad[3];
};
static_assert(sizeof(TileDesc) == 64, "two descriptors fit the 128 bytes reserved");

// Hands out production indices in increasing order to whichever engine asks next (a slow engine
// then delays one tile, not every tile of a fixed share).  The counter lives in the workspace header
// and carries the call id in its upper half, so a value left by an earlier call is recognised and
// replaced by the first asker instead of having to be cleared.
__device__ __forceinline__ uint32_t fetch_index(const FusedArgs& f)
{
    unsigned long long* ctr = reinterpret_cast<unsigned long long*>(&f.hdr->pad[40]);
    for (;;) {
        const unsigned long long v = *reinterpret_cast<volatile unsigned long long*>(ctr);
        if ((uint32_t)(v >> 32) == f.epoch) return (uint32_t)atomicAdd(ctr, 1ull);
        if (atomicCAS(ctr, v, tag(f.epoch, 1u)) == v) return 0u;
    }
}
// Describes the tile with production index i; false if there is no tile at that index (a shorter
// sequence of the round, or past the end).
__device__ bool describe_tile(const FusedArgs& f, uint32_t i, TileDesc* d)
{
    d->len = 0;
    if (i >= f.n_prod) return false;
    int r;
    if (f.round_base) {
        int lo = 0, hi = f.n_rounds - 1;   // last round with base <= i
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (f.round_base[mid] <= i) lo = mid; else hi = mid - 1;
        }
        r = lo;
    } else {
        r = (int)(i / ((uint32_t)f.a.chunks_per_seq * (uint32_t)f.Q));
    }
    const RoundInfo R = round_info(f, r);
    const uint32_t il = i - R.base;
    const int c = (int)(il / (uint32_t)R.Qr), q = (int)(il - (uint32_t)c * (uint32_t)R.Qr);
    const JobInfo J = job_info(f, r * f.Q + q);
    if (c >= J.nch) return false;
    const int pos = q * f.R + c % f.R;
    d->tok0 = J.tok_begin + (int64_t)c * kC;
    const int64_t rem = J.tok_end - d->tok0;
    d->tile = f.ring + (size_t)pos * tc::TILE_BYTES;
    d->ready = f.ready + pos;
    d->ready_val = tag(f.epoch, i + 1u);
    d->consumed = f.consumed + q * kSlices;
    // the ring position was last used by chunk c - R of this job, or by the slot's job of an earlier round
    d->need = c >= f.R ? i - (uint32_t)f.R * (uint32_t)R.Qr + 1u : R.base;
    d->h = J.h;
    d->len = rem < kC ? (int)rem : kC;
    return true;
}
// The scheduler thread's look-ahead state: the request for the index after next is in flight while
// a tile is worked on, and so is a first look at the progress of the next tile's consumers; neither
// value is touched before it is needed, so the round trips cost nothing.
struct SchedState {
    unsigned long long pending;             // return value of the counter request in flight
    unsigned long long seen[kSlices];       // progress words of the next tile's consumers, read a tile early
};
// The engine's next tile: takes the index requested a tile ago, requests the one after it, skips
// indices without a tile.  ONE thread.
__device__ void next_tile(const FusedArgs& f, SchedState& ss, TileDesc* d)
{
    unsigned long long* ctr = reinterpret_cast<unsigned long long*>(&f.hdr->pad[40]);
    for (;;) {
        // (the counter carries this call's id since the engine's first request)
        const uint32_t i = (uint32_t)(ss.pending >> 32) == f.epoch ? (uint32_t)ss.pending : 0xffffffffu;
        if (i >= f.n_prod) { d->len = 0; return; }
        ss.pending = atomicAdd(ctr, 1ull);
        if (describe_tile(f, i, d)) break;
    }
#pragma unroll
    for (int sl = 0; sl < kSlices; ++sl) ss.seen[sl] = d->need > 0 ? ptx::ld_acquire_gpu(d->consumed + sl) : 0ull;
}
// Waits (bounded) until the chain roles have finished with the previous occupant of the tile's ring
// position.  Runs in ONE thread, at a point where its engine holds no unfinished tile and has
// published every finished one: a producer that waited for its consumers while sitting on a tile
// they need would deadlock.
__device__ void wait_slot_free(const FusedArgs& f, const TileDesc& d, const SchedState& ss,
                               volatile uint32_t* abort_word)
{
    if (d.need == 0) return;
    uint64_t t0 = 0;
    for (int sl = 0; sl < kSlices; ++sl) {
        unsigned long long v = ss.seen[sl];   // the look taken a tile ago usually settles it
        for (;;) {
            if ((uint32_t)(v >> 32) == f.epoch && (uint32_t)v >= d.need) break;
            v = ptx::ld_acquire_gpu(d.consumed + sl);
            if ((uint32_t)(v >> 32) == f.epoch && (uint32_t)v >= d.need) break;
            if (t0 == 0) t0 = ptx::globaltimer_ns();
            if (*abort_word || call_aborted(f)) { *abort_word = 1; return; }
            if (ptx::globaltimer_ns() - t0 > f.a.wait_limit_ns) {
                *abort_word = 1;
                report_timeout(f, 20);
                return;
            }
            ptx::nanosleep(100);
        }
    }
    ptx::fence_proxy_async_all();   // the consumers' bulk reads of the position precede our writes
}

// ====================================================================================================
// intra-chunk engine: 256 threads (te = 0..255), named barrier `bar_id`, 256 TMEM columns at tmem_e
// ====================================================================================================
// Stand-alone use (kFused = false, the intra-chunk kernel of the two-kernel schedule): tile number
// idx of the pass = (chunk of the pass) * H + head goes to position idx of a plain tile array, the
// engines take the tiles first, first + stride, ...; nothing is waited for or published.
__device__ bool static_tile(const FusedArgs& f, uint32_t idx, TileDesc* d)
{
    d->len = 0;
    if (idx >= f.n_prod) return false;
    const uint32_t gl = idx / (uint32_t)f.a.H;
    const ChunkLoc L = locate_chunk(f.a, f.a.g0 + gl);
    d->tok0 = L.tok0;
    d->tile = f.ring + (size_t)idx * tc::TILE_BYTES;
    d->ready = nullptr;
    d->ready_val = 0;
    d->consumed = nullptr;
    d->need = 0;
    d->h = (int)(idx - gl * (uint32_t)f.a.H);
    d->len = L.len;
    return true;
}

template <bool kHasQ, bool kFused, bool kLayer = false>
__device__ void engine_run(const FusedArgs& f, uint8_t* smem, uint32_t tmem_e, int bar_id, int te,
                           uint32_t first, uint32_t stride, const CUtensorMap* tm_k,
                           const CUtensorMap* tm_q, const CUtensorMap* tm_v)
{
    constexpr bool has_q = kHasQ;
    constexpr int kNW = 8, kRPT = 8;
    constexpr int kBulkThread = 128;   // lane 0 of warp 4 issues every bulk copy; thread 0 the MMAs
    constexpr int kSchedThread = 32;   // lane 0 of warp 1 finds the next tile
    constexpr int kMma2Thread = 64;    // lane 0 of warp 2 issues half of the second MMA group
    const ChunkArgs& a = f.a;
    float* sA = reinterpret_cast<float*>(smem + E_A);
    float* sTd = reinterpret_cast<float*>(smem + E_TD);
    float* sTot = reinterpret_cast<float*>(smem + E_TD);   // [8][128] during the scan
    float* sBeta = reinterpret_cast<float*>(smem + E_BETA);
    TileDesc* desc = reinterpret_cast<TileDesc*>(smem + E_DESC);
    uint64_t* mma_bar = reinterpret_cast<uint64_t*>(smem + E_BAR);
    uint64_t* bar_k = mma_bar + 1;   // raw k has landed in the staging buffer
    uint64_t* bar_q = mma_bar + 3;   // raw q has landed in rows 64-127 of the operand image
    uint64_t* bar_v = mma_bar + 5;   // v has landed
    volatile uint32_t* abort_word = reinterpret_cast<volatile uint32_t*>(mma_bar + 2);

    const int warp = te >> 5, lane = te & 31;
    auto ebar = [&]() { ptx::named_bar_sync(bar_id, kEngThreads); };

    // thread (w, c4) owns rows 8w..8w+7 and channels 4c4..4c4+3 in the gating phase
    const int c4 = lane, d0 = c4 * 4, i0 = warp * kRPT;
    float G[kRPT][4];
    float rate = 0.f, bias[4] = {0.f, 0.f, 0.f, 0.f};   // layer mode: decay-function parameters of the tile's head
    auto prefetch_regs = [&](const TileDesc& D) {
        if (kLayer) {
            // bf16 pre-activations of the decay function; the function itself is applied at the top of
            // the tile, when the registers are next looked at
            const __nv_bfloat16* gp = reinterpret_cast<const __nv_bfloat16*>(a.log_alpha) +
                                      ((size_t)D.tok0 * a.H + D.h) * kD + d0;
#pragma unroll
            for (int r = 0; r < kRPT; ++r) {
                const int i = i0 + r;
                uint32_t lo = 0u, hi = 0u;
                if (i < D.len)
                    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];"
                                 : "=r"(lo), "=r"(hi)
                                 : "l"(gp + (size_t)i * a.H * kD));
                G[r][0] = __uint_as_float(lo << 16); G[r][1] = __uint_as_float(lo & 0xffff0000u);
                G[r][2] = __uint_as_float(hi << 16); G[r][3] = __uint_as_float(hi & 0xffff0000u);
            }
            rate = a.gate_rate[D.h];
            const float4 b4 = *reinterpret_cast<const float4*>(a.gate_bias + (size_t)D.h * kD + d0);
            bias[0] = b4.x; bias[1] = b4.y; bias[2] = b4.z; bias[3] = b4.w;
            return;
        }
        const float* gp = a.log_alpha + ((size_t)D.tok0 * a.H + D.h) * kD + d0;
#pragma unroll
        for (int r = 0; r < kRPT; ++r) {
            const int i = i0 + r;
            if (i < D.len) {
                ld_nc_f4(gp + (size_t)i * a.H * kD, G[r][0], G[r][1], G[r][2], G[r][3]);
            } else {
                G[r][0] = G[r][1] = G[r][2] = G[r][3] = 0.f;
            }
        }
    };
    // k, q, v of the NEXT tile by 2-D tiled TMA loads (128-byte swizzle), each requested as soon as
    // its destination is free: k into a staging buffer (the gating loop reads it there and writes
    // the gated image), q straight into rows 64-127 of the operand image (gated in place), v into
    // the B operand buffer of the second MMA group; beta by small asynchronous copies.  Run by the
    // bulk thread (beta: by the first 64 threads).
    auto request_k = [&](const TileDesc& D) {
        ptx::mbar_expect_tx(bar_k, 16384);
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
            ptx::tma_load_2d(smem + E_KS + hf * 8192, tm_k, D.h * kD + hf * 64, (int)D.tok0, bar_k);
    };
    auto request_q = [&](const TileDesc& D) {
        ptx::mbar_expect_tx(bar_q, 16384);
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
            ptx::tma_load_2d(smem + E_KQ + hf * E_KQ_HALF + 8192, tm_q, D.h * kD + hf * 64, (int)D.tok0, bar_q);
    };
    auto request_v = [&](const TileDesc& D) {
        ptx::mbar_expect_tx(bar_v, 16384);
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
            ptx::tma_load_2d(smem + E_V + hf * E_V_BLOCK, tm_v, D.h * kD + hf * 64, (int)D.tok0, bar_v);
    };
    auto request_beta = [&](const TileDesc& D) {
        if (te < kC) {
            const bool ok = te < D.len;
            ptx::cp_async4(sBeta + te, a.beta + (D.tok0 + (ok ? te : 0)) * a.H + D.h, ok ? 4u : 0u);
        }
        ptx::cp_async_commit();
    };

    bool timed_out = false, out_of_range = false;
    bool pend_k = false, pend_q = false, pend_v = false;   // (thread 0) requests not yet waited for
    uint32_t tma_parity = 0;
    SchedState ss = {};   // (scheduler thread)
    uint32_t next_static = first;
    bool stores_pending = false;   // (bulk thread) the previous tile's staging may still be read out
    int cur = 0;
    unsigned long long* pending_ready = nullptr;   // bulk thread: flag of the tile whose stores are in flight
    unsigned long long pending_val = 0;

    if (te == kSchedThread) {
        if (kFused) {
            ss.pending = tag(f.epoch, fetch_index(f));
            next_tile(f, ss, &desc[0]);
        } else {
            static_tile(f, next_static, &desc[0]);
            next_static += stride;
        }
    }
    ebar();
    if (desc[0].len > 0 && !*abort_word) {
        prefetch_regs(desc[0]);
        if (te == kBulkThread) {
            request_k(desc[0]);
            if (has_q) request_q(desc[0]);
            request_v(desc[0]);
        }
        request_beta(desc[0]);
        pend_k = pend_v = true;
        pend_q = has_q;
    }
    KT_DECL(10);
    while (true) {
        const TileDesc D = desc[cur];
        if (D.len == 0 || *abort_word) break;
        char* tile = D.tile;
        KT_MARK(te == 0, 0);   // loop overhead

        if (kLayer) {
            // log alpha = -exp(rate) * softplus(x + bias); rows past the end of the sequence do not decay
            const float nr = -__expf(rate);
#pragma unroll
            for (int r = 0; r < kRPT; ++r)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float x = G[r][e] + bias[e];
                    const float sp = fmaxf(x, 0.f) + __logf(1.f + __expf(-fabsf(x)));
                    G[r][e] = (i0 + r < D.len) ? nr * sp : 0.f;
                }
        }
        // ---- a1: cumulative log-decay, in the log2 domain (exponentials below are bare ex2) ---------
#pragma unroll
        for (int e = 0; e < 4; ++e) G[0][e] *= kLog2e;
#pragma unroll
        for (int r = 1; r < kRPT; ++r)
#pragma unroll
            for (int e = 0; e < 4; ++e) G[r][e] = fmaf(G[r][e], kLog2e, G[r - 1][e]);
        *reinterpret_cast<float4*>(sTot + warp * kD + d0) =
            make_float4(G[kRPT - 1][0], G[kRPT - 1][1], G[kRPT - 1][2], G[kRPT - 1][3]);
        if (!kFused && te == kBulkThread && stores_pending) ptx::bulk_wait_read0();   // staging read out
        if (kFused && te == kBulkThread && pending_ready) {
            // The previous tile is complete in global memory: hand it to the chain roles.  (This also
            // means its W' / U staging has been read out: the buffers are written again below.)  It
            // has to happen before this engine may wait for a ring position: a producer that waits
            // for its consumers while holding back a tile they need would deadlock.
            ptx::bulk_wait_all0();
            ptx::fence_proxy_async_all();
            ptx::st_release_gpu(pending_ready, pending_val);
            pending_ready = nullptr;
        }
#ifdef KDA_FUSED_TIMING
        const uint64_t ts0_ = te == kSchedThread ? ptx::globaltimer_ns() : 0;
#endif
        if (kFused && te == kSchedThread) wait_slot_free(f, D, ss, abort_word);
#ifdef KDA_FUSED_TIMING
        if (te == kSchedThread) atomicAdd(&f.hdr->pad[11], (int)((ptx::globaltimer_ns() - ts0_) >> 4));
#endif
        ptx::cp_async_wait_all();             // beta
        if (kLayer && te < kC)                // (each of these threads copied its own element)
            sBeta[te] = te < D.len ? 1.f / (1.f + __expf(-sBeta[te])) : 0.f;
        ebar();
        KT_MARK(te == 0, 1);   // scan + publish + slot wait
        if (*abort_word) break;
        float base[4] = {0.f, 0.f, 0.f, 0.f}, gref[4], glast[4] = {0.f, 0.f, 0.f, 0.f};
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
        // the true scales exp(G_C), exp(G_m) and exp(G_C - G_m) go to the tile as fp32 vectors; the
        // chain applies them to the state in fp32
        if (warp == 0) {
            *reinterpret_cast<float4*>(tile + tc::OFF_GV + d0 * 4) =
                make_float4(ex2(glast[0]), ex2(glast[1]), ex2(glast[2]), ex2(glast[3]));
            *reinterpret_cast<float4*>(tile + tc::OFF_GV + 512 + d0 * 4) =
                make_float4(ex2(gref[0]), ex2(gref[1]), ex2(gref[2]), ex2(gref[3]));
            *reinterpret_cast<float4*>(tile + tc::OFF_GV + 1024 + d0 * 4) =
                make_float4(ex2(glast[0] - gref[0]), ex2(glast[1] - gref[1]), ex2(glast[2] - gref[2]),
                            ex2(glast[3] - gref[3]));
            // a channel that decays by more than e^-160 inside this chunk leaves the range of the
            // two-factor form: flag it (the clamp below keeps everything finite)
            if (fminf(fminf(glast[0], glast[1]), fminf(glast[2], glast[3])) < -2.f * kClamp2) out_of_range = true;
        }
#ifdef KDA_FUSED_TIMING
        if (te == 0) {
            const uint64_t now_ = ptx::globaltimer_ns();
        }
#endif
        if (!ptx::mbar_wait(bar_k, tma_parity, f.a.wait_limit_ns)) timed_out = true;   // raw k, q have landed
        if (has_q && !ptx::mbar_wait(bar_q, tma_parity, f.a.wait_limit_ns)) timed_out = true;
        pend_k = pend_q = false;
        KT_MARK(te == 0, 2);   // prefix + TMA wait
        // ---- gated operands ---------------------------------------------------------------------------
        // (two copies of the loop, chosen per warp: without the clamp when no channel of the warp's
        // share of the tile can reach it, since |G_i - G_m| <= |G_C| / 2)
        float* sNorm = reinterpret_cast<float*>(smem + E_NORM);
        if (kLayer) {
            // L2Norm of k and q: the warp owns its eight rows whole (32 lanes x 4 channels)
            const int hf = c4 >> 4;
            float ssk[kRPT], ssq[kRPT];
#pragma unroll
            for (int r = 0; r < kRPT; ++r) {
                const int i = i0 + r;
                const uint32_t o2 = (uint32_t)(i * 128 + ((((c4 >> 1) & 7) ^ (i & 7)) << 4) + (c4 & 1) * 8);
                const uint2 k2 = *reinterpret_cast<const uint2*>(smem + E_KS + hf * 8192 + o2);
                uint2 q2 = make_uint2(0u, 0u);
                if (has_q) q2 = *reinterpret_cast<const uint2*>(smem + E_KQ + hf * E_KQ_HALF + o2 + 8192);
                const float k0 = __uint_as_float(k2.x << 16), k1 = __uint_as_float(k2.x & 0xffff0000u);
                const float k2f = __uint_as_float(k2.y << 16), k3 = __uint_as_float(k2.y & 0xffff0000u);
                const float q0 = __uint_as_float(q2.x << 16), q1 = __uint_as_float(q2.x & 0xffff0000u);
                const float q2f = __uint_as_float(q2.y << 16), q3 = __uint_as_float(q2.y & 0xffff0000u);
                ssk[r] = k0 * k0 + k1 * k1 + k2f * k2f + k3 * k3;
                ssq[r] = q0 * q0 + q1 * q1 + q2f * q2f + q3 * q3;
            }
#pragma unroll
            for (int s = 16; s >= 1; s >>= 1)
#pragma unroll
                for (int r = 0; r < kRPT; ++r) {
                    ssk[r] += __shfl_xor_sync(0xffffffffu, ssk[r], s);
                    ssq[r] += __shfl_xor_sync(0xffffffffu, ssq[r], s);
                }
#pragma unroll
            for (int r = 0; r < kRPT; ++r)
                if (lane == r) {   // (rows past the end of the sequence are zeroed below: keep their factor finite)
                    const bool in = i0 + r < D.len;
                    sNorm[i0 + r] = in ? rsqrtf(ssk[r] + a.l2_eps) : 0.f;
                    sNorm[kC + i0 + r] = in ? rsqrtf(ssq[r] + a.l2_eps) : 0.f;
                }
            __syncwarp();
        }
        auto gate_rows = [&](auto clamp_tag) {
            constexpr bool kClamp = decltype(clamp_tag)::value;
            const int hf = c4 >> 4;                       // K-half (channels 0-63 / 64-127)
            float off[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) off[e] = base[e] - gref[e];
#pragma unroll
            for (int r = 0; r < kRPT; ++r) {
                const int i = i0 + r;
                const uint32_t o2 = (uint32_t)(i * 128 + ((((c4 >> 1) & 7) ^ (i & 7)) << 4) + (c4 & 1) * 8);
                uint8_t* pk = smem + E_KQ + hf * E_KQ_HALF + o2;
                uint2 k2 = *reinterpret_cast<const uint2*>(smem + E_KS + hf * 8192 + o2);
                uint2 q2 = make_uint2(0u, 0u);
                if (has_q) q2 = *reinterpret_cast<const uint2*>(pk + 8192);
                if (i >= D.len) k2 = q2 = make_uint2(0u, 0u);
                const float kf[4] = {__uint_as_float(k2.x << 16), __uint_as_float(k2.x & 0xffff0000u),
                                     __uint_as_float(k2.y << 16), __uint_as_float(k2.y & 0xffff0000u)};
                const float qf[4] = {__uint_as_float(q2.x << 16), __uint_as_float(q2.x & 0xffff0000u),
                                     __uint_as_float(q2.y << 16), __uint_as_float(q2.y & 0xffff0000u)};
                float okg[4], oqg[4], oki[4];
                float rk = 1.f, rq = a.scale;
                if (kLayer) {
                    rk = sNorm[i];
                    rq = a.scale * sNorm[kC + i];
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float x = G[r][e] + off[e];
                    if (kClamp) x = fminf(fmaxf(x, -kClamp2), kClamp2);
                    const float e1 = ex2(x);                     // exp(G - G_m)
                    const float e2 = ex2(-x);                    // exp(G_m - G)
                    if (kLayer) {
                        okg[e] = kf[e] * (e1 * rk);
                        oki[e] = kf[e] * (e2 * rk);
                    } else {
                        okg[e] = kf[e] * e1;
                        oki[e] = kf[e] * e2;
                    }
                    oqg[e] = rq * qf[e] * e1;
                }
                *reinterpret_cast<uint2*>(pk) = make_uint2(pack_bf16(okg[0], okg[1]), pack_bf16(okg[2], okg[3]));
                if (has_q)
                    *reinterpret_cast<uint2*>(pk + 8192) =
                        make_uint2(pack_bf16(oqg[0], oqg[1]), pack_bf16(oqg[2], oqg[3]));
                *reinterpret_cast<uint2*>(smem + E_KI + hf * E_KI_HALF + o2) =
                    make_uint2(pack_bf16(oki[0], oki[1]), pack_bf16(oki[2], oki[3]));
            }
        };
        {
            const bool may_clamp = fminf(fminf(gref[0], gref[1]), fminf(gref[2], gref[3])) < -kClamp2;
            if (__any_sync(0xffffffffu, may_clamp)) gate_rows(std::true_type{});
            else gate_rows(std::false_type{});
        }
        ptx::fence_async_smem();
        ptx::tc_fence_before();
        ebar();
        ptx::tc_fence_after();
        KT_MARK(te == 0, 3);   // gating

        // ---- a2 + a5: [Kg ; Qg] Ki^T --------------------------------------------------------------------
        if (te == kBulkThread) {
            // Q' (rows 64-127 of both K-halves of the operand image) and K' are tile contents as they are
            if (has_q) {
                ptx::bulk_s2g(tile + tc::OFF_QW + 8192, smem + E_KQ + 8192, 8192);
                ptx::bulk_s2g(tile + tc::OFF_QW + tc::QW_HALF + 8192, smem + E_KQ + E_KQ_HALF + 8192, 8192);
            }
            ptx::bulk_s2g(tile + tc::OFF_KI, smem + E_KI, 16384);
            ptx::bulk_commit();
        }
        if (te == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16(128, 64);
            const uint32_t a0 = ptx::smem_u32(smem + E_KQ), b0 = ptx::smem_u32(smem + E_KI);
#pragma unroll
            for (int k = 0; k < 8; ++k)
                ptx::umma_bf16(tmem_e, ptx::umma_desc_sw128(a0 + (k >> 2) * E_KQ_HALF + (k & 3) * 32),
                               ptx::umma_desc_sw128(b0 + (k >> 2) * E_KI_HALF + (k & 3) * 32), idesc, k > 0);
            ptx::umma_commit(mma_bar);
        }
        if (te == kMma2Thread) ptx::umma_commit(mma_bar);   // (the barrier counts both issuing threads)
        if (te == kSchedThread) {
            if (kFused) {
                next_tile(f, ss, &desc[cur ^ 1]);
            } else {
                static_tile(f, next_static, &desc[cur ^ 1]);
                next_static += stride;
            }
        }
        if (!ptx::mbar_wait(mma_bar, 0, f.a.wait_limit_ns)) timed_out = true;
        // Q' and K' have been read out of shared memory by now: Aqk goes over the Q' rows next
        if (te == kBulkThread) ptx::bulk_wait_read0();
        ebar();
        ptx::tc_fence_after();
        KT_MARK(te == 0, 4);   // MMA A
        const TileDesc Dn = desc[cur ^ 1];
        const bool has_next = Dn.len > 0 && !*abort_word;
        if (has_next) {
            prefetch_regs(Dn);   // the next tile's log alpha: its registers are free since the gating loop
            if (te == kBulkThread) request_k(Dn);   // the staging buffer was read by the gating loop
            pend_k = true;
        }
        {
            const int q4 = warp & 3, c0 = (warp >> 2) * 32;
            const int Rr = q4 * 32 + lane;
            uint32_t r[32];
            ptx::tmem_ld_32x32b_x32(tmem_e + ((uint32_t)(q4 * 32) << 16) + c0, r);
            ptx::tmem_ld_wait();
            if (Rr < 64) {
                const int i = Rr;
                const float bi = sBeta[i];
#pragma unroll
                for (int j4 = 0; j4 < 32; j4 += 4) {
                    float x[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int j = c0 + j4 + e;
                        x[e] = (j < i) ? bi * __uint_as_float(r[j4 + e]) : 0.f;
                    }
                    *reinterpret_cast<float4*>(sA + i * LDT + c0 + j4) = make_float4(x[0], x[1], x[2], x[3]);
                }
            } else if (has_q) {
                const int i = Rr - 64;
#pragma unroll
                for (int j8 = 0; j8 < 32; j8 += 8) {
                    float x[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int j = c0 + j8 + e;
                        x[e] = (j <= i) ? __uint_as_float(r[j8 + e]) : 0.f;
                    }
                    *reinterpret_cast<uint4*>(smem + E_AQ + ptx::sw128_off(i, c0 + j8)) =
                        make_uint4(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]), pack_bf16(x[4], x[5]),
                                   pack_bf16(x[6], x[7]));
                }
            }
        }
        ptx::fence_async_smem();
        ptx::tc_fence_before();
        ebar();
        if (te == kBulkThread && has_q) {
            ptx::bulk_s2g(tile + tc::OFF_AQ, smem + E_AQ, 8192);
            ptx::bulk_commit();
        }
        KT_MARK(te == 0, 5);   // A read-out

        // ---- a3: T = (I + L)^-1, blocked forward substitution -------------------------------------------
        // T's diagonal blocks live in sTd, its sub-diagonal block (I, J) in the (J, I) position of sA
        // (the upper triangle of L is empty), so L, X and T share one 64 x 64 array.
        auto blkA = [&](int I, int J) { return sA + (I * 16) * LDT + J * 16; };
        auto blkD = [&](int I) { return sTd + I * 16 * LDD; };
        if (te < 64) {   // diagonal 16x16 blocks: one column per thread, rows unrolled in registers
            const int I = te >> 4, c = te & 15;
            const float* Lb = blkA(I, I);
            float x[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                float s = (r == c) ? 1.f : 0.f;
#pragma unroll
                for (int m = 0; m < r; ++m) s -= Lb[r * LDT + m] * x[m];
                x[r] = s;
            }
#pragma unroll
            for (int r = 0; r < 16; ++r) blkD(I)[r * LDD + c] = x[r];
        }
        ebar();
        // X_IM = T_II L_IM for the six sub-diagonal blocks (one warp each, in place), then
        // T_IJ = - sum_{M=J..I-1} X_IM T_MJ in three dependency stages; the terms of a sum that do not
        // depend on blocks still being computed are taken early (kept, un-negated, in the block's place).
        //   stage A: T10, T21, T32 final;  P20 = X20 T00,  P31 = X31 T11,  P30 = X30 T00
        //   stage B: T20 = -(P20 + X21 T10),  T31 = -(P31 + X32 T21),  P30 += X31 T10
        //   stage C: T30 = -(P30 + X32 T20)
        if (warp < 6) {
            const int I = warp < 1 ? 1 : (warp < 3 ? 2 : 3);
            const int M = warp < 1 ? 0 : (warp < 3 ? warp - 1 : warp - 3);
            float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            block16_mma(acc, blkD(I), LDD, blkA(I, M), LDT, lane);
            __syncwarp();   // every lane has read its part of L_IM before anyone overwrites it
            block16_store(blkA(I, M), acc, 1.f, LDT, lane);
            __syncwarp();
            float acc2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            block16_mma(acc2, blkA(I, M), LDT, blkD(M), LDD, lane);
            block16_store(blkA(M, I), acc2, (I - M == 1) ? -1.f : 1.f, LDT, lane);
        }
        ebar();
        if (warp < 3) {
            // warp 0: T20 (M = 1), warp 1: T31 (M = 2), warp 2: P30 += X31 T10
            const int I = warp == 0 ? 2 : 3, J = warp == 1 ? 1 : 0, M = warp == 1 ? 2 : 1;
            float acc[2][4];
            block16_load(acc, blkA(J, I), LDT, lane);
            block16_mma(acc, blkA(I, M), LDT, blkA(J, M), LDT, lane);
            block16_store(blkA(J, I), acc, warp < 2 ? -1.f : 1.f, LDT, lane);
        }
        ebar();
        if (warp == 0) {
            float acc[2][4];
            block16_load(acc, blkA(0, 3), LDT, lane);
            block16_mma(acc, blkA(3, 2), LDT, blkA(0, 2), LDT, lane);
            block16_store(blkA(0, 3), acc, -1.f, LDT, lane);
        }
        // K' (overwritten by the Mm image) and the Aqk staging have been read out: the next tile's q
        // may land over the Aqk staging
        if (te == kBulkThread) {
            ptx::bulk_wait_read0();
            if (has_next && has_q) request_q(Dn);
        }
        if (has_next) pend_q = has_q;
        if (!ptx::mbar_wait(bar_v, tma_parity, f.a.wait_limit_ns)) timed_out = true;   // v has landed
        pend_v = false;
        tma_parity ^= 1;
        if (D.len < kC) {   // short last chunk: rows past the end hold other tokens' v; zero them
            for (int idx = te; idx < (kC - D.len) * 16; idx += kEngThreads) {
                const int j = D.len + (idx >> 4), c16 = idx & 15;
                *reinterpret_cast<uint4*>(smem + E_V + (c16 >> 3) * E_V_BLOCK + j * 128 +
                                          (((c16 & 7) ^ (j & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        ebar();
        KT_MARK(te == 0, 6);   // inverse

        // ---- a4: Mm = T Diag(beta) as the A operand; [W | U] = Mm [Kg | V] ---------------------------------
        {
            const int i = te >> 2, J = te & 3, I = i >> 4;   // one 16-column block of one row per thread
            const int j0 = J * 16;
            float x[16];
            if (J > I) {
#pragma unroll
                for (int e = 0; e < 16; ++e) x[e] = 0.f;
            } else {
                const float* src = (J == I) ? blkD(I) + (i & 15) * LDD : blkA(J, I) + (i & 15) * LDT;
#pragma unroll
                for (int e4 = 0; e4 < 16; e4 += 4) {
                    const float4 tv = *reinterpret_cast<const float4*>(src + e4);
                    const float4 bv = *reinterpret_cast<const float4*>(sBeta + j0 + e4);
                    x[e4] = tv.x * bv.x; x[e4 + 1] = tv.y * bv.y; x[e4 + 2] = tv.z * bv.z; x[e4 + 3] = tv.w * bv.w;
                }
            }
#pragma unroll
            for (int c8 = 0; c8 < 2; ++c8) {
                const uint4 pk = make_uint4(pack_bf16(x[c8 * 8], x[c8 * 8 + 1]), pack_bf16(x[c8 * 8 + 2], x[c8 * 8 + 3]),
                                            pack_bf16(x[c8 * 8 + 4], x[c8 * 8 + 5]), pack_bf16(x[c8 * 8 + 6], x[c8 * 8 + 7]));
                uint8_t* dst = smem + E_KI + i * 128 + ((((j0 >> 3) + c8) ^ (i & 7)) << 4);
                *reinterpret_cast<uint4*>(dst) = pk;
                *reinterpret_cast<uint4*>(dst + 8192) = pk;   // rows 64-127 repeat rows 0-63
            }
        }
        ptx::fence_async_smem();
        ptx::tc_fence_before();
        ebar();
        if (te == 0) {
            ptx::tc_fence_after();
            const uint32_t idesc = ptx::umma_idesc_bf16(128, 128) | ptx::kIdescBMajorMN;
            const uint32_t m0 = ptx::smem_u32(smem + E_KI);
            const uint32_t kg0 = ptx::smem_u32(smem + E_KQ);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                ptx::umma_bf16(tmem_e, ptx::umma_desc_sw128(m0 + k * 32),
                               ptx::umma_desc_sw128_mn(kg0 + k * 2048, E_KQ_HALF), idesc, k > 0);
            ptx::umma_commit(mma_bar);
        }
        if (te == kMma2Thread) {   // the U half of the group is issued by a second thread at the same time
            ptx::tc_fence_after();
            const uint32_t idesc = ptx::umma_idesc_bf16(128, 128) | ptx::kIdescBMajorMN;
            const uint32_t m0 = ptx::smem_u32(smem + E_KI), v0 = ptx::smem_u32(smem + E_V);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                ptx::umma_bf16(tmem_e + 128, ptx::umma_desc_sw128(m0 + k * 32),
                               ptx::umma_desc_sw128_mn(v0 + k * 2048, E_V_BLOCK), idesc, k > 0);
            ptx::umma_commit(mma_bar);
        }
        if (!ptx::mbar_wait(mma_bar, 1, f.a.wait_limit_ns)) timed_out = true;
        KT_MARK(te == 0, 7);   // Mm + MMA B
        if (has_next) {   // V and beta are free: the next tile's may land
            if (te == kBulkThread) request_v(Dn);
            request_beta(Dn);
            pend_v = true;
        }
        ptx::tc_fence_after();
        {   // The A operand held every row twice, so TMEM lanes 0-63 and 64-127 both carry rows 0-63:
            // each warp converts rows 32 (q4 & 1) + lane of one 64-column block of [W | U].
            const int q4 = warp & 3, cbk = (warp >> 2) * 2 + (q4 >> 1);
            const int col0 = cbk * 64;             // first column inside [W | U]
            const int i = (q4 & 1) * 32 + lane;
            const uint32_t ta = tmem_e + ((uint32_t)(q4 * 32) << 16) + col0;
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                uint32_t r[32];
                ptx::tmem_ld_32x32b_x32(ta + b * 32, r);
                ptx::tmem_ld_wait();
                if (col0 < 128) {   // W' = Mm Kg: K-half col0 / 64 of the [W' ; Q'] image
                    uint8_t* dst = smem + E_KI + (col0 >> 6) * 8192;
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8)
                        *reinterpret_cast<uint4*>(dst + ptx::sw128_off(i, b * 32 + j8)) =
                            make_uint4(pack_bf16(__uint_as_float(r[j8]), __uint_as_float(r[j8 + 1])),
                                       pack_bf16(__uint_as_float(r[j8 + 2]), __uint_as_float(r[j8 + 3])),
                                       pack_bf16(__uint_as_float(r[j8 + 4]), __uint_as_float(r[j8 + 5])),
                                       pack_bf16(__uint_as_float(r[j8 + 6]), __uint_as_float(r[j8 + 7])));
                } else {            // U: 32-column block (col0 - 128) / 32 + b
                    uint8_t* dst = smem + E_A + (((col0 - 128) >> 5) + b) * tc::U_BLOCK;
#pragma unroll
                    for (int j8 = 0; j8 < 32; j8 += 8)
                        *reinterpret_cast<uint4*>(dst + tc::u_off(i, j8 >> 3)) =
                            make_uint4(pack_bf16(__uint_as_float(r[j8]), __uint_as_float(r[j8 + 1])),
                                       pack_bf16(__uint_as_float(r[j8 + 2]), __uint_as_float(r[j8 + 3])),
                                       pack_bf16(__uint_as_float(r[j8 + 4]), __uint_as_float(r[j8 + 5])),
                                       pack_bf16(__uint_as_float(r[j8 + 6]), __uint_as_float(r[j8 + 7])));
                }
            }
        }
        ptx::fence_async_smem();
        ptx::tc_fence_before();
        if (timed_out) *abort_word = 1;
        ebar();
        if (te == kBulkThread) {
            ptx::bulk_s2g(tile + tc::OFF_QW, smem + E_KI, 8192);
            ptx::bulk_s2g(tile + tc::OFF_QW + tc::QW_HALF, smem + E_KI + 8192, 8192);
            ptx::bulk_s2g(tile + tc::OFF_U, smem + E_A, 16384);
            ptx::bulk_commit();
            pending_ready = D.ready;
            pending_val = D.ready_val;
            stores_pending = true;
        }
        KT_MARK(te == 0, 8);   // epilogue
#ifdef KDA_FUSED_TIMING
        if (te == 0) kt_acc_[9] += 16;   // tiles
#endif
        cur ^= 1;
    }   // tile loop
    KT_FLUSH(te == 0, f.hdr, 0, 10);

    if (timed_out) report_timeout(f, 10);
    if (out_of_range) atomicOr(&f.hdr->flags, 1);
    if (te == kBulkThread) {
        ptx::bulk_wait_all0();   // shared memory must outlive the reads of every bulk store
        if (kFused && pending_ready && !timed_out && !*abort_word) {
            ptx::fence_proxy_async_all();
            ptx::st_release_gpu(pending_ready, pending_val);
        }
    }
    ptx::cp_async_wait_all();
    // an aborted engine may still have a TMA load in flight (requested for a tile it never started)
    if (te == 0) {
        // tma_parity is the parity of the current / next tile's K and Q loads; V's flips in the Mm phase
        if (pend_k) ptx::mbar_wait(bar_k, tma_parity, f.a.wait_limit_ns);
        if (pend_q) ptx::mbar_wait(bar_q, tma_parity, f.a.wait_limit_ns);
        if (pend_v) ptx::mbar_wait(bar_v, tma_parity, f.a.wait_limit_ns);
    }
    ptx::tc_fence_before();
    ebar();
}

// ====================================================================================================
// inter-chunk chain: a whole CTA (t = 0..511), 384 TMEM columns at tmem_c
//   warps 0-7  compute: TMEM lane quadrant = warp & 3 (token row for V_new / O, dk row for the state),
//              32-column half of the slice = warp >> 2
//   warps 8-9  lane 0 of each issues MMAs;  warp 10 lane 0 requests the operand copies
// ====================================================================================================
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&p);
}
// 32 fp32 values as bf16 into row `row` (four 16-byte chunks starting at chunk `c0`) of an MN-major
// operand image with 128-byte rows and 128-byte swizzle
__device__ __forceinline__ void store_row32(uint8_t* img, int row, int c0, const float (&x)[32]) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
        *reinterpret_cast<uint4*>(img + row * 128 + (((c0 + c) ^ (row & 7)) << 4)) =
            make_uint4(pack2(x[8 * c], x[8 * c + 1]), pack2(x[8 * c + 2], x[8 * c + 3]),
                       pack2(x[8 * c + 4], x[8 * c + 5]), pack2(x[8 * c + 6], x[8 * c + 7]));
}
// sum of the two partial accumulators (NS columns apart in TMEM) of one matrix, 32 columns
__device__ __forceinline__ void tmem_ld_sum32(uint32_t taddr, float (&acc)[32]) {
#pragma unroll
    for (int hb = 0; hb < 2; ++hb) {
        uint32_t r[16], r2[16];
        ptx::tmem_ld_32x32b_x16(taddr + hb * 16, r);
        ptx::tmem_ld_32x32b_x16(taddr + NS + hb * 16, r2);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[hb * 16 + j] = __uint_as_float(r[j]) + __uint_as_float(r2[j]);
    }
}

template <bool kHasQ>
__device__ void chain_run(const FusedArgs& f, uint8_t* smem, uint32_t tmem_c, int t, int q, int slice)
{
    const ChunkArgs& a = f.a;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C_BAR);
    uint64_t* fullA = bars;                  // [2] [W';Q'] landed
    uint64_t* fullB = fullA + 2;             // [2] K', Aqk, U landed
    uint64_t* fullG = fullB + 2;             // [3] gate vectors landed
    uint64_t* emptyA = fullG + 3;            // [2] MMA1 done with the stage
    uint64_t* emptyB = emptyA + 2;           // [2] MMA2 / output product and the U readers done with the stage
    uint64_t* emptyG = emptyB + 2;           // [3] gate vectors read
    uint64_t* mma1_bar = emptyG + 3;         // MMA1 of a chunk complete
    uint64_t* mma2_bar = mma1_bar + 1;       // MMA2 of a chunk complete
    uint64_t* out_bar = mma2_bar + 1;        // [2] output accumulator of a chunk complete (alternating)
    uint64_t* sbf_ready = out_bar + 2;       // 8 warp arrivals: bf16 state copy written
    uint64_t* vn_ready = sbf_ready + 1;      // 4 warp arrivals: V_new written
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(vn_ready + 1);
    uint8_t* sbf = smem + C_SBF;
    uint8_t* vn = smem + C_VN;

    const int warp = t >> 5, lane = t & 31;
    const int col0 = slice * NS;
    __nv_bfloat16* op = kHasQ ? reinterpret_cast<__nv_bfloat16*>(a.o) : nullptr;

    if (t == 0) {
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&fullA[s], 1);
            ptx::mbar_init(&fullB[s], 1);
            ptx::mbar_init(&emptyA[s], 2);    // one commit from each MMA-issuing thread
            ptx::mbar_init(&emptyB[s], 6);    // two commits + the four warps that read U
            ptx::mbar_init(&out_bar[s], 1);
        }
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            ptx::mbar_init(&fullG[s], 1);
            ptx::mbar_init(&emptyG[s], 8);    // the eight compute warps
        }
        ptx::mbar_init(mma1_bar, 2);
        ptx::mbar_init(mma2_bar, 2);
        ptx::mbar_init(sbf_ready, 8);
        ptx::mbar_init(vn_ready, 4);
        abort_flag[0] = 0;
        abort_flag[1] = 0;   // s_ready
        abort_flag[2] = 0;   // s_done
        abort_flag[3] = 0;   // s_exit
        ptx::fence_mbar_init();
    }
    __syncthreads();

    auto wait = [&](uint64_t* bar, uint32_t parity, int where) {
        if (*abort_flag) return;
        if (ptx::mbar_try(bar, parity)) return;
        const uint64_t t0 = ptx::globaltimer_ns();
        uint32_t spins = 0;
        while (!ptx::mbar_try(bar, parity)) {
            if ((++spins & 15u) == 0) {
                if (*abort_flag) return;
                if (call_aborted(f)) { *abort_flag = 1; return; }
                if (ptx::globaltimer_ns() - t0 > f.a.wait_limit_ns) {
                    *abort_flag = 1;
                    report_timeout(f, where);
                    return;
                }
            }
        }
    };
    // TMEM columns: D1 {parity 0,1} x {part 0,1} (NS each), then the two D3 parts
    const uint32_t d1c = tmem_c, d3c = tmem_c + 4 * NS;

    // two words the loader and the flag thread talk through (shared memory, CTA-scope ordering)
    volatile uint32_t* s_ready = abort_flag + 1;   // chunks (running number) whose tiles are complete in the ring
    volatile uint32_t* s_done = abort_flag + 2;    // progress value to publish for the engines
    volatile uint32_t* s_exit = abort_flag + 3;    // the loader has finished
    if (warp == 11) {
        // ================= flag thread: all traffic with the flag words in global memory =================
        // An acquire load or a release store at GPU scope costs of the order of a microsecond; done by
        // the loader they would sit on the chain's path once per chunk.  This thread confirms tiles
        // ahead of the loader (up to the ring depth) and publishes the loader's progress behind it.
        if (lane == 0) {
            unsigned long long* cw = f.consumed + q * kSlices + slice;
            uint32_t pr = 0, published = 0;
            int r = 0, c = 0;
            bool jobs_left = r * f.Q + q < f.J;
            RoundInfo R = {0, 1};
            JobInfo J = {};
            auto load_job = [&]() {
                while (jobs_left) {
                    R = round_info(f, r);
                    J = job_info(f, r * f.Q + q);
                    if (J.nch > 0) break;
                    ++r;
                    jobs_left = r * f.Q + q < f.J;
                }
                c = 0;
            };
            load_job();
            uint64_t t0 = 0;
            while (!*abort_flag) {
                bool progressed = false;
                if (jobs_left) {
                    const int pos = q * f.R + c % f.R;
                    const uint32_t idx = R.base + (uint32_t)c * (uint32_t)R.Qr + (uint32_t)q;
                    if (ptx::ld_acquire_gpu(f.ready + pos) == tag(f.epoch, idx + 1u)) {
                        ++pr;
                        __threadfence_block();
                        *s_ready = pr;
                        progressed = true;
                        if (++c == J.nch) {
                            ++r;
                            jobs_left = r * f.Q + q < f.J;
                            load_job();
                        }
                    }
                }
                const uint32_t d = *s_done;
                if (d != published) {
                    __threadfence_block();
                    ptx::st_release_gpu(cw, tag(f.epoch, d));
                    published = d;
                    progressed = true;
                }
                if (progressed) {
                    t0 = 0;
                } else {
                    if (*s_exit && *s_done == published) break;
                    if (t0 == 0) t0 = ptx::globaltimer_ns();
                    if (call_aborted(f)) { *abort_flag = 1; break; }
                    if (jobs_left && ptx::globaltimer_ns() - t0 > f.a.wait_limit_ns) {
                        *abort_flag = 1;
                        report_timeout(f, 30);
                        break;
                    }
                    ptx::nanosleep(32);
                }
            }
        }
    } else if (warp == 10) {
        // ================= loader: one thread requests every piece as early as its buffer frees up =======
        if (lane == 0) {
            uint32_t p = 0;                       // running chunk number of this chain role
            uint32_t nG = 0, nA = 0, nB = 0;      // pieces requested so far
            // production index + 1 of the last two chunks; a chunk counts as consumed (its ring
            // position may be overwritten) once its copies have landed, which is certain when the
            // stage it went to is free again, i.e. two chunks later.  A ring of fewer than four
            // positions cannot afford that lag: there the landing is waited for.
            uint32_t done1 = 0, done2 = 0;
            const bool lazy = f.R >= 4;
            KT_DECL(6);
            auto landed = [&](uint32_t pp) {
                wait(&fullG[pp % 3], (pp / 3) & 1u, 31);
                wait(&fullA[pp & 1], (pp >> 1) & 1u, 32);
                wait(&fullB[pp & 1], (pp >> 1) & 1u, 33);
            };
            for (int r = 0; r * f.Q + q < f.J && !*abort_flag; ++r) {
                const RoundInfo R = round_info(f, r);
                const JobInfo J = job_info(f, r * f.Q + q);
                const uint32_t p0 = p;
                for (int c = 0; c < J.nch && !*abort_flag; ++c, ++p) {
                    const int pos = q * f.R + c % f.R;
                    const char* tile = f.ring + (size_t)pos * tc::TILE_BYTES;
                    const uint32_t idx = R.base + (uint32_t)c * (uint32_t)R.Qr + (uint32_t)q;
                    KT_MARK(true, 0);
                    {   // the engines have completed the tile (confirmed by the flag thread)
                        uint64_t t0 = 0;
                        while (*s_ready <= p) {
                            if (t0 == 0) t0 = ptx::globaltimer_ns();
                            if (*abort_flag) break;
                            if (ptx::globaltimer_ns() - t0 > 2 * f.a.wait_limit_ns) {   // (the flag thread gives up first)
                                *abort_flag = 1;
                                report_timeout(f, 37);
                                break;
                            }
                        }
                        if (*abort_flag) break;
                        __threadfence_block();
                        ptx::fence_proxy_async_all();
                    }
                    KT_MARK(true, 1);   // tile ready
                    const uint32_t s2 = p & 1, s3 = p % 3;
                    uint8_t* sb = smem + s2 * C_STAGE;
                    wait(&emptyG[s3], ((p / 3) & 1u) ^ 1u, 34);
                    if (*abort_flag) break;
                    ptx::mbar_expect_tx(&fullG[s3], tc::GV_BYTES);
                    ptx::bulk_g2s(smem + C_GV + s3 * tc::GV_BYTES, tile + tc::OFF_GV, tc::GV_BYTES, &fullG[s3]);
                    ++nG;
                    wait(&emptyA[s2], ((p >> 1) & 1u) ^ 1u, 35);
                    if (*abort_flag) break;
                    if (kHasQ) {
                        ptx::mbar_expect_tx(&fullA[s2], 32768);
                        ptx::bulk_g2s(sb + C_QW, tile + tc::OFF_QW, 32768, &fullA[s2]);
                    } else {   // state-only call: only the W' rows exist
                        ptx::mbar_expect_tx(&fullA[s2], 16384);
                        ptx::bulk_g2s(sb + C_QW, tile + tc::OFF_QW, 8192, &fullA[s2]);
                        ptx::bulk_g2s(sb + C_QW + tc::QW_HALF, tile + tc::OFF_QW + tc::QW_HALF, 8192, &fullA[s2]);
                    }
                    ++nA;
                    wait(&emptyB[s2], ((p >> 1) & 1u) ^ 1u, 36);
                    if (*abort_flag) break;
                    ptx::mbar_expect_tx(&fullB[s2], (kHasQ ? 24576u : 16384u) + C_UBYTES);
                    ptx::bulk_g2s(sb + C_KT, tile + tc::OFF_KI, kHasQ ? 24576u : 16384u, &fullB[s2]);
                    ptx::bulk_g2s(sb + C_U, tile + tc::OFF_U + (size_t)slice * C_UBYTES, C_UBYTES, &fullB[s2]);
                    ++nB;
                    KT_MARK(true, 2);   // buffers free + requests
                    if (lazy) {
                        // stage s2 was free: the chunk that used it two steps ago (if of this job) has landed
                        if (p >= p0 + 2) *s_done = done2;
                    } else if (p > p0) {
                        landed(p - 1);
                        if (!*abort_flag) *s_done = done1;
                    }
                    done2 = done1;
                    done1 = idx + 1u;
                    KT_MARK(true, 3);   // progress handed to the flag thread
                }
                if (*abort_flag) break;
                // the job is over for this slice: once its last copies have landed, everything of this
                // round counts as consumed
                if (p > p0) landed(p - 1);
                if (p > p0 + 1) landed(p - 2);
                if (!*abort_flag) *s_done = (r + 1 < f.n_rounds) ? round_info(f, r + 1).base : f.n_prod;
            }
            __threadfence_block();
            *s_exit = 1;
            KT_FLUSH(true, f.hdr, 24, 4);
            if (*abort_flag) {
                // drain: the copies already requested must land before the shared memory goes away
                // (bounded waits without the abort short-cut; a completed phase returns at once)
                for (uint32_t pp = (nG > 3 ? nG - 3 : 0); pp < nG; ++pp)
                    ptx::mbar_wait(&fullG[pp % 3], (pp / 3) & 1u, f.a.wait_limit_ns / 8);
                for (uint32_t pp = (nA > 2 ? nA - 2 : 0); pp < nA; ++pp)
                    ptx::mbar_wait(&fullA[pp & 1], (pp >> 1) & 1u, f.a.wait_limit_ns / 8);
                for (uint32_t pp = (nB > 2 ? nB - 2 : 0); pp < nB; ++pp)
                    ptx::mbar_wait(&fullB[pp & 1], (pp >> 1) & 1u, f.a.wait_limit_ns / 8);
            }
        }
    } else if (warp == 8 || warp == 9) {
        // ================= control warps: lane 0 of each issues MMAs =================
        // Issuing one tcgen05.mma costs the issuing thread several tens of cycles whatever the tile
        // size, and both products on the sequential chain are small, so each is split along its
        // summation index between the two control threads, into one accumulator each; the
        // accumulators are added when they are read back.  The first thread also issues the output
        // product.
        const int half = warp - 8;
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16(128, NS) | ptx::kIdescBMajorMN;
            const uint32_t sbf_a = ptx::smem_u32(sbf), vn_a = ptx::smem_u32(vn);
            uint32_t g = 0, last_out = 0;
            bool any_out = false;
            KT_DECL(8);
            for (int r = 0; r * f.Q + q < f.J && !*abort_flag; ++r) {
                const JobInfo J = job_info(f, r * f.Q + q);
                for (int c = 0; c < J.nch && !*abort_flag; ++c, ++g) {
                    const uint32_t s2 = g & 1;
                    const uint32_t sb = ptx::smem_u32(smem + s2 * C_STAGE);
                    const uint32_t d1 = d1c + (uint32_t)((g & 1) * 2 + half) * NS;
                    // MMA1(g): D1 = [W' ; Q'] (exp(G_m) . S), this thread's half of the sum over dk
                    KT_MARK(half == 0, 0);
                    wait(&fullA[s2], (g >> 1) & 1u, 1);
                    KT_MARK(half == 0, 1);   // operands A
                    wait(sbf_ready, g & 1u, 4);
                    KT_MARK(half == 0, 2);   // state copy
                    ptx::tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int kk = half * 4 + k;   // 16-wide step of the sum over dk
                        ptx::umma_bf16(d1, ptx::umma_desc_sw128(sb + C_QW + (kk >> 2) * tc::QW_HALF + (kk & 3) * 32),
                                       ptx::umma_desc_sw128_mn(sbf_a + kk * 2048, 8192), idesc, k > 0);
                    }
                    ptx::umma_commit(mma1_bar);
                    ptx::umma_commit(&emptyA[s2]);
                    KT_MARK(half == 0, 3);   // MMA1 issue
                    // MMA2(g): D3 = K'^T V_new (K' token-major = MN-major A operand), this thread's half of
                    // the sum over the chunk's tokens; the state product sits on the sequential chain, so it
                    // is issued and committed first
                    wait(vn_ready, g & 1u, 5);
                    KT_MARK(half == 0, 4);   // V_new
                    wait(&fullB[s2], (g >> 1) & 1u, 6);
                    KT_MARK(half == 0, 5);   // operands B
                    ptx::tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        const int kk = half * 2 + k;   // 16-wide step of the sum over tokens
                        ptx::umma_bf16(d3c + half * NS,
                                       ptx::umma_desc_sw128_mn(sb + C_KT + kk * 2048, tc::KI_HALF),
                                       ptx::umma_desc_sw128_mn(vn_a + kk * 2048, 8192), idesc | ptx::kIdescAMajorMN,
                                       k > 0);
                    }
                    ptx::umma_commit(mma2_bar);
                    if (half == 0 && op) {
                        // D1[64:128] += Aqk V_new.  The 128-row A operand starts 64 rows before Aqk: those
                        // rows (the tail of the K' image) only touch accumulator rows 0-63, which are dead
                        // once V_new has been taken.
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            ptx::umma_bf16(d1, ptx::umma_desc_sw128(sb + C_AQ - 8192 + k * 32),
                                           ptx::umma_desc_sw128_mn(vn_a + k * 2048, 8192), idesc, 1);
                        ptx::umma_commit(&out_bar[g & 1]);
                        last_out = g;
                        any_out = true;
                    }
                    ptx::umma_commit(&emptyB[s2]);
                    KT_MARK(half == 0, 6);   // MMA2 + output issue
#ifdef KDA_FUSED_TIMING
                    kt_acc_[7] += 16;
#endif
                }
            }
            KT_FLUSH(half == 0, f.hdr, 16, 8);
            // every MMA of this thread has completed before the TMEM goes away
            if (half == 0 && any_out) wait(&out_bar[last_out & 1], (last_out >> 1) & 1u, 7);
            else if (g > 0) wait(&emptyB[(g - 1) & 1], ((g - 1) >> 1) & 1u, 8);
        }
    } else if (warp < 8) {
        // ================= compute warps =================
        const int quad = warp & 3, ch = warp >> 2;       // TMEM lane quadrant, 32-column half of the slice
        const int tid = quad * 32 + lane;                // 0..127: token row for V_new / O, dk row for the state
        const uint32_t tmem_lane = ((uint32_t)(quad * 32) << 16) + (uint32_t)ch * 32;
        auto warp_arrive = [&](uint64_t* bar) {
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar);
        };
        float S[32];
        uint32_t g = 0;
        for (int r = 0; r * f.Q + q < f.J; ++r) {
            const JobInfo J = job_info(f, r * f.Q + q);
            const size_t sbase = ((size_t)J.n * a.H + J.h) * (size_t)(kD * kD) + (size_t)tid * kD + col0 + ch * 32;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (a.S_in) x = *reinterpret_cast<const float4*>(a.S_in + sbase + j);
                S[j] = x.x; S[j + 1] = x.y; S[j + 2] = x.z; S[j + 3] = x.w;
            }
            auto ref_scale_of = [&](uint32_t gg) {   // exp(G_m) of the chunk with running number gg
                wait(&fullG[gg % 3], (gg / 3) & 1u, 8);
                return reinterpret_cast<const float*>(smem + C_GV + (gg % 3) * tc::GV_BYTES + 512)[tid];
            };
            auto store_scaled = [&](float cgn) {
                float z[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) z[j] = cgn * S[j];
                store_row32(sbf, tid, ch * 4, z);
            };
            if (J.nch > 0) {
                store_scaled(ref_scale_of(g));
                ptx::fence_async_smem();
                warp_arrive(sbf_ready);
            }
            for (int c = 0; c < J.nch; ++c, ++g) {
                const uint32_t s2 = g & 1, par = g & 1u;
                const uint8_t* sb = smem + s2 * C_STAGE;
                const uint32_t d1 = d1c + tmem_lane + (uint32_t)(g & 1) * 2 * NS;
                if (quad < 2) {   // a6: V_new = U - W S  (token row = tid)
                    wait(&fullB[s2], (g >> 1) & 1u, 1);
                    uint4 uq[4];   // this token's 32 values of U
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        uq[cc] = *reinterpret_cast<const uint4*>(sb + C_U + ch * tc::U_BLOCK + tc::u_off(tid, cc));
                    warp_arrive(&emptyB[s2]);
                    const __nv_bfloat16* U = reinterpret_cast<const __nv_bfloat16*>(uq);
                    wait(mma1_bar, par, 2);
                    ptx::tc_fence_after();
                    float x[32];
                    tmem_ld_sum32(d1, x);
#pragma unroll
                    for (int j = 0; j < 32; ++j) x[j] = __bfloat162float(U[j]) - x[j];
                    store_row32(vn, tid, ch * 4, x);
                    ptx::fence_async_smem();
                    ptx::tc_fence_before();
                    warp_arrive(vn_ready);
                }
                wait(&fullG[g % 3], (g / 3) & 1u, 9);
                const float* gv = reinterpret_cast<const float*>(smem + C_GV + (g % 3) * tc::GV_BYTES);
                const float gc = gv[tid];          // gamma^C
                const float ct = gv[256 + tid];    // exp(G_C - G_m)
                const bool more = c + 1 < J.nch;
                const float cgn = more ? ref_scale_of(g + 1) : 0.f;   // fetched off the chain, before the wait below
                warp_arrive(&emptyG[g % 3]);
                // S_new = gc . S + ct . D3; the part that does not need D3 is formed before the wait.  (The
                // scales are applied one after the other: ct . D3 is of ordinary size although ct can be
                // e^-80 and D3 e^+80, whereas a pre-multiplied cgn * ct would underflow.)
#pragma unroll
                for (int j = 0; j < 32; ++j) S[j] *= gc;
                wait(mma2_bar, par, 3);
                ptx::tc_fence_after();
                {   // a8: S <- gamma^C . S + exp(G_C - G_m) . (K'^T V_new) ; refresh the bf16 operand copy
                    float ds[32];
                    tmem_ld_sum32(d3c + tmem_lane, ds);
#pragma unroll
                    for (int j = 0; j < 32; ++j) S[j] = fmaf(ct, ds[j], S[j]);
                    if (more) {
                        store_scaled(cgn);   // next chunk's operand copy: bf16(exp(G_m') . S_new)
                        ptx::fence_async_smem();
                    }
                    ptx::tc_fence_before();
                    if (more) warp_arrive(sbf_ready);
                }
                if (quad >= 2 && op) {   // a7: O = (Gamma.Q) S + Aqk V_new  (token row = tid - 64)
                    const int i = tid - 64;
                    const int64_t tok0 = J.tok_begin + (int64_t)c * kC;
                    const int len = (J.tok_end - tok0) < kC ? (int)(J.tok_end - tok0) : kC;
                    __nv_bfloat16* orow = op + ((tok0 + i) * a.H + J.h) * kD + col0 + ch * 32;
                    wait(&out_bar[g & 1], (g >> 1) & 1u, 6);
                    ptx::tc_fence_after();
                    float ov[32];
                    tmem_ld_sum32(d1, ov);
                    if (i < len && !*abort_flag) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            *reinterpret_cast<uint4*>(orow + j) =
                                make_uint4(pack2(ov[j], ov[j + 1]), pack2(ov[j + 2], ov[j + 3]),
                                           pack2(ov[j + 4], ov[j + 5]), pack2(ov[j + 6], ov[j + 7]));
                    }
                    ptx::tc_fence_before();
                }
            }
            if (*abort_flag) break;
            if (a.S_out) {
                float* so = a.S_out + sbase;
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(so + j) = make_float4(S[j], S[j + 1], S[j + 2], S[j + 3]);
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
}

template <bool kHasQ>
__global__ void __launch_bounds__(kThreads, 1)
kda_fused_tc(const __grid_constant__ FusedArgs f, const __grid_constant__ CUtensorMap tm_k,
             const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_v,
             int clear_status)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int t = threadIdx.x, warp = t >> 5;
    const bool chain_cta = (int)blockIdx.x < f.n_chain_cta;
    // (the TMEM slot sits in a spare word of the barrier block of either layout)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + (chain_cta ? C_BAR + 248 : E_BAR + 32));

    if (clear_status && blockIdx.x == 0 && t == 0) {
        f.hdr->status = 0;      // (an equal-length call has no prologue kernel to do this)
        f.hdr->where = 0;
        f.hdr->flags = 0;
    }
    // barriers of the engines
    if (!chain_cta && (t == 0 || t == kEngThreads)) {
        uint64_t* mb = reinterpret_cast<uint64_t*>(smem + (t ? E_BYTES : 0) + E_BAR);
        ptx::mbar_init(mb, 2);       // MMA group complete (two issuing threads)
        ptx::mbar_init(mb + 1, 1);   // k landed
        ptx::mbar_init(mb + 3, 1);   // q landed
        ptx::mbar_init(mb + 5, 1);   // v landed
        *reinterpret_cast<volatile uint32_t*>(mb + 2) = 0;
        ptx::fence_mbar_init();
        if (t == 0) {
            ptx::prefetch_tmap(&tm_k);
            ptx::prefetch_tmap(&tm_q);
            ptx::prefetch_tmap(&tm_v);
        }
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const bool aligned = (ptx::smem_u32(smem) & 1023u) == 0;   // the operand images need 1024-byte alignment
    if (!aligned) {
        if (t == 0) report_timeout(f, 90);
    } else if (chain_cta) {
        chain_run<kHasQ>(f, smem, tmem_base, t, (int)blockIdx.x / kSlices, (int)blockIdx.x % kSlices);
    } else {
        // two engines per CTA
        if (t < kEngThreads)
            engine_run<kHasQ, true>(f, smem, tmem_base, 1, t, 0, 0, &tm_k, &tm_q, &tm_v);
        else
            engine_run<kHasQ, true>(f, smem + E_BYTES, tmem_base + 256, 2, t - kEngThreads, 0, 0, &tm_k, &tm_q, &tm_v);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem_base, kTmemCols);
}

// ---- the intra-chunk stage alone (first kernel of the two-kernel schedule) --------------------------------
// Persistent CTAs of one engine each, two per SM; the tiles of the pass go to a plain array.
template <bool kHasQ, bool kLayer>
__global__ void __launch_bounds__(kEngThreads, 2)
kda_intra_tc(const __grid_constant__ FusedArgs f, const __grid_constant__ CUtensorMap tm_k,
             const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_v,
             int clear_status)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int t = threadIdx.x, warp = t >> 5;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + E_BAR + 32);
    ptx::grid_dep_launch();   // the inter-chunk kernel may set itself up while this one drains
    if (clear_status && blockIdx.x == 0 && t == 0) {
        f.hdr->status = 0;      // (an equal-length call has no prologue kernel to do this)
        f.hdr->where = 0;
        f.hdr->flags = 0;
    }
    if (t == 0) {
        uint64_t* mb = reinterpret_cast<uint64_t*>(smem + E_BAR);
        ptx::mbar_init(mb, 2);       // MMA group complete (two issuing threads)
        ptx::mbar_init(mb + 1, 1);   // k landed
        ptx::mbar_init(mb + 3, 1);   // q landed
        ptx::mbar_init(mb + 5, 1);   // v landed
        *reinterpret_cast<volatile uint32_t*>(mb + 2) = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tm_k);
        ptx::prefetch_tmap(&tm_q);
        ptx::prefetch_tmap(&tm_v);
    }
    if (warp == 0) {
        ptx::tmem_alloc(tmem_slot, 256);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if ((ptx::smem_u32(smem) & 1023u) != 0) {
        if (t == 0) report_timeout(f, 90);   // the operand images need 1024-byte alignment
    } else {
        engine_run<kHasQ, false, kLayer>(f, smem, tmem_base, 1, t, blockIdx.x, gridDim.x, &tm_k, &tm_q, &tm_v);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tmem_base, 256);
}

// ---- prologue of a packed batch: status word + production-index base of every round ----------------------
__global__ void kda_fused_prep_kernel(WsHeader* hdr, const int32_t* __restrict__ cu, uint32_t* __restrict__ round_base,
                                      int n_seqs, int H, int Q, int n_rounds)
{
    // one CTA; thread i handles rounds i, i + blockDim.x, ...; a running offset chains the passes
    __shared__ uint32_t s_part[1024];
    __shared__ uint32_t s_carry;
    const int t = threadIdx.x;
    if (t == 0) {
        hdr->status = 0;
        hdr->where = 0;
        hdr->flags = 0;
        s_carry = 0;
    }
    __syncthreads();
    const int J = n_seqs * H;
    for (int r0 = 0; r0 < n_rounds; r0 += (int)blockDim.x) {
        const int r = r0 + t;
        uint32_t cnt = 0;
        if (r < n_rounds) {
            const int j0 = r * Q, j1 = (j0 + Q < J ? j0 + Q : J) - 1;
            int maxlen = 0;
            for (int n = j0 / H; n <= j1 / H; ++n) {
                const int len = (cu[n + 1] - cu[n] + kC - 1) / kC;
                maxlen = len > maxlen ? len : maxlen;
            }
            cnt = (uint32_t)maxlen * (uint32_t)(j1 - j0 + 1);
        }
        s_part[t] = cnt;
        __syncthreads();
        // inclusive scan (Hillis-Steele)
        for (int off = 1; off < (int)blockDim.x; off <<= 1) {
            uint32_t v = 0;
            if (t >= off) v = s_part[t - off];
            __syncthreads();
            s_part[t] += v;
            __syncthreads();
        }
        if (r < n_rounds) round_base[r] = s_carry + s_part[t] - cnt;
        __syncthreads();
        if (t == (int)blockDim.x - 1) s_carry += s_part[t];
        __syncthreads();
    }
    if (t == 0) round_base[n_rounds] = s_carry;
}

// cuTensorMapEncodeTiled through the runtime's driver entry-point query (no link dependency on
// libcuda, so the library still loads on a machine without a driver)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;   // (the entry point is the same for every device: benign race)
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

// [total_tokens, H*128] bf16 matrix, boxes of `rows` tokens x `cols` channels, no swizzle (rows of the
// box land back to back); used for the output-gate blocks of the layer wrap
kda_status_t make_plain_tmap(CUtensorMap* tm, const void* base, int64_t total_tokens, int H, int cols, int rows)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return fail(KDA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const cuuint64_t dims[2] = {(cuuint64_t)H * kD, (cuuint64_t)total_tokens};
    const cuuint64_t strides[1] = {(cuuint64_t)H * kD * 2};
    const cuuint32_t box[2] = {(cuuint32_t)cols, (cuuint32_t)rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(KDA_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return KDA_OK;
}

// (tc_tile_bytes is defined beside the two-kernel path)

kda_status_t launch_fused_prep(WsHeader* hdr, const int32_t* cu_seqlens, uint32_t* round_base, int n_seqs,
                               int H, int Q, int n_rounds, cudaStream_t st)
{
    ProfScope ps(PROF_PREP, st);
    kda_fused_prep_kernel<<<1, 1024, 0, st>>>(hdr, cu_seqlens, round_base, n_seqs, H, Q, n_rounds);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

// chain CTAs: kSlices per running (sequence, head); at least half of the SMs stay with the engines
kda_status_t launch_intra_tc(const ChunkArgs& a, void* tiles, WsHeader* hdr, bool clear_status,
                             cudaStream_t st)
{
    int n_sm = 0;
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (!lk.st->attr_done[1]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_tc<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)E_BYTES));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_tc<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)E_BYTES));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_tc<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)E_BYTES));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_tc<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)E_BYTES));
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
    FusedArgs f = {};
    f.a = a;
    f.ring = static_cast<char*>(tiles);
    f.hdr = hdr;
    f.n_prod = (uint32_t)n_tiles;
    const bool has_q = a.q != nullptr && a.o != nullptr;
    CUtensorMap tm_k, tm_q, tm_v;
    kda_status_t rc = make_tmap(&tm_k, a.k, a.total_tokens, a.H);
    if (rc == KDA_OK) rc = make_tmap(&tm_v, a.v, a.total_tokens, a.H);
    if (rc == KDA_OK) rc = make_tmap(&tm_q, has_q ? a.q : a.k, a.total_tokens, a.H);
    if (rc != KDA_OK) return rc;
    const int64_t resident = 2 * (int64_t)n_sm;   // two CTAs per SM
    const unsigned grid = (unsigned)(n_tiles < resident ? n_tiles : resident);
    ProfScope ps(PROF_INTRA, st);
    const bool layer = a.gate_rate != nullptr;
    if (layer && has_q)
        kda_intra_tc<true, true><<<grid, kEngThreads, E_BYTES, st>>>(f, tm_k, tm_q, tm_v, clear_status ? 1 : 0);
    else if (layer)
        kda_intra_tc<false, true><<<grid, kEngThreads, E_BYTES, st>>>(f, tm_k, tm_q, tm_v, clear_status ? 1 : 0);
    else if (has_q)
        kda_intra_tc<true, false><<<grid, kEngThreads, E_BYTES, st>>>(f, tm_k, tm_q, tm_v, clear_status ? 1 : 0);
    else
        kda_intra_tc<false, false><<<grid, kEngThreads, E_BYTES, st>>>(f, tm_k, tm_q, tm_v, clear_status ? 1 : 0);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

int fused_max_slots(int n_sm) { return n_sm / (2 * kSlices); }
int fused_slices() { return kSlices; }

kda_status_t launch_fused_tc(FusedArgs f, bool has_q, bool clear_status, cudaStream_t st)
{
    int n_sm = 0;
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (lk.st->n_sm == 0) {
            int dev = 0, coop = 0;
            KDA_CUDA_TRY(cudaGetDevice(&dev));
            KDA_CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
            if (!coop) return fail(KDA_ERR_UNSUPPORTED, "the device does not support cooperative launches");
            KDA_CUDA_TRY(cudaDeviceGetAttribute(&lk.st->n_sm, cudaDevAttrMultiProcessorCount, dev));
        }
        if (!lk.st->attr_done[0]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_fused_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kSmemBytes));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_fused_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kSmemBytes));
            lk.st->attr_done[0] = true;
        }
        n_sm = lk.st->n_sm;
    }
    if (f.a.total_tokens > 0x7fffffff)
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: more than 2^31 tokens in one call");
    CUtensorMap tm_k, tm_q, tm_v;
    kda_status_t rc = make_tmap(&tm_k, f.a.k, f.a.total_tokens, f.a.H);
    if (rc == KDA_OK) rc = make_tmap(&tm_v, f.a.v, f.a.total_tokens, f.a.H);
    if (rc == KDA_OK) rc = make_tmap(&tm_q, has_q ? f.a.q : f.a.k, f.a.total_tokens, f.a.H);
    if (rc != KDA_OK) return rc;
    if (f.n_chain_cta >= n_sm)
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: %d chain CTAs leave no SM of %d for the engines",
                    f.n_chain_cta, n_sm);
    int cs = clear_status ? 1 : 0;
    void* args[] = {(void*)&f, (void*)&tm_k, (void*)&tm_q, (void*)&tm_v, (void*)&cs};
    const void* fn = has_q ? (const void*)kda_fused_tc<true> : (const void*)kda_fused_tc<false>;
    ProfScope ps(PROF_FUSED, st);
    KDA_CUDA_TRY(cudaLaunchCooperativeKernel(fn, dim3((unsigned)n_sm), dim3(kThreads), args, kSmemBytes, st));
    count_launch();
    return KDA_OK;
}

}  // namespace kda
