// Backward pass of the KDA recurrence (gradients of paper Eq. 1; the paper trains with this operator,
// Section 5, but gives no backward algorithm, so the adjoint is taken of Eq. 1 itself).
//
// For L = sum_t <d_o_t, o_t> + <dS_T, S_T> and the forward step written as
//     S' = Diag(alpha_t) S_{t-1},   r = v_t - S'^T k_t,   S_t = S' + beta_t k_t r^T,   o_t = scale S_t^T q_t
// the adjoint Lam of the state runs backwards in time:
//     Lam += scale q_t d_o_t^T          dq_t = scale S_t d_o_t
//     dbeta_t = k_t^T Lam r             dk_t  = beta_t Lam r - S' dr
//     dr = beta_t Lam^T k_t = dv_t      Lam' = Lam - k_t dr^T
//     dlog_alpha_t = rowsum(Lam' . S')  Lam <- Diag(alpha_t) Lam'
//
// Columns of S and of Lam never mix, so dv is cut into four 32-column slices: one CTA of eight warps
// per (sequence, head, slice), thread = (column, block of 16 rows), both matrices in registers.  The
// sums over columns (dq, dk, dlog_alpha, dbeta) are formed per slice and added by a second kernel,
// in a fixed order.  Forward states are not stored for the whole sequence: a first sweep keeps the
// state at the start of every block of 8 tokens, the reverse sweep recomputes one block at a time into
// shared memory (8 decayed states of this slice, 128 KB) and runs the adjoint through it.  All
// arithmetic is fp32 FMA; q, k, v, d_o may be stored as bf16.
#include <vector>

#include "kda_common.cuh"

namespace kda {
namespace {

constexpr int NS = 32;                 // state columns per CTA
constexpr int kSlices = kD / NS;
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRows = kD / kWarps;      // state rows per thread (the warp's block of rows)
constexpr int kB = 8;                  // tokens per recomputation block
constexpr int kBlocksPerChunk = kC / kB;
constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct BwdArgs {
    const void* q; const void* k; const void* v; const void* d_o;
    const float* log_alpha; const float* beta;
    const float* S0; const float* dS_T;
    float* dv; float* dS0;
    const int32_t* cu_seqlens; const int32_t* chunk_cu;
    float* ckpt;        // [total_chunks * 8][H][128][128]: state at the start of every block of 8 tokens
    float* part_q; float* part_k; float* part_g;   // [kSlices][T][H][128]
    float* part_b;      // [kSlices][T][H]
    int n_seqs, H;
    int64_t total_tokens, seq_len, chunks_per_seq;
    float scale;
};

// shared memory of the sweep kernel (floats)
constexpr int M_SD = 0;                      // [8][128][NS] decayed states S' of the block in flight
constexpr int M_K = M_SD + kB * kD * NS;     // [8][128] k
constexpr int M_Q = M_K + kB * kD;           // [8][128] q
constexpr int M_A = M_Q + kB * kD;           // [8][128] alpha = exp(log alpha)
constexpr int M_V = M_A + kB * kD;           // [8][NS] v slice
constexpr int M_DO = M_V + kB * NS;          // [8][NS] d_o slice
constexpr int M_R = M_DO + kB * NS;          // [8][NS] residuals r_t
constexpr int M_B = M_R + kB * NS;           // [8] beta
constexpr int M_RED = M_B + kB;              // [2][warps][NS] cross-warp column sums
constexpr int M_DB = M_RED + 2 * kWarps * NS;   // [8][warps] dbeta per warp
constexpr int M_FLOATS = M_DB + kB * kWarps;
constexpr size_t kSweepSmem = (size_t)M_FLOATS * sizeof(float);
static_assert(kSweepSmem <= 232448, "fits the shared memory of one SM");

// sum over the 32 lanes of kRows per-lane values each: afterwards lane l holds the total of x[l % kRows]
__device__ __forceinline__ float lane_transpose_sum(float (&x)[kRows], int lane) {
#pragma unroll
    for (int s = kRows / 2; s >= 1; s >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int j = 0; j < s; ++j) {
            const float send = up ? x[j] : x[j + s];
            const float keep = up ? x[j + s] : x[j];
            x[j] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    float v = x[0];
#pragma unroll
    for (int s = kRows; s < 32; s <<= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
    return v;
}
__device__ __forceinline__ float sum_db(const float* p) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) v += p[w];
    return v;
}
__device__ __forceinline__ float sum_partials(const float* red, int lane) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) v += red[w * NS + lane];
    return v;
}

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T>
__global__ void __launch_bounds__(kThreads, 1) kda_bwd_sweep(BwdArgs a)
{
    extern __shared__ __align__(16) float sm[];
    const int t = threadIdx.x, lane = t & 31, rg = t >> 5;
    const int slice = blockIdx.x, h = blockIdx.y, n = blockIdx.z;
    const int col = slice * NS + lane;
    const int i0 = rg * kRows;                 // first of this thread's rows

    int64_t tok_begin, tok_end, chunk0;
    if (a.cu_seqlens) {
        tok_begin = a.cu_seqlens[n]; tok_end = a.cu_seqlens[n + 1];
        chunk0 = a.chunk_cu[n];
    } else {
        tok_begin = (int64_t)n * a.seq_len; tok_end = tok_begin + a.seq_len;
        chunk0 = (int64_t)n * a.chunks_per_seq;
    }
    const int nblk = (int)((tok_end - tok_begin + kB - 1) / kB);
    const T* qp = reinterpret_cast<const T*>(a.q);
    const T* kp = reinterpret_cast<const T*>(a.k);
    const T* vp = reinterpret_cast<const T*>(a.v);
    const T* gp = reinterpret_cast<const T*>(a.d_o);
    const size_t sbase = ((size_t)n * a.H + h) * (size_t)(kD * kD);
    float* sSd = sm + M_SD;

    float S[kRows], Lam[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) S[r] = a.S0 ? a.S0[sbase + (size_t)(i0 + r) * kD + col] : 0.f;

    // loads the vectors of block b into shared memory; returns its number of tokens
    auto load_block = [&](int b, bool with_q) {
        const int64_t tok0 = tok_begin + (int64_t)b * kB;
        const int len = (tok_end - tok0) < kB ? (int)(tok_end - tok0) : kB;
        __syncthreads();   // the previous block's readers are done
        for (int idx = t; idx < len * kD; idx += kThreads) {
            const int j = idx >> 7, d = idx & 127;
            const size_t off = ((size_t)(tok0 + j) * a.H + h) * kD + d;
            sm[M_K + idx] = ldf<T>(kp + off);
            sm[M_A + idx] = __expf(a.log_alpha[off]);
            if (with_q) sm[M_Q + idx] = ldf<T>(qp + off);
        }
        for (int idx = t; idx < len * NS; idx += kThreads) {
            const int j = idx >> 5, cc = idx & 31;
            const size_t off = ((size_t)(tok0 + j) * a.H + h) * kD + slice * NS + cc;
            sm[M_V + idx] = ldf<T>(vp + off);
            if (with_q) sm[M_DO + idx] = gp ? ldf<T>(gp + off) : 0.f;
        }
        if (t < len) sm[M_B + t] = a.beta[(size_t)(tok0 + t) * a.H + h];
        __syncthreads();
        return len;
    };
    // one forward token on the register state; optionally keeps S' and r in shared memory
    auto forward_token = [&](int j, bool keep) {
        const float* kj = sm + M_K + j * kD + i0;
        const float* aj = sm + M_A + j * kD + i0;
        float p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
#pragma unroll
        for (int r = 0; r < kRows; r += 4) {
            S[r] *= aj[r]; S[r + 1] *= aj[r + 1]; S[r + 2] *= aj[r + 2]; S[r + 3] *= aj[r + 3];
            p0 = fmaf(kj[r], S[r], p0); p1 = fmaf(kj[r + 1], S[r + 1], p1);
            p2 = fmaf(kj[r + 2], S[r + 2], p2); p3 = fmaf(kj[r + 3], S[r + 3], p3);
        }
        if (keep) {
#pragma unroll
            for (int r = 0; r < kRows; ++r) sSd[((size_t)j * kD + i0 + r) * NS + lane] = S[r];
        }
        float* red = sm + M_RED + (j & 1) * kWarps * NS;
        red[rg * NS + lane] = (p0 + p1) + (p2 + p3);
        __syncthreads();
        const float res = sm[M_V + j * NS + lane] - sum_partials(red, lane);
        if (keep && rg == 0) sm[M_R + j * NS + lane] = res;
        const float br = sm[M_B + j] * res;
#pragma unroll
        for (int r = 0; r < kRows; ++r) S[r] = fmaf(kj[r], br, S[r]);
    };
    auto ckpt_of = [&](int b) {   // (a chunk of 64 tokens owns eight block slots)
        return a.ckpt + ((size_t)(chunk0 * kBlocksPerChunk + b) * a.H + h) * (size_t)(kD * kD);
    };

    // ---- sweep 1: forward, keeping the state at every block start -----------------------------------
    for (int b = 0; b < nblk; ++b) {
        float* ck = ckpt_of(b);
#pragma unroll
        for (int r = 0; r < kRows; ++r) ck[(size_t)(i0 + r) * kD + col] = S[r];
        const int len = load_block(b, false);
        for (int j = 0; j < len; ++j) forward_token(j, false);
    }

    // ---- sweep 2: blocks in reverse; recompute the block, then run the adjoint through it ------------
#pragma unroll
    for (int r = 0; r < kRows; ++r) Lam[r] = a.dS_T ? a.dS_T[sbase + (size_t)(i0 + r) * kD + col] : 0.f;
    for (int b = nblk - 1; b >= 0; --b) {
        const int64_t tok0 = tok_begin + (int64_t)b * kB;
        const float* ck = ckpt_of(b);
#pragma unroll
        for (int r = 0; r < kRows; ++r) S[r] = ck[(size_t)(i0 + r) * kD + col];
        const int len = load_block(b, true);
        for (int j = 0; j < len; ++j) forward_token(j, true);
        __syncthreads();   // r_t of every token is in shared memory (a thread reads back its own S' only)
        for (int j = len - 1; j >= 0; --j) {
            const float* kj = sm + M_K + j * kD + i0;
            const float* qj = sm + M_Q + j * kD + i0;
            const float* aj = sm + M_A + j * kD + i0;
            const float res = sm[M_R + j * NS + lane], go = sm[M_DO + j * NS + lane];
            const float bt = sm[M_B + j];
            float Sd[kRows], x[kRows];
#pragma unroll
            for (int r = 0; r < kRows; ++r) Sd[r] = sSd[((size_t)j * kD + i0 + r) * NS + lane];
            // o_t = scale S_t^T q_t
            const float sgo = a.scale * go, br = bt * res;
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                Lam[r] = fmaf(qj[r], sgo, Lam[r]);
                x[r] = fmaf(kj[r], br, Sd[r]) * sgo;          // S_t[i][c] * scale * d_o[c]
            }
            const float dq_i = lane_transpose_sum(x, lane);
            // S_t = S' + beta k r^T
            float p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
#pragma unroll
            for (int r = 0; r < kRows; r += 4) {
                x[r] = Lam[r] * res; x[r + 1] = Lam[r + 1] * res; x[r + 2] = Lam[r + 2] * res; x[r + 3] = Lam[r + 3] * res;
                p0 = fmaf(Lam[r], kj[r], p0); p1 = fmaf(Lam[r + 1], kj[r + 1], p1);
                p2 = fmaf(Lam[r + 2], kj[r + 2], p2); p3 = fmaf(Lam[r + 3], kj[r + 3], p3);
            }
            const float lr_i = lane_transpose_sum(x, lane);    // (Lam r)_i
            float* red = sm + M_RED + (j & 1) * kWarps * NS;
            red[rg * NS + lane] = (p0 + p1) + (p2 + p3);
            __syncthreads();
            const float dr = bt * sum_partials(red, lane);
            if (rg == 0) a.dv[((size_t)(tok0 + j) * a.H + h) * kD + col] = dr;
            // r = v - S'^T k ;  S' = Diag(alpha) S_{t-1}
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                Lam[r] = fmaf(-kj[r], dr, Lam[r]);             // Lam'
                x[r] = Sd[r] * dr;
            }
            const float sdr_i = lane_transpose_sum(x, lane);   // (S' dr)_i
#pragma unroll
            for (int r = 0; r < kRows; ++r) {
                x[r] = Lam[r] * Sd[r];
                Lam[r] *= aj[r];
            }
            const float dg_i = lane_transpose_sum(x, lane);
            // lanes l and l + 16 now hold the slice's share of row i0 + l
            const int rl = lane & (kRows - 1);
            const float k_i = sm[M_K + j * kD + i0 + rl];
            if (lane < kRows) {
                const size_t po = (((size_t)slice * a.total_tokens + (size_t)(tok0 + j)) * a.H + h) * kD + i0 + lane;
                a.part_q[po] = dq_i;
                a.part_k[po] = bt * lr_i - sdr_i;
                a.part_g[po] = dg_i;
            }
            float db = lane < kRows ? k_i * lr_i : 0.f;
#pragma unroll
            for (int s = 16; s >= 1; s >>= 1) db += __shfl_xor_sync(0xffffffffu, db, s);
            if (lane == 0) sm[M_DB + j * kWarps + rg] = db;
        }
        __syncthreads();
        if (t < len)
            a.part_b[((size_t)slice * a.total_tokens + (size_t)(tok0 + t)) * a.H + h] =
                sum_db(sm + M_DB + t * kWarps);
    }
    if (a.dS0) {
#pragma unroll
        for (int r = 0; r < kRows; ++r) a.dS0[sbase + (size_t)(i0 + r) * kD + col] = Lam[r];
    }
}

// adds the four slices' shares, in slice order
__global__ void kda_bwd_reduce(const float* __restrict__ part_q, const float* __restrict__ part_k,
                               const float* __restrict__ part_g, const float* __restrict__ part_b,
                               float* __restrict__ dq, float* __restrict__ dk, float* __restrict__ dg,
                               float* __restrict__ dbeta, size_t n_vec, size_t n_tok)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec / 4; i += stride) {
        float4 sq = make_float4(0.f, 0.f, 0.f, 0.f), sk = sq, sg = sq;
#pragma unroll
        for (int s = 0; s < kSlices; ++s) {
            const float4 x = reinterpret_cast<const float4*>(part_q + s * n_vec)[i];
            const float4 y = reinterpret_cast<const float4*>(part_k + s * n_vec)[i];
            const float4 z = reinterpret_cast<const float4*>(part_g + s * n_vec)[i];
            sq.x += x.x; sq.y += x.y; sq.z += x.z; sq.w += x.w;
            sk.x += y.x; sk.y += y.y; sk.z += y.z; sk.w += y.w;
            sg.x += z.x; sg.y += z.y; sg.z += z.z; sg.w += z.w;
        }
        reinterpret_cast<float4*>(dq)[i] = sq;
        reinterpret_cast<float4*>(dk)[i] = sk;
        reinterpret_cast<float4*>(dg)[i] = sg;
    }
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_tok; i += stride) {
        float s = 0.f;
#pragma unroll
        for (int sl = 0; sl < kSlices; ++sl) s += part_b[sl * n_tok + i];
        dbeta[i] = s;
    }
}

struct BwdLayout {
    size_t off_table, off_ckpt, off_pq, off_pk, off_pg, off_pb, total;
};
BwdLayout bwd_layout(int64_t T, int n_seqs, int H)
{
    BwdLayout L;
    const size_t chunks = (size_t)((T + kC - 1) / kC + n_seqs);
    const size_t vec = (size_t)T * H * kD * sizeof(float);
    L.off_table = sizeof(WsHeader);
    L.off_ckpt = L.off_table + align_up((size_t)(n_seqs + 1) * sizeof(int32_t));
    L.off_pq = L.off_ckpt + align_up(chunks * kBlocksPerChunk * H * kD * kD * sizeof(float));
    L.off_pk = L.off_pq + align_up(kSlices * vec);
    L.off_pg = L.off_pk + align_up(kSlices * vec);
    L.off_pb = L.off_pg + align_up(kSlices * vec);
    L.total = L.off_pb + align_up((size_t)kSlices * T * H * sizeof(float));
    return L;
}

}  // namespace
}  // namespace kda

using namespace kda;

extern "C" {

size_t kda_chunk_bwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk)
{
    if (dk != kD || dv != kD || chunk != kC || total_tokens < 0 || n_seqs < 0 || H <= 0) return 0;
    return bwd_layout(total_tokens, n_seqs, H).total;
}

kda_status_t kda_chunk_bwd(const void* q, const void* k, const void* v, const float* log_alpha,
                           const float* beta, const float* S0, const void* d_o, const float* dS_T,
                           float* dq, float* dk_out, float* dv_out, float* dlog_alpha, float* dbeta,
                           float* dS0, const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host,
                           int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk, float scale,
                           kda_dtype_t dt, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (dk != kD || dv != kD || chunk != kC || (dt != KDA_F32 && dt != KDA_BF16))
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_bwd: only dk=dv=128, chunk=64, dt in {f32,bf16} are "
                    "supported (got dk=%d dv=%d chunk=%d dt=%d)", dk, dv, chunk, (int)dt);
    if (n_seqs < 0 || total_tokens < 0 || H <= 0 || H > 65535 || n_seqs > 65535)
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: bad sizes n_seqs=%d total_tokens=%lld H=%d", n_seqs,
                    (long long)total_tokens, H);
    if ((cu_seqlens_dev == nullptr) != (cu_seqlens_host == nullptr))
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: cu_seqlens_dev and cu_seqlens_host must be given "
                    "together");
    if (n_seqs == 0) {
        if (total_tokens != 0)
            return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: n_seqs=0 with total_tokens=%lld",
                        (long long)total_tokens);
        return KDA_OK;
    }
    if (total_tokens > 0 && (!q || !k || !v || !log_alpha || !beta || !dq || !dk_out || !dv_out ||
                             !dlog_alpha || !dbeta))
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: q, k, v, log_alpha, beta and the five token "
                    "gradients must not be NULL");
    const void* ptrs[] = {q, k, v, log_alpha, beta, S0, d_o, dS_T, dq, dk_out, dv_out, dlog_alpha, dbeta, dS0,
                          cu_seqlens_dev};
    for (const void* p : ptrs)
        if (!aligned16(p)) return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: pointer %p is not 16-byte "
                                       "aligned", p);
    int64_t seq_len = 0, chunks_per_seq = 0;
    if (cu_seqlens_host) {
        if (cu_seqlens_host[0] != 0 || (int64_t)cu_seqlens_host[n_seqs] != total_tokens)
            return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: cu_seqlens must start at 0 and end at "
                        "total_tokens");
        for (int n = 0; n < n_seqs; ++n)
            if (cu_seqlens_host[n + 1] < cu_seqlens_host[n])
                return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: cu_seqlens decreases at %d", n);
    } else {
        if (total_tokens % n_seqs != 0)
            return fail(KDA_ERR_INVALID_ARG, "kda_chunk_bwd: total_tokens not divisible by n_seqs for an "
                        "equal-length batch");
        seq_len = total_tokens / n_seqs;
        chunks_per_seq = (seq_len + kC - 1) / kC;
    }
    const BwdLayout L = bwd_layout(total_tokens, n_seqs, H);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) || workspace_bytes < L.total)
        return fail(KDA_ERR_WORKSPACE, "kda_chunk_bwd: workspace must be 256-byte aligned and at least %zu "
                    "bytes (got %zu)", L.total, workspace_bytes);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws);
    int32_t* chunk_cu_dev = reinterpret_cast<int32_t*>(ws + L.off_table);
    kda_status_t rc = launch_prep(hdr, cu_seqlens_dev, chunk_cu_dev, n_seqs, st);
    if (rc != KDA_OK) return rc;
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (!lk.st->attr_done[8]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_bwd_sweep<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kSweepSmem));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_bwd_sweep<__nv_bfloat16>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSweepSmem));
            lk.st->attr_done[8] = true;
        }
    }
    BwdArgs a;
    a.q = q; a.k = k; a.v = v; a.d_o = d_o; a.log_alpha = log_alpha; a.beta = beta;
    a.S0 = S0; a.dS_T = dS_T; a.dv = dv_out; a.dS0 = dS0;
    a.cu_seqlens = cu_seqlens_dev; a.chunk_cu = cu_seqlens_dev ? chunk_cu_dev : nullptr;
    a.ckpt = reinterpret_cast<float*>(ws + L.off_ckpt);
    a.part_q = reinterpret_cast<float*>(ws + L.off_pq);
    a.part_k = reinterpret_cast<float*>(ws + L.off_pk);
    a.part_g = reinterpret_cast<float*>(ws + L.off_pg);
    a.part_b = reinterpret_cast<float*>(ws + L.off_pb);
    a.n_seqs = n_seqs; a.H = H; a.total_tokens = total_tokens; a.seq_len = seq_len;
    a.chunks_per_seq = chunks_per_seq; a.scale = scale;
    if (total_tokens > 0 || dS0) {
        dim3 grid(kSlices, (unsigned)H, (unsigned)n_seqs);
        ProfScope ps(PROF_INTER, st);
        if (dt == KDA_BF16) kda_bwd_sweep<__nv_bfloat16><<<grid, kThreads, kSweepSmem, st>>>(a);
        else kda_bwd_sweep<float><<<grid, kThreads, kSweepSmem, st>>>(a);
        count_launch();
        KDA_CUDA_TRY(cudaGetLastError());
    }
    if (total_tokens > 0) {
        const size_t n_vec = (size_t)total_tokens * H * kD, n_tok = (size_t)total_tokens * H;
        ProfScope ps(PROF_INTRA, st);
        kda_bwd_reduce<<<1184, 256, 0, st>>>(a.part_q, a.part_k, a.part_g, a.part_b, dq, dk_out, dlog_alpha,
                                             dbeta, n_vec, n_tok);
        count_launch();
        KDA_CUDA_TRY(cudaGetLastError());
    }
    return KDA_OK;
}

}  // extern "C"
