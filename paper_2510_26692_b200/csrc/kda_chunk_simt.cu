// fp32 FMA path of the chunkwise KDA forward (paper Section 3.1; steps follow Appendix C's order).
// Used for dt = KDA_F32 (tolerance 1e-4 rules out tf32/bf16 tensor-core products); it also accepts
// bf16 storage of q/k/v/o and then computes in fp32.
//
// Two kernels per pass over a range of chunks:
//   intra  one CTA per (chunk, head): cumulative log-decay G (a1), gated Gram matrices
//          Akk = Diag(beta) StrictTril((Gamma.K)(K/Gamma)^T) (a2) and Aqk = Tril((Gamma.Q)(K/Gamma)^T)
//          (a5), T = (I + Akk)^-1 by forward substitution (a3), W = T Diag(beta) (Gamma.K),
//          U = T Diag(beta) V (a4).  Writes W, U, Gamma.Q, (gamma^C/Gamma).K, Aqk, gamma^C to a
//          scratch tile.
//   inter  one CTA per (sequence, head, 16-column slice of dv), sequential over the chunks:
//          V_new = U - W S (a6), O = (Gamma.Q) S + Aqk V_new (a7),
//          S <- Diag(gamma^C) S + ((gamma^C/Gamma).K)^T V_new (a8).  State columns are independent,
//          which is what lets dv be sliced across CTAs.
//
// The decay ratios exp(G_i - G_j) are factored around G_m = G_C / 2 (per channel) as
// exp(G_i - G_m) * exp(G_m - G_j), with each exponent clamped to [-80, 80], so no product
// overflows fp32; entries above the diagonal are never used (selected to zero, not multiplied).
#include "kda_common.cuh"

namespace kda {
namespace {

constexpr int LD = kD + 4;           // padded fp32 row (keeps float4 alignment, spreads banks)
constexpr int LDA = kC + 1;
constexpr float kClamp = 80.f;

// scratch tile (floats)
constexpr int T_W = 0;
constexpr int T_U = T_W + kC * kD;
constexpr int T_QG = T_U + kC * kD;
constexpr int T_KT = T_QG + kC * kD;
constexpr int T_AQK = T_KT + kC * kD;
constexpr int T_GC = T_AQK + kC * kC;
constexpr int T_FLOATS = T_GC + kD;

constexpr size_t kIntraSmem = (size_t)(5 * kC * LD + 2 * kC * LDA + kC) * sizeof(float);
constexpr int NS = 16;               // dv columns per inter-chunk CTA
constexpr size_t kInterSmem =
    (size_t)(3 * kC * LD + kC * LDA + kD * NS + 2 * kC * NS + kD) * sizeof(float);

__device__ __forceinline__ float clampf(float x) { return fminf(fmaxf(x, -kClamp), kClamp); }

template <typename T>
__global__ void __launch_bounds__(256, 1) kda_intra_simt(ChunkArgs a, float* __restrict__ tiles, WsHeader* hdr)
{
    extern __shared__ __align__(16) float smem[];
    float* sG = smem;                    // log-decay cumsum, later V
    float* sKg = sG + kC * LD;           // K * exp(G - G_ref)
    float* sKi = sKg + kC * LD;          // K * exp(G_ref - G)
    float* sQg = sKi + kC * LD;          // scale * Q * exp(G - G_ref)
    float* sKG = sQg + kC * LD;          // K * exp(G)        (Gamma . K)
    float* sA = sKG + kC * LD;           // Akk
    float* sT = sA + kC * LDA;           // (I + Akk)^-1
    float* sB = sT + kC * LDA;           // beta

    const int t = threadIdx.x;
    const int h = blockIdx.y;
    const int64_t g = a.g0 + blockIdx.x;
    const ChunkLoc L = locate_chunk(a, g);
    const T* qp = reinterpret_cast<const T*>(a.q);
    const T* kp = reinterpret_cast<const T*>(a.k);
    const T* vp = reinterpret_cast<const T*>(a.v);
    float* tile = tiles + ((size_t)(g - a.g0) * a.H + h) * T_FLOATS;

    // a1: load log alpha (identity padding past the sequence end), then scan over the tokens
    for (int idx = t; idx < kC * (kD / 4); idx += 256) {
        const int i = idx >> 5, c = (idx & 31) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < L.len) x = IO<float>::load4(a.log_alpha + ((L.tok0 + i) * a.H + h) * kD + c);
        *reinterpret_cast<float4*>(sG + i * LD + c) = x;
    }
    if (t < kC) sB[t] = (t < L.len) ? a.beta[(L.tok0 + t) * a.H + h] : 0.f;
    __syncthreads();
    if (t < kD) {
        float acc = 0.f;
        for (int i = 0; i < kC; ++i) {
            acc += sG[i * LD + t];
            sG[i * LD + t] = acc;
        }
    }
    __syncthreads();

    // gated operands
    for (int idx = t; idx < kC * (kD / 4); idx += 256) {
        const int i = idx >> 5, c = (idx & 31) * 4;
        float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), qv = kv;
        if (i < L.len) {
            const size_t off = ((L.tok0 + i) * a.H + h) * kD + c;
            kv = IO<T>::load4(kp + off);
            if (qp) qv = IO<T>::load4(qp + off);
        }
        const float4 G = *reinterpret_cast<const float4*>(sG + i * LD + c);
        const float4 Gl = *reinterpret_cast<const float4*>(sG + (kC - 1) * LD + c);
        const float4 Gr = make_float4(0.5f * Gl.x, 0.5f * Gl.y, 0.5f * Gl.z, 0.5f * Gl.w);   // reference: G_C / 2
        const float kk[4] = {kv.x, kv.y, kv.z, kv.w}, qq[4] = {qv.x, qv.y, qv.z, qv.w};
        const float gg[4] = {G.x, G.y, G.z, G.w}, gr[4] = {Gr.x, Gr.y, Gr.z, Gr.w};
        const float gl[4] = {Gl.x, Gl.y, Gl.z, Gl.w};
        float okg[4], oki[4], oqg[4], oKG[4], oQG[4], oKT[4], ogc[4];
        // a channel that decays by more than e^-160 inside the chunk leaves the range of the
        // two-factor form (the clamp keeps everything finite): flag the call
        if (fminf(fminf(gl[0], gl[1]), fminf(gl[2], gl[3])) < -2.f * kClamp) atomicOr(&hdr->flags, 1);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float e1 = expf(clampf(gg[e] - gr[e]));
            const float e2 = expf(clampf(gr[e] - gg[e]));
            const float eG = expf(gg[e]);
            okg[e] = kk[e] * e1;
            oki[e] = kk[e] * e2;
            oqg[e] = a.scale * qq[e] * e1;
            oKG[e] = kk[e] * eG;
            oQG[e] = a.scale * qq[e] * eG;
            oKT[e] = kk[e] * expf(gl[e] - gg[e]);
            ogc[e] = expf(gl[e]);
        }
        *reinterpret_cast<float4*>(sKg + i * LD + c) = make_float4(okg[0], okg[1], okg[2], okg[3]);
        *reinterpret_cast<float4*>(sKi + i * LD + c) = make_float4(oki[0], oki[1], oki[2], oki[3]);
        *reinterpret_cast<float4*>(sQg + i * LD + c) = make_float4(oqg[0], oqg[1], oqg[2], oqg[3]);
        *reinterpret_cast<float4*>(sKG + i * LD + c) = make_float4(oKG[0], oKG[1], oKG[2], oKG[3]);
        *reinterpret_cast<float4*>(tile + T_QG + i * kD + c) = make_float4(oQG[0], oQG[1], oQG[2], oQG[3]);
        *reinterpret_cast<float4*>(tile + T_KT + i * kD + c) = make_float4(oKT[0], oKT[1], oKT[2], oKT[3]);
        if (i == 0)
            *reinterpret_cast<float4*>(tile + T_GC + c) = make_float4(ogc[0], ogc[1], ogc[2], ogc[3]);
    }
    __syncthreads();

    // V into the buffer that held G
    for (int idx = t; idx < kC * (kD / 4); idx += 256) {
        const int i = idx >> 5, c = (idx & 31) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < L.len) x = IO<T>::load4(vp + ((L.tok0 + i) * a.H + h) * kD + c);
        *reinterpret_cast<float4*>(sG + i * LD + c) = x;
    }

    // a2 + a5: Akk (strictly lower, row-scaled by beta) and Aqk (lower incl. diagonal)
    {
        const int i = t >> 2, jq = t & 3;
        const float bi = sB[i];
        for (int m = 0; m < kC / 4; ++m) {
            const int j = jq + 4 * m;
            float akk = 0.f, aqk = 0.f;
            if (j <= i) {
                const float4* ki = reinterpret_cast<const float4*>(sKi + j * LD);
                const float4* kg = reinterpret_cast<const float4*>(sKg + i * LD);
                const float4* qg = reinterpret_cast<const float4*>(sQg + i * LD);
#pragma unroll 8
                for (int d = 0; d < kD / 4; ++d) {
                    const float4 b = ki[d], x = kg[d], y = qg[d];
                    akk += x.x * b.x + x.y * b.y + x.z * b.z + x.w * b.w;
                    aqk += y.x * b.x + y.y * b.y + y.z * b.z + y.w * b.w;
                }
            }
            sA[i * LDA + j] = (j < i) ? bi * akk : 0.f;
            tile[T_AQK + i * kC + j] = aqk;
        }
    }
    __syncthreads();

    // a3: T = (I + Akk)^-1, one column per thread by forward substitution
    if (t < kC) {
        const int j = t;
        for (int i = 0; i < kC; ++i) {
            float x = (i == j) ? 1.f : 0.f;
            for (int m = j; m < i; ++m) x -= sA[i * LDA + m] * sT[m * LDA + j];
            sT[i * LDA + j] = (i < j) ? 0.f : x;
        }
    }
    __syncthreads();

    // a4: W = T Diag(beta) (Gamma.K), U = T Diag(beta) V
    {
        const int i = t >> 2, cq = t & 3;
        float4 w[8], u[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) w[m] = u[m] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j <= i; ++j) {
            const float mij = sT[i * LDA + j] * sB[j];
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const int c = cq * 4 + 16 * m;
                const float4 x = *reinterpret_cast<const float4*>(sKG + j * LD + c);
                const float4 y = *reinterpret_cast<const float4*>(sG + j * LD + c);
                w[m].x += mij * x.x; w[m].y += mij * x.y; w[m].z += mij * x.z; w[m].w += mij * x.w;
                u[m].x += mij * y.x; u[m].y += mij * y.y; u[m].z += mij * y.z; u[m].w += mij * y.w;
            }
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) {
            const int c = cq * 4 + 16 * m;
            *reinterpret_cast<float4*>(tile + T_W + i * kD + c) = w[m];
            *reinterpret_cast<float4*>(tile + T_U + i * kD + c) = u[m];
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256, 1)
kda_inter_simt(ChunkArgs a, const float* __restrict__ tiles, int n_begin)
{
    extern __shared__ __align__(16) float smem[];
    float* sW = smem;
    float* sQ = sW + kC * LD;
    float* sK = sQ + kC * LD;
    float* sAqk = sK + kC * LD;
    float* sS = sAqk + kC * LDA;       // [128][NS]
    float* sVn = sS + kD * NS;         // [64][NS]
    float* sU = sVn + kC * NS;         // [64][NS]
    float* sgC = sU + kC * NS;         // [128]

    const int t = threadIdx.x;
    const int slice = blockIdx.x, h = blockIdx.y, n = n_begin + blockIdx.z;
    const int col0 = slice * NS;
    T* op = reinterpret_cast<T*>(a.o);

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

    const size_t sbase = ((size_t)n * a.H + h) * (size_t)(kD * kD);
    for (int idx = t; idx < kD * NS / 4; idx += 256) {
        const int kk = idx >> 2, c = (idx & 3) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (a.S_in) x = *reinterpret_cast<const float4*>(a.S_in + sbase + kk * kD + col0 + c);
        *reinterpret_cast<float4*>(sS + kk * NS + c) = x;
    }

    for (int64_t g = cb; g < ce; ++g) {
        const float* tile = tiles + ((size_t)(g - a.g0) * a.H + h) * T_FLOATS;
        const int64_t tok0 = tok_begin + (g - seq_c0) * kC;
        const int len = (tok_end - tok0) < kC ? (int)(tok_end - tok0) : kC;
        __syncthreads();   // previous iteration's readers are done
        for (int idx = t; idx < kC * (kD / 4); idx += 256) {
            const int i = idx >> 5, c = (idx & 31) * 4;
            *reinterpret_cast<float4*>(sW + i * LD + c) =
                *reinterpret_cast<const float4*>(tile + T_W + i * kD + c);
            *reinterpret_cast<float4*>(sQ + i * LD + c) =
                *reinterpret_cast<const float4*>(tile + T_QG + i * kD + c);
            *reinterpret_cast<float4*>(sK + i * LD + c) =
                *reinterpret_cast<const float4*>(tile + T_KT + i * kD + c);
        }
        for (int idx = t; idx < kC * kC; idx += 256)
            sAqk[(idx >> 6) * LDA + (idx & 63)] = tile[T_AQK + idx];
        for (int idx = t; idx < kC * NS; idx += 256)
            sU[idx] = tile[T_U + (idx / NS) * kD + col0 + (idx % NS)];
        if (t < kD) sgC[t] = tile[T_GC + t];
        __syncthreads();

        // a6: V_new = U - W S ;  inter-chunk part of a7: (Gamma.Q) S
        const int r = t >> 2, cg = (t & 3) * 4;
        float vn[4], oq[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) { vn[e] = sU[r * NS + cg + e]; oq[e] = 0.f; }
        for (int kk = 0; kk < kD; ++kk) {
            const float w = sW[r * LD + kk], qv = sQ[r * LD + kk];
            const float4 s = *reinterpret_cast<const float4*>(sS + kk * NS + cg);
            vn[0] -= w * s.x; vn[1] -= w * s.y; vn[2] -= w * s.z; vn[3] -= w * s.w;
            oq[0] += qv * s.x; oq[1] += qv * s.y; oq[2] += qv * s.z; oq[3] += qv * s.w;
        }
        *reinterpret_cast<float4*>(sVn + r * NS + cg) = make_float4(vn[0], vn[1], vn[2], vn[3]);
        __syncthreads();

        // a7: O = (Gamma.Q) S + Aqk V_new
        if (op) {
            for (int j = 0; j <= r; ++j) {
                const float aq = sAqk[r * LDA + j];
                const float4 x = *reinterpret_cast<const float4*>(sVn + j * NS + cg);
                oq[0] += aq * x.x; oq[1] += aq * x.y; oq[2] += aq * x.z; oq[3] += aq * x.w;
            }
            if (r < len)
                IO<T>::store4(op + ((tok0 + r) * a.H + h) * kD + col0 + cg,
                              make_float4(oq[0], oq[1], oq[2], oq[3]));
        }

        // a8: S <- Diag(gamma^C) S + ((gamma^C/Gamma).K)^T V_new
        const int kk = t >> 1, c8 = (t & 1) * 8;
        float sn[8];
        {
            const float gc = sgC[kk];
#pragma unroll
            for (int e = 0; e < 8; ++e) sn[e] = gc * sS[kk * NS + c8 + e];
            for (int j = 0; j < kC; ++j) {
                const float kt = sK[j * LD + kk];
                const float4 x0 = *reinterpret_cast<const float4*>(sVn + j * NS + c8);
                const float4 x1 = *reinterpret_cast<const float4*>(sVn + j * NS + c8 + 4);
                sn[0] += kt * x0.x; sn[1] += kt * x0.y; sn[2] += kt * x0.z; sn[3] += kt * x0.w;
                sn[4] += kt * x1.x; sn[5] += kt * x1.y; sn[6] += kt * x1.z; sn[7] += kt * x1.w;
            }
        }
        // every thread owns its 8 state entries; the reads of sS in a6 finished at the barrier above
#pragma unroll
        for (int e = 0; e < 8; ++e) sS[kk * NS + c8 + e] = sn[e];
    }
    __syncthreads();
    for (int idx = t; idx < kD * NS / 4; idx += 256) {
        const int kk = idx >> 2, c = (idx & 3) * 4;
        *reinterpret_cast<float4*>(a.S_out + sbase + kk * kD + col0 + c) =
            *reinterpret_cast<const float4*>(sS + kk * NS + c);
    }
}

__global__ void kda_prep_kernel(WsHeader* hdr, const int32_t* __restrict__ cu,
                                int32_t* __restrict__ chunk_cu, int n_seqs)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        hdr->status = 0;
        hdr->where = 0;
        hdr->flags = 0;
        if (cu) {
            int acc = 0;
            chunk_cu[0] = 0;
            for (int n = 0; n < n_seqs; ++n) {
                acc += (cu[n + 1] - cu[n] + kC - 1) / kC;
                chunk_cu[n + 1] = acc;
            }
        }
    }
}

template <typename T>
kda_status_t launch_simt_t(const ChunkArgs& a, float* tiles, int n_begin, int n_count, WsHeader* hdr,
                           cudaStream_t st)
{
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (!lk.st->attr_done[4]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_intra_simt<T>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kIntraSmem));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_inter_simt<T>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kInterSmem));
            lk.st->attr_done[4] = true;
        }
    }
    if (n_count > 65535)
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: more than 65535 sequences in one fp32 call");
    const int64_t n_chunks = a.g1 - a.g0;
    if (n_chunks > 0) {
        dim3 grid((unsigned)n_chunks, (unsigned)a.H);
        ProfScope ps(PROF_INTRA, st);
        kda_intra_simt<T><<<grid, 256, kIntraSmem, st>>>(a, tiles, hdr);
        count_launch();
        KDA_CUDA_TRY(cudaGetLastError());
    }
    if (n_count > 0) {
        dim3 grid(kD / NS, (unsigned)a.H, (unsigned)n_count);
        ProfScope ps(PROF_INTER, st);
        kda_inter_simt<T><<<grid, 256, kInterSmem, st>>>(a, tiles, n_begin);
        count_launch();
        KDA_CUDA_TRY(cudaGetLastError());
    }
    return KDA_OK;
}

}  // namespace

size_t simt_tile_bytes() { return (size_t)T_FLOATS * sizeof(float); }

kda_status_t launch_chunk_simt(const ChunkArgs& a, kda_dtype_t dt, void* tiles, int n_begin,
                               int n_count, WsHeader* hdr, cudaStream_t st)
{
    if (dt != KDA_F32) return fail(KDA_ERR_UNSUPPORTED, "the FMA path serves fp32 storage only");
    return launch_simt_t<float>(a, (float*)tiles, n_begin, n_count, hdr, st);
}

kda_status_t launch_prep(WsHeader* hdr, const int32_t* cu_seqlens, int32_t* chunk_cu, int n_seqs,
                         cudaStream_t st)
{
    ProfScope ps(PROF_PREP, st);
    kda_prep_kernel<<<1, 32, 0, st>>>(hdr, cu_seqlens, chunk_cu, n_seqs);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

}  // namespace kda
