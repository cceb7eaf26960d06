// Recurrent decode step of KDA (paper Section 3, Eq. 1, one token per sequence and head):
//     Sd = Diag(alpha) S;  r = v - Sd^T k;  S = Sd + beta k r^T;  o = scale S^T q
// evaluated in ONE pass over the 128x128 fp32 state using the identity
//     o = scale (Sd^T q + beta (q.k) r),
// so that both column reductions (Sd^T k and Sd^T q) are taken while the state streams through
// registers, and the state is written back exactly once.  HBM-bound: 64 KiB read + 64 KiB written
// per (sequence, head).
//
// One CTA of 256 threads owns one state.  Thread (warp w, lane l) holds rows w, w+8, ... and the
// four columns 4l..4l+3 of each: every warp-level access is one fully coalesced 512-byte row, and
// all 16 loads of a thread are issued before the first use (64 KiB in flight per CTA).
#include "kda_common.cuh"

namespace kda {
namespace {

__device__ __forceinline__ float4 ld_stream(const float* p) {
    float4 r;
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream(float* p, float4 x) {
    asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(x.x),
                 "f"(x.y), "f"(x.z), "f"(x.w)
                 : "memory");
}
// packed fp32 arithmetic (two independent round-to-nearest operations per instruction on sm_100):
// the multi-token kernel is bound by instruction issue, not by HBM
__device__ __forceinline__ void mul4(float4& x, float a) {
    const float2 aa = make_float2(a, a);
    const float2 lo = __fmul2_rn(make_float2(x.x, x.y), aa), hi = __fmul2_rn(make_float2(x.z, x.w), aa);
    x = make_float4(lo.x, lo.y, hi.x, hi.y);
}
__device__ __forceinline__ void fma4(float4& acc, float a, const float4& x) {   // acc += a * x
    const float2 aa = make_float2(a, a);
    const float2 lo = __ffma2_rn(aa, make_float2(x.x, x.y), make_float2(acc.x, acc.y));
    const float2 hi = __ffma2_rn(aa, make_float2(x.z, x.w), make_float2(acc.z, acc.w));
    acc = make_float4(lo.x, lo.y, hi.x, hi.y);
}
template <typename T> __device__ __forceinline__ float to_f(T x);
template <> __device__ __forceinline__ float to_f<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 x) {
    return __bfloat162float(x);
}

// Layer mode (kda_layer_decode_step, paper Section 4 "Neural Parameterization"): q and k arrive
// un-normalised, `log_alpha` points to the bf16 pre-activations of the decay function, `beta` to the
// pre-activations of beta, and the output row goes through the head-wise RMSNorm and the sigmoid
// output gate before it is stored.  All of it is arithmetic on 128-vectors beside a 64 KiB state
// stream: free at the HBM bound.
struct DecodeLayer {
    const float* A_log;        // [H]
    const float* dt_bias;      // [H, dk]
    const void* g_o;           // bf16 [n_seqs, H, dv]
    const float* rms_weight;   // [dv]
    float l2_eps, rms_eps;
};

template <typename T, bool kLayer>
__global__ void __launch_bounds__(256, 2)
kda_decode_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                  const float* __restrict__ log_alpha, const float* __restrict__ beta, float* S,
                  const int32_t* __restrict__ slot, T* __restrict__ o, int H, float scale, DecodeLayer lay)
{
    __shared__ float s_a[kD], s_k[kD], s_q[kD];
    __shared__ float4 s_red[2][8][32];
    const int item = blockIdx.x;
    const int n = item / H, h = item - n * H;
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const size_t sl = slot ? (size_t)slot[n] : (size_t)n;
    float* Sp = S + (sl * H + h) * (size_t)(kD * kD) + lane * 4;

    float4 x[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) x[m] = ld_stream(Sp + (size_t)(warp + 8 * m) * kD);

    const size_t vec = (size_t)item * kD;
    if (t < kD) {
        if (kLayer) {
            const float z = to_f<T>(reinterpret_cast<const T*>(log_alpha)[vec + t]) + lay.dt_bias[(size_t)h * kD + t];
            const float sp = fmaxf(z, 0.f) + log1pf(expf(-fabsf(z)));
            s_a[t] = expf(-expf(lay.A_log[h]) * sp);
        } else {
            s_a[t] = expf(log_alpha[vec + t]);
        }
        s_k[t] = to_f<T>(k[vec + t]);
        s_q[t] = to_f<T>(q[vec + t]);
    }
    __syncthreads();

    // q.k, redundantly per warp (4 rows per lane, butterfly reduce); layer mode: the norms as well
    float qk = 0.f, ssk = 0.f, ssq = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float kv = s_k[lane * 4 + i], qv = s_q[lane * 4 + i];
        qk += qv * kv;
        if (kLayer) {
            ssk += kv * kv;
            ssq += qv * qv;
        }
    }
#pragma unroll
    for (int ofs = 16; ofs > 0; ofs >>= 1) {
        qk += __shfl_xor_sync(0xffffffffu, qk, ofs);
        if (kLayer) {
            ssk += __shfl_xor_sync(0xffffffffu, ssk, ofs);
            ssq += __shfl_xor_sync(0xffffffffu, ssq, ofs);
        }
    }
    const float rk = kLayer ? rsqrtf(ssk + lay.l2_eps) : 1.f;   // 1 / |k|, 1 / |q| (L2Norm)
    const float rq = kLayer ? rsqrtf(ssq + lay.l2_eps) : 1.f;
    if (kLayer) qk *= rk * rq;

    float4 p = make_float4(0.f, 0.f, 0.f, 0.f), s = p;
#pragma unroll
    for (int m = 0; m < 16; ++m) {
        const int row = warp + 8 * m;
        const float a = s_a[row], kk = kLayer ? s_k[row] * rk : s_k[row], qq = kLayer ? s_q[row] * rq : s_q[row];
        x[m].x *= a; x[m].y *= a; x[m].z *= a; x[m].w *= a;
        p.x += kk * x[m].x; p.y += kk * x[m].y; p.z += kk * x[m].z; p.w += kk * x[m].w;
        s.x += qq * x[m].x; s.y += qq * x[m].y; s.z += qq * x[m].z; s.w += qq * x[m].w;
    }
    s_red[0][warp][lane] = p;
    s_red[1][warp][lane] = s;
    __syncthreads();
    p = s_red[0][0][lane];
    s = s_red[1][0][lane];
#pragma unroll
    for (int w = 1; w < 8; ++w) {   // fixed order: bitwise reproducible
        float4 a = s_red[0][w][lane], b = s_red[1][w][lane];
        p.x += a.x; p.y += a.y; p.z += a.z; p.w += a.w;
        s.x += b.x; s.y += b.y; s.z += b.z; s.w += b.w;
    }
    const float bt = kLayer ? 1.f / (1.f + expf(-beta[item])) : beta[item];
    float4 vv = IO<T>::load4(v + vec + lane * 4);
    float4 r = make_float4(vv.x - p.x, vv.y - p.y, vv.z - p.z, vv.w - p.w);
    if (warp == 0) {
        const float c = bt * qk;
        float4 ov = make_float4(scale * (s.x + c * r.x), scale * (s.y + c * r.y),
                                scale * (s.z + c * r.z), scale * (s.w + c * r.w));
        if (kLayer) {   // head-wise RMSNorm over the 128 values of the row (4 per lane), weight, sigmoid gate
            float ss = ov.x * ov.x + ov.y * ov.y + ov.z * ov.z + ov.w * ov.w;
#pragma unroll
            for (int ofs = 16; ofs > 0; ofs >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, ofs);
            const float rstd = rsqrtf(ss * (1.f / kD) + lay.rms_eps);
            const float4 w4 = *reinterpret_cast<const float4*>(lay.rms_weight + lane * 4);
            const float4 g4 = IO<T>::load4(reinterpret_cast<const T*>(lay.g_o) + vec + lane * 4);
            ov.x *= rstd * w4.x / (1.f + expf(-g4.x));
            ov.y *= rstd * w4.y / (1.f + expf(-g4.y));
            ov.z *= rstd * w4.z / (1.f + expf(-g4.z));
            ov.w *= rstd * w4.w / (1.f + expf(-g4.w));
        }
        IO<T>::store4(o + vec + lane * 4, ov);
    }
#pragma unroll
    for (int m = 0; m < 16; ++m) {
        const int row = warp + 8 * m;
        const float c = kLayer ? bt * s_k[row] * rk : bt * s_k[row];
        x[m].x += c * r.x; x[m].y += c * r.y; x[m].z += c * r.z; x[m].w += c * r.w;
        st_stream(Sp + (size_t)row * kD, x[m]);
    }
}

// Multi-token decode: the same recurrence for T consecutive tokens of each sequence (speculative
// decoding, continuation of a chunked prefill by a few tokens) with the state held in registers
// across the tokens: it crosses HBM once in each direction per call instead of once per token.
// Layout: q, k, log_alpha [n_seqs, T, H, 128], v, o [n_seqs, T, H, 128], beta [n_seqs, T, H].
// Thread layout of the multi-token kernel: warp w owns the 16 state columns 16w..16w+15 for ALL 128
// dk rows; lane (rg, cg) = (lane >> 2, lane & 3) holds rows rg, rg + 8, ..., rg + 120 and the four
// columns 16w + 4cg .. +3.  The two column reductions of a token (S^T k and S^T q, over the dk rows)
// then stay inside the warp: 16 rows in the thread's registers, the 8 row groups by three
// butterfly shuffles.  No shared-memory reduction and no CTA-wide barrier per token (the
// single-token kernel keeps its fully coalesced row layout: it has no token loop to protect).
//
// The token loop is bound by instruction issue, so a CTA that only started to fetch its state when
// it began would leave HBM idle while it computes.  CTAs are therefore persistent (two per SM) and
// fetch the NEXT state into shared memory with asynchronous 16-byte copies while they work on the
// current one; every thread copies exactly the elements it will own into its own slots, so the
// hand-over needs no barrier: a thread waits for its own copies only.
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src_gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)),
                 "l"(src_gmem)
                 : "memory");
}
// Dynamic shared memory of the multi-token kernel
template <typename T> struct MultiSmem {
    static constexpr int GT = 8;                        // tokens staged together
    static constexpr int kState = 16 * 256 * 16;        // the prefetched state: element m of thread t at [m][t]
    static constexpr int kAkq = GT * kD * 16;           // per token and dk row: (alpha, k, q, beta k)
    static constexpr int kV = GT * kD * 4;
    static constexpr int kRawA = GT * kD * 4;           // raw log alpha of the next item's first tokens
    static constexpr int kRawX = GT * kD * (int)sizeof(T);   // raw k / q / v of the same tokens
    static constexpr int oAkq = kState, oV = oAkq + kAkq, oRawA = oV + kV, oRawK = oRawA + kRawA,
                         oRawQ = oRawK + kRawX, oRawV = oRawQ + kRawX, oRawB = oRawV + kRawX,
                         kTotal = oRawB + 64;
};
__device__ __forceinline__ void cp_async4b(void* dst_smem, const void* src_gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)),
                 "l"(src_gmem)
                 : "memory");
}

template <typename T>
__global__ void __launch_bounds__(256, 2)
kda_decode_multi_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                        const float* __restrict__ log_alpha, const float* __restrict__ beta, float* S,
                        const int32_t* __restrict__ slot, T* __restrict__ o, int H, int n_tok, float scale,
                        int n_items)
{
    using L = MultiSmem<T>;
    constexpr int GT = L::GT;
    extern __shared__ __align__(16) unsigned char sm[];
    float4* s_next = reinterpret_cast<float4*>(sm);
    float4 (*s_akq)[kD] = reinterpret_cast<float4(*)[kD]>(sm + L::oAkq);
    float (*s_v)[kD] = reinterpret_cast<float(*)[kD]>(sm + L::oV);
    float (*r_a)[kD] = reinterpret_cast<float(*)[kD]>(sm + L::oRawA);
    T (*r_k)[kD] = reinterpret_cast<T(*)[kD]>(sm + L::oRawK);
    T (*r_q)[kD] = reinterpret_cast<T(*)[kD]>(sm + L::oRawQ);
    T (*r_v)[kD] = reinterpret_cast<T(*)[kD]>(sm + L::oRawV);
    float* r_b = reinterpret_cast<float*>(sm + L::oRawB);
    __shared__ float s_b[GT], s_qk[GT];
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const int rg = lane >> 2, cg = lane & 3, col = warp * 16 + cg * 4;
    const int gfirst = n_tok < GT ? n_tok : GT;   // tokens of an item's first group

    auto state_of = [&](int item) {
        const int n = item / H, h = item - n * H;
        const size_t sl = slot ? (size_t)slot[n] : (size_t)n;
        return S + (sl * H + h) * (size_t)(kD * kD) + col;
    };
    // Everything the next item needs first -- its state and the vectors of its first tokens -- is
    // requested with asynchronous copies while the current item is worked on.
    auto fetch = [&](int item) {
        const float* Sp = state_of(item);   // a copy instruction of a warp covers 8 consecutive rows x 64 contiguous bytes
#pragma unroll
        for (int m = 0; m < 16; ++m) cp_async16(&s_next[m * 256 + t], Sp + (size_t)(rg + 8 * m) * kD);
        const int n = item / H, h = item - n * H;
        constexpr int CA = kD * 4 / 16, CX = kD * (int)sizeof(T) / 16;   // 16-byte pieces per token
        for (int idx = t; idx < gfirst * (CA + 3 * CX); idx += 256) {
            const int tok = idx / (CA + 3 * CX), j = idx - tok * (CA + 3 * CX);
            const size_t vec = ((size_t)(n * n_tok + tok) * H + h) * kD;
            if (j < CA) cp_async16(&r_a[tok][j * 4], log_alpha + vec + j * 4);
            else if (j < CA + CX) cp_async16(&r_k[tok][(j - CA) * (16 / (int)sizeof(T))], k + vec + (j - CA) * (16 / (int)sizeof(T)));
            else if (j < CA + 2 * CX) cp_async16(&r_q[tok][(j - CA - CX) * (16 / (int)sizeof(T))], q + vec + (j - CA - CX) * (16 / (int)sizeof(T)));
            else cp_async16(&r_v[tok][(j - CA - 2 * CX) * (16 / (int)sizeof(T))], v + vec + (j - CA - 2 * CX) * (16 / (int)sizeof(T)));
        }
        if (t < gfirst) cp_async4b(&r_b[t], beta + (size_t)(n * n_tok + t) * H + h);
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    int item = blockIdx.x;
    if (item < n_items) fetch(item);
    for (; item < n_items; item += gridDim.x) {
        const int n = item / H, h = item - n * H;
        float* Sp = state_of(item);
        float4 x[16];
        asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
        for (int m = 0; m < 16; ++m) x[m] = s_next[m * 256 + t];   // (each thread reads back its own copies)
        __syncthreads();   // the raw vectors were copied by other threads; the previous item's vectors are no longer read
        auto vec_of = [&](int tt) { return ((size_t)(n * n_tok + tt) * H + h) * kD; };
        for (int g0 = 0; g0 < n_tok; g0 += GT) {
            const int gn = (n_tok - g0) < GT ? (n_tok - g0) : GT;
            {   // thread (half, c): channel c of tokens half, half + 2, ...
                const int c = t & (kD - 1), half = t >> 7;
                if (g0 == 0) {   // from the prefetched raw vectors
#pragma unroll
                    for (int j = 0; j < GT / 2; ++j) {
                        const int tok = half + 2 * j;
                        if (tok < gn) {
                            const float kk = to_f<T>(r_k[tok][c]), bb = r_b[tok];
                            s_akq[tok][c] = make_float4(expf(r_a[tok][c]), kk, to_f<T>(r_q[tok][c]), bb * kk);
                            s_v[tok][c] = to_f<T>(r_v[tok][c]);
                            if (c == 0) s_b[tok] = bb;
                        }
                    }
                } else {         // later groups of a long call: straight from global memory, loads first
                    __syncthreads();   // the previous group's vectors are no longer read
                    float la[GT / 2], kk[GT / 2], qq[GT / 2], vv[GT / 2], bb[GT / 2];
#pragma unroll
                    for (int j = 0; j < GT / 2; ++j) {
                        const int tok = half + 2 * j;
                        if (tok < gn) {
                            const size_t vec = vec_of(g0 + tok) + c;
                            la[j] = log_alpha[vec];
                            kk[j] = to_f<T>(k[vec]);
                            qq[j] = to_f<T>(q[vec]);
                            vv[j] = to_f<T>(v[vec]);
                            bb[j] = beta[(size_t)(n * n_tok + g0 + tok) * H + h];
                        }
                    }
#pragma unroll
                    for (int j = 0; j < GT / 2; ++j) {
                        const int tok = half + 2 * j;
                        if (tok < gn) {
                            s_akq[tok][c] = make_float4(expf(la[j]), kk[j], qq[j], bb[j] * kk[j]);
                            s_v[tok][c] = vv[j];
                            if (c == 0) s_b[tok] = bb[j];
                        }
                    }
                }
            }
            __syncthreads();
            // the raw buffers and the state buffer are free: the next item's data may stream in
            if (g0 == 0 && item + (int)gridDim.x < n_items) fetch(item + gridDim.x);
            if (warp < gn) {   // q.k of token `warp` (4 channels per lane, butterfly reduce)
                float qk = 0.f;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 e = s_akq[warp][lane * 4 + i];
                    qk += e.z * e.y;
                }
#pragma unroll
                for (int ofs = 16; ofs > 0; ofs >>= 1) qk += __shfl_xor_sync(0xffffffffu, qk, ofs);
                if (lane == 0) s_qk[warp] = qk;
            }
            __syncthreads();
            for (int tok = 0; tok < gn; ++tok) {
                float4 p = make_float4(0.f, 0.f, 0.f, 0.f), s = p;
#pragma unroll
                for (int m4 = 0; m4 < 16; m4 += 4) {
                    float4 e[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) e[j] = s_akq[tok][rg + 8 * (m4 + j)];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        mul4(x[m4 + j], e[j].x);
                        fma4(p, e[j].y, x[m4 + j]);
                        fma4(s, e[j].z, x[m4 + j]);
                    }
                    asm volatile("" ::: "memory");   // keeps the loads of later rows from being hoisted (registers)
                }
                // the eight row groups of a column group: lanes that differ in bits 2..4 (fixed order)
#pragma unroll
                for (int ofs = 4; ofs < 32; ofs <<= 1) {
                    p.x += __shfl_xor_sync(0xffffffffu, p.x, ofs); p.y += __shfl_xor_sync(0xffffffffu, p.y, ofs);
                    p.z += __shfl_xor_sync(0xffffffffu, p.z, ofs); p.w += __shfl_xor_sync(0xffffffffu, p.w, ofs);
                    s.x += __shfl_xor_sync(0xffffffffu, s.x, ofs); s.y += __shfl_xor_sync(0xffffffffu, s.y, ofs);
                    s.z += __shfl_xor_sync(0xffffffffu, s.z, ofs); s.w += __shfl_xor_sync(0xffffffffu, s.w, ofs);
                }
                const float4 vv = *reinterpret_cast<const float4*>(&s_v[tok][col]);
                const float4 r = make_float4(vv.x - p.x, vv.y - p.y, vv.z - p.z, vv.w - p.w);
                if (rg == 0) {
                    const float c = s_b[tok] * s_qk[tok];
                    IO<T>::store4(o + vec_of(g0 + tok) + col,
                                  make_float4(scale * (s.x + c * r.x), scale * (s.y + c * r.y),
                                              scale * (s.z + c * r.z), scale * (s.w + c * r.w)));
                }
#pragma unroll
                for (int m4 = 0; m4 < 16; m4 += 4) {
                    float bk[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) bk[j] = s_akq[tok][rg + 8 * (m4 + j)].w;
#pragma unroll
                    for (int j = 0; j < 4; ++j) fma4(x[m4 + j], bk[j], r);
                    asm volatile("" ::: "memory");
                }
            }
        }
#pragma unroll
        for (int m = 0; m < 16; ++m) st_stream(Sp + (size_t)(rg + 8 * m) * kD, x[m]);
    }
}

}  // namespace

kda_status_t launch_decode(const void* q, const void* k, const void* v, const float* log_alpha,
                           const float* beta, float* S, const int32_t* slot, void* o, int n_seqs,
                           int H, float scale, kda_dtype_t dt, cudaStream_t st)
{
    if (n_seqs == 0) return KDA_OK;
    const unsigned grid = (unsigned)((size_t)n_seqs * H);
    ProfScope ps(PROF_DECODE, st);
    if (dt == KDA_BF16) {
        using T = __nv_bfloat16;
        kda_decode_kernel<T, false><<<grid, 256, 0, st>>>((const T*)q, (const T*)k, (const T*)v,
                                                          log_alpha, beta, S, slot, (T*)o, H, scale, DecodeLayer());
    } else {
        kda_decode_kernel<float, false><<<grid, 256, 0, st>>>((const float*)q, (const float*)k,
                                                              (const float*)v, log_alpha, beta, S, slot,
                                                              (float*)o, H, scale, DecodeLayer());
    }
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

kda_status_t launch_layer_decode(const void* q_c, const void* k_c, const void* v, const void* g_a,
                                 const float* b_pre, const void* g_o, const float* A_log, const float* dt_bias,
                                 const float* rms_weight, float l2_eps, float rms_eps, float* S,
                                 const int32_t* slot, void* y, int n_seqs, int H, float scale, cudaStream_t st)
{
    if (n_seqs == 0) return KDA_OK;
    using T = __nv_bfloat16;
    DecodeLayer lay;
    lay.A_log = A_log; lay.dt_bias = dt_bias; lay.g_o = g_o; lay.rms_weight = rms_weight;
    lay.l2_eps = l2_eps; lay.rms_eps = rms_eps;
    const unsigned grid = (unsigned)((size_t)n_seqs * H);
    ProfScope ps(PROF_DECODE, st);
    kda_decode_kernel<T, true><<<grid, 256, 0, st>>>((const T*)q_c, (const T*)k_c, (const T*)v,
                                                     reinterpret_cast<const float*>(g_a), b_pre, S, slot, (T*)y, H,
                                                     scale, lay);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

kda_status_t launch_decode_multi(const void* q, const void* k, const void* v, const float* log_alpha,
                                 const float* beta, float* S, const int32_t* slot, void* o, int n_seqs,
                                 int n_tok, int H, float scale, kda_dtype_t dt, cudaStream_t st)
{
    if (n_seqs == 0 || n_tok == 0) return KDA_OK;
    int n_sm = 0;
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (!lk.st->attr_done[6]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_decode_multi_kernel<__nv_bfloat16>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              MultiSmem<__nv_bfloat16>::kTotal));
            KDA_CUDA_TRY(cudaFuncSetAttribute(kda_decode_multi_kernel<float>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              MultiSmem<float>::kTotal));
            lk.st->attr_done[6] = true;
        }
        if (lk.st->n_sm == 0) {
            int dev = 0;
            KDA_CUDA_TRY(cudaGetDevice(&dev));
            KDA_CUDA_TRY(cudaDeviceGetAttribute(&lk.st->n_sm, cudaDevAttrMultiProcessorCount, dev));
        }
        n_sm = lk.st->n_sm;
    }
    const int n_items = n_seqs * H;
    const unsigned grid = (unsigned)(n_items < 2 * n_sm ? n_items : 2 * n_sm);   // persistent, two CTAs per SM
    ProfScope ps(PROF_DECODE, st);
    if (dt == KDA_BF16) {
        using T = __nv_bfloat16;
        kda_decode_multi_kernel<T><<<grid, 256, MultiSmem<T>::kTotal, st>>>((const T*)q, (const T*)k, (const T*)v, log_alpha,
                                                                  beta, S, slot, (T*)o, H, n_tok, scale, n_items);
    } else {
        kda_decode_multi_kernel<float><<<grid, 256, MultiSmem<float>::kTotal, st>>>((const float*)q, (const float*)k,
                                                                      (const float*)v, log_alpha, beta, S, slot,
                                                                      (float*)o, H, n_tok, scale, n_items);
    }
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

}  // namespace kda
