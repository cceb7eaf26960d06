// Chunkwise forward of the GENERAL diagonal-plus-low-rank recurrence (paper Section 6.1, "Relation to
// DPLR"; Section 3.2's kernel-time comparison), fp32 FMA path:
//
//     S_t = (Diag(exp(g_t)) + b_t a_t^T) S_{t-1} + k_t v_t^T ,      o_t = scale * S_t^T q_t .
//
// It is the comparison workload for the KDA kernels: same chunk length, same two-kernel structure
// and the same arithmetic style as the fp32 KDA path (kda_chunk_simt.cu), so that the ratio of the
// two run times shows what binding a and b to k saves (Section 6.1 counts four second-level Gram
// matrices against two, and three more matrix products in the inter-chunk and output stage).
//
//   intra  one CTA per (chunk, head): cumulative log-decay G; the four gated Gram matrices
//          Aab[i,j] = sum_d a_i exp(G_{i-1} - G_j) b_j,  Aak (with k_j)        (j <  i)
//          Aqb[i,j] = sum_d q_i exp(G_i     - G_j) b_j,  Aqk (with k_j)        (j <= i);
//          T = (I - Aab)^-1 by forward substitution;  w = T (a . exp(G_{i-1})),  u = T (Aak V).
//          Writes w, u, q . exp(G), k . exp(G_C - G), b . exp(G_C - G), Aqk, Aqb, exp(G_C) to a tile.
//   inter  one CTA per (sequence, head, 16-column slice of dv), sequential over the chunks:
//          X = u + w S,   O = (q . exp(G)) S + Aqb X + Aqk V,
//          S <- Diag(exp(G_C)) S + (k . exp(G_C - G))^T V + (b . exp(G_C - G))^T X.
//
// The decay ratios are factored around G_m = G_C / 2 per channel, exponents clamped to [-80, 80], as
// in the KDA path; entries above the diagonal are selected to zero, never multiplied.
#include <vector>

#include "kda_common.cuh"

namespace kda {
namespace {

constexpr int LD = kD + 4;
constexpr int LDA = kC + 1;
constexpr float kClamp = 80.f;
constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// scratch tile (floats)
constexpr int T_W = 0;
constexpr int T_U = T_W + kC * kD;
constexpr int T_QG = T_U + kC * kD;
constexpr int T_KT = T_QG + kC * kD;
constexpr int T_BT = T_KT + kC * kD;
constexpr int T_AQK = T_BT + kC * kD;
constexpr int T_AQB = T_AQK + kC * kC;
constexpr int T_GC = T_AQB + kC * kC;
constexpr int T_FLOATS = T_GC + kD;

constexpr size_t kIntraSmem = (size_t)(5 * kC * LD + 3 * kC * LDA) * sizeof(float);
constexpr int NS = 16;               // dv columns per inter-chunk CTA
constexpr size_t kInterSmem =
    (size_t)(4 * kC * LD + 2 * kC * LDA + kD * NS + 3 * kC * NS + kD) * sizeof(float);
static_assert(kIntraSmem <= 232448 && kInterSmem <= 232448, "fits the shared memory of one SM");

struct DplrArgs {
    ChunkArgs c;        // log_alpha = g; beta unused
    const float* a;
    const float* b;
};

__device__ __forceinline__ float clampf(float x) { return fminf(fmaxf(x, -kClamp), kClamp); }

__global__ void __launch_bounds__(256, 1) dplr_intra_simt(DplrArgs p, float* __restrict__ tiles, WsHeader* hdr)
{
    extern __shared__ __align__(16) float smem[];
    float* sG = smem;                    // cumulative log-decay, later V
    float* sQ1 = sG + kC * LD;           // scale q exp(G - G_m); later a . exp(G_{i-1})
    float* sA1 = sQ1 + kC * LD;          // a exp(G_{i-1} - G_m)
    float* sK2 = sA1 + kC * LD;          // k exp(G_m - G); later Aak V
    float* sB2 = sK2 + kC * LD;          // b exp(G_m - G)
    float* sAab = sB2 + kC * LD;
    float* sT = sAab + kC * LDA;         // (I - Aab)^-1
    float* sAak = sT + kC * LDA;

    const ChunkArgs& a = p.c;
    const int t = threadIdx.x;
    const int h = blockIdx.y;
    const int64_t g = a.g0 + blockIdx.x;
    const ChunkLoc L = locate_chunk(a, g);
    const float* qp = reinterpret_cast<const float*>(a.q);
    const float* kp = reinterpret_cast<const float*>(a.k);
    const float* vp = reinterpret_cast<const float*>(a.v);
    float* tile = tiles + ((size_t)(g - a.g0) * a.H + h) * T_FLOATS;

    // cumulative log-decay (identity padding past the sequence end)
    for (int idx = t; idx < kC * (kD / 4); idx += 256) {
        const int i = idx >> 5, c = (idx & 31) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < L.len) x = *reinterpret_cast<const float4*>(a.log_alpha + ((L.tok0 + i) * a.H + h) * kD + c);
        *reinterpret_cast<float4*>(sG + i * LD + c) = x;
    }
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
        float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), qv = kv, av = kv, bv = kv;
        if (i < L.len) {
            const size_t off = ((L.tok0 + i) * a.H + h) * kD + c;
            kv = *reinterpret_cast<const float4*>(kp + off);
            if (qp) qv = *reinterpret_cast<const float4*>(qp + off);
            av = *reinterpret_cast<const float4*>(p.a + off);
            bv = *reinterpret_cast<const float4*>(p.b + off);
        }
        const float4 G = *reinterpret_cast<const float4*>(sG + i * LD + c);
        float4 Gp = make_float4(0.f, 0.f, 0.f, 0.f);   // G_{i-1}
        if (i > 0) Gp = *reinterpret_cast<const float4*>(sG + (i - 1) * LD + c);
        const float4 Gl = *reinterpret_cast<const float4*>(sG + (kC - 1) * LD + c);
        const float kk[4] = {kv.x, kv.y, kv.z, kv.w}, qq[4] = {qv.x, qv.y, qv.z, qv.w};
        const float aa[4] = {av.x, av.y, av.z, av.w}, bb[4] = {bv.x, bv.y, bv.z, bv.w};
        const float gg[4] = {G.x, G.y, G.z, G.w}, gp[4] = {Gp.x, Gp.y, Gp.z, Gp.w};
        const float gl[4] = {Gl.x, Gl.y, Gl.z, Gl.w};
        if (fminf(fminf(gl[0], gl[1]), fminf(gl[2], gl[3])) < -2.f * kClamp) atomicOr(&hdr->flags, 1);
        float oq1[4], oa1[4], ok2[4], ob2[4], oQG[4], oKT[4], oBT[4], ogc[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float gr = 0.5f * gl[e];
            const float e1 = expf(clampf(gg[e] - gr));
            const float e1m = expf(clampf(gp[e] - gr));
            const float e2 = expf(clampf(gr - gg[e]));
            const float tail = expf(gl[e] - gg[e]);
            oq1[e] = a.scale * qq[e] * e1;
            oa1[e] = aa[e] * e1m;
            ok2[e] = kk[e] * e2;
            ob2[e] = bb[e] * e2;
            oQG[e] = a.scale * qq[e] * expf(gg[e]);
            oKT[e] = kk[e] * tail;
            oBT[e] = bb[e] * tail;
            ogc[e] = expf(gl[e]);
        }
        *reinterpret_cast<float4*>(sQ1 + i * LD + c) = make_float4(oq1[0], oq1[1], oq1[2], oq1[3]);
        *reinterpret_cast<float4*>(sA1 + i * LD + c) = make_float4(oa1[0], oa1[1], oa1[2], oa1[3]);
        *reinterpret_cast<float4*>(sK2 + i * LD + c) = make_float4(ok2[0], ok2[1], ok2[2], ok2[3]);
        *reinterpret_cast<float4*>(sB2 + i * LD + c) = make_float4(ob2[0], ob2[1], ob2[2], ob2[3]);
        *reinterpret_cast<float4*>(tile + T_QG + i * kD + c) = make_float4(oQG[0], oQG[1], oQG[2], oQG[3]);
        *reinterpret_cast<float4*>(tile + T_KT + i * kD + c) = make_float4(oKT[0], oKT[1], oKT[2], oKT[3]);
        *reinterpret_cast<float4*>(tile + T_BT + i * kD + c) = make_float4(oBT[0], oBT[1], oBT[2], oBT[3]);
        if (i == 0)
            *reinterpret_cast<float4*>(tile + T_GC + c) = make_float4(ogc[0], ogc[1], ogc[2], ogc[3]);
    }
    __syncthreads();

    // the four Gram matrices
    {
        const int i = t >> 2, jq = t & 3;
        for (int m = 0; m < kC / 4; ++m) {
            const int j = jq + 4 * m;
            float aqk = 0.f, aqb = 0.f, aab = 0.f, aak = 0.f;
            if (j <= i) {
                const float4* k2 = reinterpret_cast<const float4*>(sK2 + j * LD);
                const float4* b2 = reinterpret_cast<const float4*>(sB2 + j * LD);
                const float4* q1 = reinterpret_cast<const float4*>(sQ1 + i * LD);
                const float4* a1 = reinterpret_cast<const float4*>(sA1 + i * LD);
#pragma unroll 4
                for (int d = 0; d < kD / 4; ++d) {
                    const float4 kx = k2[d], bx = b2[d], qx = q1[d], ax = a1[d];
                    aqk += qx.x * kx.x + qx.y * kx.y + qx.z * kx.z + qx.w * kx.w;
                    aqb += qx.x * bx.x + qx.y * bx.y + qx.z * bx.z + qx.w * bx.w;
                    aab += ax.x * bx.x + ax.y * bx.y + ax.z * bx.z + ax.w * bx.w;
                    aak += ax.x * kx.x + ax.y * kx.y + ax.z * kx.z + ax.w * kx.w;
                }
            }
            sAab[i * LDA + j] = (j < i) ? aab : 0.f;
            sAak[i * LDA + j] = (j < i) ? aak : 0.f;
            tile[T_AQK + i * kC + j] = aqk;
            tile[T_AQB + i * kC + j] = aqb;
        }
    }
    __syncthreads();

    // a . exp(G_{i-1}) over the buffer that held the gated q (G is still in sG)
    for (int idx = t; idx < kC * (kD / 4); idx += 256) {
        const int i = idx >> 5, c = (idx & 31) * 4;
        float4 av = make_float4(0.f, 0.f, 0.f, 0.f), Gp = av;
        if (i < L.len) av = *reinterpret_cast<const float4*>(p.a + ((L.tok0 + i) * a.H + h) * kD + c);
        if (i > 0) Gp = *reinterpret_cast<const float4*>(sG + (i - 1) * LD + c);
        *reinterpret_cast<float4*>(sQ1 + i * LD + c) =
            make_float4(av.x * expf(Gp.x), av.y * expf(Gp.y), av.z * expf(Gp.z), av.w * expf(Gp.w));
    }
    __syncthreads();
    // V into the buffer that held G
    for (int idx = t; idx < kC * (kD / 4); idx += 256) {
        const int i = idx >> 5, c = (idx & 31) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < L.len) x = *reinterpret_cast<const float4*>(vp + ((L.tok0 + i) * a.H + h) * kD + c);
        *reinterpret_cast<float4*>(sG + i * LD + c) = x;
    }
    // T = (I - Aab)^-1, one column per thread by forward substitution
    if (t < kC) {
        const int j = t;
        for (int i = 0; i < kC; ++i) {
            float x = (i == j) ? 1.f : 0.f;
            for (int m = j; m < i; ++m) x += sAab[i * LDA + m] * sT[m * LDA + j];
            sT[i * LDA + j] = (i < j) ? 0.f : x;
        }
    }
    __syncthreads();

    // Y = Aak V over the buffer that held the gated k
    {
        const int i = t >> 2, cq = t & 3;
        float4 y[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) y[m] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j < i; ++j) {
            const float w = sAak[i * LDA + j];
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const float4 x = *reinterpret_cast<const float4*>(sG + j * LD + cq * 4 + 16 * m);
                y[m].x += w * x.x; y[m].y += w * x.y; y[m].z += w * x.z; y[m].w += w * x.w;
            }
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) *reinterpret_cast<float4*>(sK2 + i * LD + cq * 4 + 16 * m) = y[m];
    }
    __syncthreads();

    // w = T (a . exp(G_{i-1})),  u = T Y
    {
        const int i = t >> 2, cq = t & 3;
        float4 w[8], u[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) w[m] = u[m] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int j = 0; j <= i; ++j) {
            const float tij = sT[i * LDA + j];
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const int c = cq * 4 + 16 * m;
                const float4 x = *reinterpret_cast<const float4*>(sQ1 + j * LD + c);
                const float4 y = *reinterpret_cast<const float4*>(sK2 + j * LD + c);
                w[m].x += tij * x.x; w[m].y += tij * x.y; w[m].z += tij * x.z; w[m].w += tij * x.w;
                u[m].x += tij * y.x; u[m].y += tij * y.y; u[m].z += tij * y.z; u[m].w += tij * y.w;
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

__global__ void __launch_bounds__(256, 1)
dplr_inter_simt(DplrArgs p, const float* __restrict__ tiles, int n_begin)
{
    extern __shared__ __align__(16) float smem[];
    float* sW = smem;
    float* sQ = sW + kC * LD;
    float* sK = sQ + kC * LD;
    float* sB = sK + kC * LD;
    float* sAqk = sB + kC * LD;
    float* sAqb = sAqk + kC * LDA;
    float* sS = sAqb + kC * LDA;       // [128][NS]
    float* sX = sS + kD * NS;          // [64][NS]
    float* sU = sX + kC * NS;          // [64][NS]
    float* sV = sU + kC * NS;          // [64][NS]
    float* sgC = sV + kC * NS;         // [128]

    const ChunkArgs& a = p.c;
    const int t = threadIdx.x;
    const int slice = blockIdx.x, h = blockIdx.y, n = n_begin + blockIdx.z;
    const int col0 = slice * NS;
    float* op = reinterpret_cast<float*>(a.o);
    const float* vp = reinterpret_cast<const float*>(a.v);

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
            *reinterpret_cast<float4*>(sW + i * LD + c) = *reinterpret_cast<const float4*>(tile + T_W + i * kD + c);
            *reinterpret_cast<float4*>(sQ + i * LD + c) = *reinterpret_cast<const float4*>(tile + T_QG + i * kD + c);
            *reinterpret_cast<float4*>(sK + i * LD + c) = *reinterpret_cast<const float4*>(tile + T_KT + i * kD + c);
            *reinterpret_cast<float4*>(sB + i * LD + c) = *reinterpret_cast<const float4*>(tile + T_BT + i * kD + c);
        }
        for (int idx = t; idx < kC * kC; idx += 256) {
            sAqk[(idx >> 6) * LDA + (idx & 63)] = tile[T_AQK + idx];
            sAqb[(idx >> 6) * LDA + (idx & 63)] = tile[T_AQB + idx];
        }
        for (int idx = t; idx < kC * NS; idx += 256) {
            const int i = idx / NS, c = idx % NS;
            sU[idx] = tile[T_U + i * kD + col0 + c];
            sV[idx] = (i < len) ? vp[((tok0 + i) * a.H + h) * kD + col0 + c] : 0.f;
        }
        if (t < kD) sgC[t] = tile[T_GC + t];
        __syncthreads();

        // X = u + w S ;  the state part of the output: (q . exp(G)) S
        const int r = t >> 2, cg = (t & 3) * 4;
        float x[4], oq[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) { x[e] = sU[r * NS + cg + e]; oq[e] = 0.f; }
        for (int kk = 0; kk < kD; ++kk) {
            const float w = sW[r * LD + kk], qv = sQ[r * LD + kk];
            const float4 s = *reinterpret_cast<const float4*>(sS + kk * NS + cg);
            x[0] += w * s.x; x[1] += w * s.y; x[2] += w * s.z; x[3] += w * s.w;
            oq[0] += qv * s.x; oq[1] += qv * s.y; oq[2] += qv * s.z; oq[3] += qv * s.w;
        }
        *reinterpret_cast<float4*>(sX + r * NS + cg) = make_float4(x[0], x[1], x[2], x[3]);
        __syncthreads();

        // O = (q . exp(G)) S + Aqb X + Aqk V
        if (op) {
            for (int j = 0; j <= r; ++j) {
                const float ab = sAqb[r * LDA + j], ak = sAqk[r * LDA + j];
                const float4 xx = *reinterpret_cast<const float4*>(sX + j * NS + cg);
                const float4 vv = *reinterpret_cast<const float4*>(sV + j * NS + cg);
                oq[0] += ab * xx.x + ak * vv.x; oq[1] += ab * xx.y + ak * vv.y;
                oq[2] += ab * xx.z + ak * vv.z; oq[3] += ab * xx.w + ak * vv.w;
            }
            if (r < len)
                *reinterpret_cast<float4*>(op + ((tok0 + r) * a.H + h) * kD + col0 + cg) =
                    make_float4(oq[0], oq[1], oq[2], oq[3]);
        }

        // S <- Diag(exp(G_C)) S + (k . exp(G_C - G))^T V + (b . exp(G_C - G))^T X
        const int kk = t >> 1, c8 = (t & 1) * 8;
        float sn[8];
        {
            const float gc = sgC[kk];
#pragma unroll
            for (int e = 0; e < 8; ++e) sn[e] = gc * sS[kk * NS + c8 + e];
            for (int j = 0; j < kC; ++j) {
                const float kt = sK[j * LD + kk], bt = sB[j * LD + kk];
                const float4 v0 = *reinterpret_cast<const float4*>(sV + j * NS + c8);
                const float4 v1 = *reinterpret_cast<const float4*>(sV + j * NS + c8 + 4);
                const float4 x0 = *reinterpret_cast<const float4*>(sX + j * NS + c8);
                const float4 x1 = *reinterpret_cast<const float4*>(sX + j * NS + c8 + 4);
                sn[0] += kt * v0.x + bt * x0.x; sn[1] += kt * v0.y + bt * x0.y;
                sn[2] += kt * v0.z + bt * x0.z; sn[3] += kt * v0.w + bt * x0.w;
                sn[4] += kt * v1.x + bt * x1.x; sn[5] += kt * v1.y + bt * x1.y;
                sn[6] += kt * v1.z + bt * x1.z; sn[7] += kt * v1.w + bt * x1.w;
            }
        }
        // (the reads of sS for X finished at the barrier above; each thread owns its 8 entries)
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

struct DplrLayout {
    size_t off_table, off_state, off_tiles;
};
DplrLayout dplr_layout(int n_seqs, int H)
{
    DplrLayout L;
    L.off_table = sizeof(WsHeader);
    L.off_state = L.off_table + align_up((size_t)(n_seqs + 1) * sizeof(int32_t));
    L.off_tiles = L.off_state + align_up((size_t)n_seqs * H * kD * kD * sizeof(float));
    return L;
}
constexpr size_t kTileBytes = (size_t)T_FLOATS * sizeof(float);
constexpr size_t kWorkspaceCap = (size_t)8 << 30;
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace kda

using namespace kda;

extern "C" {

size_t kda_dplr_chunk_fwd_min_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk)
{
    if (dk != kD || dv != kD || chunk != kC || total_tokens < 0 || n_seqs < 0 || H <= 0) return 0;
    return dplr_layout(n_seqs, H).off_tiles + align_up((size_t)H * kTileBytes);
}

size_t kda_dplr_chunk_fwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk)
{
    if (dk != kD || dv != kD || chunk != kC || total_tokens < 0 || n_seqs < 0 || H <= 0) return 0;
    const size_t lo = kda_dplr_chunk_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk);
    const size_t chunks = (size_t)((total_tokens + kC - 1) / kC + n_seqs);
    size_t want = dplr_layout(n_seqs, H).off_tiles + align_up(chunks * H * kTileBytes);
    if (want > kWorkspaceCap) want = kWorkspaceCap;
    return want < lo ? lo : want;
}

kda_status_t kda_dplr_chunk_fwd(const float* q, const float* k, const float* v, const float* a,
                                const float* b, const float* g, const float* S0, float* o, float* S_T,
                                const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host,
                                int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk,
                                float scale, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (dk != kD || dv != kD || chunk != kC)
        return fail(KDA_ERR_UNSUPPORTED, "kda_dplr_chunk_fwd: only dk=dv=128, chunk=64 are supported "
                    "(got dk=%d dv=%d chunk=%d)", dk, dv, chunk);
    if (n_seqs < 0 || total_tokens < 0 || H <= 0 || H > 65535 || n_seqs > 65535)
        return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: bad sizes n_seqs=%d total_tokens=%lld H=%d",
                    n_seqs, (long long)total_tokens, H);
    if ((cu_seqlens_dev == nullptr) != (cu_seqlens_host == nullptr))
        return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: cu_seqlens_dev and cu_seqlens_host must be "
                    "given together");
    if (n_seqs == 0) {
        if (total_tokens != 0)
            return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: n_seqs=0 with total_tokens=%lld",
                        (long long)total_tokens);
        return KDA_OK;
    }
    if (total_tokens > 0 && (!k || !v || !a || !b || !g))
        return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: k, v, a, b, g must not be NULL");
    if (o && total_tokens > 0 && !q)
        return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: q is NULL but o is requested");
    const void* ptrs[] = {q, k, v, a, b, g, S0, o, S_T, cu_seqlens_dev};
    for (const void* ptr : ptrs)
        if (!aligned16(ptr)) return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: pointer %p is not "
                                         "16-byte aligned", ptr);

    std::vector<int64_t> chunk_cu((size_t)n_seqs + 1, 0);
    int64_t seq_len = 0, chunks_per_seq = 0;
    if (cu_seqlens_host) {
        if (cu_seqlens_host[0] != 0 || (int64_t)cu_seqlens_host[n_seqs] != total_tokens)
            return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: cu_seqlens must start at 0 and end at "
                        "total_tokens");
        for (int n = 0; n < n_seqs; ++n) {
            const int64_t len = (int64_t)cu_seqlens_host[n + 1] - cu_seqlens_host[n];
            if (len < 0) return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: cu_seqlens decreases at %d", n);
            chunk_cu[n + 1] = chunk_cu[n] + (len + kC - 1) / kC;
        }
    } else {
        if (total_tokens % n_seqs != 0)
            return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: total_tokens not divisible by n_seqs for "
                        "an equal-length batch");
        seq_len = total_tokens / n_seqs;
        chunks_per_seq = (seq_len + kC - 1) / kC;
        for (int n = 0; n < n_seqs; ++n) chunk_cu[n + 1] = chunk_cu[n] + chunks_per_seq;
    }
    const int64_t total_chunks = chunk_cu[n_seqs];
    if (total_chunks > 0x7fffffff) return fail(KDA_ERR_INVALID_ARG, "kda_dplr_chunk_fwd: too many chunks");

    const DplrLayout L = dplr_layout(n_seqs, H);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) ||
        workspace_bytes < L.off_tiles + (size_t)H * kTileBytes)
        return fail(KDA_ERR_WORKSPACE, "kda_dplr_chunk_fwd: workspace must be 256-byte aligned and at least "
                    "%zu bytes (got %zu)", L.off_tiles + (size_t)H * kTileBytes, workspace_bytes);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    int64_t cap = (int64_t)((workspace_bytes - L.off_tiles) / ((size_t)H * kTileBytes));
    if (cap > 0x7fffffff) cap = 0x7fffffff;
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws);
    int32_t* chunk_cu_dev = reinterpret_cast<int32_t*>(ws + L.off_table);
    kda_status_t rc = launch_prep(hdr, cu_seqlens_dev, chunk_cu_dev, n_seqs, st);
    if (rc != KDA_OK) return rc;
    if (!o && !S_T) return KDA_OK;
    {
        DeviceLock lk;
        if (!lk.st) return lk.rc;
        if (!lk.st->attr_done[7]) {
            KDA_CUDA_TRY(cudaFuncSetAttribute(dplr_intra_simt, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kIntraSmem));
            KDA_CUDA_TRY(cudaFuncSetAttribute(dplr_inter_simt, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)kInterSmem));
            lk.st->attr_done[7] = true;
        }
    }

    float* state = S_T ? S_T : reinterpret_cast<float*>(ws + L.off_state);
    DplrArgs p;
    p.a = a; p.b = b;
    p.c.q = q; p.c.k = k; p.c.v = v; p.c.log_alpha = g; p.c.beta = nullptr;
    p.c.o = o; p.c.cu_seqlens = cu_seqlens_dev; p.c.chunk_cu = cu_seqlens_dev ? chunk_cu_dev : nullptr;
    p.c.n_seqs = n_seqs; p.c.H = H; p.c.total_tokens = total_tokens; p.c.seq_len = seq_len;
    p.c.chunks_per_seq = chunks_per_seq; p.c.scale = scale;
    p.c.S_out = state;
    float* tiles = reinterpret_cast<float*>(ws + L.off_tiles);

    int64_t g0 = 0;
    bool first = true;
    do {
        const int64_t g1 = (total_chunks - g0 > cap) ? g0 + cap : total_chunks;
        p.c.g0 = g0; p.c.g1 = g1;
        p.c.S_in = first ? S0 : state;
        int n_begin = 0, n_count = n_seqs;
        if (!first) {   // only the sequences that own a chunk of this pass
            while (n_begin < n_seqs && chunk_cu[n_begin + 1] <= g0) ++n_begin;
            int n_end = n_begin;
            while (n_end < n_seqs && chunk_cu[n_end] < g1) ++n_end;
            n_count = n_end - n_begin;
        }
        if (g1 > g0) {
            dim3 grid((unsigned)(g1 - g0), (unsigned)H);
            ProfScope ps(PROF_INTRA, st);
            dplr_intra_simt<<<grid, 256, kIntraSmem, st>>>(p, tiles, hdr);
            count_launch();
            KDA_CUDA_TRY(cudaGetLastError());
        }
        if (n_count > 0) {
            dim3 grid(kD / NS, (unsigned)H, (unsigned)n_count);
            ProfScope ps(PROF_INTER, st);
            dplr_inter_simt<<<grid, 256, kInterSmem, st>>>(p, tiles, n_begin);
            count_launch();
            KDA_CUDA_TRY(cudaGetLastError());
        }
        g0 = g1;
        first = false;
    } while (g0 < total_chunks);
    return KDA_OK;
}

}  // extern "C"
