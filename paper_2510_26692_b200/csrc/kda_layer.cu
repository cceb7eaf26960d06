// Output stage of the KDA layer (paper Section 4, "Neural Parameterization", last equation): the
// head-wise RMSNorm over the dv values of one (token, head) row, its learned weight, and the
// data-dependent sigmoid gate,   y = sigmoid(g_o) . RMSNorm(o) . w ,   applied in place to the bf16
// output of the chunk kernels.  Rows are spread over a grid sized to the device; HBM-bound: 256 B
// read + 256 B gate + 256 B written per row.
#include "kda_common.cuh"

namespace kda {
namespace {

__device__ __forceinline__ void unpack8(uint4 r, float (&x)[8]) {
    x[0] = __uint_as_float(r.x << 16); x[1] = __uint_as_float(r.x & 0xffff0000u);
    x[2] = __uint_as_float(r.y << 16); x[3] = __uint_as_float(r.y & 0xffff0000u);
    x[4] = __uint_as_float(r.z << 16); x[5] = __uint_as_float(r.z & 0xffff0000u);
    x[6] = __uint_as_float(r.w << 16); x[7] = __uint_as_float(r.w & 0xffff0000u);
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&p);
}

// Half a warp per row (eight values = one 16-byte access per lane); every warp iteration covers
// kRows consecutive pairs of rows, all of whose loads are issued before the first is used.
constexpr int kRows = 4;

__global__ void __launch_bounds__(256) kda_layer_epilogue_kernel(__nv_bfloat16* __restrict__ y,
                                                                 const __nv_bfloat16* __restrict__ g_o,
                                                                 const float* __restrict__ w, float eps,
                                                                 int64_t n_rows)
{
    const int lane = threadIdx.x & 31, sub = lane & 15, half = lane >> 4;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const float4 wa = *reinterpret_cast<const float4*>(w + sub * 8);
    const float4 wb = *reinterpret_cast<const float4*>(w + sub * 8 + 4);
    const float ww[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
    const int64_t n_groups = (n_rows + 2 * kRows - 1) / (2 * kRows);
    for (int64_t grp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); grp < n_groups; grp += warps) {
        uint4 ro[kRows], rg[kRows];
#pragma unroll
        for (int u = 0; u < kRows; ++u) {
            const int64_t row = (grp * kRows + u) * 2 + half;
            ro[u] = rg[u] = make_uint4(0u, 0u, 0u, 0u);
            if (row < n_rows) {
                ro[u] = *reinterpret_cast<const uint4*>(y + row * kD + sub * 8);
                rg[u] = *reinterpret_cast<const uint4*>(g_o + row * kD + sub * 8);
            }
        }
#pragma unroll
        for (int u = 0; u < kRows; ++u) {
            const int64_t row = (grp * kRows + u) * 2 + half;
            float o[8], g[8];
            unpack8(ro[u], o);
            unpack8(rg[u], g);
            float ss = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(o[e], o[e], ss);
#pragma unroll
            for (int s = 8; s >= 1; s >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, s);
            const float rstd = rsqrtf(ss * (1.f / kD) + eps);
            float r[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) r[e] = o[e] * rstd * ww[e] / (1.f + __expf(-g[e]));
            if (row < n_rows)
                *reinterpret_cast<uint4*>(y + row * kD + sub * 8) =
                    make_uint4(pack2(r[0], r[1]), pack2(r[2], r[3]), pack2(r[4], r[5]), pack2(r[6], r[7]));
        }
    }
}

}  // namespace

kda_status_t launch_layer_epilogue(void* y, const void* g_o, const float* w, float eps, int64_t n_rows,
                                   cudaStream_t st)
{
    if (n_rows <= 0) return KDA_OK;
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
    int64_t blocks = (n_rows + 8 * 2 * kRows - 1) / (8 * 2 * kRows);   // 8 warps per block, 2 kRows rows per warp step
    if (blocks > (int64_t)n_sm * 64) blocks = (int64_t)n_sm * 64;
    ProfScope ps(PROF_DECODE, st);
    kda_layer_epilogue_kernel<<<(unsigned)blocks, 256, 0, st>>>(static_cast<__nv_bfloat16*>(y),
                                                                 static_cast<const __nv_bfloat16*>(g_o), w, eps,
                                                                 n_rows);
    count_launch();
    KDA_CUDA_TRY(cudaGetLastError());
    return KDA_OK;
}

}  // namespace kda
