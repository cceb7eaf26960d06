// Layout of the per-(chunk, head) scratch tile that the intra-chunk stage hands to the inter-chunk
// stage on the bf16 tensor-core path.  Every matrix operand is stored as the exact shared-memory
// image the tcgen05 MMA expects (K-major, 128-byte swizzle, see ptx::sw128_off), so the consumer
// brings it in with plain 1-D bulk copies.
#pragma once
#include <stdint.h>

namespace kda {
namespace tc {
// All gated quantities in a tile are relative to the chunk's middle row m (the reference of the
// decay factorisation): W' = W / exp(G_m) and Q' = scale Q exp(G - G_m) column-wise, K' = K exp(G_m - G).
// The consumer restores the true scale in fp32: it feeds the products with exp(G_m) . S and scales
// the state increment by exp(G_C - G_m), so nothing here can underflow before it is used.
//
// A operand of  [ W' ; Q' ] (exp(G_m) . S): two K-halves of [128 rows][64], rows 0-63 = W', rows 64-127 = Q'
constexpr uint32_t OFF_QW = 0;
constexpr uint32_t QW_HALF = 128 * 128;
// K' as two dk-halves of [64 tokens][64 channels]: the MN-major A operand of the state product K'^T V_new
constexpr uint32_t OFF_KI = 32768;
constexpr uint32_t KI_HALF = 64 * 128;
// A operand of the intra-chunk output term: Aqk [64][64] (lower triangular incl. diagonal)
constexpr uint32_t OFF_AQ = 49152;
// three fp32 vectors of 128 (directly after the operand images: one bulk copy fetches everything):
// gamma^C = exp(G_C), exp(G_m), exp(G_C - G_m)
constexpr uint32_t OFF_GV = 57344;
constexpr uint32_t GV_BYTES = 3 * 512;
// U in four column blocks of [64 tokens][32 columns] bf16 (64-byte rows).  It is read with plain
// loads; the 16-byte chunks of a row are XOR-swizzled with (row >> 1) & 3 only to keep the
// producer's row-per-thread stores free of shared-memory bank conflicts (see u_off).
constexpr uint32_t OFF_U = OFF_GV + GV_BYTES;
constexpr uint32_t U_BLOCK = 64 * 64;
__host__ __device__ __forceinline__ constexpr uint32_t u_off(uint32_t row, uint32_t chunk) {
    return row * 64u + ((chunk ^ ((row >> 1) & 3u)) << 4);
}
constexpr uint32_t TILE_BYTES = OFF_U + 4 * U_BLOCK;
static_assert(TILE_BYTES % 256 == 0, "tiles stay 256-byte aligned");
}  // namespace tc
}  // namespace kda
