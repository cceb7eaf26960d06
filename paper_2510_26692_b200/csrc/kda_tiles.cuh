// Layout of the per-(chunk, head) scratch tile that the intra-chunk stage hands to the inter-chunk
// stage on the bf16 tensor-core path.  Every matrix operand is stored as the exact shared-memory
// image the tcgen05 MMA expects (K-major, 128-byte swizzle, see ptx::sw128_off), so the consumer
// brings it in with plain 1-D bulk copies.
#pragma once
#include <stdint.h>

namespace kda {
namespace tc {
// A operand of  [ W ; (Gamma.Q) ] S : two K-halves of [128 rows][64], rows 0-63 = W,
// rows 64-127 = scale*Gamma.Q
constexpr uint32_t OFF_QW = 0;
constexpr uint32_t QW_HALF = 128 * 128;
// A operand of the state update: ((gamma^C/Gamma).K)^T as [128 dk][64 tokens]
constexpr uint32_t OFF_KT = 32768;
// A operand of the intra-chunk output term: Aqk [64][64] (lower triangular incl. diagonal)
constexpr uint32_t OFF_AQ = 49152;
// gamma^C: 128 fp32 (directly after the three operand images: one bulk copy fetches all four)
constexpr uint32_t OFF_GC = 57344;
// U in four column blocks of [64 tokens][32 columns] bf16 (64-byte rows).  It is read with plain
// loads; the 16-byte chunks of a row are XOR-swizzled with (row >> 1) & 3 only to keep the
// producer's row-per-thread stores free of shared-memory bank conflicts (see u_off).
constexpr uint32_t OFF_U = 57856;
constexpr uint32_t U_BLOCK = 64 * 64;
__host__ __device__ __forceinline__ constexpr uint32_t u_off(uint32_t row, uint32_t chunk) {
    return row * 64u + ((chunk ^ ((row >> 1) & 3u)) << 4);
}
constexpr uint32_t TILE_BYTES = 74240;
static_assert(TILE_BYTES % 256 == 0, "tiles stay 256-byte aligned");
}  // namespace tc
}  // namespace kda
