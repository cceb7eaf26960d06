// Internal helpers shared by the translation units of the KDA library (host side error plumbing,
// launch accounting, workspace header layout, small device utilities).  Not part of the C ABI.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kda.h"

namespace kda {

constexpr int kD = 128;      // dk = dv (head size fixed by the paper's models)
constexpr int kC = 64;       // chunk length (Section 3.1 uses C = 64)

// ---- host-side plumbing (defined in kda_api.cu) -------------------------------------------------
kda_status_t fail(kda_status_t code, const char* fmt, ...);
void count_launch(int n = 1);
#define KDA_CUDA_TRY(expr)                                                                   \
    do {                                                                                     \
        cudaError_t e__ = (expr);                                                            \
        if (e__ != cudaSuccess)                                                              \
            return ::kda::fail(KDA_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

// Optional per-kernel timing (kda_profile_*): when enabled, every launch site is bracketed by a pair
// of CUDA events on the launching stream.  A no-op when disabled.
enum ProfKind { PROF_PREP = 0, PROF_INTRA = 1, PROF_INTER = 2, PROF_DECODE = 3, PROF_FUSED = 4, PROF_KINDS = 8 };
struct ProfScope {
    ProfScope(int kind, cudaStream_t st);
    ~ProfScope();
    int slot;
    cudaStream_t st;
};

// ---- workspace header ---------------------------------------------------------------------------
// The first 256 bytes of the caller's workspace hold a status word (set by device code whose
// bounded wait ran out); the chunk table follows.
struct WsHeader {
    int status;       // 0 = ok, otherwise a kda_status_t
    int where;        // implementation-defined location code of the first failure
    unsigned int abort_epoch;   // call id of a fused-kernel call that gave up (its waiters return at once)
    int flags;        // bit 0: a decay factor left the supported range in some chunk (see kda.h)
    int pad[60];
};
static_assert(sizeof(WsHeader) == 256, "header is one 256-byte block");

// Work description of one chunk-forward pass, passed by value to the kernels.
struct ChunkArgs {
    const void* q;
    const void* k;
    const void* v;
    const float* log_alpha;
    const float* beta;
    const float* S_in;        // state entering this pass ([n_seqs,H,dk,dv]) or nullptr = zeros
    float* S_out;             // state leaving this pass (may equal S_in), never nullptr
    void* o;                  // or nullptr
    const int32_t* cu_seqlens;  // device, or nullptr = equal lengths
    const int32_t* chunk_cu;    // device [n_seqs+1]: first global chunk index of each sequence
    int n_seqs;
    int H;
    int64_t total_tokens;
    int64_t seq_len;          // equal-length case
    int64_t chunks_per_seq;   // equal-length case
    int64_t g0, g1;           // global chunk range of this pass
    float scale;
    // Layer mode (kda_layer_fwd, bf16 tensor-core path only), off when gate_rate is nullptr: q and k
    // arrive un-normalised, `log_alpha` points to the bf16 pre-activations of the decay function and
    // `beta` to the fp32 pre-activations of beta; the intra-chunk kernel applies L2Norm, the decay
    // function -exp(gate_rate[h]) * softplus(x + gate_bias[h, d]) and the sigmoid itself.
    const float* gate_rate = nullptr;   // [H]
    const float* gate_bias = nullptr;   // [H, dk]
    float l2_eps = 0.f;
    // Output stage of the layer wrap inside the inter-chunk kernel (off when out_gate is nullptr):
    // o is replaced by sigmoid(out_gate) . RMSNorm(o) . rms_weight before it is stored.
    // Upper bound of every device-side wait of the tensor-core kernels (ns); set from the environment
    // variable KDA_WAIT_LIMIT_MS by the host entry points (default 1 s).
    unsigned long long wait_limit_ns = 1000000000ull;
    const void* out_gate = nullptr;     // bf16 [T_total, H, dv]
    const float* rms_weight = nullptr;  // [dv]
    float rms_eps = 0.f;
};

// Work description of the fused bf16 chunk-forward kernel (one cooperative launch per call).
//
// Jobs are (sequence, head) pairs in natural order j = n * H + h.  Q of them run at a time ("round"
// r covers jobs [r Q, (r + 1) Q)); slot q of a round is served by the chain CTAs 2 q and 2 q + 1
// (one 64-column slice of the state each); the other CTAs run two intra-chunk engines each.  The intra-chunk engines of all CTAs
// produce the tiles of a round chunk by chunk (production index = base_r + c * Q_r + q) into a ring
// of R tiles per slot; `ready` holds (epoch << 32 | production index + 1) per ring position and
// `consumed` (epoch << 32 | number of production indices the slice has finished with) per chain
// role, so nothing has to be cleared between calls.
struct FusedArgs {
    ChunkArgs a;                     // g0, g1 unused
    char* ring;                      // [Q][R] tiles
    unsigned long long* ready;       // [Q * R]
    unsigned long long* consumed;    // [Q * fused_slices()]
    const uint32_t* round_base;      // packed batches: [n_rounds + 1] production index base per round; else nullptr
    WsHeader* hdr;
    int Q, R, J, n_rounds;
    uint32_t n_prod;                 // production indices in total (equal lengths; packed: round_base[n_rounds])
    uint32_t epoch;                  // call id, never 0
    int n_chain_cta;                 // chain CTAs: fused_slices() per slot
};

// ---- dtype helpers ------------------------------------------------------------------------------
template <typename T> struct IO;
template <> struct IO<float> {
    __device__ static __forceinline__ float4 load4(const float* p) {
        return *reinterpret_cast<const float4*>(p);
    }
    __device__ static __forceinline__ void store4(float* p, float4 x) {
        *reinterpret_cast<float4*>(p) = x;
    }
};
template <> struct IO<__nv_bfloat16> {
    __device__ static __forceinline__ float4 load4(const __nv_bfloat16* p) {
        uint2 r = *reinterpret_cast<const uint2*>(p);
        __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&r.x);
        __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&r.y);
        float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
        return make_float4(fa.x, fa.y, fb.x, fb.y);
    }
    __device__ static __forceinline__ void store4(__nv_bfloat16* p, float4 x) {
        __nv_bfloat162 a = __floats2bfloat162_rn(x.x, x.y), b = __floats2bfloat162_rn(x.z, x.w);
        uint2 r;
        r.x = *reinterpret_cast<uint32_t*>(&a);
        r.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(p) = r;
    }
};

// Locate global chunk g: sequence index, first token, number of valid tokens (1..64).
struct ChunkLoc {
    int n;
    int64_t tok0;
    int len;
    int64_t c;   // chunk index inside the sequence
};
__device__ __forceinline__ ChunkLoc locate_chunk(const ChunkArgs& a, int64_t g) {
    ChunkLoc L;
    if (a.cu_seqlens == nullptr) {
        L.n = (int)(g / a.chunks_per_seq);
        L.c = g - (int64_t)L.n * a.chunks_per_seq;
        int64_t t = L.c * kC;
        L.tok0 = (int64_t)L.n * a.seq_len + t;
        int64_t rem = a.seq_len - t;
        L.len = rem < kC ? (int)rem : kC;
    } else {
        int lo = 0, hi = a.n_seqs - 1;   // last n with chunk_cu[n] <= g
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if ((int64_t)a.chunk_cu[mid] <= g) lo = mid; else hi = mid - 1;
        }
        L.n = lo;
        L.c = g - a.chunk_cu[lo];
        int64_t b = a.cu_seqlens[lo], e = a.cu_seqlens[lo + 1];
        L.tok0 = b + L.c * kC;
        int64_t rem = e - L.tok0;
        L.len = rem < kC ? (int)rem : kC;
    }
    return L;
}

// ---- launchers implemented by the kernel translation units --------------------------------------
kda_status_t launch_decode(const void* q, const void* k, const void* v, const float* log_alpha,
                           const float* beta, float* S, const int32_t* slot, void* o, int n_seqs,
                           int H, float scale, kda_dtype_t dt, cudaStream_t st);

kda_status_t launch_layer_decode(const void* q_c, const void* k_c, const void* v, const void* g_a,
                                 const float* b_pre, const void* g_o, const float* A_log, const float* dt_bias,
                                 const float* rms_weight, float l2_eps, float rms_eps, float* S,
                                 const int32_t* slot, void* y, int n_seqs, int H, float scale, cudaStream_t st);

kda_status_t launch_decode_multi(const void* q, const void* k, const void* v, const float* log_alpha,
                                 const float* beta, float* S, const int32_t* slot, void* o, int n_seqs,
                                 int n_tok, int H, float scale, kda_dtype_t dt, cudaStream_t st);

// fp32 FMA path (also accepts bf16 storage): per-tile scratch size and pass launcher
size_t simt_tile_bytes();
kda_status_t launch_chunk_simt(const ChunkArgs& a, kda_dtype_t dt, void* tiles, int n_begin,
                               int n_count, WsHeader* hdr, cudaStream_t st);

// bf16 tensor-core path (tcgen05 + bulk copies): per-tile scratch size and pass launcher
size_t tc_tile_bytes();
kda_status_t launch_chunk_tc(const ChunkArgs& a, void* tiles, int n_begin, int n_count,
                             WsHeader* hdr, bool clear_status, cudaStream_t st);
bool inter_can_fuse_epilogue(int64_t groups);
unsigned long long wait_limit_ns();   // KDA_WAIT_LIMIT_MS (1 .. 600000) in ns, default 1 s
kda_status_t make_plain_tmap(CUtensorMap* tm, const void* base, int64_t total_tokens, int H, int cols, int rows);

// fused bf16 path: workspace bytes besides the ring (flags and round table), and the launcher
size_t fused_fixed_bytes(int n_seqs, int H);
int fused_max_slots(int n_sm);
int fused_slices();
kda_status_t launch_fused_tc(FusedArgs f, bool has_q, bool clear_status, cudaStream_t st);
kda_status_t launch_fused_prep(WsHeader* hdr, const int32_t* cu_seqlens, uint32_t* round_base, int n_seqs,
                               int H, int Q, int n_rounds, cudaStream_t st);

// ---- per-device library state ---------------------------------------------------------------------
// Everything the library caches about a device (SM count, which kernels already carry their
// dynamic-shared-memory attribute, helper streams) lives in one slot per device ordinal, created
// on first use under a mutex.
constexpr int kMaxDevices = 64;
constexpr int kAttrSlots = 16;
struct DeviceState {
    int n_sm = 0;
    bool attr_done[kAttrSlots] = {};
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    int max_clusters = -1;   // resident 4-CTA clusters of the inter-chunk kernel with the output stage (-1: not asked yet)
};
// Locks the table and returns the slot of the calling thread's current device (nullptr + error set
// on failure); the lock is released by ~DeviceLock.
struct DeviceLock {
    DeviceLock();
    ~DeviceLock();
    DeviceState* st;      // nullptr if the device could not be identified
    kda_status_t rc;
};
// The slot table itself, without any CUDA call (unit-testable on a machine without a GPU).
DeviceState* device_slot(int ordinal);

// output stage of the layer wrap: y = sigmoid(g_o) . RMSNorm(y) . w in place, rows of kD bf16 values
kda_status_t launch_layer_epilogue(void* y, const void* g_o, const float* w, float eps, int64_t n_rows,
                                   cudaStream_t st);

kda_status_t launch_wait_selftest(WsHeader* hdr, uint64_t limit_ns, cudaStream_t st);

// clears the status word and (packed batches) builds chunk_cu[n_seqs+1] from cu_seqlens
kda_status_t launch_prep(WsHeader* hdr, const int32_t* cu_seqlens, int32_t* chunk_cu, int n_seqs,
                         cudaStream_t st);

}  // namespace kda
