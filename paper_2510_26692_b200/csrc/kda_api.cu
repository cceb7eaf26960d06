// C ABI of the KDA library: argument validation, workspace carving, pass scheduling.  Every step
// of the computation runs in the kernels of the other translation units; this file only decides
// what to launch.
#include <atomic>
#include <chrono>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <random>
#include <vector>

#include "kda_common.cuh"

namespace kda {

static thread_local char g_err[512] = "";
static std::atomic<uint64_t> g_launches{0};

kda_status_t fail(kda_status_t code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

unsigned long long wait_limit_ns()
{
    static const unsigned long long v = [] {
        const char* e = std::getenv("KDA_WAIT_LIMIT_MS");
        long ms = e ? std::strtol(e, nullptr, 10) : 0;
        if (ms < 1 || ms > 600000) ms = 1000;
        return (unsigned long long)ms * 1000000ull;
    }();
    return v;
}

// ---- per-device state -------------------------------------------------------------------------------
namespace {
std::mutex g_dev_mu;
DeviceState g_dev[kMaxDevices];
}  // namespace
DeviceState* device_slot(int ordinal)
{
    return (ordinal >= 0 && ordinal < kMaxDevices) ? &g_dev[ordinal] : nullptr;
}
DeviceLock::DeviceLock() : st(nullptr), rc(KDA_OK)
{
    g_dev_mu.lock();
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) {
        rc = fail(KDA_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
        return;
    }
    st = device_slot(dev);
    if (!st) rc = fail(KDA_ERR_UNSUPPORTED, "device ordinal %d is outside the supported range 0..%d", dev,
                       kMaxDevices - 1);
}
DeviceLock::~DeviceLock() { g_dev_mu.unlock(); }

// ---- per-kernel event timing ------------------------------------------------------------------------
namespace {
constexpr int kProfMax = 8192;
struct ProfState {
    std::mutex mu;
    bool on = false;
    int used = 0;
    std::vector<cudaEvent_t> ev0, ev1;
    std::vector<int> kind;
} g_prof;
}  // namespace

ProfScope::ProfScope(int kind, cudaStream_t s) : slot(-1), st(s)
{
    if (!g_prof.on) return;
    std::lock_guard<std::mutex> lk(g_prof.mu);
    if (g_prof.used >= kProfMax) return;
    if ((int)g_prof.ev0.size() <= g_prof.used) {
        cudaEvent_t a, b;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
        g_prof.ev0.push_back(a);
        g_prof.ev1.push_back(b);
        g_prof.kind.push_back(0);
    }
    slot = g_prof.used++;
    g_prof.kind[slot] = kind;
    cudaEventRecord(g_prof.ev0[slot], st);
}
ProfScope::~ProfScope()
{
    if (slot >= 0) cudaEventRecord(g_prof.ev1[slot], st);
}

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kWorkspaceCap = (size_t)8 << 30;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t esize(kda_dtype_t dt) { return dt == KDA_BF16 ? 2 : 4; }

bool shape_ok(int dk, int dv, int chunk, kda_dtype_t dt)
{
    return dk == kD && dv == kD && chunk == kC && (dt == KDA_F32 || dt == KDA_BF16);
}

size_t tile_bytes(kda_dtype_t dt)
{
    return dt == KDA_BF16 ? tc_tile_bytes() : simt_tile_bytes();
}

struct WsLayout {
    size_t off_table, off_state, off_tiles, fixed;
};
WsLayout ws_layout(int n_seqs, int H)
{
    WsLayout L;
    L.off_table = sizeof(WsHeader);
    L.off_state = L.off_table + align_up((size_t)(n_seqs + 1) * sizeof(int32_t));
    L.off_tiles = L.off_state + align_up((size_t)n_seqs * H * kD * kD * sizeof(float));
    L.fixed = L.off_tiles;
    return L;
}
int64_t max_chunks(int64_t total_tokens, int n_seqs)
{
    return (total_tokens + kC - 1) / kC + n_seqs;
}

// ---- fused bf16 path: workspace = header | flag words | round table | ring of tiles ---------------------
constexpr int kSlotCap = 64;      // upper bound of concurrently running (sequence, head) chains
constexpr int kRingMax = 16;      // tiles per chain the engines may run ahead
constexpr size_t kFlagBytes = (size_t)kSlotCap * kRingMax * 8 + (size_t)kSlotCap * 4 * 8;
struct FusedLayout {
    size_t off_ready, off_consumed, off_table, off_ring;
};
FusedLayout fused_layout(int64_t J)
{
    FusedLayout L;
    L.off_ready = sizeof(WsHeader);
    L.off_consumed = L.off_ready + (size_t)kSlotCap * kRingMax * 8;
    L.off_table = L.off_ready + kFlagBytes;
    L.off_ring = L.off_table + align_up((size_t)(J + 1) * sizeof(uint32_t));
    return L;
}
// Call counter that tags the flag words of the fused kernel.  It starts at a value drawn per process:
// device memory handed from one process to the next may still hold the flag words of the earlier
// one, and a counter that restarted at 1 could meet its own tags there.
uint32_t epoch_seed()
{
    std::random_device rd;
    const uint64_t t = (uint64_t)std::chrono::steady_clock::now().time_since_epoch().count();
    return (uint32_t)rd() ^ (uint32_t)(t * 0x9E3779B97F4A7C15ull >> 32);
}
std::atomic<uint32_t> g_epoch{epoch_seed()};

// Schedule of the fused kernel: Q chains run side by side (one round), each with a ring of R tiles;
// n_prod counts the production indices, a round taking (longest chain) x (chains of the round).
struct FusedPlan {
    int64_t Q, R, n_rounds;
    uint64_t n_prod;
};
FusedPlan fused_plan(const std::vector<int64_t>& chunk_cu, int n_seqs, int H, int64_t avail_tiles, int n_sm)
{
    FusedPlan P{0, 0, 0, 0};
    const int64_t J = (int64_t)n_seqs * H;
    int Qmax = fused_max_slots(n_sm);
    if (Qmax > kSlotCap) Qmax = kSlotCap;
    if (Qmax < 1 || avail_tiles < 2 || J < 1) return P;
    // whole sequences per round when the heads of one fit, so that the chains of a round have
    // equal lengths
    int64_t Q = (H <= Qmax) ? (int64_t)H * (Qmax / H) : Qmax;
    if (Q > J) Q = J;
    if (Q * 2 > avail_tiles) Q = avail_tiles / 2;
    int64_t R = avail_tiles / Q;
    if (R > kRingMax) R = kRingMax;
    P.Q = Q; P.R = R; P.n_rounds = (J + Q - 1) / Q;
    for (int64_t r = 0; r < P.n_rounds; ++r) {
        const int64_t j0 = r * Q, j1 = (j0 + Q < J ? j0 + Q : J) - 1;
        int64_t maxlen = 0;
        for (int64_t n = j0 / H; n <= j1 / H; ++n) {
            const int64_t len = chunk_cu[n + 1] - chunk_cu[n];
            maxlen = len > maxlen ? len : maxlen;
        }
        P.n_prod += (uint64_t)maxlen * (uint64_t)(j1 - j0 + 1);
    }
    return P;
}
std::atomic<int> g_chunk_path{0};
std::atomic<int> g_fuse_output{1};  // kda_layer_fwd: 1 = output stage inside the inter-chunk kernel when possible   // 0 = automatic, 1 = always two kernels, 2 = always the fused kernel

}  // namespace
}  // namespace kda

using namespace kda;

extern "C" {

const char* kda_last_error(void) { return g_err; }
uint64_t kda_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
const char* kda_version(void) { return "kda-b200 sm_100a"; }

int kda_selftest_device_table(void)
{
    // the slot table alone (no CUDA call): distinct slots for distinct ordinals, stable addresses,
    // nothing for ordinals outside the table, and mutual exclusion of the lock
    DeviceState* s0 = device_slot(0);
    DeviceState* s1 = device_slot(1);
    if (!s0 || !s1 || s0 == s1 || device_slot(0) != s0) return 1;
    if (device_slot(-1) || device_slot(kMaxDevices)) return 2;
    DeviceState* last = device_slot(kMaxDevices - 1);
    if (!last || last == s0) return 3;
    const bool a0 = s0->attr_done[5];
    s1->attr_done[5] = !a0;
    if (s0->attr_done[5] != a0) return 4;   // a write to one device's slot leaves the others alone
    s1->attr_done[5] = false;
    if (!g_dev_mu.try_lock()) return 5;     // (not held by this thread)
    g_dev_mu.unlock();
    return 0;
}

int kda_selftest_fused_plan(const int32_t* chunks_per_seq, int n_seqs, int H, int64_t avail_tiles,
                            int n_sm, int64_t out[4])
{
    if (!chunks_per_seq || !out || n_seqs < 1 || H < 1) return 1;
    std::vector<int64_t> chunk_cu((size_t)n_seqs + 1, 0);
    for (int n = 0; n < n_seqs; ++n) chunk_cu[n + 1] = chunk_cu[n] + chunks_per_seq[n];
    const FusedPlan P = fused_plan(chunk_cu, n_seqs, H, avail_tiles, n_sm);
    out[0] = P.Q; out[1] = P.R; out[2] = P.n_rounds; out[3] = (int64_t)P.n_prod;
    return 0;
}

uint64_t kda_wait_limit_ns(void) { return wait_limit_ns(); }

kda_status_t kda_set_chunk_path(int mode)
{
    if (mode < 0 || mode > 2) return fail(KDA_ERR_INVALID_ARG, "kda_set_chunk_path: mode must be 0, 1 or 2");
    g_chunk_path.store(mode, std::memory_order_relaxed);
    return KDA_OK;
}

size_t kda_chunk_fwd_min_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                         int chunk, kda_dtype_t dt)
{
    if (!shape_ok(dk, dv, chunk, dt) || total_tokens < 0 || n_seqs < 0 || H <= 0) return 0;
    // fp32: state scratch + one tile per head (the call then walks the chunks one at a time).
    // bf16: what the fused kernel needs -- header, flag words, round table and a ring of two tiles.
    if (dt != KDA_BF16) return ws_layout(n_seqs, H).fixed + align_up((size_t)H * tile_bytes(dt));
    return fused_layout((int64_t)n_seqs * H).off_ring + 2 * tc_tile_bytes();
}

size_t kda_chunk_fwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                     int chunk, kda_dtype_t dt)
{
    if (!shape_ok(dk, dv, chunk, dt) || total_tokens < 0 || n_seqs < 0 || H <= 0) return 0;
    const size_t lo = kda_chunk_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, dt);
    const size_t fixed = ws_layout(n_seqs, H).fixed;
    size_t want = fixed + align_up((size_t)max_chunks(total_tokens, n_seqs) * H * tile_bytes(dt));
    if (want > kWorkspaceCap) want = kWorkspaceCap;
    if (dt == KDA_BF16) {
        // never below a full ring for the fused kernel (the path of a capped workspace)
        const int64_t J = (int64_t)n_seqs * H;
        const size_t ring = fused_layout(J).off_ring + (size_t)(J < kSlotCap ? J : kSlotCap) * kRingMax * tc_tile_bytes();
        if (want < ring) want = ring;
    }
    return want < lo ? lo : want;
}

}  // extern "C"

namespace kda {
namespace {
// decay-function parameters of a layer-mode call (kda_layer_fwd); rate == nullptr = plain call
struct LayerMode {
    const float* rate = nullptr;
    const float* bias = nullptr;
    float l2_eps = 0.f;
    const void* out_gate = nullptr;     // non-null: the output stage runs inside the inter-chunk kernel
    const float* rms_weight = nullptr;
    float rms_eps = 0.f;
};

kda_status_t chunk_fwd_impl(const void* q, const void* k, const void* v, const float* log_alpha,
                            const float* beta, const float* S0, void* o, float* S_T,
                            const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host,
                            int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk,
                            float scale, kda_dtype_t dt, void* workspace, size_t workspace_bytes,
                            void* cuda_stream, const LayerMode& lm)
{
    if (!shape_ok(dk, dv, chunk, dt))
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: only dk=dv=128, chunk=64, dt in {f32,bf16} "
                    "are supported (got dk=%d dv=%d chunk=%d dt=%d)", dk, dv, chunk, (int)dt);
    if (n_seqs < 0 || total_tokens < 0 || H <= 0 || H > 65535)
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: bad sizes n_seqs=%d total_tokens=%lld H=%d",
                    n_seqs, (long long)total_tokens, H);
    if ((cu_seqlens_dev == nullptr) != (cu_seqlens_host == nullptr))
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: cu_seqlens_dev and cu_seqlens_host must be "
                    "given together");
    if (n_seqs == 0) {
        if (total_tokens != 0)
            return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: n_seqs=0 with total_tokens=%lld",
                        (long long)total_tokens);
        return KDA_OK;
    }
    if (total_tokens > 0 && (!k || !v || !log_alpha || !beta))
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: k, v, log_alpha, beta must not be NULL");
    if (o && total_tokens > 0 && !q)
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: q is NULL but o is requested");
    const void* ptrs[] = {q, k, v, log_alpha, beta, S0, o, S_T, cu_seqlens_dev};
    for (const void* p : ptrs)
        if (!aligned16(p)) return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: pointer %p is not "
                                       "16-byte aligned", p);
    if (total_tokens * (int64_t)H > ((int64_t)1 << 40))
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: total_tokens*H too large");

    // chunk table on the host (validation + scheduling)
    std::vector<int64_t> chunk_cu((size_t)n_seqs + 1, 0);
    int64_t seq_len = 0, chunks_per_seq = 0;
    if (cu_seqlens_host) {
        if (cu_seqlens_host[0] != 0 || (int64_t)cu_seqlens_host[n_seqs] != total_tokens)
            return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: cu_seqlens must start at 0 and end at "
                        "total_tokens");
        for (int n = 0; n < n_seqs; ++n) {
            const int64_t len = (int64_t)cu_seqlens_host[n + 1] - cu_seqlens_host[n];
            if (len < 0) return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: cu_seqlens decreases at %d", n);
            chunk_cu[n + 1] = chunk_cu[n] + (len + kC - 1) / kC;
        }
    } else {
        if (total_tokens % n_seqs != 0)
            return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: total_tokens not divisible by n_seqs "
                        "for an equal-length batch");
        seq_len = total_tokens / n_seqs;
        chunks_per_seq = (seq_len + kC - 1) / kC;
        for (int n = 0; n < n_seqs; ++n) chunk_cu[n + 1] = chunk_cu[n] + chunks_per_seq;
    }
    const int64_t total_chunks = chunk_cu[n_seqs];
    if (total_chunks > 0x7fffffff)
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: too many chunks");

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // bf16: two paths.  With room for every tile of the call, the intra-chunk stage runs as one
    // kernel over all SMs followed by the inter-chunk kernel (fastest on this device).  With less
    // room, one fused cooperative kernel hands the tiles over through a small ring that stays in L2
    // instead of walking the chunks in several passes.
    bool fused = false;
    if (dt == KDA_BF16) {
        const int mode = g_chunk_path.load(std::memory_order_relaxed);
        const WsLayout L2p = ws_layout(n_seqs, H);
        const bool one_pass = workspace_bytes >= L2p.fixed &&
                              (int64_t)((workspace_bytes - L2p.fixed) / ((size_t)H * tc_tile_bytes())) >= total_chunks;
        fused = !lm.rate && (mode == 2 || (mode == 0 && !one_pass));
    }
    if (fused) {
        // ---- one fused cooperative kernel ----
        const int64_t J = (int64_t)n_seqs * H;
        const FusedLayout FL = fused_layout(J);
        const size_t tbf = tc_tile_bytes();
        if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) ||
            workspace_bytes < FL.off_ring + 2 * tbf)
            return fail(KDA_ERR_WORKSPACE, "kda_chunk_fwd: workspace must be 256-byte aligned and at "
                        "least %zu bytes (got %zu)", FL.off_ring + 2 * tbf, workspace_bytes);
        if (J > 0x3fffffff) return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd: n_seqs*H too large");
        char* wsb = static_cast<char*>(workspace);
        WsHeader* hdrf = reinterpret_cast<WsHeader*>(wsb);
        if (!o && !S_T) {   // nothing observable to produce: only leave a clean status word
            KDA_CUDA_TRY(cudaMemsetAsync(hdrf, 0, sizeof(WsHeader), st));
            return KDA_OK;
        }
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
        const int64_t avail = (int64_t)((workspace_bytes - FL.off_ring) / tbf);
        const FusedPlan P = fused_plan(chunk_cu, n_seqs, H, avail, n_sm);
        if (P.Q < 1) return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: the device has too few SMs");
        const int64_t Q = P.Q, R = P.R, n_rounds = P.n_rounds;
        const uint64_t n_prod = P.n_prod;
        if (n_prod > 0x7fffffffull)
            return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd: too many (chunk, head) tiles in one call");
        FusedArgs f;
        f.a.q = q; f.a.k = k; f.a.v = v; f.a.log_alpha = log_alpha; f.a.beta = beta;
        f.a.S_in = S0; f.a.S_out = S_T; f.a.o = o;
        f.a.cu_seqlens = cu_seqlens_dev; f.a.chunk_cu = nullptr;
        f.a.n_seqs = n_seqs; f.a.H = H; f.a.total_tokens = total_tokens; f.a.seq_len = seq_len;
        f.a.chunks_per_seq = chunks_per_seq; f.a.g0 = 0; f.a.g1 = total_chunks; f.a.scale = scale;
        f.a.wait_limit_ns = wait_limit_ns();
        f.ring = wsb + FL.off_ring;
        f.ready = reinterpret_cast<unsigned long long*>(wsb + FL.off_ready);
        f.consumed = reinterpret_cast<unsigned long long*>(wsb + FL.off_consumed);
        f.round_base = cu_seqlens_dev ? reinterpret_cast<const uint32_t*>(wsb + FL.off_table) : nullptr;
        f.hdr = hdrf;
        f.Q = (int)Q; f.R = (int)R; f.J = (int)J; f.n_rounds = (int)n_rounds;
        f.n_prod = (uint32_t)n_prod;
        uint32_t ep = g_epoch.fetch_add(1, std::memory_order_relaxed) + 1;
        if (ep == 0) ep = g_epoch.fetch_add(1, std::memory_order_relaxed) + 1;
        f.epoch = ep;
        f.n_chain_cta = (int)(fused_slices() * Q);
        kda_status_t rcf = KDA_OK;
        if (cu_seqlens_dev)
            rcf = launch_fused_prep(hdrf, cu_seqlens_dev, reinterpret_cast<uint32_t*>(wsb + FL.off_table),
                                    n_seqs, H, (int)Q, (int)n_rounds, st);
        if (rcf != KDA_OK) return rcf;
        return launch_fused_tc(f, q != nullptr && o != nullptr, cu_seqlens_dev == nullptr, st);
    }

    const WsLayout L = ws_layout(n_seqs, H);
    const size_t tb = tile_bytes(dt);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) ||
        workspace_bytes < L.fixed + (size_t)H * tb)
        return fail(KDA_ERR_WORKSPACE, "kda_chunk_fwd: workspace must be 256-byte aligned and at "
                    "least %zu bytes (got %zu)", L.fixed + (size_t)H * tb, workspace_bytes);
    char* ws = static_cast<char*>(workspace);
    int64_t cap = (int64_t)((workspace_bytes - L.fixed) / ((size_t)H * tb));
    if (cap > 0x7fffffff) cap = 0x7fffffff;

    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws);
    int32_t* chunk_cu_dev = reinterpret_cast<int32_t*>(ws + L.off_table);
    // The prologue kernel clears the status word and builds the chunk table of a packed batch.  An
    // equal-length bf16 call with work to do skips it: its first intra-chunk kernel clears the word.
    const bool tc_clears = dt == KDA_BF16 && !cu_seqlens_dev && total_chunks > 0 && (o || S_T);
    kda_status_t rc = KDA_OK;
    if (!tc_clears) rc = launch_prep(hdr, cu_seqlens_dev, chunk_cu_dev, n_seqs, st);
    if (rc != KDA_OK) return rc;
    if (!o && !S_T) return KDA_OK;   // nothing observable to produce

    float* state = S_T ? S_T : reinterpret_cast<float*>(ws + L.off_state);
    ChunkArgs a;
    a.q = q; a.k = k; a.v = v; a.log_alpha = log_alpha; a.beta = beta;
    a.o = o; a.cu_seqlens = cu_seqlens_dev; a.chunk_cu = cu_seqlens_dev ? chunk_cu_dev : nullptr;
    a.n_seqs = n_seqs; a.H = H; a.total_tokens = total_tokens; a.seq_len = seq_len;
    a.chunks_per_seq = chunks_per_seq; a.scale = scale;
    a.S_out = state;
    a.gate_rate = lm.rate; a.gate_bias = lm.bias; a.l2_eps = lm.l2_eps;
    a.wait_limit_ns = wait_limit_ns();
    a.out_gate = lm.out_gate; a.rms_weight = lm.rms_weight; a.rms_eps = lm.rms_eps;

    int64_t g0 = 0;
    bool first = true;
    do {
        const int64_t g1 = (total_chunks - g0 > cap) ? g0 + cap : total_chunks;
        a.g0 = g0; a.g1 = g1;
        a.S_in = first ? S0 : state;
        int n_begin = 0, n_count = n_seqs;
        if (!first) {   // only the sequences that own a chunk of this pass
            n_begin = 0;
            while (n_begin < n_seqs && chunk_cu[n_begin + 1] <= g0) ++n_begin;
            int n_end = n_begin;
            while (n_end < n_seqs && chunk_cu[n_end] < g1) ++n_end;
            n_count = n_end - n_begin;
        }
        if (dt == KDA_BF16)
            rc = launch_chunk_tc(a, ws + L.off_tiles, n_begin, n_count, hdr, tc_clears && first, st);
        else
            rc = launch_chunk_simt(a, dt, ws + L.off_tiles, n_begin, n_count, hdr, st);
        if (rc != KDA_OK) return rc;
        g0 = g1;
        first = false;
    } while (g0 < total_chunks);
    return KDA_OK;
}

}  // namespace
}  // namespace kda

extern "C" {

kda_status_t kda_chunk_fwd(const void* q, const void* k, const void* v, const float* log_alpha,
                           const float* beta, const float* S0, void* o, float* S_T,
                           const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host,
                           int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk,
                           float scale, kda_dtype_t dt, void* workspace, size_t workspace_bytes,
                           void* cuda_stream)
{
    return chunk_fwd_impl(q, k, v, log_alpha, beta, S0, o, S_T, cu_seqlens_dev, cu_seqlens_host, n_seqs,
                          total_tokens, H, dk, dv, chunk, scale, dt, workspace, workspace_bytes, cuda_stream,
                          LayerMode());
}

kda_status_t kda_layer_set_fused_output(int on)
{
    g_fuse_output.store(on ? 1 : 0, std::memory_order_relaxed);
    return KDA_OK;
}

size_t kda_layer_fwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk)
{
    return kda_chunk_fwd_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, KDA_BF16);
}

size_t kda_layer_fwd_min_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk)
{
    if (!shape_ok(dk, dv, chunk, KDA_BF16) || total_tokens < 0 || n_seqs < 0 || H <= 0) return 0;
    return ws_layout(n_seqs, H).fixed + align_up((size_t)H * tc_tile_bytes());
}

kda_status_t kda_layer_fwd(const void* q_c, const void* k_c, const void* v, const void* g_a,
                           const float* b_pre, const void* g_o, const float* A_log, const float* dt_bias,
                           const float* rms_weight, float l2_eps, float rms_eps, const float* S0, void* y,
                           float* S_T, const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host,
                           int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk, float scale,
                           void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!A_log || !dt_bias)
        return fail(KDA_ERR_INVALID_ARG, "kda_layer_fwd: A_log and dt_bias must not be NULL");
    if (y && total_tokens > 0 && (!g_o || !rms_weight))
        return fail(KDA_ERR_INVALID_ARG, "kda_layer_fwd: g_o and rms_weight must not be NULL when y is "
                    "requested");
    const void* ptrs[] = {g_o, A_log, dt_bias, rms_weight};
    for (const void* p : ptrs)
        if (!aligned16(p)) return fail(KDA_ERR_INVALID_ARG, "kda_layer_fwd: pointer %p is not 16-byte "
                                       "aligned", p);
    LayerMode lm;
    lm.rate = A_log; lm.bias = dt_bias; lm.l2_eps = l2_eps;
    // The output stage runs inside the inter-chunk kernel when the device can hold the clusters this
    // needs (the slices of a row exchange their sums of squares), else as a pass of its own.
    const bool fuse_out = y && total_tokens > 0 && n_seqs > 0 && g_fuse_output.load(std::memory_order_relaxed) &&
                          inter_can_fuse_epilogue((int64_t)n_seqs * H);
    if (fuse_out) {
        lm.out_gate = g_o; lm.rms_weight = rms_weight; lm.rms_eps = rms_eps;
    }
    kda_status_t rc = chunk_fwd_impl(q_c, k_c, v, reinterpret_cast<const float*>(g_a), b_pre, S0, y, S_T,
                                     cu_seqlens_dev, cu_seqlens_host, n_seqs, total_tokens, H, dk, dv, chunk,
                                     scale, KDA_BF16, workspace, workspace_bytes, cuda_stream, lm);
    if (rc != KDA_OK || !y || total_tokens == 0 || n_seqs == 0 || fuse_out) return rc;
    return launch_layer_epilogue(y, g_o, rms_weight, rms_eps, total_tokens * H,
                                 static_cast<cudaStream_t>(cuda_stream));
}

kda_status_t kda_decode_step(const void* q, const void* k, const void* v, const float* log_alpha,
                             const float* beta, float* S, const int32_t* state_slot, void* o,
                             int n_seqs, int H, int dk, int dv, float scale, kda_dtype_t dt,
                             void* cuda_stream)
{
    if (dk != kD || dv != kD || (dt != KDA_F32 && dt != KDA_BF16))
        return fail(KDA_ERR_UNSUPPORTED, "kda_decode_step: only dk=dv=128, dt in {f32,bf16} are "
                    "supported (got dk=%d dv=%d dt=%d)", dk, dv, (int)dt);
    if (n_seqs < 0 || H <= 0 || (int64_t)n_seqs * H > 0x7fffffff)
        return fail(KDA_ERR_INVALID_ARG, "kda_decode_step: bad sizes n_seqs=%d H=%d", n_seqs, H);
    if (n_seqs == 0) return KDA_OK;
    if (!q || !k || !v || !log_alpha || !beta || !S || !o)
        return fail(KDA_ERR_INVALID_ARG, "kda_decode_step: NULL pointer argument");
    const void* ptrs[] = {q, k, v, log_alpha, beta, S, o, state_slot};
    for (const void* p : ptrs)
        if (!aligned16(p)) return fail(KDA_ERR_INVALID_ARG, "kda_decode_step: pointer %p is not "
                                       "16-byte aligned", p);
    return launch_decode(q, k, v, log_alpha, beta, S, state_slot, o, n_seqs, H, scale, dt,
                         static_cast<cudaStream_t>(cuda_stream));
}

kda_status_t kda_layer_decode_step(const void* q_c, const void* k_c, const void* v, const void* g_a,
                                   const float* b_pre, const void* g_o, const float* A_log,
                                   const float* dt_bias, const float* rms_weight, float l2_eps, float rms_eps,
                                   float* S, const int32_t* state_slot, void* y, int n_seqs, int H, int dk,
                                   int dv, float scale, void* cuda_stream)
{
    if (dk != kD || dv != kD)
        return fail(KDA_ERR_UNSUPPORTED, "kda_layer_decode_step: only dk=dv=128 is supported (got dk=%d dv=%d)",
                    dk, dv);
    if (n_seqs < 0 || H <= 0 || (int64_t)n_seqs * H > 0x7fffffff)
        return fail(KDA_ERR_INVALID_ARG, "kda_layer_decode_step: bad sizes n_seqs=%d H=%d", n_seqs, H);
    if (n_seqs == 0) return KDA_OK;
    if (!q_c || !k_c || !v || !g_a || !b_pre || !g_o || !A_log || !dt_bias || !rms_weight || !S || !y)
        return fail(KDA_ERR_INVALID_ARG, "kda_layer_decode_step: NULL pointer argument");
    const void* ptrs[] = {q_c, k_c, v, g_a, b_pre, g_o, A_log, dt_bias, rms_weight, S, y, state_slot};
    for (const void* p : ptrs)
        if (!aligned16(p)) return fail(KDA_ERR_INVALID_ARG, "kda_layer_decode_step: pointer %p is not "
                                       "16-byte aligned", p);
    return launch_layer_decode(q_c, k_c, v, g_a, b_pre, g_o, A_log, dt_bias, rms_weight, l2_eps, rms_eps, S,
                               state_slot, y, n_seqs, H, scale, static_cast<cudaStream_t>(cuda_stream));
}

kda_status_t kda_decode_multi(const void* q, const void* k, const void* v, const float* log_alpha,
                              const float* beta, float* S, const int32_t* state_slot, void* o,
                              int n_seqs, int n_tokens, int H, int dk, int dv, float scale,
                              kda_dtype_t dt, void* cuda_stream)
{
    if (dk != kD || dv != kD || (dt != KDA_F32 && dt != KDA_BF16))
        return fail(KDA_ERR_UNSUPPORTED, "kda_decode_multi: only dk=dv=128, dt in {f32,bf16} are "
                    "supported (got dk=%d dv=%d dt=%d)", dk, dv, (int)dt);
    if (n_seqs < 0 || H <= 0 || n_tokens < 0 || n_tokens > 64 || (int64_t)n_seqs * H > 0x7fffffff)
        return fail(KDA_ERR_INVALID_ARG, "kda_decode_multi: bad sizes n_seqs=%d n_tokens=%d H=%d "
                    "(n_tokens must be 0..64)", n_seqs, n_tokens, H);
    if (n_seqs == 0 || n_tokens == 0) return KDA_OK;
    if (!q || !k || !v || !log_alpha || !beta || !S || !o)
        return fail(KDA_ERR_INVALID_ARG, "kda_decode_multi: NULL pointer argument");
    const void* ptrs[] = {q, k, v, log_alpha, beta, S, o, state_slot};
    for (const void* p : ptrs)
        if (!aligned16(p)) return fail(KDA_ERR_INVALID_ARG, "kda_decode_multi: pointer %p is not "
                                       "16-byte aligned", p);
    return launch_decode_multi(q, k, v, log_alpha, beta, S, state_slot, o, n_seqs, n_tokens, H, scale, dt,
                               static_cast<cudaStream_t>(cuda_stream));
}

// ---- host-buffer variants -------------------------------------------------------------------------

namespace {
struct HostChunkLayout {
    size_t q, k, v, g, b, s0, o, st, cu, inner, total;
};
HostChunkLayout host_chunk_layout(int64_t T, int n_seqs, int H, kda_dtype_t dt, size_t inner_bytes)
{
    HostChunkLayout L;
    const size_t e = esize(dt), td = (size_t)T * H * kD;
    size_t off = 0;
    L.q = off; off += align_up(td * e);
    L.k = off; off += align_up(td * e);
    L.v = off; off += align_up(td * e);
    L.g = off; off += align_up(td * 4);
    L.b = off; off += align_up((size_t)T * H * 4);
    L.s0 = off; off += align_up((size_t)n_seqs * H * kD * kD * 4);
    L.o = off; off += align_up(td * e);
    L.st = off; off += align_up((size_t)n_seqs * H * kD * kD * 4);
    L.cu = off; off += align_up((size_t)(n_seqs + 1) * 4);
    L.inner = off; off += inner_bytes;
    L.total = off;
    return L;
}
}  // namespace

size_t kda_chunk_fwd_host_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                          int chunk, kda_dtype_t dt)
{
    const size_t inner = kda_chunk_fwd_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, dt);
    if (inner == 0) return 0;
    return host_chunk_layout(total_tokens, n_seqs, H, dt, inner).total;
}

kda_status_t kda_chunk_fwd_host(const void* q_host, const void* k_host, const void* v_host,
                                const float* log_alpha_host, const float* beta_host,
                                const float* S0_host, void* o_host, float* S_T_host,
                                const int32_t* cu_seqlens_host, int n_seqs, int64_t total_tokens,
                                int H, int dk, int dv, int chunk, float scale, kda_dtype_t dt,
                                void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!shape_ok(dk, dv, chunk, dt))
        return fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd_host: unsupported shape or dtype");
    if (n_seqs < 0 || total_tokens < 0 || H <= 0)
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd_host: bad sizes");
    const size_t inner_min =
        kda_chunk_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, dt);
    const HostChunkLayout L0 = host_chunk_layout(total_tokens, n_seqs, H, dt, 0);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) ||
        workspace_bytes < L0.total + inner_min)
        return fail(KDA_ERR_WORKSPACE, "kda_chunk_fwd_host: workspace must be 256-byte aligned and "
                    "at least %zu bytes (got %zu)", L0.total + inner_min, workspace_bytes);
    if (total_tokens > 0 && (!k_host || !v_host || !log_alpha_host || !beta_host))
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd_host: NULL input");
    if (o_host && total_tokens > 0 && !q_host)
        return fail(KDA_ERR_INVALID_ARG, "kda_chunk_fwd_host: q is NULL but o is requested");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    const size_t e = esize(dt), td = (size_t)total_tokens * H * kD;
    const size_t sb = (size_t)n_seqs * H * kD * kD * 4;

    // One long sequence: copy-in, compute and copy-out are pipelined over a few segments of the
    // sequence (the state handed from one segment to the next is exactly the resume property of
    // the recurrence), on two helper streams owned by the library, so that the host link is busy
    // in both directions while the kernels run.
    constexpr int64_t kMinSegTokens = 512;
    if (n_seqs == 1 && !cu_seqlens_host && total_tokens >= 2 * kMinSegTokens) {
        cudaStream_t c_in = nullptr, c_out = nullptr;   // helper streams of the calling thread's current device
        {
            DeviceLock lk;
            if (!lk.st) return lk.rc;
            if (!lk.st->copy_in)
                KDA_CUDA_TRY(cudaStreamCreateWithFlags(&lk.st->copy_in, cudaStreamNonBlocking));
            if (!lk.st->copy_out)
                KDA_CUDA_TRY(cudaStreamCreateWithFlags(&lk.st->copy_out, cudaStreamNonBlocking));
            c_in = lk.st->copy_in;
            c_out = lk.st->copy_out;
        }
        int nseg = (int)(total_tokens / kMinSegTokens);
        if (nseg > 4) nseg = 4;
        const int64_t seg = ((total_tokens + nseg - 1) / nseg + kC - 1) / kC * kC;
        std::vector<cudaEvent_t> evs;
        auto new_event = [&](cudaEvent_t* ev) {
            cudaError_t err = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
            if (err == cudaSuccess) evs.push_back(*ev);
            return err;
        };
        kda_status_t rc = KDA_OK;
        cudaError_t cerr = cudaSuccess;
#define KDA_PIPE_TRY(expr)                                                          \
    if (rc == KDA_OK && cerr == cudaSuccess) {                                      \
        cerr = (expr);                                                              \
        if (cerr != cudaSuccess)                                                    \
            rc = fail(KDA_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(cerr)); \
    }
        cudaEvent_t fork = nullptr, join = nullptr;
        KDA_PIPE_TRY(new_event(&fork));
        KDA_PIPE_TRY(cudaEventRecord(fork, st));
        KDA_PIPE_TRY(cudaStreamWaitEvent(c_in, fork, 0));
        if (S0_host) KDA_PIPE_TRY(cudaMemcpyAsync(ws + L0.s0, S0_host, sb, cudaMemcpyHostToDevice, c_in));
        float* state = reinterpret_cast<float*>(ws + L0.st);
        for (int64_t t0 = 0, k = 0; t0 < total_tokens && rc == KDA_OK; t0 += seg, ++k) {
            const int64_t t1 = (t0 + seg < total_tokens) ? t0 + seg : total_tokens;
            const size_t r0 = (size_t)t0 * H * kD, rn = (size_t)(t1 - t0) * H * kD;
            if (q_host)
                KDA_PIPE_TRY(cudaMemcpyAsync(ws + L0.q + r0 * e, (const char*)q_host + r0 * e, rn * e, cudaMemcpyHostToDevice, c_in));
            KDA_PIPE_TRY(cudaMemcpyAsync(ws + L0.k + r0 * e, (const char*)k_host + r0 * e, rn * e, cudaMemcpyHostToDevice, c_in));
            KDA_PIPE_TRY(cudaMemcpyAsync(ws + L0.v + r0 * e, (const char*)v_host + r0 * e, rn * e, cudaMemcpyHostToDevice, c_in));
            KDA_PIPE_TRY(cudaMemcpyAsync(ws + L0.g + r0 * 4, (const char*)log_alpha_host + r0 * 4, rn * 4, cudaMemcpyHostToDevice, c_in));
            KDA_PIPE_TRY(cudaMemcpyAsync(ws + L0.b + (size_t)t0 * H * 4, (const char*)beta_host + (size_t)t0 * H * 4,
                                         (size_t)(t1 - t0) * H * 4, cudaMemcpyHostToDevice, c_in));
            cudaEvent_t in_done = nullptr, out_ready = nullptr;
            KDA_PIPE_TRY(new_event(&in_done));
            KDA_PIPE_TRY(cudaEventRecord(in_done, c_in));
            KDA_PIPE_TRY(cudaStreamWaitEvent(st, in_done, 0));
            if (rc == KDA_OK)
                rc = kda_chunk_fwd(q_host ? ws + L0.q + r0 * e : nullptr, ws + L0.k + r0 * e, ws + L0.v + r0 * e,
                                   reinterpret_cast<float*>(ws + L0.g) + r0, reinterpret_cast<float*>(ws + L0.b) + (size_t)t0 * H,
                                   k == 0 ? (S0_host ? reinterpret_cast<float*>(ws + L0.s0) : nullptr) : state,
                                   o_host ? ws + L0.o + r0 * e : nullptr, state, nullptr, nullptr, 1, t1 - t0, H, dk, dv,
                                   chunk, scale, dt, ws + L0.inner, workspace_bytes - L0.inner, st);
            if (o_host) {
                KDA_PIPE_TRY(new_event(&out_ready));
                KDA_PIPE_TRY(cudaEventRecord(out_ready, st));
                KDA_PIPE_TRY(cudaStreamWaitEvent(c_out, out_ready, 0));
                KDA_PIPE_TRY(cudaMemcpyAsync((char*)o_host + r0 * e, ws + L0.o + r0 * e, rn * e, cudaMemcpyDeviceToHost, c_out));
            }
        }
        if (o_host) {   // the caller's stream completes only after the last copy-out
            KDA_PIPE_TRY(new_event(&join));
            KDA_PIPE_TRY(cudaEventRecord(join, c_out));
            KDA_PIPE_TRY(cudaStreamWaitEvent(st, join, 0));
        }
        if (S_T_host) KDA_PIPE_TRY(cudaMemcpyAsync(S_T_host, state, sb, cudaMemcpyDeviceToHost, st));
#undef KDA_PIPE_TRY
        for (cudaEvent_t ev : evs) cudaEventDestroy(ev);   // released once the work that uses them is done
        return rc;
    }

    if (q_host && td) KDA_CUDA_TRY(cudaMemcpyAsync(ws + L0.q, q_host, td * e, cudaMemcpyHostToDevice, st));
    if (td) {
        KDA_CUDA_TRY(cudaMemcpyAsync(ws + L0.k, k_host, td * e, cudaMemcpyHostToDevice, st));
        KDA_CUDA_TRY(cudaMemcpyAsync(ws + L0.v, v_host, td * e, cudaMemcpyHostToDevice, st));
        KDA_CUDA_TRY(cudaMemcpyAsync(ws + L0.g, log_alpha_host, td * 4, cudaMemcpyHostToDevice, st));
        KDA_CUDA_TRY(cudaMemcpyAsync(ws + L0.b, beta_host, (size_t)total_tokens * H * 4,
                                     cudaMemcpyHostToDevice, st));
    }
    if (S0_host && sb) KDA_CUDA_TRY(cudaMemcpyAsync(ws + L0.s0, S0_host, sb, cudaMemcpyHostToDevice, st));
    if (cu_seqlens_host)
        KDA_CUDA_TRY(cudaMemcpyAsync(ws + L0.cu, cu_seqlens_host, (size_t)(n_seqs + 1) * 4,
                                     cudaMemcpyHostToDevice, st));
    kda_status_t rc = kda_chunk_fwd(
        q_host ? ws + L0.q : nullptr, ws + L0.k, ws + L0.v, reinterpret_cast<float*>(ws + L0.g),
        reinterpret_cast<float*>(ws + L0.b), S0_host ? reinterpret_cast<float*>(ws + L0.s0) : nullptr,
        o_host ? ws + L0.o : nullptr, S_T_host ? reinterpret_cast<float*>(ws + L0.st) : nullptr,
        cu_seqlens_host ? reinterpret_cast<int32_t*>(ws + L0.cu) : nullptr, cu_seqlens_host, n_seqs,
        total_tokens, H, dk, dv, chunk, scale, dt, ws + L0.inner, workspace_bytes - L0.inner, st);
    if (rc != KDA_OK) return rc;
    if (o_host && td) KDA_CUDA_TRY(cudaMemcpyAsync(o_host, ws + L0.o, td * e, cudaMemcpyDeviceToHost, st));
    if (S_T_host && sb) KDA_CUDA_TRY(cudaMemcpyAsync(S_T_host, ws + L0.st, sb, cudaMemcpyDeviceToHost, st));
    return KDA_OK;
}

size_t kda_decode_step_host_workspace_bytes(int n_seqs, int H, int dk, int dv, kda_dtype_t dt)
{
    if (dk != kD || dv != kD || n_seqs < 0 || H <= 0) return 0;
    const size_t e = esize(dt), nd = (size_t)n_seqs * H * kD;
    return 4 * align_up(nd * e) + align_up(nd * 4) + align_up((size_t)n_seqs * H * 4) +
           align_up((size_t)n_seqs * 4) + kAlign;
}

kda_status_t kda_decode_step_host(const void* q_host, const void* k_host, const void* v_host,
                                  const float* log_alpha_host, const float* beta_host,
                                  float* S_dev, const int32_t* state_slot_host, void* o_host,
                                  int n_seqs, int H, int dk, int dv, float scale, kda_dtype_t dt,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    const size_t need = kda_decode_step_host_workspace_bytes(n_seqs, H, dk, dv, dt);
    if (need == 0) return fail(KDA_ERR_UNSUPPORTED, "kda_decode_step_host: unsupported shape");
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) || workspace_bytes < need)
        return fail(KDA_ERR_WORKSPACE, "kda_decode_step_host: workspace must be 256-byte aligned and "
                    "at least %zu bytes", need);
    if (n_seqs == 0) return KDA_OK;
    if (!q_host || !k_host || !v_host || !log_alpha_host || !beta_host || !S_dev || !o_host)
        return fail(KDA_ERR_INVALID_ARG, "kda_decode_step_host: NULL pointer argument");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    const size_t e = esize(dt), nd = (size_t)n_seqs * H * kD;
    size_t off = 0;
    char* dq = ws + off; off += align_up(nd * e);
    char* dkk = ws + off; off += align_up(nd * e);
    char* dvv = ws + off; off += align_up(nd * e);
    char* dout = ws + off; off += align_up(nd * e);
    char* dg = ws + off; off += align_up(nd * 4);
    char* db = ws + off; off += align_up((size_t)n_seqs * H * 4);
    char* ds = ws + off;
    KDA_CUDA_TRY(cudaMemcpyAsync(dq, q_host, nd * e, cudaMemcpyHostToDevice, st));
    KDA_CUDA_TRY(cudaMemcpyAsync(dkk, k_host, nd * e, cudaMemcpyHostToDevice, st));
    KDA_CUDA_TRY(cudaMemcpyAsync(dvv, v_host, nd * e, cudaMemcpyHostToDevice, st));
    KDA_CUDA_TRY(cudaMemcpyAsync(dg, log_alpha_host, nd * 4, cudaMemcpyHostToDevice, st));
    KDA_CUDA_TRY(cudaMemcpyAsync(db, beta_host, (size_t)n_seqs * H * 4, cudaMemcpyHostToDevice, st));
    if (state_slot_host)
        KDA_CUDA_TRY(cudaMemcpyAsync(ds, state_slot_host, (size_t)n_seqs * 4, cudaMemcpyHostToDevice, st));
    kda_status_t rc = kda_decode_step(dq, dkk, dvv, reinterpret_cast<float*>(dg),
                                      reinterpret_cast<float*>(db), S_dev,
                                      state_slot_host ? reinterpret_cast<int32_t*>(ds) : nullptr, dout,
                                      n_seqs, H, dk, dv, scale, dt, st);
    if (rc != KDA_OK) return rc;
    KDA_CUDA_TRY(cudaMemcpyAsync(o_host, dout, nd * e, cudaMemcpyDeviceToHost, st));
    return KDA_OK;
}

kda_status_t kda_selftest_wait_timeout(void* workspace, int limit_ms, void* cuda_stream)
{
    if (!workspace || limit_ms <= 0 || limit_ms > 1000)
        return fail(KDA_ERR_INVALID_ARG, "kda_selftest_wait_timeout: workspace NULL or limit outside 1..1000 ms");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    KDA_CUDA_TRY(cudaMemsetAsync(workspace, 0, sizeof(WsHeader), st));
    return launch_wait_selftest(reinterpret_cast<WsHeader*>(workspace), (uint64_t)limit_ms * 1000000ull, st);
}

void kda_profile_enable(int on)
{
    std::lock_guard<std::mutex> lk(g_prof.mu);
    g_prof.on = on != 0;
    g_prof.used = 0;
}

kda_status_t kda_profile_read(int kind, double* total_ms, int* launches)
{
    if (kind < 0 || kind >= PROF_KINDS || !total_ms || !launches)
        return fail(KDA_ERR_INVALID_ARG, "kda_profile_read: bad argument");
    KDA_CUDA_TRY(cudaDeviceSynchronize());
    std::lock_guard<std::mutex> lk(g_prof.mu);
    double sum = 0.0;
    int cnt = 0;
    for (int i = 0; i < g_prof.used; ++i) {
        if (g_prof.kind[i] != kind) continue;
        float ms = 0.f;
        KDA_CUDA_TRY(cudaEventElapsedTime(&ms, g_prof.ev0[i], g_prof.ev1[i]));
        sum += ms;
        ++cnt;
    }
    *total_ms = sum;
    *launches = cnt;
    return KDA_OK;
}

kda_status_t kda_check_status(void* workspace, void* cuda_stream)
{
    if (!workspace) return fail(KDA_ERR_INVALID_ARG, "kda_check_status: NULL workspace");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    WsHeader h;
    KDA_CUDA_TRY(cudaMemcpyAsync(&h, workspace, sizeof(h), cudaMemcpyDeviceToHost, st));
    KDA_CUDA_TRY(cudaStreamSynchronize(st));
    if (h.status != 0 || (h.flags & 1)) {
        // only the words the device reports through are cleared (a fused call keeps a counter
        // further down in the header)
        KDA_CUDA_TRY(cudaMemsetAsync(workspace, 0, 16, st));
        if (h.status != 0)
            return fail((kda_status_t)h.status, "device code reported status %d at location %d",
                        h.status, h.where);
        return fail(KDA_ERR_GATE_RANGE, "a channel decayed by more than e^-160 within one 64-token "
                    "chunk: its intra-chunk terms were formed from clamped factors and are not exact");
    }
    return KDA_OK;
}

}  // extern "C"
