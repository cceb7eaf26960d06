// kda_chunk_fwd_static: the chunkwise forward for callers that cannot allocate device memory.
//
// Some hosts of this library are not allowed to call cudaMalloc (or any allocating routine) at the
// point where they need a prefill: code running inside a serving loop whose memory pool is fixed
// at start-up, a plug-in that is handed tensors but no allocator, a process whose device memory is
// fully reserved by its framework.  For them the scratch that kda_chunk_fwd normally receives from
// the caller lives here, in a fixed array that is part of the loaded module.
#include <mutex>

#include "kda_common.cuh"

namespace {

// Every GPU that loads this library holds this array until the process exits.
constexpr size_t kStaticScratchBytes = (size_t)16 << 20;   // 16 MiB
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mu;
void* g_scratch_addr[kMaxDevices] = {};   // device address of the array, per device ordinal

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the
// address a kernel can use has to be asked for, once per device, with that device current.
kda_status_t scratch_address(void** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess)
        return kda::fail(KDA_ERR_CUDA, "kda_chunk_fwd_static: cudaGetDevice failed: %s",
                         cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices)
        return kda::fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd_static: device ordinal %d out of range", dev);
    std::lock_guard<std::mutex> lk(g_setup_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p)
            return kda::fail(KDA_ERR_CUDA, "kda_chunk_fwd_static: cudaGetSymbolAddress failed: %s",
                             cudaGetErrorString(e));
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return KDA_OK;
}

}  // namespace

extern "C" {

size_t kda_chunk_fwd_static_max_bytes(void) { return kStaticScratchBytes; }

kda_status_t kda_chunk_fwd_static_check_status(void* cuda_stream)
{
    void* scratch = nullptr;
    kda_status_t rc = scratch_address(&scratch);
    if (rc != KDA_OK) return rc;
    return kda_check_status(scratch, cuda_stream);
}

kda_status_t kda_chunk_fwd_static(const void* q, const void* k, const void* v, const float* log_alpha,
                                  const float* beta, const float* S0, void* o, float* S_T,
                                  const int32_t* cu_seqlens_dev, const int32_t* cu_seqlens_host,
                                  int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk,
                                  float scale, kda_dtype_t dt, void* cuda_stream)
{
    const size_t need =
        kda_chunk_fwd_min_workspace_bytes(total_tokens, n_seqs, H, dk, dv, chunk, dt);
    if (need == 0)
        return kda::fail(KDA_ERR_UNSUPPORTED, "kda_chunk_fwd_static: unsupported shape or dtype "
                         "(dk=%d dv=%d chunk=%d dt=%d)", dk, dv, chunk, (int)dt);
    if (need > kStaticScratchBytes)
        return kda::fail(KDA_ERR_WORKSPACE, "kda_chunk_fwd_static: this call needs at least %zu bytes "
                         "of scratch but the built-in scratch holds %zu; use kda_chunk_fwd with a "
                         "caller-provided workspace (n_seqs=%d, H=%d)", need, kStaticScratchBytes,
                         n_seqs, H);
    void* scratch = nullptr;
    kda_status_t rc = scratch_address(&scratch);
    if (rc != KDA_OK) return rc;
    // The status word at the start of the scratch is the only part that must start at zero; the
    // forward call clears it on the stream before any kernel reads it.  Everything else is written
    // before it is read within the call.
    return kda_chunk_fwd(q, k, v, log_alpha, beta, S0, o, S_T, cu_seqlens_dev, cu_seqlens_host, n_seqs,
                         total_tokens, H, dk, dv, chunk, scale, dt, scratch, kStaticScratchBytes,
                         cuda_stream);
}

}  // extern "C"
