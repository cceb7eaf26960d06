/*
 * kda.h -- C ABI of the B200 (sm_100a) Kimi Delta Attention hot path.
 *
 * Two operations, both per sequence n and head h independently, with a dk x dv state S:
 *
 *   kda_chunk_fwd    chunkwise-parallel forward (prefill) of the recurrence
 *                      S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T
 *                      o_t = scale * S_t^T q_t
 *                    (Kimi Linear paper, Section 3, Eq. 1) evaluated with the chunkwise algorithm
 *                    of Section 3.1: per-chunk cumulative log-decay, WY representation, UT
 *                    transform, pseudo-values U - W S, output equation and chunk state update.
 *   kda_decode_step  the same recurrence for ONE new token per sequence, state updated in place
 *                    (Section 6.3 "Inference strategy": prefill uses the chunk kernel, generation
 *                    the recurrent kernel).
 *
 * Conventions
 *   - All tensors are dense, innermost dimension contiguous, token-major:
 *       q, k, log_alpha : [total_tokens, H, dk]     v, o : [total_tokens, H, dv]
 *       beta            : [total_tokens, H]         S0, S_T, S : [n, H, dk, dv]  (dv contiguous)
 *   - alpha_t = exp(log_alpha_t), log_alpha <= 0 (a decay).  The cumulative log-decay of a channel
 *     over one 64-token chunk must stay above -160 (a factor e^-160).  The decay ratio
 *     exp(G_i - G_j) of two tokens of a chunk is formed as exp(G_i - G_m) * exp(G_m - G_j) around the
 *     middle G_m of the chunk's log-decay range, each exponent clamped to +-80.  Inside the limit
 *     that is exact.  Beyond it a pair of tokens that both lie more than 80 from G_m on the same
 *     side gets the product of two clamped factors, i.e. a ratio that is TOO LARGE (up to 1 where
 *     the true ratio is smaller): the results stay finite but that channel's intra-chunk terms are
 *     wrong.  The library detects the condition per chunk and channel and reports it through
 *     kda_check_status as KDA_ERR_GATE_RANGE.
 *   - dt selects the storage type of q, k, v and o (fp32 or bf16).  Gates, beta and states are
 *     always fp32.  dt = KDA_BF16 runs the contractions on bf16 tensor cores with fp32
 *     accumulation; dt = KDA_F32 runs everything in fp32 FMA arithmetic.
 *   - Supported shapes: dk = dv = 128, chunk = 64.  Anything else returns KDA_ERR_UNSUPPORTED;
 *     there is no fallback path of any kind.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer, 16-byte aligned, owned by
 *     the caller.  The library allocates no device memory: scratch comes from the caller's
 *     workspace.  Calls are asynchronous and ordered on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the default stream); the caller keeps every buffer alive until the stream has
 *     finished the call.
 *   - Errors: every entry point returns a kda_status_t; nothing throws, aborts or traps.  Argument
 *     errors are detected on the host before anything is launched.  kda_last_error() returns a
 *     description of the calling thread's most recent failure.
 */
#ifndef KDA_H_
#define KDA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KDA_OK = 0,
    KDA_ERR_INVALID_ARG = 1, /* NULL/misaligned pointer, bad size, non-monotone cu_seqlens */
    KDA_ERR_UNSUPPORTED = 2, /* shape or dtype outside the supported set */
    KDA_ERR_WORKSPACE = 3,   /* workspace NULL or smaller than the minimum */
    KDA_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed */
    KDA_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out (reported by kda_check_status) */
    KDA_ERR_GATE_RANGE = 6   /* a channel decayed by more than e^-160 inside one chunk: results are
                                finite but not exact (reported by kda_check_status) */
} kda_status_t;

typedef enum { KDA_F32 = 0, KDA_BF16 = 1 } kda_dtype_t;

/*
 * Workspace size that lets kda_chunk_fwd keep every (chunk, head) tile of the call at once (the
 * fastest schedule on this device: one kernel per stage), capped at 8 GiB.  Any workspace of at
 * least kda_chunk_fwd_min_workspace_bytes() works: with less than the full size a bf16 call runs
 * as one fused kernel whose stages exchange tiles through a ring (of up to 16 tiles per running
 * head) inside the workspace, and an fp32 call proceeds in several passes over ranges of chunks
 * with the state carried between them.  Both return 0 for an unsupported shape.
 */
size_t kda_chunk_fwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                     int chunk, kda_dtype_t dt);
size_t kda_chunk_fwd_min_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                         int chunk, kda_dtype_t dt);

/*
 * Chunkwise forward (Section 3.1; pseudo-code in Appendix C).
 *
 *   q, k        [total_tokens,H,dk] dt      q may be NULL when o is NULL
 *   v           [total_tokens,H,dv] dt
 *   log_alpha   [total_tokens,H,dk] fp32    per-channel log decay of each token
 *   beta        [total_tokens,H]    fp32
 *   S0          [n_seqs,H,dk,dv]    fp32    initial states, or NULL = zeros
 *   o           [total_tokens,H,dv] dt      output, or NULL = not produced (state-only mode)
 *   S_T         [n_seqs,H,dk,dv]    fp32    state after each sequence's last token, or NULL
 *   cu_seqlens_dev   [n_seqs+1] int32 device token offsets of a packed batch (cu[0] = 0,
 *                    cu[n_seqs] = total_tokens, non-decreasing), or NULL = n_seqs sequences of
 *                    equal length total_tokens / n_seqs
 *   cu_seqlens_host  the same values in host memory (used for validation and scheduling); NULL
 *                    exactly when cu_seqlens_dev is NULL
 *   scale       multiplies q (the paper's pseudo-code uses dk^-0.5; pass 1 for pre-scaled q)
 *   workspace   device scratch of workspace_bytes bytes, 256-byte aligned
 *
 * Chunks restart at every sequence start; a sequence whose length is not a multiple of 64 ends in
 * a short chunk; a zero-length sequence yields S_T = S0 and no rows of o.  S0 and S_T may alias.
 * Returns KDA_OK once all work is enqueued on the stream.
 */
kda_status_t kda_chunk_fwd(const void *q, const void *k, const void *v, const float *log_alpha,
                           const float *beta, const float *S0, void *o, float *S_T,
                           const int32_t *cu_seqlens_dev, const int32_t *cu_seqlens_host,
                           int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk,
                           float scale, kda_dtype_t dt, void *workspace, size_t workspace_bytes,
                           void *cuda_stream);

/*
 * kda_chunk_fwd without a workspace argument, for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a deployment convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc and every allocating routine are off limits -- a
 * serving loop whose memory pool was fixed at start-up, a plug-in that receives tensors but no
 * allocator, a process whose framework has reserved all device memory.  The scratch that
 * kda_chunk_fwd takes from the caller is replaced by a fixed array of
 * kda_chunk_fwd_static_max_bytes() = 16 MiB that is part of the library image: every GPU that
 * loads the library holds those 16 MiB until the process exits.
 *
 * Same arguments, results and error codes as kda_chunk_fwd, with these differences:
 *   - A call whose minimum scratch (kda_chunk_fwd_min_workspace_bytes) exceeds the 16 MiB is
 *     rejected with KDA_ERR_WORKSPACE and a message naming both sizes; nothing is launched.  For
 *     bf16 the minimum is a few hundred KiB plus 4 bytes per (sequence, head), so practically every
 *     batch fits: the call runs as the fused kernel with a ring of about 220 tiles (e.g. 6 tiles
 *     ahead for each of 32 concurrently running heads).  For fp32 the minimum holds 64 KiB of state
 *     scratch per (sequence, head), which limits that path to about 200 of them.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress, with the calling thread's current device).  Make that first call
 *     before starting any stream capture.
 *   - The entry point calls no cudaMalloc, cudaFree or allocating library routine.
 *   - All calls on one device share the one array, and it keeps the previous call's contents.
 *     Nothing in it has to be cleared by the caller (every call clears or re-tags what it reads),
 *     but two calls that overlap on the GPU -- different streams, or one stream per thread -- race
 *     on it: serialise them.
 *   - The status word lives in the array: kda_chunk_fwd_static_check_status(stream) reads and
 *     clears it exactly as kda_check_status does for a caller's workspace (it synchronises the
 *     stream; it allocates nothing either).
 */
size_t kda_chunk_fwd_static_max_bytes(void);
kda_status_t kda_chunk_fwd_static_check_status(void *cuda_stream);
kda_status_t kda_chunk_fwd_static(const void *q, const void *k, const void *v,
                                  const float *log_alpha, const float *beta, const float *S0,
                                  void *o, float *S_T, const int32_t *cu_seqlens_dev,
                                  const int32_t *cu_seqlens_host, int n_seqs, int64_t total_tokens,
                                  int H, int dk, int dv, int chunk, float scale, kda_dtype_t dt,
                                  void *cuda_stream);

/*
 * The KDA operator with the layer's surrounding element-wise stages (paper Section 4, "Neural
 * Parameterization"), from the activations that leave the short convolutions to the input of the
 * output projection, bf16 tensor-core path:
 *
 *     q, k      = L2Norm(q_c), L2Norm(k_c)                      x / sqrt(sum x^2 + l2_eps), over dk
 *     log alpha = -exp(A_log[h]) * softplus(g_a + dt_bias[h,:])  (the decay function f; the paper
 *                 names its family only -- "similar to GDN and Mamba" -- this is that form)
 *     beta      = sigmoid(b_pre)
 *     o         = KDA(q, k, v, alpha, beta)                      Eq. 1, with `scale` on q
 *     y         = sigmoid(g_o) . RMSNorm(o) . rms_weight         o / sqrt(mean o^2 + rms_eps), over dv
 *
 * The normalisation, the decay function and the sigmoid of beta are computed inside the
 * intra-chunk kernel from the half-precision pre-activations (no fp32 gate tensor and no
 * normalised copy of q and k ever exists in memory).  The output stage runs inside the inter-chunk
 * kernel: the CTAs that hold the column slices of one (sequence, head) are launched as a thread-block
 * cluster and exchange each row's sums of squares through distributed shared memory.  Where the
 * device cannot keep as many clusters resident as the call has work for (or after
 * kda_layer_set_fused_output(0)), the stage runs as a separate pass over the bf16 output, in place;
 * the results of the two forms differ by rounding only (the separate pass normalises the rounded
 * bf16 output).
 *
 *   q_c, k_c, g_a [T_total,H,dk], v, g_o, y [T_total,H,dv]   bf16 device
 *   b_pre [T_total,H]                                        fp32 device
 *   A_log [H], dt_bias [H,dk], rms_weight [dv]               fp32 device
 *   S0, S_T, cu_seqlens_dev, cu_seqlens_host, n_seqs, total_tokens, H, scale: as in kda_chunk_fwd;
 *   y may be NULL (final state only; q_c, g_o, rms_weight are then unused)
 *   workspace: as for kda_chunk_fwd with dt = KDA_BF16, at least kda_layer_fwd_min_workspace_bytes
 *              (the call always runs the two-kernel schedule, in several passes if need be).
 * Only dk = dv = 128 and chunk = 64.  Asynchronous; nothing is allocated; errors and the status
 * word as for kda_chunk_fwd.
 */
/* Process-wide switch (default 1): 0 makes kda_layer_fwd always run its output stage as a pass of its own. */
kda_status_t kda_layer_set_fused_output(int on);
size_t kda_layer_fwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk);
size_t kda_layer_fwd_min_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk);
kda_status_t kda_layer_fwd(const void *q_c, const void *k_c, const void *v, const void *g_a,
                           const float *b_pre, const void *g_o, const float *A_log,
                           const float *dt_bias, const float *rms_weight, float l2_eps, float rms_eps,
                           const float *S0, void *y, float *S_T, const int32_t *cu_seqlens_dev,
                           const int32_t *cu_seqlens_host, int n_seqs, int64_t total_tokens, int H,
                           int dk, int dv, int chunk, float scale, void *workspace,
                           size_t workspace_bytes, void *cuda_stream);

/*
 * Decode step of the layer wrap: kda_decode_step with the same element-wise stages as kda_layer_fwd
 * (L2Norm of q_c and k_c, the decay function on g_a, sigmoid on b_pre, head-wise RMSNorm and sigmoid
 * output gate on the output row) computed inside the decode kernel; one token per sequence.
 *
 *   q_c, k_c, g_a [n_seqs,H,dk], v, g_o, y [n_seqs,H,dv]   bf16 device;  b_pre [n_seqs,H] fp32 device
 *   A_log [H], dt_bias [H,dk], rms_weight [dv]              fp32 device
 *   S, state_slot, scale                                    as in kda_decode_step (state in place)
 * Only dk = dv = 128.  Asynchronous on `cuda_stream`; errors as for kda_decode_step.
 */
kda_status_t kda_layer_decode_step(const void *q_c, const void *k_c, const void *v, const void *g_a,
                                   const float *b_pre, const void *g_o, const float *A_log,
                                   const float *dt_bias, const float *rms_weight, float l2_eps,
                                   float rms_eps, float *S, const int32_t *state_slot, void *y,
                                   int n_seqs, int H, int dk, int dv, float scale, void *cuda_stream);

/*
 * Backward pass of kda_chunk_fwd: gradients of Eq. 1 (the operator is trained end to end, Section 5;
 * the paper prints no backward algorithm, so this is the adjoint of Eq. 1 itself).  For
 *
 *     L = sum_t <d_o_t, o_t> + <dS_T, S_T>
 *
 * it returns dL/dq, dL/dk, dL/dv, dL/dlog_alpha, dL/dbeta and dL/dS0.  The forward pass is
 * recomputed inside (nothing has to be kept from kda_chunk_fwd): a first sweep stores the state at
 * the start of every block of 8 tokens, a reverse sweep recomputes one block at a time (in shared
 * memory) and runs the adjoint through
 * it token by token; fp32 arithmetic throughout.
 *
 *   q, k [T_total,H,dk], v, d_o [T_total,H,dv]   device, element type `dt` (KDA_F32 or KDA_BF16)
 *   log_alpha [T_total,H,dk], beta [T_total,H]   fp32 device
 *   S0, dS_T  [n_seqs,H,dk,dv] fp32 device or NULL (= zeros);  d_o may be NULL (= zeros)
 *   dq, dk, dlog_alpha [T_total,H,dk], dv [T_total,H,dv], dbeta [T_total,H]   fp32 device, written
 *   dS0 [n_seqs,H,dk,dv] fp32 device, written, or NULL
 *   cu_seqlens_dev / cu_seqlens_host, n_seqs, total_tokens, H, scale: as in kda_chunk_fwd
 *   workspace: device memory, 256-byte aligned, at least kda_chunk_bwd_workspace_bytes(...) (chunk
 *              states at the start of every block of 8 tokens and the
 *              per-slice shares of the gradients that are summed over dv; about 0.45 MB per token
 *              at H = 32).  Its first 256 bytes hold the status word that kda_check_status reads.
 * Only dk = dv = 128 and chunk = 64.  Asynchronous on `cuda_stream`; nothing is allocated; results
 * are deterministic (fixed summation order).  Errors: KDA_ERR_INVALID_ARG, KDA_ERR_UNSUPPORTED,
 * KDA_ERR_WORKSPACE, KDA_ERR_CUDA.
 */
size_t kda_chunk_bwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv, int chunk);
kda_status_t kda_chunk_bwd(const void *q, const void *k, const void *v, const float *log_alpha,
                           const float *beta, const float *S0, const void *d_o, const float *dS_T,
                           float *dq, float *dk_out, float *dv_out, float *dlog_alpha, float *dbeta,
                           float *dS0, const int32_t *cu_seqlens_dev, const int32_t *cu_seqlens_host,
                           int n_seqs, int64_t total_tokens, int H, int dk, int dv, int chunk,
                           float scale, kda_dtype_t dt, void *workspace, size_t workspace_bytes,
                           void *cuda_stream);

/*
 * Comparison workload: chunkwise forward of the GENERAL diagonal-plus-low-rank recurrence (paper
 * Section 6.1 "Relation to DPLR" and its chunkwise DPLR pseudo-code; the kernel-time comparison of
 * Section 3.2), per sequence and head:
 *
 *     S_t = (Diag(exp(g_t)) + b_t a_t^T) S_{t-1} + k_t v_t^T ,      o_t = scale * S_t^T q_t
 *
 * (a_t is contracted with the state the previous token left; with a = alpha . k, b = -beta k and
 * the key beta k this is Eq. 1).  fp32 storage and arithmetic only, in the same two-kernel FMA
 * style as kda_chunk_fwd with dt = KDA_F32, so that the two run times compare like with like.
 *
 *   q, k, a, b, g  [T_total, H, dk] fp32 device;  v, o [T_total, H, dv] fp32 device
 *   S0, S_T, cu_seqlens_dev, cu_seqlens_host, n_seqs, total_tokens, H, scale: as in kda_chunk_fwd
 *   workspace: device memory, 256-byte aligned, at least ..._min_workspace_bytes (the call then
 *              walks the chunks in several passes); ..._workspace_bytes gives room for one pass.
 *              Its first 256 bytes hold the status word that kda_check_status reads.
 * Only dk = dv = 128 and chunk = 64.  Asynchronous on `cuda_stream`; nothing is allocated.  Errors
 * as for kda_chunk_fwd (KDA_ERR_INVALID_ARG, KDA_ERR_UNSUPPORTED, KDA_ERR_WORKSPACE, KDA_ERR_CUDA);
 * a channel that decays by more than e^-160 inside one chunk raises the KDA_ERR_GATE_RANGE flag.
 */
size_t kda_dplr_chunk_fwd_min_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                              int chunk);
size_t kda_dplr_chunk_fwd_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                          int chunk);
kda_status_t kda_dplr_chunk_fwd(const float *q, const float *k, const float *v, const float *a,
                                const float *b, const float *g, const float *S0, float *o,
                                float *S_T, const int32_t *cu_seqlens_dev,
                                const int32_t *cu_seqlens_host, int n_seqs, int64_t total_tokens,
                                int H, int dk, int dv, int chunk, float scale, void *workspace,
                                size_t workspace_bytes, void *cuda_stream);

/*
 * Chooses how kda_chunk_fwd schedules a bf16 call (process-wide; no counterpart in the paper).
 *   0  automatic (default): when the workspace has room for every (chunk, head) tile of the call,
 *      the intra-chunk stage (Section 3.1: gates, UT transform) runs as one kernel and the
 *      inter-chunk stage (state and output equations) as a second one; with a smaller workspace
 *      one fused cooperative kernel runs both stages at once and hands the tiles over through a
 *      ring of a few tiles per (sequence, head) that stays in the L2 cache.
 *   1  always the two kernels (a small workspace then makes the call walk the chunks in passes)
 *   2  always the fused kernel
 * All three give the same results up to the rounding of the chunk states' bf16 operand copies
 * (identical arithmetic per tile).  Returns KDA_ERR_INVALID_ARG for any other mode.
 */
kda_status_t kda_set_chunk_path(int mode);

/*
 * Recurrent decode step (Eq. 1 for one token per sequence).
 *
 *   q, k, log_alpha  [n_seqs,H,dk]   v, o  [n_seqs,H,dv]   beta  [n_seqs,H]
 *   S           [n_slots,H,dk,dv] fp32, read and written IN PLACE
 *   state_slot  [n_seqs] int32 device: sequence n uses S[state_slot[n]]; NULL = identity.  Slots
 *               must be distinct within a call and < n_slots (not checked on the device).
 * Needs no workspace.
 */
kda_status_t kda_decode_step(const void *q, const void *k, const void *v, const float *log_alpha,
                             const float *beta, float *S, const int32_t *state_slot, void *o,
                             int n_seqs, int H, int dk, int dv, float scale, kda_dtype_t dt,
                             void *cuda_stream);

/*
 * Multi-token decode: Eq. 1 for n_tokens (1..64) consecutive tokens of every sequence in one call,
 * e.g. the verification step of speculative decoding or a few tokens appended to a prefill
 * (Section 6.3: generation uses the recurrent kernel; the paper's serving integration is the use
 * case).  The state is read and written once per call, not once per token.
 *
 *   q, k, log_alpha  [n_seqs, n_tokens, H, dk]   v, o  [n_seqs, n_tokens, H, dv]
 *   beta             [n_seqs, n_tokens, H]
 *   S, state_slot    as in kda_decode_step
 * Equivalent to n_tokens calls of kda_decode_step on the tokens in order.
 */
kda_status_t kda_decode_multi(const void *q, const void *k, const void *v, const float *log_alpha,
                              const float *beta, float *S, const int32_t *state_slot, void *o,
                              int n_seqs, int n_tokens, int H, int dk, int dv, float scale,
                              kda_dtype_t dt, void *cuda_stream);

/*
 * Host-buffer variants: same operations with q, k, v, log_alpha, beta, S0 (chunk) and o, S_T read
 * from / written to HOST memory (pinned memory makes the copies asynchronous).  The device copies
 * live in the caller's device workspace, so these allocate nothing either.  cu_seqlens is given on
 * the host only.  For decode the states stay on the device (they are the resident cache);
 * state_slot is a host array or NULL.  Outputs are valid after `cuda_stream` is synchronised.  For
 * one long sequence (n_seqs = 1, at least 1024 tokens) kda_chunk_fwd_host pipelines copy-in,
 * compute and copy-out over up to four segments of the sequence, using two helper streams that the
 * library creates once per process; everything is still ordered after prior work on `cuda_stream`
 * and complete when `cuda_stream` is.
 */
size_t kda_chunk_fwd_host_workspace_bytes(int64_t total_tokens, int n_seqs, int H, int dk, int dv,
                                          int chunk, kda_dtype_t dt);
kda_status_t kda_chunk_fwd_host(const void *q_host, const void *k_host, const void *v_host,
                                const float *log_alpha_host, const float *beta_host,
                                const float *S0_host, void *o_host, float *S_T_host,
                                const int32_t *cu_seqlens_host, int n_seqs, int64_t total_tokens,
                                int H, int dk, int dv, int chunk, float scale, kda_dtype_t dt,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);
size_t kda_decode_step_host_workspace_bytes(int n_seqs, int H, int dk, int dv, kda_dtype_t dt);
kda_status_t kda_decode_step_host(const void *q_host, const void *k_host, const void *v_host,
                                  const float *log_alpha_host, const float *beta_host,
                                  float *S_dev, const int32_t *state_slot_host, void *o_host,
                                  int n_seqs, int H, int dk, int dv, float scale, kda_dtype_t dt,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Reads back (synchronising the stream) the status word that device code sets when one of its
 * bounded waits runs out, and the flag that marks a decay outside the supported range (see the
 * conventions at the top), and clears both.  They live at the start of the workspace passed to
 * kda_chunk_fwd.  Returns KDA_OK, KDA_ERR_TIMEOUT or KDA_ERR_GATE_RANGE (a timeout wins).
 */
kda_status_t kda_check_status(void *workspace, void *cuda_stream);

/*
 * Self-test of the bounded-wait mechanism every tensor-core kernel of this library relies on (no
 * counterpart in the paper).  Launches one warp that waits, for at most limit_ms (1..1000), on a
 * barrier that nothing ever completes; the wait must give up and record KDA_ERR_TIMEOUT in the
 * status word at the start of `workspace` (>= 256 bytes, device), which kda_check_status then
 * reports.  The CUDA context stays usable.
 */
kda_status_t kda_selftest_wait_timeout(void *workspace, int limit_ms, void *cuda_stream);

/*
 * Optional per-kernel timing for benchmarks.  While enabled, every kernel launch of this library
 * is bracketed by CUDA events on the launching stream (at most 8192 launches are recorded; enabling
 * resets the record).  kda_profile_read synchronises the device and returns the summed duration and
 * the launch count of one kernel kind: 0 = prologue, 1 = intra-chunk, 2 = inter-chunk, 3 = decode.
 */
void kda_profile_enable(int on);
kda_status_t kda_profile_read(int kind, double *total_ms, int *launches);

/*
 * Self-test of the table in which the library keeps what it caches per device (SM count, kernel
 * attributes already set, helper streams), one slot per device ordinal behind a mutex; no CUDA call
 * is made, so it runs on a machine without a GPU.  Returns 0 when the table behaves (no counterpart
 * in the paper).
 */
int kda_selftest_device_table(void);

/*
 * The schedule that the fused bf16 prefill kernel of kda_chunk_fwd would use for a batch whose
 * sequence n has chunks_per_seq[n] chunks (HOST array of n_seqs entries), with H heads, room for
 * avail_tiles tiles in the workspace and n_sm multiprocessors: out[0] = Q, the (sequence, head)
 * chains that run side by side in one round; out[1] = R, the tiles per chain that the intra-chunk
 * stage (Section 3.1, the WY / UT part) may run ahead of the state recurrence; out[2] = rounds;
 * out[3] = production indices handed out in total (a round takes its longest chain times its number
 * of chains).  Host arithmetic only: no CUDA call, runs without a GPU.  Returns 0, or 1 on a bad
 * argument; Q = 0 in out[] means that no schedule exists (fewer than two tiles, or too few SMs).
 */
int kda_selftest_fused_plan(const int32_t *chunks_per_seq, int n_seqs, int H, int64_t avail_tiles,
                            int n_sm, int64_t out[4]);

/*
 * Upper bound, in nanoseconds, of every wait inside the tensor-core kernels (on a barrier, a flag or
 * a peer CTA); a wait that runs out makes its kernel return with KDA_ERR_TIMEOUT in the status word.
 * Default 1 s; the environment variable KDA_WAIT_LIMIT_MS (1 .. 600000), read once per process,
 * overrides it.  No counterpart in the paper.
 */
uint64_t kda_wait_limit_ns(void);

/* Description of the calling thread's last error ("" if none); static storage, never NULL. */
const char *kda_last_error(void);

/* Number of kernel launches issued by this library in the calling process (for accounting). */
uint64_t kda_launch_count(void);

/* Library build tag, e.g. "kda-b200 sm_100a". */
const char *kda_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KDA_H_ */
