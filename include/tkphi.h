/*
 * tkphi.h -- C ABI of libtkphi: decode-step Top-K+phi residual-mass attention
 * and its prefill summary build, as hand-written CUDA kernels for sm_100a.
 *
 * Method (arXiv 2604.05438, "Residual-Mass Accounting for Partial-KV Decoding"):
 * for one attention layer and each decode query head the library
 *   (1) scores the query against every mid-region key, s_i = q.k_i / sqrt(d_h)
 *       (Sec. 3, Eq. full_attention), and selects the K highest-scoring
 *       mid-region indices K(q) (exhaustive Top-K control selector, Sec. 5.1);
 *   (2) forms the exact unnormalised terms nu_E, Z_E over E = A U K(q), A the
 *       sink/tail anchors (Sec. 3, Eq. partition and Eq. exact_terms);
 *   (3) removes the retrieved tokens' feature contributions from the prefill
 *       summaries (S, u) (Sec. 4.2, Eq. subtraction);
 *   (4) evaluates the residual estimate nu_hat_R = S_R phi_q(q),
 *       Z_hat_R = phi_q(q)^T u_R (Sec. 4.3);
 *   (5) returns y = (nu_E + nu_hat_R) / (Z_E + Z_hat_R) (Sec. 4.3, Eq. hybrid_merge).
 * The prefill pass builds S = sum_{i in M} v_i phi_k(k_i)^T, u = sum_{i in M} phi_k(k_i)
 * over the mid-region M (Sec. 4.1, Eq. natural_cache).
 *
 * Feature maps: phi(x) = exp(W x + b - gamma ||x||^2) elementwise, W in R^{r x d};
 * one map per query head (phi_q) and one per KV head (phi_k) (Sec. 4.1; positivity
 * by exponentiation, App. C.1).
 *
 * General rules
 *  - Every tensor pointer is a DEVICE pointer unless its comment says "host".
 *    The caller owns all memory; the library allocates nothing, keeps nothing
 *    between calls, and enqueues its work on the caller's stream (a
 *    cudaStream_t passed as void*; NULL is the default stream).
 *  - Functions return after enqueuing.  The return value reports host-side
 *    validation and launch errors only; invalid arguments are rejected before
 *    anything is launched.  tkphi_last_error() gives a message for the last
 *    failing call of the calling thread.
 *  - Small per-sequence arrays (cu_seqlens, topk) are passed twice: a host copy
 *    (validated, used for sizing) and a device copy with the same contents (read
 *    by the kernels), so that no call needs a device-to-host synchronisation.
 *  - Inputs must be finite.  Results for NaN/Inf inputs are unspecified.
 *  - One call processes one attention layer; a model stack is a host loop.
 */
#ifndef TKPHI_H
#define TKPHI_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TKPHI_OK = 0,
  TKPHI_ERR_INVALID_ARG = -1,  /* bad pointer, size, stride or range */
  TKPHI_ERR_UNSUPPORTED = -2,  /* legal problem the library has no kernel for */
  TKPHI_ERR_WORKSPACE = -3,    /* workspace NULL, misaligned or too small */
  TKPHI_ERR_CUDA = -4,         /* a CUDA runtime/driver call failed */
  TKPHI_ERR_TIMEOUT = -5       /* a bounded device-side wait ran out (see tkphi_device_status) */
} tkphi_status;

/* Which entry point a workspace is sized for. */
enum { TKPHI_WS_BUILD = 0, TKPHI_WS_TOPK_DECODE = 1, TKPHI_WS_DECODE_STEP = 2, TKPHI_WS_MLP_KEY_FEATURES = 3 };

/* Flags of tkphi_decode_step. */
enum {
  TKPHI_FLAG_NONE = 0,
  TKPHI_FLAG_NOSUB = 1 /* skip the retrieved-token subtraction (the paper's NoSub ablation, Sec. 5.1) */
};

/*
 * One attention layer's K/V cache for `batch` ragged sequences (Sec. 3: keys and
 * values (k_i, v_i), i < L, per KV head).  Sequence b owns cache rows
 * cu_seqlens[b] .. cu_seqlens[b+1]-1; its prefill length is L_b = cu_seqlens[b+1]
 * - cu_seqlens[b] >= 1.  Element (head h, row t, dim c) of k is at
 * k + h*kv_stride_head + t*kv_stride_token + c (in bf16 elements); v uses the
 * same strides.  Requirements: 1 <= batch <= 1024; head_dim in {64, 128}; n_q_heads a multiple of
 * n_kv_heads with group size <= 8; n_feat in {64, 128}; k and v 16-byte aligned;
 * both strides multiples of 8 elements; kv_stride_token >= head_dim; total rows
 * < 2^31; at most 2,097,152 mid-region rows per sequence for the decode entry points.
 * With more than one KV head the heads must not share memory: either kv_stride_head >=
 * rows * kv_stride_token (head-major) or kv_stride_head >= head_dim and kv_stride_token >=
 * (n_kv_heads - 1) * kv_stride_head + head_dim (token-major); anything else, a zero head
 * stride included, is TKPHI_ERR_INVALID_ARG.
 * Query head h_q uses KV head h_q / (n_q_heads / n_kv_heads).
 * Any strides within these rules work.  Head-major caches (kv_stride_head a multiple of
 * kv_stride_token) and token-major ones (kv_stride_token a multiple of kv_stride_head) also
 * let the decode entry points fetch the rows of the exact support by TMA row gathers, which
 * calls with many retrieved rows (more 256-token pieces of support lists than SMs) use.
 * Anchors (Eq. partition): the first n_sink and the last n_tail rows of each
 * sequence (their union when L_b < n_sink + n_tail); the mid-region is what lies
 * between, |M_b| = max(0, L_b - n_sink - n_tail).
 * n_tail_seq_host / n_tail_seq_dev (optional; both NULL or both given, the same [batch]
 * values >= 0 on the host and on the device) give every sequence a tail-anchor count of its
 * own, which then replaces n_tail everywhere: sequences that have generated different
 * numbers of tokens share a decode call this way (see tkphi_decode_step).
 */
typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim;
  int32_t n_feat;                 /* r = d_phi */
  int32_t n_sink, n_tail;         /* >= 0 */
  const int64_t* cu_seqlens_host; /* host,   [batch+1], cu[0] = 0, non-decreasing */
  const int64_t* cu_seqlens_dev;  /* device, same contents */
  const void* k;                  /* device, bf16 */
  const void* v;                  /* device, bf16 */
  int64_t kv_stride_head, kv_stride_token; /* in elements */
  const int32_t* n_tail_seq_host; /* host,   [batch] or NULL */
  const int32_t* n_tail_seq_dev;  /* device, [batch] or NULL */
} tkphi_kv_desc;

/* phi(x) = exp(W x + b - gamma ||x||^2); row-major fp32 parameters on the device; w_q and
 * w_k 16-byte aligned (as are S and u where a call takes them).
 *
 * phi_k_cache (optional, NULL to leave out) is the cached-feature variant that Sec. 4.2
 * names as a way to avoid recomputing the retrieved keys' feature maps at decode time:
 * device fp32 [n_kv_heads][T_total][n_feat], T_total = cu_seqlens[batch], 16-byte aligned,
 * owned by the caller.  tkphi_build_summaries, given a non-NULL pointer, also writes
 * phi_k(k_i) of every mid-region token i of every sequence to row cu_seqlens[b] + i of each
 * KV head (rows of anchor tokens are left untouched).  tkphi_decode_step, given a non-NULL
 * pointer, takes the retrieved tokens' feature rows from it instead of recomputing them from
 * the keys (Eq. subtraction is unchanged: the same phi_k(k_i) enter it); the rows must hold
 * what the build wrote for the same cache, anchors and parameters (w_k, b_k and gamma_k are
 * then not read by the decode step).  tkphi_topk_decode and the NoSub flag ignore it. */
typedef struct {
  const float* w_q; /* [n_q_heads][n_feat][head_dim] */
  const float* b_q; /* [n_q_heads][n_feat] */
  const float* w_k; /* [n_kv_heads][n_feat][head_dim] */
  const float* b_k; /* [n_kv_heads][n_feat] */
  float gamma_q, gamma_k;
  float* phi_k_cache; /* optional, [n_kv_heads][T_total][n_feat] */
} tkphi_phi_desc;

/*
 * Bytes of workspace the given entry point needs for this problem (0 on invalid
 * arguments; tkphi_last_error() then says why).  topk_host (host, [batch]) may be
 * NULL for TKPHI_WS_BUILD.  The workspace must be 256-byte aligned device memory.
 * Its contents on entry do not matter and are undefined on exit.
 */
size_t tkphi_workspace_bytes(const tkphi_kv_desc* kv, const int32_t* topk_host,
                             int32_t topk_max, int which);

/*
 * Prefill summary build (Sec. 4.1, Eq. natural_cache): for every sequence b and KV
 * head h, S[b][h] = sum_{i in M_b} v_i phi_k(k_i)^T (row-major [head_dim][n_feat],
 * fp32) and u[b][h] = sum_{i in M_b} phi_k(k_i) ([n_feat], fp32); both zero when the
 * mid-region is empty.  Only phi->w_k, b_k and gamma_k are read.
 * S: [batch][n_kv_heads][head_dim][n_feat], u: [batch][n_kv_heads][n_feat], written in full.
 */
tkphi_status tkphi_build_summaries(const tkphi_kv_desc* kv, const tkphi_phi_desc* phi,
                                   float* S, float* u,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Prefill summary build without any caller-provided workspace (the paper has no
 * counterpart; this serves a deployment constraint).  Some callers cannot obtain
 * device memory at call time: plug-ins of a serving process whose memory pool is sized
 * and handed out once at start-up, runtimes that forbid cudaMalloc (an implicit
 * device-wide synchronisation) on the latency-critical path, and hosts whose policy
 * allows allocation only during initialisation.  For them this entry point
 * computes exactly what tkphi_build_summaries computes, on the same kernel, but takes
 * its scratch from a fixed array of TKPHI_STATIC_SCRATCH_BYTES that is part of the
 * library's device image.  It calls no allocating routine of CUDA or of any library.
 *  - Limit: problems whose tkphi_workspace_bytes(kv, NULL, 0, TKPHI_WS_BUILD) exceeds
 *    TKPHI_STATIC_SCRATCH_BYTES are rejected with TKPHI_ERR_WORKSPACE before anything
 *    is enqueued (the message names both sizes); use tkphi_build_summaries for those.
 *  - Cost: the array is part of the library's device code.  Every GPU on which that code
 *    is loaded holds the array until the process exits.  The CUDA runtime loads it on a
 *    device when the library is first used there (at the latest by this function's first
 *    call on the device, which therefore is also where the device's free memory drops by
 *    the array's size).
 *  - First call on each device: looks up the array's device address (a host-side
 *    runtime query, done with that device current and cached).  Make that first call
 *    at initialisation, before any stream capture begins on the device.
 *  - Sharing: all calls on a device use the same array.  The array keeps the previous
 *    call's contents; the build needs none of it cleared (the kernel sets the status word
 *    at the head of the array itself and overwrites every partial sum before it is read).
 *    Two calls whose GPU work overlaps (different streams, or different host threads)
 *    race on it and give undefined results: serialise them.
 *  - Device-side errors: tkphi_static_device_status reads the status word of the last
 *    static call on the current device (the array's address is not exposed, so
 *    tkphi_device_status cannot be used): 0, or TKPHI_ERR_TIMEOUT if a bounded wait of the
 *    build kernel ran out, in which case (S, u) are not valid.  Waits for the stream;
 *    *status_out is a host int.  TKPHI_ERR_INVALID_ARG if no static call has been made on
 *    the device yet.
 * Arguments, outputs and error reporting otherwise as for tkphi_build_summaries;
 * tkphi_static_last_error() gives the message of the last failing call of the thread.
 */
#define TKPHI_STATIC_SCRATCH_BYTES (8u << 20)
tkphi_status tkphi_build_summaries_static(const tkphi_kv_desc* kv, const tkphi_phi_desc* phi,
                                          float* S, float* u, void* cuda_stream);
tkphi_status tkphi_static_device_status(void* cuda_stream, int32_t* status_out);
const char* tkphi_static_last_error(void);

/*
 * Selection-only Top-K decode (Sec. 3, Eq. exact_terms and y_TopK = nu_E / Z_E), steps
 * (1)-(2) above.
 *   q         bf16 [batch][n_q_heads][head_dim], one decode query per sequence and head.
 *   topk_host host int32 [batch]; topk_dev device copy.  0 <= topk[b] <= |M_b|
 *             (larger is TKPHI_ERR_INVALID_ARG); topk_max >= max_b topk[b].
 *   idx_out   int32 [batch][n_q_heads][topk_max] or NULL: the retrieved positions
 *             within the sequence (n_sink <= i < L_b - n_tail), ascending, padded
 *             with -1.  Equal scores are broken towards the lower index.
 *   y_out     fp32 [batch][n_q_heads][head_dim].
 * A sequence needs at least one anchor or one retrieved token (else INVALID_ARG).
 */
tkphi_status tkphi_topk_decode(const tkphi_kv_desc* kv, const void* q,
                               const int32_t* topk_host, const int32_t* topk_dev, int32_t topk_max,
                               int32_t* idx_out, float* y_out,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Length of one dbg_out row of tkphi_decode_step for a given head_dim. */
#define TKPHI_DBG_STRIDE(head_dim) (4 + (head_dim))

/*
 * Top-K+phi decode step (Sec. 4.2-4.3), steps (1)-(5) above, for summaries (S, u)
 * laid out as tkphi_build_summaries writes them.
 *   dbg_out   fp32 [batch][n_q_heads][TKPHI_DBG_STRIDE(head_dim)] or NULL.  Per query
 *             head: [0] m_E = max_{i in E} s_i, [1] sum_{i in E} exp(s_i - m_E),
 *             [2] log Z_hat_R (-inf when the residual was clamped away), [3] the
 *             common log-scale of the merge, [4..] nu_hat_R / Z_hat_R (zeros when clamped).
 *   flags     TKPHI_FLAG_*.
 * Clamp: a residual denominator Z_hat_R <= 0 (a finite-precision artefact of the
 * subtraction, App. C.1) drops both residual terms, so y falls back to nu_E / Z_E.
 * With no anchor and no retrieved token the output is nu_hat_R / Z_hat_R; if that is
 * clamped as well the output row is zero.
 * Generated tokens (Sec. 4.3, Eq. implemented_decode: tokens produced after the prefill
 * stay in the exact branch): append their rows to the cache and pass n_tail + n_gen as the
 * tail-anchor count of the decode call; the mid-region, and with it the meaning of (S, u)
 * built at prefill time with n_tail, is unchanged.  Sequences with different n_gen share a
 * call through n_tail_seq (entry b = n_tail + n_gen_b).
 * Other arguments as for tkphi_topk_decode.
 */
tkphi_status tkphi_decode_step(const tkphi_kv_desc* kv, const tkphi_phi_desc* phi, const void* q,
                               const int32_t* topk_host, const int32_t* topk_dev, int32_t topk_max,
                               const float* S, const float* u,
                               int32_t* idx_out, float* y_out, float* dbg_out, uint32_t flags,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The paper's own feature map (App. C.2, "Head-wise phi architecture"): a one-block ReZero MLP of
 * hidden width d_emb per head,
 *   g0 = W_s x + b_s;  Delta = W_2 GeLU(W_1 g0 + b_1) + b_2;  g1 = g0 + alpha Delta;  phi(x) = exp(W_o g1 + b_o),
 * GeLU(t) = t Phi(t) with the normal CDF (erf form).  One descriptor holds the maps of one side:
 * n_heads = n_q_heads for phi_q, n_kv_heads for phi_k.  Row-major fp32 device parameters, every
 * pointer 16-byte aligned; d_emb a multiple of 128, at most 512.
 */
typedef struct {
  int32_t d_emb, n_heads;
  const float* w_s; const float* b_s; /* [n_heads][d_emb][head_dim], [n_heads][d_emb] */
  const float* w_1; const float* b_1; /* [n_heads][d_emb][d_emb],    [n_heads][d_emb] */
  const float* w_2; const float* b_2; /* [n_heads][d_emb][d_emb],    [n_heads][d_emb] */
  const float* alpha;                 /* [n_heads] */
  const float* w_o; const float* b_o; /* [n_heads][n_feat][d_emb],   [n_heads][n_feat] */
} tkphi_mlp_desc;

/*
 * Key features of the MLP map (App. C.2) for a whole cache: phi_k(k_t) of EVERY cache row t of every
 * KV head (anchor rows included) is written to phi_k_cache, fp32 [n_kv_heads][T_total][n_feat]
 * (layout as in tkphi_phi_desc).  The four layers run as tensor-core GEMMs over all tokens with
 * bf16 operands (weights and the activations between the layers are rounded to bf16), fp32
 * accumulation, biases, residual and exponent.  Workspace: tkphi_workspace_bytes(kv, NULL, 0,
 * TKPHI_WS_MLP_KEY_FEATURES).  Feed the cache to tkphi_build_summaries_cached and
 * tkphi_decode_step_mlp.
 */
tkphi_status tkphi_mlp_key_features(const tkphi_kv_desc* kv, const tkphi_mlp_desc* mlp_k, float* phi_k_cache,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Prefill summary build (Sec. 4.1, Eq. natural_cache) from stored key features: S[b][h] = sum_{i in M_b}
 * v_i phi_k(k_i)^T, u[b][h] = sum phi_k(k_i) with phi_k(k_i) read from row cu_seqlens[b] + i of
 * phi_k_cache (as tkphi_mlp_key_features, or tkphi_build_summaries with a cache, wrote it).  kv->k is
 * validated like every descriptor field (a valid device pointer) but its rows are not read.
 * Outputs, workspace (TKPHI_WS_BUILD) and errors as for tkphi_build_summaries.
 */
tkphi_status tkphi_build_summaries_cached(const tkphi_kv_desc* kv, const float* phi_k_cache, float* S, float* u,
                                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Top-K+phi decode step (Sec. 4.2-4.3) with the paper's MLP feature maps (App. C.2): phi_q(q) is
 * evaluated by the library from mlp_q (n_heads = n_q_heads), the retrieved keys' features are taken
 * from phi_k_cache (the MLP is never re-evaluated for keys at decode time).  With TKPHI_FLAG_NOSUB the
 * cache is not read and may be NULL.  Everything else as for tkphi_decode_step; workspace
 * TKPHI_WS_DECODE_STEP.
 */
tkphi_status tkphi_decode_step_mlp(const tkphi_kv_desc* kv, const tkphi_mlp_desc* mlp_q, const float* phi_k_cache,
                                   const void* q, const int32_t* topk_host, const int32_t* topk_dev, int32_t topk_max,
                                   const float* S, const float* u, int32_t* idx_out, float* y_out, float* dbg_out,
                                   uint32_t flags, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Reads the device status word that the kernels of the last call using this
 * workspace set (0 = fine; TKPHI_ERR_TIMEOUT if a bounded wait ran out).  Waits
 * for the stream.  *status_out is a host int.
 */
tkphi_status tkphi_device_status(const void* workspace, void* cuda_stream, int32_t* status_out);

/*
 * Self-test of the error path of the bounded device-side waits (no counterpart in the
 * paper).  Every wait inside the kernels (on a TMA copy, an MMA completion, a hand-off
 * between warps) gives up after a fixed number of polls, raises a flag that makes the
 * other warps of its CTA leave their loops, and the CTA stores TKPHI_ERR_TIMEOUT in the
 * status word at the head of the workspace before it returns.  This entry point runs a
 * one-CTA kernel through exactly that path: one warp waits, with a limit of 4096 polls, on
 * a barrier that nothing ever arrives on, a second warp waits on a barrier the first one
 * would have signalled.  The kernel returns by itself within microseconds; afterwards
 * tkphi_device_status(workspace) reads TKPHI_ERR_TIMEOUT, and the next ordinary call on
 * the same workspace sets the word back to 0.  workspace: device memory, 256-byte
 * aligned, at least 256 bytes.
 */
tkphi_status tkphi_selftest_timeout(void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Optional per-kernel timing for benchmarks (no counterpart in the paper).  While
 * enabled, every launch the library makes is bracketed by CUDA events on the caller's
 * stream (the events are host objects; no device memory is allocated).  Not
 * thread-safe; leave it off in production.  tkphi_kernel_timing_read waits for the
 * recorded events, adds up milliseconds and launch counts per kernel kind into the
 * two host arrays of TKPHI_KERNEL_KINDS entries, and clears the record.
 */
enum {
  TKPHI_KERNEL_SCORE = 0,           /* key scoring (streams the mid-region keys) */
  TKPHI_KERNEL_SELECT = 1,          /* exact Top-K over the score rows; query-side feature work */
  TKPHI_KERNEL_EXACT_RESIDUAL = 2,  /* exact branch, subtraction, residual, merge */
  TKPHI_KERNEL_BUILD = 3,           /* prefill summary build */
  TKPHI_KERNEL_MEMSET = 4,          /* clearing counters when there is nothing to score */
  TKPHI_KERNEL_CACHED_Z = 5,        /* <phi_q, cached phi_k row> of the retrieved tokens (phi_k_cache given) */
  TKPHI_KERNEL_MLP = 6,             /* the layers of the MLP key feature map (weight conversion included) */
  TKPHI_KERNEL_KINDS = 7
};
void tkphi_kernel_timing_enable(int32_t on);
tkphi_status tkphi_kernel_timing_read(float* ms_out, int32_t* count_out);

/* Message for the last error returned on the calling thread ("" if none). */
const char* tkphi_last_error(void);

/* Library version, e.g. 100 for 0.1.0. */
int32_t tkphi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TKPHI_H */
