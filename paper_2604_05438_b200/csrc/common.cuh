// Shared declarations of the libtkphi kernels: problem description, workspace
// layout, small device helpers.  sm_100a only.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <stddef.h>

namespace tkphi {

constexpr int kHistBits = 12;                 // leading bits of the ordered score key
constexpr int kHistBins = 1 << kHistBits;     // bins of the fused first-pass histogram
constexpr int kLowBits = 32 - kHistBits;      // bits refined inside the threshold bin
constexpr int kMaxBatch = 1024;               // sequences per call
constexpr int kSlice = 128;                   // exact-support tokens per CTA of the exact/residual kernel (= MMA M)
constexpr float kLog2e = 1.4426950408889634f;

// Device status word values (first word of the workspace).
constexpr int kStatusOk = 0;
constexpr int kStatusTimeout = -5;

// Device pointers of one side's ReZero-MLP feature maps (App. C.2); w_s == nullptr: not used.
struct MlpParams {
  int d_emb;
  const float* w_s; const float* b_s;      // [heads][d_emb][head_dim], [heads][d_emb]
  const float* w_1; const float* b_1;      // [heads][d_emb][d_emb],   [heads][d_emb]
  const float* w_2; const float* b_2;
  const float* alpha;                      // [heads]
  const float* w_o; const float* b_o;      // [heads][n_feat][d_emb],  [heads][n_feat]
};

// Everything the kernels need to know about one layer call.
struct Problem {
  int batch, n_q_heads, n_kv_heads, head_dim, n_feat, n_sink, n_tail, group;
  const int* n_tail_seq;           // device [batch] per-sequence tail-anchor counts, or null: n_tail for all
  const long long* cu_seqlens;     // device [batch+1]
  const int* topk;                 // device [batch] (null for the build)
  int topk_max;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  long long stride_head, stride_token;   // elements
  const __nv_bfloat16* q;          // [batch][n_q_heads][head_dim]
  // feature maps
  const float* w_q; const float* b_q; const float* w_k; const float* b_k;
  float gamma_q, gamma_k;
  MlpParams mlp_q;                 // query-side MLP maps (mlp_q.w_s != nullptr: used instead of w_q, b_q, gamma_q)
  float* mlp_vec;                  // their per-row layer outputs: [rows][g0 (E) | h (E) | g1 (E) | log phi_q (r)]
  // cached key features (optional): phi_k rows [n_kv_heads][total_tokens][n_feat], and where the
  // decode step keeps z_i = <phi_q, phi_k(k_i)> / exp(m_q) of the retrieved tokens: [rows][topk_max]
  const float* phi_cache; long long total_tokens;
  float* zbuf;                     // null: the features of the retrieved keys are recomputed
  // summaries
  const float* S; const float* u;
  // row gather of the exact support through 2-D tensor maps over the k and v caches:
  // gather_mode 0: row = kv head * gather_ratio + cache row; 1: row = cache row * gather_ratio + kv head;
  // -1: the cache strides do not form a 2-D tensor, rows are gathered with 16-byte copies
  int gather_mode; long long gather_ratio; long long gather_rows;
  // outputs
  int* idx_out; float* y_out; float* dbg_out;
  unsigned flags;
  int with_phi;                    // 0: selection-only, 1: Top-K+phi
  // workspace pieces (device pointers)
  int* status;                     // first word of the workspace
  size_t zero_bytes;               // head of the workspace that must be zero before the selection kernels
  unsigned* row_counter;           // [batch*n_q_heads]
  float* scores;                   // [n_q_heads * total_tokens]
  __nv_bfloat16* wk_img;           // [n_kv_heads][2][r*d] W_k split into bf16 hi / lo, stored as MMA operand tiles
  int* idx;                        // [rows][topk_max] ascending retrieved positions
  float* aq;                       // [rows][aq_stride]: w = exp(a_q - m_q), m_q, w.u_M, S_M w, log2 w
  float* partials;                 // [rows][max_slices][partial_stride]
  int max_slices, partial_stride;
  float scale;                     // 1/sqrt(head_dim)
};

struct BuildProblem {
  int batch, n_kv_heads, head_dim, n_feat, n_sink, n_tail;
  const int* n_tail_seq;           // as in Problem
  const long long* cu_seqlens;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  long long stride_head, stride_token;
  const float* w_k; const float* b_k; float gamma_k;
  float* phi_cache;                // optional: phi_k rows of the mid-region tokens are also written here ...
  int from_cache;                  // ... or, if set, read from here instead of being computed
  long long total_tokens;
  float* S; float* u;
  int* status;
  float* partials;                 // [units][chunks_per_unit][d*r + r]
  int chunks_per_unit;             // upper bound over sequences
};

// Host-side byte offsets of the workspace pieces.
struct WsLayout {
  size_t status, row_counter, zero_end;
  size_t scores, wk_img, idx, aq, partials, zbuf, mlp_vec, total;
  int max_slices, partial_stride;
  // build
  size_t b_partials; int chunks_per_unit;
};

// Row length of Problem::aq: [0, r) w; [r] m_q; [r+1] w.u_M; [r+4, r+4+d) S_M w; [r+4+d, 2r+4+d) log2 w.
__host__ __device__ inline int aq_stride(int r, int d) { return 2 * r + d + 4; }
__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// keys per TMA tile of the scoring kernel (32 KB of bf16 rows)
__host__ __device__ inline int score_tile_keys(int head_dim) { return head_dim == 64 ? 256 : 128; }

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ int mid_len(long long n, int n_sink, int n_tail) {
  long long m = n - n_sink - n_tail;
  return m > 0 ? (int)m : 0;
}
// Tail-anchor count of sequence b (P: Problem or BuildProblem).
template <typename P>
__device__ __forceinline__ int tail_of(const P& p, int b) {
  return p.n_tail_seq ? __ldg(p.n_tail_seq + b) : p.n_tail;
}

// Order-preserving map from fp32 to uint32: larger float <=> larger key.
__device__ __forceinline__ unsigned ordered_key(float f) {
  unsigned u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float bf16_lo(unsigned packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(unsigned packed) { return __uint_as_float(packed & 0xffff0000u); }

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ int warp_sum_int(int x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// Exclusive prefix sum of one int per thread over the block; returns the
// exclusive prefix, *total gets the block sum.  `scratch` holds >= 33 ints.
// All threads of the block must call it; blockDim.x is a multiple of 32, <= 1024.
__device__ __forceinline__ int block_exclusive_scan(int x, int* scratch, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  int incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();                     // scratch may still be in use by a previous scan
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = lane < nwarp ? scratch[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    scratch[lane] = wi - w;            // exclusive prefix of warp sums
    if (lane == 31) scratch[32] = wi;
  }
  __syncthreads();
  int res = scratch[warp] + incl - x;
  *total = scratch[32];
  return res;
}

// Offsets that follow from cu_seqlens alone (no per-call prefix arrays needed):
// the score row of (b, hq) starts at element H_q*cu[b] + hq*L_b.
__device__ __forceinline__ long long score_row_base(const Problem& p, int b, int hq, long long cu_b, long long len_b) {
  return (long long)p.n_q_heads * cu_b + (long long)hq * len_b;
}
// Launch with programmatic stream serialization: the kernel may begin (up to its
// pdl_wait()) while the previous kernel of the stream is still finishing.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---------------------------------------------------------------- per-device host state
// A process may drive several GPUs: what is configured or queried per device is kept per
// device ordinal of the calling thread's current device.
constexpr int kMaxDevices = 64;
struct PerDeviceFlag { bool done[kMaxDevices] = {}; };
// cudaFuncAttributeMaxDynamicSharedMemorySize of `kernel`, set once on the current device.
cudaError_t set_max_dynamic_smem(PerDeviceFlag& flag, const void* kernel, size_t bytes);
// Multiprocessor count of the current device (148 if it cannot be read).
int sm_count_current_device();

// ---------------------------------------------------------------- host launchers
// Each returns cudaGetLastError() after enqueuing on `stream`.
cudaError_t launch_score(const Problem& p, const CUtensorMap& tmap_k, int n_sm, cudaStream_t stream);
cudaError_t launch_select(const Problem& p, int max_mid, int n_sm, cudaStream_t stream);
cudaError_t launch_exact_residual(const Problem& p, const CUtensorMap& gk, const CUtensorMap& gv, long long n_pairs, int n_sm,
                                  cudaStream_t stream);
cudaError_t launch_cached_z(const Problem& p, cudaStream_t stream);
cudaError_t launch_mlp_query(const Problem& p, cudaStream_t stream);

// One dense layer of the MLP feature map on the tensor cores (mlp_features.cu):
// out[h][m][n] = epilogue(sum_k A[h][m][k] W[h][n][k] + bias[h][n]).
enum { kEpiBias = 0, kEpiGelu = 1, kEpiResidual = 2, kEpiExp = 3 };
struct GemmArgs {
  int M, N, K, heads;                  // rows, output columns, reduction length (K a multiple of 64), matrix sets
  int epi;
  const float* bias;                   // [heads][N]
  const float* alpha;                  // [heads] (kEpiResidual)
  const __nv_bfloat16* resid;          // [heads][M][N] (kEpiResidual): out = resid + alpha (acc + bias)
  void* out;                           // bf16 [heads][M][N], or fp32 for kEpiExp
  long long out_head_stride;           // elements between heads of out (and of resid)
  int* status;
};
// Output columns per tile of the MLP GEMM kernel (also the row count of the weight tensor map's box).
inline int mlp_gemm_bn(int N) { return N % 256 == 0 ? 256 : N % 128 == 0 ? 128 : N == 64 ? 64 : 0; }
cudaError_t launch_mlp_gemm(const CUtensorMap& map_a, const CUtensorMap& map_w, const GemmArgs& g, cudaStream_t stream);
cudaError_t launch_f32_to_bf16(const float* src, __nv_bfloat16* dst, size_t n, cudaStream_t stream);
cudaError_t launch_build(const BuildProblem& p, const CUtensorMap& tmap_k, const CUtensorMap& tmap_v, cudaStream_t stream);

}  // namespace tkphi
