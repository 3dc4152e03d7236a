// Cached key features at decode time (Sec. 4.2 mentions a cached implementation as a way around
// the retrieved-key feature recompute): when the caller keeps the phi_k rows that the summary build
// wrote, the retrieved tokens' z_i = <phi_q(q), phi_k(k_i)> are plain dot products of those rows
// with w = exp(a_q - m_q) (z_i is carried in units of exp(m_q), like every residual term).
// One warp per retrieved token: the lanes read the row coalesced and reduce in a fixed order.
// The exact/residual kernels then take z_i from the buffer this kernel fills and skip the key
// gather of retrieved tokens, the W_k tiles and the tensor-core recompute.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr int kZThreads = 256;

template <int R>
__global__ void __launch_bounds__(kZThreads) cached_z_kernel(const Problem p) {
  constexpr int LPR = R / 4;                     // lanes per feature row (float4 each): 32 or 16
  constexpr int RPW = 32 / LPR;                  // rows per warp and load
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.y, b = row / p.n_q_heads, hq = row % p.n_q_heads, kvh = hq / p.group;
  pdl_launch_next();
  const int K = p.topk[b];
  const long long cu_b = p.cu_seqlens[b];
  pdl_wait();                                    // the retrieved lists and the query-side features
  const float4 w = __ldcg(reinterpret_cast<const float4*>(p.aq + (size_t)row * aq_stride(R, p.head_dim)) + lane % LPR);
  const float* fbase = p.phi_cache + ((size_t)kvh * p.total_tokens + (size_t)cu_b) * R;
  const int* idx = p.idx + (size_t)row * p.topk_max;
  float* z = p.zbuf + (size_t)row * p.topk_max;
  const int per_block = (kZThreads / 32) * RPW;
  const int stride = gridDim.x * per_block;
  constexpr int U = 4;                           // tokens in flight per warp slot: the index and row loads are latency-bound
  for (int i0 = blockIdx.x * per_block + warp * RPW; i0 < K; i0 += U * stride) {
    int ti[U];
    float acc[U];
#pragma unroll
    for (int n = 0; n < U; ++n) {
      const int i = i0 + n * stride + lane / LPR;
      ti[n] = i < K ? __ldcg(idx + i) : -1;
    }
#pragma unroll
    for (int n = 0; n < U; ++n) {
      acc[n] = 0.f;
      if (ti[n] >= 0) {
        const float4 f = __ldcs(reinterpret_cast<const float4*>(fbase + (size_t)ti[n] * R) + lane % LPR);
        acc[n] = fmaf(w.x, f.x, fmaf(w.y, f.y, fmaf(w.z, f.z, w.w * f.w)));
      }
    }
#pragma unroll
    for (int n = 0; n < U; ++n) {
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) acc[n] += __shfl_xor_sync(0xffffffffu, acc[n], o);
      const int i = i0 + n * stride + lane / LPR;
      if (i < K && lane % LPR == 0) z[i] = acc[n];
    }
  }
}

cudaError_t launch_cached_z(const Problem& p, cudaStream_t st) {
  const int rows = p.batch * p.n_q_heads;
  const int per_block = (kZThreads / 32) * (p.n_feat == 64 ? 2 : 1);
  int bx = (p.topk_max + per_block - 1) / per_block;
  if (bx > 64) bx = 64;
  if (bx < 1) bx = 1;
  if (p.n_feat == 64) return launch_pdl(cached_z_kernel<64>, dim3(bx, rows), dim3(kZThreads), 0, st, p);
  if (p.n_feat == 128) return launch_pdl(cached_z_kernel<128>, dim3(bx, rows), dim3(kZThreads), 0, st, p);
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
