// Prefill summary build (Sec. 4.1, Eq. natural_cache):
//   S = sum_{i in M} v_i phi_k(k_i)^T  (d_v x d_phi),   u = sum_{i in M} phi_k(k_i),
//   phi_k(k) = exp(W_k k + b_k - gamma_k |k|^2).
// CUDA-core fp32 version: each CTA owns a contiguous chunk of the mid-region of one
// (sequence, KV head) unit, keeps its share of S in registers, and writes one
// partial; the last CTA of the unit (atomic ticket) adds the partials in chunk order.
#include "common.cuh"

namespace tkphi {

constexpr int kBuildThreads = 256;
constexpr int kBuildTile = 32;      // tokens per inner tile

template <int D, int R>
struct BuildSmem {
  static constexpr int WT_LD = R + 1;
  static constexpr size_t wt = 0;                                       // float [D][R+1]
  static constexpr size_t kf = wt + sizeof(float) * D * WT_LD;           // float [D][tile]
  static constexpr size_t vf = kf + sizeof(float) * D * kBuildTile;      // float [tile][D]
  static constexpr size_t ph = vf + sizeof(float) * D * kBuildTile;      // float [tile][R]
  static constexpr size_t kn = ph + sizeof(float) * R * kBuildTile;      // float [tile]
  static constexpr size_t total = kn + sizeof(float) * (kBuildTile + 8);
};

template <int D, int R>
__global__ void __launch_bounds__(kBuildThreads) build_kernel(const BuildProblem p) {
  using L = BuildSmem<D, R>;
  extern __shared__ __align__(16) unsigned char smem[];
  float* Wt = reinterpret_cast<float*>(smem + L::wt);
  float* kf = reinterpret_cast<float*>(smem + L::kf);
  float* vf = reinterpret_cast<float*>(smem + L::vf);
  float* ph = reinterpret_cast<float*>(smem + L::ph);
  float* knorm = reinterpret_cast<float*>(smem + L::kn);
  __shared__ int s_last;

  constexpr int TD = D / 16, TR = R / 16;          // register tile of S per thread
  const int tid = threadIdx.x;
  const int b = blockIdx.z, kvh = blockIdx.y, chunk = blockIdx.x;
  const int unit = b * p.n_kv_heads + kvh;
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  const int n_chunks = (n_mid + p.chunk_len - 1) / p.chunk_len;
  float* S_out = p.S + (size_t)unit * D * R;
  float* u_out = p.u + (size_t)unit * R;
  if (n_mid == 0) {
    if (chunk == 0) {
      for (int i = tid; i < D * R; i += kBuildThreads) S_out[i] = 0.f;
      for (int i = tid; i < R; i += kBuildThreads) u_out[i] = 0.f;
    }
    return;
  }
  if (chunk >= n_chunks) return;
  const int m0 = chunk * p.chunk_len;
  const int m1 = min(n_mid, m0 + p.chunk_len);

  const float* W = p.w_k + (size_t)kvh * R * D;
  for (int i = tid; i < R * D; i += kBuildThreads) Wt[(i % D) * L::WT_LD + (i / D)] = W[i];

  const __nv_bfloat16* kbase = p.k + (long long)kvh * p.stride_head + (cu_b + p.n_sink) * p.stride_token;
  const __nv_bfloat16* vbase = p.v + (long long)kvh * p.stride_head + (cu_b + p.n_sink) * p.stride_token;

  // phase-1 mapping: feature j, token group tg
  constexpr int NG = kBuildThreads / R, TPG = kBuildTile / NG;
  const int j = tid % R, tg = tid / R, t0 = tg * TPG;
  const float bj = p.b_k[(size_t)kvh * R + j];
  // phase-2 mapping: S rows [TD*ti, +TD), columns [TR*tj, +TR)
  const int ti = tid / 16, tj = tid % 16;
  float acc[TD][TR];
#pragma unroll
  for (int a = 0; a < TD; ++a)
#pragma unroll
    for (int c = 0; c < TR; ++c) acc[a][c] = 0.f;
  float uacc = 0.f;

  constexpr int CPR = D / 8;
  for (int base = m0; base < m1; base += kBuildTile) {
    __syncthreads();
    for (int i = tid; i < kBuildTile * CPR; i += kBuildThreads) {
      const int t = i / CPR, c = i % CPR;
      uint4 kraw = make_uint4(0, 0, 0, 0), vraw = make_uint4(0, 0, 0, 0);
      if (base + t < m1) {
        kraw = *reinterpret_cast<const uint4*>(kbase + (long long)(base + t) * p.stride_token + c * 8);
        vraw = *reinterpret_cast<const uint4*>(vbase + (long long)(base + t) * p.stride_token + c * 8);
      }
      const unsigned kw[4] = {kraw.x, kraw.y, kraw.z, kraw.w};
      const unsigned vw[4] = {vraw.x, vraw.y, vraw.z, vraw.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        kf[(c * 8 + 2 * e) * kBuildTile + t] = bf16_lo(kw[e]);
        kf[(c * 8 + 2 * e + 1) * kBuildTile + t] = bf16_hi(kw[e]);
        vf[t * D + c * 8 + 2 * e] = bf16_lo(vw[e]);
        vf[t * D + c * 8 + 2 * e + 1] = bf16_hi(vw[e]);
      }
    }
    __syncthreads();
    if (tid < kBuildTile) {
      float kn = 0.f;
      for (int c = 0; c < D; ++c) { const float x = kf[c * kBuildTile + tid]; kn = fmaf(x, x, kn); }
      knorm[tid] = kn;
    }
    // phi_k for the tile
    float a[TPG];
#pragma unroll
    for (int t = 0; t < TPG; ++t) a[t] = 0.f;
    for (int c = 0; c < D; ++c) {
      const float w = Wt[c * L::WT_LD + j];
      const float4* kp = reinterpret_cast<const float4*>(kf + c * kBuildTile + t0);
#pragma unroll
      for (int t4 = 0; t4 < TPG / 4; ++t4) {
        const float4 kv = kp[t4];
        a[4 * t4 + 0] = fmaf(w, kv.x, a[4 * t4 + 0]);
        a[4 * t4 + 1] = fmaf(w, kv.y, a[4 * t4 + 1]);
        a[4 * t4 + 2] = fmaf(w, kv.z, a[4 * t4 + 2]);
        a[4 * t4 + 3] = fmaf(w, kv.w, a[4 * t4 + 3]);
      }
    }
    __syncthreads();                                   // knorm visible
#pragma unroll
    for (int t = 0; t < TPG; ++t) {
      const float f = (base + t0 + t < m1) ? expf(a[t] + bj - p.gamma_k * knorm[t0 + t]) : 0.f;
      ph[(t0 + t) * R + j] = f;
    }
    __syncthreads();
    // S += V^T Phi, u += column sums of Phi
    for (int t = 0; t < kBuildTile; ++t) {
      float vv[TD], pp[TR];
#pragma unroll
      for (int x = 0; x < TD; x += 4) {
        const float4 q4 = *reinterpret_cast<const float4*>(vf + t * D + TD * ti + x);
        vv[x] = q4.x; vv[x + 1] = q4.y; vv[x + 2] = q4.z; vv[x + 3] = q4.w;
      }
#pragma unroll
      for (int x = 0; x < TR; x += 4) {
        const float4 q4 = *reinterpret_cast<const float4*>(ph + t * R + TR * tj + x);
        pp[x] = q4.x; pp[x + 1] = q4.y; pp[x + 2] = q4.z; pp[x + 3] = q4.w;
      }
#pragma unroll
      for (int x = 0; x < TD; ++x)
#pragma unroll
        for (int y = 0; y < TR; ++y) acc[x][y] = fmaf(vv[x], pp[y], acc[x][y]);
    }
    if (tid < R) {
      for (int t = 0; t < kBuildTile; ++t) uacc += ph[t * R + tid];
    }
  }

  // ---- partial of this chunk
  float* part = p.partials + ((size_t)unit * p.chunks_per_unit + chunk) * (D * R + R);
#pragma unroll
  for (int x = 0; x < TD; ++x)
#pragma unroll
    for (int y = 0; y < TR; ++y) part[(TD * ti + x) * R + TR * tj + y] = acc[x][y];
  if (tid < R) part[D * R + tid] = uacc;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&p.unit_counter[unit], 1u) == (unsigned)(n_chunks - 1));
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float* parts = p.partials + (size_t)unit * p.chunks_per_unit * (D * R + R);
  for (int i = tid; i < D * R + R; i += kBuildThreads) {
    float s = 0.f;
    for (int c = 0; c < n_chunks; ++c) s += __ldcg(parts + (size_t)c * (D * R + R) + i);
    if (i < D * R) S_out[i] = s; else u_out[i - D * R] = s;
  }
}

template <int D, int R>
static cudaError_t launch_build_t(const BuildProblem& p, cudaStream_t st) {
  static bool configured = false;
  const size_t smem = BuildSmem<D, R>::total;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(build_kernel<D, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(p.chunks_per_unit, p.n_kv_heads, p.batch);
  build_kernel<D, R><<<grid, kBuildThreads, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_build(const BuildProblem& p, cudaStream_t st) {
  if (p.head_dim == 64 && p.n_feat == 64) return launch_build_t<64, 64>(p, st);
  if (p.head_dim == 64 && p.n_feat == 128) return launch_build_t<64, 128>(p, st);
  if (p.head_dim == 128 && p.n_feat == 64) return launch_build_t<128, 64>(p, st);
  if (p.head_dim == 128 && p.n_feat == 128) return launch_build_t<128, 128>(p, st);
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
