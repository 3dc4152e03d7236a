// The paper's head-wise feature map (App. C.2), a one-block ReZero MLP of hidden width d_emb = 512:
//   g0 = W_s x + b_s;  Delta = W_2 GeLU(W_1 g0 + b_1) + b_2;  g1 = g0 + alpha Delta;  phi(x) = exp(W_o g1 + b_o).
// Key side: phi_k of every cache row is four dense layers over all tokens, i.e. four GEMMs per KV head
// ([tokens x K] . [N x K]^T); they run on the tensor cores (tcgen05.mma, accumulators in tensor memory,
// both operands staged by TMA into a 2-stage ring, three CTAs per SM), each followed by its layer's epilogue (bias,
// GeLU, the gated residual, the exponential).  Activations between the layers are bf16 in the caller's
// workspace; accumulation, biases and the exponent are fp32.  The rows of phi_k go to the caller's
// feature cache, from which the summaries are built (build_summaries.cu, cached variant) and the
// decode step takes the retrieved tokens' rows (cached_features.cu).
// Query side: one vector per head and decode step: mlp_query.cu.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr int kGemmThreads = 320;      // warp 0: TMA producer, warp 1: MMA issuer, warps 2..9: epilogue (two per lane quadrant)
constexpr int kGemmStages = 2;
constexpr int kGemmBM = 128;           // rows (tokens) per CTA = MMA M = tensor-memory lanes
constexpr int kGemmBK = 64;            // reduction elements per stage: one 128-byte swizzled row

__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }

// out[h][m][n] = epilogue(sum_k A[h][m][k] W[h][n][k] + bias[h][n]); grid (N / BN, ceil(M / 128), heads).
template <int BN>
__global__ void __launch_bounds__(kGemmThreads)
mlp_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const GemmArgs g) {
  constexpr int A_BYTES = kGemmBM * 128, W_BYTES = BN * 128, STAGE = A_BYTES + W_BYTES;
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kGemmStages * STAGE);
  uint64_t* full = bars;
  uint64_t* empty = bars + kGemmStages;
  uint64_t* done = bars + 2 * kGemmStages;
  float* s_bias = reinterpret_cast<float*>(bars + 2 * kGemmStages + 1);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_bias + BN);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bias + BN + 1);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * kGemmBM, h = blockIdx.z;
  const int n_kb = g.K / kGemmBK;
  if (tid == 0) {
    for (int s = 0; s < kGemmStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(done, 1);
    mbar_fence_init();
    *s_abort = 0;
  }
  if (warp == 1) tmem_alloc(s_tmem, BN);
  for (int i = tid; i < BN; i += kGemmThreads) s_bias[i] = g.bias[(size_t)h * g.N + n0 + i];
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;

  if (warp == 0) {
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_last();         // both operands are read by several CTAs
      int kb = 0;
      for (; kb < n_kb; ++kb) {
        const int s = kb % kGemmStages;
        if (!mbar_wait(&empty[s], (((uint32_t)(kb / kGemmStages)) & 1u) ^ 1u, s_abort)) break;
        mbar_expect_tx(&full[s], STAGE);
        tma_load_3d(smem + s * STAGE, &map_a, &full[s], kb * kGemmBK, m0, h, pol);
        tma_load_3d(smem + s * STAGE + A_BYTES, &map_w, &full[s], kb * kGemmBK, n0, h, pol);
      }
      if (kb < n_kb) {                                     // gave up: let the copies in flight land
        for (int j = (kb > kGemmStages ? kb - kGemmStages : 0); j < kb; ++j)
          for (uint32_t w = 0; w < kWaitPolls; ++w) {
            if (mbar_try_wait(&full[j % kGemmStages], (uint32_t)(j / kGemmStages) & 1u)) break;
            __nanosleep(64);
          }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kGemmBM, BN, 0, 0);
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kGemmStages;
        ok = mbar_wait(&full[s], (uint32_t)(kb / kGemmStages) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t ad = umma_smem_desc(smem_u32(smem + s * STAGE), 16, 1024);
        const uint64_t wd = umma_smem_desc(smem_u32(smem + s * STAGE + A_BYTES), 16, 1024);
#pragma unroll
        for (int k = 0; k < kGemmBK / 16; ++k)
          umma_ss(tmem_base, ad + (uint64_t)((k * 32) >> 4), wd + (uint64_t)((k * 32) >> 4), idesc, (kb | k) ? 1u : 0u);
        tc_commit(&empty[s]);
      }
      if (ok) tc_commit(done);
    }
  } else {
    // ---- epilogue: thread = output row (tensor-memory lane 32 (warp % 4) + lane) x one half of the columns
    const int quad = warp & 3, half = (warp - 2) >> 2, row = quad * 32 + lane, m = m0 + row;
    const bool ok = __all_sync(0xffffffffu, mbar_wait(done, 0, s_abort));
    if (ok) {
      tc_fence_after_sync();
      const float al = g.epi == kEpiResidual ? g.alpha[h] : 0.f;
      const size_t o = (size_t)h * g.out_head_stride + (size_t)m * g.N + n0;
#pragma unroll
      for (int cc = 0; cc < BN / 64; ++cc) {
        const int c = half * (BN / 64) + cc;
        float v[32];
        tmem_ld_x32(tmem_addr(tmem_base, quad * 32, c * 32), v);
        tc_wait_ld();
        if (m < g.M) {
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] += s_bias[c * 32 + e];
          if (g.epi == kEpiExp) {
            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(g.out) + o + c * 32);
#pragma unroll
            for (int e = 0; e < 8; ++e)
              dst[e] = make_float4(__expf(v[4 * e]), __expf(v[4 * e + 1]), __expf(v[4 * e + 2]), __expf(v[4 * e + 3]));
          } else {
            if (g.epi == kEpiGelu) {
#pragma unroll
              for (int e = 0; e < 32; ++e) v[e] = gelu_erf(v[e]);
            } else if (g.epi == kEpiResidual) {
              const uint4* rs = reinterpret_cast<const uint4*>(g.resid + o + c * 32);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint4 raw = rs[e];
                const unsigned w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                  v[8 * e + 2 * t] = fmaf(al, v[8 * e + 2 * t], bf16_lo(w[t]));
                  v[8 * e + 2 * t + 1] = fmaf(al, v[8 * e + 2 * t + 1], bf16_hi(w[t]));
                }
              }
            }
            uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(g.out) + o + c * 32);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              unsigned w[4];
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(v[8 * e + 2 * t], v[8 * e + 2 * t + 1]);
                w[t] = *reinterpret_cast<const unsigned*>(&pr);
              }
              dst[e] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (*s_abort && tid == 0) atomicExch(g.status, kStatusTimeout);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, BN);
  }
}

__global__ void f32_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = __float2bfloat16_rn(src[i]);
}

cudaError_t launch_f32_to_bf16(const float* src, __nv_bfloat16* dst, size_t n, cudaStream_t st) {
  const int blocks = (int)((n + 255) / 256 < 1184 ? (n + 255) / 256 : 1184);
  f32_to_bf16_kernel<<<blocks, 256, 0, st>>>(src, dst, n);
  return cudaGetLastError();
}

template <int BN>
static cudaError_t launch_gemm_t(const CUtensorMap& ma, const CUtensorMap& mw, const GemmArgs& g, int heads, cudaStream_t st) {
  static PerDeviceFlag configured;
  const size_t smem = (size_t)kGemmStages * (kGemmBM * 128 + BN * 128) + (2 * kGemmStages + 1) * 8 + BN * 4 + 64;
  cudaError_t e = set_max_dynamic_smem(configured, reinterpret_cast<const void*>(mlp_gemm_kernel<BN>), smem);
  if (e != cudaSuccess) return e;
  dim3 grid(g.N / BN, (g.M + kGemmBM - 1) / kGemmBM, heads);
  mlp_gemm_kernel<BN><<<grid, kGemmThreads, smem, st>>>(ma, mw, g);
  return cudaGetLastError();
}

cudaError_t launch_mlp_gemm(const CUtensorMap& ma, const CUtensorMap& mw, const GemmArgs& g, int heads, cudaStream_t st) {
  if (g.N % 128 == 0) return launch_gemm_t<128>(ma, mw, g, heads, st);
  if (g.N == 64) return launch_gemm_t<64>(ma, mw, g, heads, st);
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
