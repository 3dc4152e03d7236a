// The paper's head-wise feature map (App. C.2), a one-block ReZero MLP of hidden width d_emb = 512:
//   g0 = W_s x + b_s;  Delta = W_2 GeLU(W_1 g0 + b_1) + b_2;  g1 = g0 + alpha Delta;  phi(x) = exp(W_o g1 + b_o).
// Key side: phi_k of every cache row is four dense layers over all tokens, i.e. four GEMMs per KV head
// ([tokens x K] . [N x K]^T); they run on the tensor cores (tcgen05.mma, two accumulators in tensor memory,
// both operands staged by TMA into a ring that runs ahead across tiles, one persistent CTA per SM), each
// followed by its layer's epilogue (bias, GeLU, the gated residual, the exponential), which overlaps the
// next tile's MMAs.  Activations between the layers are bf16 in the caller's
// workspace; accumulation, biases and the exponent are fp32.  The rows of phi_k go to the caller's
// feature cache, from which the summaries are built (build_summaries.cu, cached variant) and the
// decode step takes the retrieved tokens' rows (cached_features.cu).
// Query side: one vector per head and decode step: mlp_query.cu.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr int kGemmThreads = 576;      // warp 0: TMA producer, warp 1: MMA issuer, warps 2..17: epilogue (four per lane quadrant)
constexpr int kGemmBM = 128;           // rows (tokens) per tile = MMA M = tensor-memory lanes
constexpr int kGemmBK = 64;            // reduction elements per stage: one 128-byte swizzled row

__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }

// Output columns per tile: 256 where the layer width allows (fewer tiles re-read the activation rows), else 128 or 64.
__host__ __device__ constexpr int gemm_stages(int BN) { return BN == 256 ? 4 : 6; }

// out[h][m][n] = epilogue(sum_k A[h][m][k] W[h][n][k] + bias[h][n]).  Persistent: one CTA per SM walks the tiles
// (head, row block, column block; column block fastest, so that the CTAs running at the same time share the
// activation rows in L2).  Two accumulators in tensor memory: the epilogue of a tile runs while the MMAs of the
// next tile fill the other one, and the TMA ring runs ahead across tile boundaries.
template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
mlp_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const GemmArgs g) {
  constexpr int NST = gemm_stages(BN);
  constexpr int A_BYTES = kGemmBM * 128, W_BYTES = BN * 128, STAGE = A_BYTES + W_BYTES;
  constexpr int ACC_COLS = BN < 128 ? 128 : BN;            // column distance of the two accumulators
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NST * STAGE);
  uint64_t* full = bars;                 // [NST]
  uint64_t* empty = bars + NST;          // [NST]
  uint64_t* acc_full = bars + 2 * NST;   // [2] the MMAs of a tile are complete
  uint64_t* acc_free = acc_full + 2;     // [2] the epilogue warps have read the accumulator
  volatile int* s_abort = reinterpret_cast<volatile int*>(acc_free + 2);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(const_cast<int*>(s_abort) + 1);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_kb = g.K / kGemmBK;
  const int tiles_n = g.N / BN, tiles_m = (g.M + kGemmBM - 1) / kGemmBM;
  const long long n_tiles = (long long)g.heads * tiles_m * tiles_n;
  if (tid == 0) {
    for (int s = 0; s < NST; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_free[s], kGemmThreads / 32 - 2); }
    mbar_fence_init();
    *s_abort = 0;
  }
  if (warp == 1) tmem_alloc(s_tmem, 2 * ACC_COLS);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;

  if (warp == 0) {
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_last();         // both operands are read by several CTAs
      long long it = 0;                                    // k-blocks issued so far, over all tiles of this CTA
      bool ok = true;
      for (long long t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        const int n0 = (int)(t % tiles_n) * BN, m0 = (int)((t / tiles_n) % tiles_m) * kGemmBM, h = (int)(t / ((long long)tiles_n * tiles_m));
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = (int)(it % NST);
          ok = mbar_wait(&empty[s], (((uint32_t)(it / NST)) & 1u) ^ 1u, s_abort);
          if (!ok) break;
          mbar_expect_tx(&full[s], STAGE);
          tma_load_3d(smem + s * STAGE, &map_a, &full[s], kb * kGemmBK, m0, h, pol);
          tma_load_3d(smem + s * STAGE + A_BYTES, &map_w, &full[s], kb * kGemmBK, n0, h, pol);
        }
      }
      if (!ok) {                                           // gave up: let the copies in flight land
        for (long long j = (it > NST ? it - NST : 0); j < it; ++j)
          for (uint32_t w = 0; w < kWaitPolls; ++w) {
            if (mbar_try_wait(&full[j % NST], (uint32_t)(j / NST) & 1u)) break;
            __nanosleep(64);
          }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kGemmBM, BN, 0, 0);
      long long it = 0, i = 0;                             // k-blocks, tiles of this CTA so far
      bool ok = true;
      for (long long t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
        const int acc = (int)(i & 1);
        // the accumulator is free once the epilogue warps have read the tile before the last
        ok = i < 2 || mbar_wait(&acc_free[acc], (uint32_t)((i - 2) >> 1) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after_sync();
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int s = (int)(it % NST);
          ok = mbar_wait(&full[s], (uint32_t)(it / NST) & 1u, s_abort);
          if (!ok) break;
          tc_fence_after_sync();
          const uint64_t ad = umma_smem_desc(smem_u32(smem + s * STAGE), 16, 1024);
          const uint64_t wd = umma_smem_desc(smem_u32(smem + s * STAGE + A_BYTES), 16, 1024);
#pragma unroll
          for (int k = 0; k < kGemmBK / 16; ++k)
            umma_ss(tmem_base + acc * ACC_COLS, ad + (uint64_t)((k * 32) >> 4), wd + (uint64_t)((k * 32) >> 4), idesc, (kb | k) ? 1u : 0u);
          tc_commit(&empty[s]);
        }
        if (ok) tc_commit(&acc_full[acc]);
      }
    }
  } else {
    // ---- epilogue: thread = output row (tensor-memory lane 32 (warp % 4) + lane) x every fourth 32-column chunk
    // (sixteen warps: the GeLU layer's epilogue is a long dependent chain per element and needs the occupancy)
    const int quad = warp & 3, sub = (warp - 2) >> 2, row = quad * 32 + lane;
    constexpr int NCH = BN / 32;                           // chunks of the tile
    const int last_c = sub + ((NCH - 1 - sub) / 4) * 4;    // this warp's last chunk (sub >= NCH: none)
    bool ok = true;
    long long i = 0;
    for (long long t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
      const int n0 = (int)(t % tiles_n) * BN, m0 = (int)((t / tiles_n) % tiles_m) * kGemmBM, h = (int)(t / ((long long)tiles_n * tiles_m));
      const int acc = (int)(i & 1), m = m0 + row;
      ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[acc], (uint32_t)(i >> 1) & 1u, s_abort));
      if (!ok) break;
      tc_fence_after_sync();
      const float al = g.epi == kEpiResidual ? __ldg(g.alpha + h) : 0.f;
      const float* bias = g.bias + (size_t)h * g.N + n0;
      const size_t o = (size_t)h * g.out_head_stride + (size_t)m * g.N + n0;
      if (sub >= NCH) {                                    // narrow tiles: nothing for this warp to read
        if (lane == 0) mbar_arrive(&acc_free[acc]);
        continue;
      }
      for (int c = sub; c < NCH; c += 4) {
        float v[32];
        tmem_ld_x32(tmem_addr(tmem_base, quad * 32, acc * ACC_COLS + c * 32), v);
        tc_wait_ld();
        if (c == last_c) {                                 // this warp has read its whole share of the tile
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_free[acc]);
        }
        if (m < g.M) {
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float4 b4 = __ldg(reinterpret_cast<const float4*>(bias + c * 32) + e);
            v[4 * e] += b4.x; v[4 * e + 1] += b4.y; v[4 * e + 2] += b4.z; v[4 * e + 3] += b4.w;
          }
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
                for (int q = 0; q < 4; ++q) {
                  v[8 * e + 2 * q] = fmaf(al, v[8 * e + 2 * q], bf16_lo(w[q]));
                  v[8 * e + 2 * q + 1] = fmaf(al, v[8 * e + 2 * q + 1], bf16_hi(w[q]));
                }
              }
            }
            uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(g.out) + o + c * 32);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              unsigned w[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(v[8 * e + 2 * q], v[8 * e + 2 * q + 1]);
                w[q] = *reinterpret_cast<const unsigned*>(&pr);
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
    tmem_dealloc(tmem_base, 2 * ACC_COLS);
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
static cudaError_t launch_gemm_t(const CUtensorMap& ma, const CUtensorMap& mw, const GemmArgs& g, cudaStream_t st) {
  static PerDeviceFlag configured;
  const size_t smem = (size_t)gemm_stages(BN) * (kGemmBM * 128 + BN * 128) + (2 * gemm_stages(BN) + 4) * 8 + 64;
  cudaError_t e = set_max_dynamic_smem(configured, reinterpret_cast<const void*>(mlp_gemm_kernel<BN>), smem);
  if (e != cudaSuccess) return e;
  const long long n_tiles = (long long)g.heads * ((g.M + kGemmBM - 1) / kGemmBM) * (g.N / BN);
  const int n_sm = sm_count_current_device();
  const int grid = (int)(n_tiles < n_sm ? n_tiles : n_sm);
  mlp_gemm_kernel<BN><<<grid > 0 ? grid : 1, kGemmThreads, smem, st>>>(ma, mw, g);
  return cudaGetLastError();
}

cudaError_t launch_mlp_gemm(const CUtensorMap& ma, const CUtensorMap& mw, const GemmArgs& g, cudaStream_t st) {
  switch (mlp_gemm_bn(g.N)) {
    case 256: return launch_gemm_t<256>(ma, mw, g, st);
    case 128: return launch_gemm_t<128>(ma, mw, g, st);
    case 64: return launch_gemm_t<64>(ma, mw, g, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
