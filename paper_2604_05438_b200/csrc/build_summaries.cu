// Prefill summary build (Sec. 4.1, Eq. natural_cache):
//   S = sum_{i in M} v_i phi_k(k_i)^T  (d_v x d_phi),   u = sum_{i in M} phi_k(k_i),
//   phi_k(k) = exp(W_k k + b_k - gamma_k |k|^2).
//
// Both contractions of the build are dense, so both run on the tensor cores
// (tcgen05.mma, accumulators in tensor memory).  Per tile of 128 mid-region tokens:
//   GEMM 1   A^T[j][t] = sum_c W_k[j][c] k_t[c]      A operand: W_k (split into bf16
//            hi + lo, rows = features, zero padded to 128), B operand: the key tile as
//            TMA lands it.  The fp32 result sits in tensor memory with one feature per
//            lane and one token per column.
//   features Phi^T[j][t] = exp2(A^T + b_j - gamma |k_t|^2) (everything pre-scaled by
//            log2 e).  Eight warps read the accumulator, add u_j += Phi (fp32), split
//            Phi into bf16 hi + lo (error ~2^-17) and store both back to tensor memory.
//   GEMM 2   S^T[j][c] += sum_t Phi^T[j][t] v_t[c]   A operand: Phi^T hi, then lo,
//            straight from tensor memory; B operand: the value tile as TMA lands it
//            (tokens along K, dims contiguous).  S^T accumulates in tensor memory over
//            all tiles of the CTA.
// With a feature cache (Sec. 4.2 notes that a cached implementation avoids the decode-side
// recompute) the feature warps also write every phi_k row they produce to global memory.
// Warp roles: 0 TMA producer, 1 MMA issuer, 2..9 feature warps, 10..13 key norms.
// GEMM 1 of tile i+1 is issued before GEMM 2 of tile i, so the tensor pipe works while
// the feature warps are busy.  Each CTA owns a contiguous range of tiles of one
// (sequence, KV head) unit and writes one partial; a second small kernel adds the
// partials in chunk order.  Every device-side wait is bounded and reports through the
// status word.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr int kBuildThreads = 448;
constexpr int kBT = 128;                 // tokens per tile
constexpr int kBuildTmemCols = 512;
constexpr int kColD1 = 0;                // two GEMM-1 accumulators of 128 columns (Phi hi overwrites them)
constexpr int kColD2 = 256;              // S^T accumulator, head_dim columns
constexpr int kColLo = 384;              // Phi lo, 64 columns per buffer

template <int D>
struct BuildCfg {
  static constexpr int BOXES = D / 64;
  static constexpr int BOX = kBT * 128;                    // bytes of one 64-dim column block of a tile
  static constexpr int TILE = BOXES * BOX;                 // 32 KB (d = 128) or 16 KB (d = 64)
  static constexpr int KS = D == 128 ? 2 : 3;              // key ring stages
  static constexpr int VS = D == 128 ? 2 : 3;              // value ring stages
  static constexpr size_t whi = 0;
  static constexpr size_t wlo = whi + TILE;
  static constexpr size_t kring = wlo + TILE;
  static constexpr size_t vring = kring + (size_t)KS * TILE;
  static constexpr size_t small = vring + (size_t)VS * TILE;
  // small: barriers (<= 32), snorm[2][128], ucomb[2][128], misc
  static constexpr size_t total = small + 32 * 8 + 4 * (2 * 128 + 2 * 128 + 16);
};

__device__ __forceinline__ void tmem_st_x16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// MODE 0: features computed; 1: computed and also stored to the feature cache; 2: read from the
// feature cache (no key tiles, no GEMM 1): for feature maps evaluated elsewhere (mlp_features.cu).
template <int D, int MODE>
__global__ void __launch_bounds__(kBuildThreads, 1)
build_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
             const BuildProblem p) {
  using C = BuildCfg<D>;
  constexpr int KS = C::KS, VS = C::VS, BOXES = C::BOXES;
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* whi = smem + C::whi;
  unsigned char* wlo = smem + C::wlo;
  unsigned char* kring = smem + C::kring;
  unsigned char* vring = smem + C::vring;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::small);
  uint64_t* k_full = bars;                 // [KS] key tile landed
  uint64_t* k_empty = k_full + KS;         // [KS] GEMM 1 and the norm warps are done with it
  uint64_t* v_full = k_empty + KS;         // [VS]
  uint64_t* v_empty = v_full + VS;         // [VS] GEMM 2 is done with it
  uint64_t* d1_full = v_empty + VS;        // [2]  GEMM 1 accumulator complete
  uint64_t* p_ready = d1_full + 2;         // [2]  features stored to tensor memory
  uint64_t* n_ready = p_ready + 2;         // [2]  key norms of the tile in shared memory
  uint64_t* d2_full = n_ready + 2;         // [1]  last GEMM 2 complete
  uint64_t* g2_done = d2_full + 1;         // [2]  GEMM 2 of the tile that used this feature buffer is complete
  float* snorm = reinterpret_cast<float*>(bars + 32);        // [2][128]  -gamma log2e |k_t|^2, -inf if masked
  float* ucomb = snorm + 2 * 128;                            // [2][128]
  int* misc = reinterpret_cast<int*>(ucomb + 2 * 128);
  volatile int* s_abort = misc;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc + 1);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.z, kvh = blockIdx.y, chunk = blockIdx.x;
  const int R = p.n_feat;
  const int unit = b * p.n_kv_heads + kvh;
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  float* S_out = p.S + (size_t)unit * D * R;
  float* u_out = p.u + (size_t)unit * R;
  if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) *p.status = kStatusOk;
  if (n_mid == 0) {
    if (chunk == 0) {
      for (int i = tid; i < D * R; i += kBuildThreads) S_out[i] = 0.f;
      for (int i = tid; i < R; i += kBuildThreads) u_out[i] = 0.f;
    }
    return;
  }
  const int n_tiles = (n_mid + kBT - 1) / kBT;
  const int n_chunks = n_tiles < p.chunks_per_unit ? n_tiles : p.chunks_per_unit;
  if (chunk >= n_chunks) return;
  const int t0 = (int)((long long)n_tiles * chunk / n_chunks);
  const int t1 = (int)((long long)n_tiles * (chunk + 1) / n_chunks);
  const int n_my = t1 - t0;                                   // >= 1
  const int row0 = (int)(cu_b + p.n_sink);                    // cache row of mid token 0

  // ---- set-up: barriers, tensor memory, W_k operand tiles (scaled by log2 e, hi + lo)
  if (tid == 0) {
    for (int s = 0; s < KS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 5); }
    for (int s = 0; s < VS; ++s) { mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&d1_full[s], 1); mbar_init(&p_ready[s], 8); mbar_init(&n_ready[s], 4);
    }
    mbar_init(d2_full, 1);
    mbar_init(&g2_done[0], 1); mbar_init(&g2_done[1], 1);
    mbar_fence_init();
    *s_abort = 0;
  }
  if (warp == 1) tmem_alloc(s_tmem, kBuildTmemCols);
  if (MODE != 2) {
    const float* W = p.w_k + (size_t)kvh * R * D;
    constexpr int CPR = D / 8;
    for (int i = tid; i < 128 * CPR; i += kBuildThreads) {
      const int row = i / CPR, c = i % CPR;
      unsigned hw[4] = {0, 0, 0, 0}, lw[4] = {0, 0, 0, 0};
      if (row < R) {
        const float4 w0 = *reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8);
        const float4 w1 = *reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8 + 4);
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float a0 = w[2 * e] * kLog2e, a1 = w[2 * e + 1] * kLog2e;
          const __nv_bfloat16 h0 = __float2bfloat16_rn(a0), h1 = __float2bfloat16_rn(a1);
          const __nv_bfloat16 l0 = __float2bfloat16_rn(a0 - __bfloat162float(h0));
          const __nv_bfloat16 l1 = __float2bfloat16_rn(a1 - __bfloat162float(h1));
          hw[e] = (unsigned)__bfloat16_as_ushort(h0) | ((unsigned)__bfloat16_as_ushort(h1) << 16);
          lw[e] = (unsigned)__bfloat16_as_ushort(l0) | ((unsigned)__bfloat16_as_ushort(l1) << 16);
        }
      }
      const uint32_t off = (c >> 3) * C::BOX + swz128(row, c & 7);
      *reinterpret_cast<uint4*>(whi + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      *reinterpret_cast<uint4*>(wlo + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
  }
  fence_proxy_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;

  if (warp == 0) {
    // ================================================================ TMA producer
    if (lane == 0) {
      bool ok = true;
      const uint64_t pol = l2_policy_evict_first();        // K and V are read once
      for (int it = 0; it < n_my && ok; ++it) {
        const int row = row0 + (t0 + it) * kBT;
        const int ks = it % KS, vs = it % VS;
        if (MODE != 2) {
          ok = mbar_wait(&k_empty[ks], ((uint32_t)(it / KS) & 1u) ^ 1u, s_abort);
          if (!ok) break;
          mbar_expect_tx(&k_full[ks], C::TILE);
#pragma unroll
          for (int x = 0; x < BOXES; ++x)
            tma_load_3d(kring + ks * C::TILE + x * C::BOX, &tmap_k, &k_full[ks], x * 64, row, kvh, pol);
        }
        ok = mbar_wait(&v_empty[vs], ((uint32_t)(it / VS) & 1u) ^ 1u, s_abort);
        if (!ok && MODE == 2) break;
        if (!ok) {
          // the key copy just issued must land before shared memory is released
          for (uint32_t w = 0; w < kWaitPolls; ++w) {
            if (mbar_try_wait(&k_full[ks], (uint32_t)(it / KS) & 1u)) break;
            __nanosleep(64);
          }
          break;
        }
        mbar_expect_tx(&v_full[vs], C::TILE);
#pragma unroll
        for (int x = 0; x < BOXES; ++x)
          tma_load_3d(vring + vs * C::TILE + x * C::BOX, &tmap_v, &v_full[vs], x * 64, row, kvh, pol);
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc1 = umma_idesc_bf16(128, kBT, 0, 0);
      constexpr uint32_t idesc2 = umma_idesc_bf16(128, D, 0, 1);
      const uint64_t whi_d = umma_smem_desc(smem_u32(whi), 16, 1024);
      const uint64_t wlo_d = umma_smem_desc(smem_u32(wlo), 16, 1024);
      const uint64_t k_d = umma_smem_desc(smem_u32(kring), 16, 1024);
      // value tile as an MN-major operand: 64-dim column blocks BOX bytes apart, groups of
      // eight token rows 1024 bytes apart
      const uint64_t v_d = umma_smem_desc(smem_u32(vring), C::BOX, 1024);
      bool ok = true;
      auto gemm2 = [&](int j) {
        const int buf = j & 1, vs = j % VS;
        ok = mbar_wait(&p_ready[buf], (uint32_t)(j >> 1) & 1u, s_abort) &&
             mbar_wait(&v_full[vs], (uint32_t)(j / VS) & 1u, s_abort);
        if (!ok) return;
        tc_fence_after_sync();
        const uint64_t vd = v_d + (uint64_t)((vs * C::TILE) >> 4);
#pragma unroll
        for (int kk = 0; kk < kBT / 16; ++kk) {
          // tokens 16 kk .. 16 kk + 15: eight packed columns of Phi hi, then of Phi lo
          const uint32_t hi_col = kColD1 + buf * 128 + (kk >> 2) * 64 + ((kk >> 1) & 1) * 16 + (kk & 1) * 8;
          const uint32_t lo_col = kColLo + buf * 64 + (kk >> 2) * 32 + ((kk >> 1) & 1) * 16 + (kk & 1) * 8;
          const uint64_t bd = vd + (uint64_t)((kk * 16 * 128) >> 4);
          umma_ts(tmem_base + kColD2, tmem_base + hi_col, bd, idesc2, (j > 0 || kk > 0) ? 1u : 0u);
          umma_ts(tmem_base + kColD2, tmem_base + lo_col, bd, idesc2, 1u);
        }
        tc_commit(&v_empty[vs]);
        tc_commit(&g2_done[buf]);
      };
      if (MODE == 2) {
        for (int it = 0; it + 1 < n_my && ok; ++it) gemm2(it);
      }
      for (int it = 0; MODE != 2 && it < n_my && ok; ++it) {
        const int buf = it & 1, ks = it % KS;
        // No wait for GEMM 2 of tile it-2, whose A operand lives where this accumulator goes:
        // MMAs issued by one thread execute in issue order, and the feature warps touch the
        // buffer only after d1_full of this tile.
        ok = mbar_wait(&k_full[ks], (uint32_t)(it / KS) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t kd = k_d + (uint64_t)((ks * C::TILE) >> 4);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint64_t wd = half == 0 ? whi_d : wlo_d;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint64_t off = (uint64_t)(((k >> 2) * C::BOX + (k & 3) * 32) >> 4);
            umma_ss(tmem_base + kColD1 + buf * 128, wd + off, kd + off, idesc1, (half | k) ? 1u : 0u);
          }
        }
        tc_commit(&d1_full[buf]);
        tc_commit(&k_empty[ks]);
        if (it > 0) gemm2(it - 1);
      }
      if (ok) gemm2(n_my - 1);
      if (ok) tc_commit(d2_full);
    }
  } else if (warp < 10) {
    // ================================================================ feature warps
    const int quad = warp & 3;                     // tensor-memory lane quadrant
    const int h = (warp - 2) >> 2;                 // which 64 tokens of the tile
    const int j = quad * 32 + lane;                // feature
    const float bj = (MODE != 2 && j < R) ? p.b_k[(size_t)kvh * R + j] * kLog2e : 0.f;
    float u_acc = 0.f;                             // sum of feature j over this thread's tokens
    // feature cache (written in mode 1, read in mode 2): row of mid token 0 of this head, column j
    float* cache_j = (MODE != 0 && j < R) ? p.phi_cache + ((size_t)kvh * p.total_tokens + (size_t)row0) * R + j : nullptr;
    bool ok = true;
    for (int it = 0; it < n_my && ok; ++it) {
      const int buf = it & 1;
      const uint32_t ph = (uint32_t)(it >> 1) & 1u;
      if (MODE == 2) {
        // the feature buffer is free once GEMM 2 of tile it - 2 has read it; snorm says which tokens are in the mid-region
        ok = mbar_wait(&n_ready[buf], ph, s_abort) && (it < 2 || mbar_wait(&g2_done[buf], ph ^ 1u, s_abort));
      } else {
        ok = mbar_wait(&d1_full[buf], ph, s_abort) && mbar_wait(&n_ready[buf], ph, s_abort);
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const float* sn = snorm + buf * 128 + h * 64;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float v[32];
        if (MODE == 2) {
          const int tok0 = (t0 + it) * kBT + h * 64 + c * 32;
#pragma unroll
          for (int e = 0; e < 32; ++e)
            v[e] = (cache_j != nullptr && sn[c * 32 + e] == 0.f) ? __ldcs(cache_j + (size_t)(tok0 + e) * R) : 0.f;
        } else {
          tmem_ld_x32(tmem_addr(tmem_base, quad * 32, kColD1 + buf * 128 + h * 64 + c * 32), v);
          tc_wait_ld();
        }
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float f0 = MODE == 2 ? v[2 * e] : ex2_approx(v[2 * e] + bj + sn[c * 32 + 2 * e]);
          const float f1 = MODE == 2 ? v[2 * e + 1] : ex2_approx(v[2 * e + 1] + bj + sn[c * 32 + 2 * e + 1]);
          u_acc += f0;
          u_acc += f1;
          const __nv_bfloat162 hp = __floats2bfloat162_rn(f0, f1);          // .x (low half) = even token
          const __nv_bfloat162 lp =
              __floats2bfloat162_rn(f0 - __bfloat162float(hp.x), f1 - __bfloat162float(hp.y));
          hi[e] = *reinterpret_cast<const uint32_t*>(&hp);
          lo[e] = *reinterpret_cast<const uint32_t*>(&lp);
          if (MODE == 1 && cache_j) {
            // one token per store: the 32 lanes of the warp write 32 consecutive features
            const int tok = (t0 + it) * kBT + h * 64 + c * 32 + 2 * e;
            if (tok < n_mid) __stcs(cache_j + (size_t)tok * R, f0);
            if (tok + 1 < n_mid) __stcs(cache_j + (size_t)(tok + 1) * R, f1);
          }
        }
        // hi goes over columns of this thread's own region that it has already read
        tmem_st_x16(tmem_addr(tmem_base, quad * 32, kColD1 + buf * 128 + h * 64 + c * 16), hi);
        tmem_st_x16(tmem_addr(tmem_base, quad * 32, kColLo + buf * 64 + h * 32 + c * 16), lo);
      }
      tc_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_ready[buf]);
    }
    // ---- S^T of this CTA's tiles -> partial (thread = feature, h = half of the dims)
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(d2_full, 0, s_abort));
    if (ok) {
      tc_fence_after_sync();
      float* part = p.partials + ((size_t)unit * p.chunks_per_unit + chunk) * ((size_t)D * R + R);
      constexpr int HALF = D / 2;
#pragma unroll
      for (int c = 0; c < HALF / 32; ++c) {
        float v[32];
        tmem_ld_x32(tmem_addr(tmem_base, quad * 32, kColD2 + h * HALF + c * 32), v);
        tc_wait_ld();
        if (j < R) {
#pragma unroll
          for (int e = 0; e < 32; ++e) part[(size_t)(h * HALF + c * 32 + e) * R + j] = v[e];
        }
      }
      ucomb[h * 128 + j] = u_acc;
    }
  } else {
    // ================================================================ key norms and masking
    const int t = (warp - 10) * 32 + lane;         // token of the tile
    const float g2 = p.gamma_k * kLog2e;
    bool ok = true;
    for (int it = 0; it < n_my && ok; ++it) {
      const int buf = it & 1, ks = it % KS;
      // snorm[buf] was last read by the feature warps for tile it-2: wait for their p_ready
      ok = (MODE == 2 || mbar_wait(&k_full[ks], (uint32_t)(it / KS) & 1u, s_abort)) &&
           mbar_wait(&p_ready[buf], ((uint32_t)(it >> 1) & 1u) ^ 1u, s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const unsigned char* tile = kring + ks * C::TILE;
      float kn = 0.f;
#pragma unroll
      for (int c = 0; MODE != 2 && c < D / 8; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(tile + (c >> 3) * C::BOX + swz128(t, c & 7));
        const unsigned w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float x0 = bf16_lo(w[e]), x1 = bf16_hi(w[e]);
          kn = fmaf(x0, x0, kn);
          kn = fmaf(x1, x1, kn);
        }
      }
      const bool valid = (t0 + it) * kBT + t < n_mid;
      snorm[buf * 128 + t] = valid ? -g2 * kn : -INFINITY;   // exp2(-inf) = 0 removes rows outside the mid-region
      __syncwarp();
      if (lane == 0) { mbar_arrive(&n_ready[buf]); if (MODE != 2) mbar_arrive(&k_empty[ks]); }
    }
  }

  // ---- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kBuildTmemCols);
  }
  if (*s_abort) {
    if (tid == 0) atomicExch(p.status, kStatusTimeout);
    return;
  }
  float* part = p.partials + ((size_t)unit * p.chunks_per_unit + chunk) * ((size_t)D * R + R);
  if (tid < R) part[(size_t)D * R + tid] = ucomb[tid] + ucomb[128 + tid];
}

// Adds the chunk partials of every unit in chunk order (fixed order: run-to-run identical).
constexpr int kRedThreads = 256;
__global__ void __launch_bounds__(kRedThreads) build_reduce_kernel(const BuildProblem p) {
  const int unit = blockIdx.y, b = unit / p.n_kv_heads;
  const int D = p.head_dim, R = p.n_feat, n_out = D * R + R;
  const long long len_b = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  if (n_mid == 0) return;                              // the build kernel wrote zeros
  const int n_tiles = (n_mid + kBT - 1) / kBT;
  const int n_chunks = n_tiles < p.chunks_per_unit ? n_tiles : p.chunks_per_unit;
  const float* parts = p.partials + (size_t)unit * p.chunks_per_unit * n_out;
  float* S_out = p.S + (size_t)unit * D * R;
  float* u_out = p.u + (size_t)unit * R;
  for (int i = blockIdx.x * kRedThreads + threadIdx.x; i < n_out; i += gridDim.x * kRedThreads) {
    float s = 0.f;
    int c = 0;
    for (; c + 8 <= n_chunks; c += 8) {
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = __ldcg(parts + (size_t)(c + e) * n_out + i);
#pragma unroll
      for (int e = 0; e < 8; ++e) s += v[e];
    }
    for (; c < n_chunks; ++c) s += __ldcg(parts + (size_t)c * n_out + i);
    if (i < D * R) S_out[i] = s; else u_out[i - D * R] = s;
  }
}

template <int D, int MODE>
static cudaError_t launch_build_t(const BuildProblem& p, const CUtensorMap& tk, const CUtensorMap& tv,
                                  cudaStream_t st) {
  static PerDeviceFlag configured;
  const size_t smem = BuildCfg<D>::total;
  cudaError_t e = set_max_dynamic_smem(configured, reinterpret_cast<const void*>(build_kernel<D, MODE>), smem);
  if (e != cudaSuccess) return e;
  dim3 grid(p.chunks_per_unit, p.n_kv_heads, p.batch);
  build_kernel<D, MODE><<<grid, kBuildThreads, smem, st>>>(tk, tv, p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  // one output per thread: every thread's loads of all chunk partials are in flight at once
  const int n_out = p.head_dim * p.n_feat + p.n_feat;
  build_reduce_kernel<<<dim3((n_out + kRedThreads - 1) / kRedThreads, p.n_kv_heads * p.batch), kRedThreads, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_build(const BuildProblem& p, const CUtensorMap& tk, const CUtensorMap& tv, cudaStream_t st) {
  const int mode = !p.phi_cache ? 0 : (p.from_cache ? 2 : 1);
  if (p.head_dim == 64)
    return mode == 0 ? launch_build_t<64, 0>(p, tk, tv, st) : mode == 1 ? launch_build_t<64, 1>(p, tk, tv, st) : launch_build_t<64, 2>(p, tk, tv, st);
  if (p.head_dim == 128)
    return mode == 0 ? launch_build_t<128, 0>(p, tk, tv, st) : mode == 1 ? launch_build_t<128, 1>(p, tk, tv, st) : launch_build_t<128, 2>(p, tk, tv, st);
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
