// Prefill summary build (Sec. 4.1, Eq. natural_cache):
//   S = sum_{i in M} v_i phi_k(k_i)^T  (d_v x d_phi),   u = sum_{i in M} phi_k(k_i),
//   phi_k(k) = exp(W_k k + b_k - gamma_k |k|^2).
//
// Both contractions of the build are dense, so both run on the tensor cores
// (tcgen05.mma, accumulators in tensor memory).  The features never leave tensor memory: they
// are written over the accumulator they were computed from and read from there as the A
// operand of the second GEMM.  Per tile of 128 mid-region tokens:
//   GEMM 1   A^T[j][t] = sum_c W_k[j][c] k_t[c]      A operand: W_k (split into bf16
//            hi + lo, rows = features, zero padded to 128) in shared memory, B operand:
//            the key tile as TMA lands it.  The fp32 result sits in tensor memory with one
//            feature per lane and one token per column.
//   features Phi^T[j][t] = exp2(A^T + b_j - gamma |k_t|^2) (everything pre-scaled by
//            log2 e).  The feature warps read the accumulator into registers, add u_j += Phi
//            (fp32), split Phi into bf16 hi + lo (error ~2^-17) and store both over the
//            accumulator columns they have read, as A operands (two tokens per column).
//            There are three such accumulator / operand buffers, used by the tiles in turn.
//   GEMM 2   S^T[j][c] += sum_t Phi^T[j][t] v_t[c]   A operand: Phi^T hi, then lo, from
//            tensor memory; B operand: the value tile as TMA lands it (MN-major: dims
//            contiguous, tokens along K).  S^T accumulates in tensor memory over all tiles
//            of the CTA.
// (Stacking hi and lo along N, with the features passing through shared memory, was measured:
// an MMA with N = 256 takes twice as long as one with N = 128, and the extra shared-memory
// traffic slowed every MMA down.)
// With a feature cache (Sec. 4.2 notes that a cached implementation avoids the decode-side
// recompute) the feature warps also write every phi_k row they produce to global memory.
// Warp roles: 0 TMA producer, 1 GEMM-1 issuer, then the feature warps, four key-norm warps, the GEMM-2 issuer (an
// issuing thread advances only as fast as its MMAs execute, so with one issuer every barrier wait between
// the two GEMMs of a tile was idle time of the tensor pipe).
// Key and value tiles share one ring of shared-memory slots, filled in the order in which the
// tensor pipe consumes them.  GEMM 1 of tiles i+1 and i+2 runs into the other buffers while the
// feature warps work on tile i and GEMM 2 of tile i waits for them, so the tensor pipe works
// while the feature warps are busy.  Each CTA
// owns a contiguous range of tiles of one (sequence, KV head) unit (at most 256 tiles, which also
// bounds the rounding bias of a tensor-memory accumulation chain) and writes one partial; a second
// small kernel, launched as a programmatic dependent, adds the
// partials in chunk order.  Every device-side wait is bounded and reports through the
// status word.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr int kFWarps = 16;              // feature warps: four per tensor-memory lane quadrant
constexpr int kTPT = 128 * 4 / kFWarps;  // tokens of a tile per feature thread (its feature, a contiguous token group)
constexpr int kNG = kFWarps / 4;         // token groups of a tile
constexpr int kWarpNorm = 2 + kFWarps;   // first of the four norm warps
constexpr int kWarpG2 = kWarpNorm + 4;   // GEMM-2 issuer
constexpr int kBuildThreads = (kWarpG2 + 1) * 32;
constexpr int kBT = 128;                 // tokens per tile
constexpr int kBuildTmemCols = 512;
constexpr int kNB = 3;                   // accumulator / operand buffers in tensor memory
constexpr int kColBuf = 0;               // kNB buffers of 128 columns: GEMM-1 accumulator, then Phi^T hi / lo as the A operand
                                         // of GEMM 2 (per token group of a feature thread: its packed columns hi, then lo)
constexpr int kColD2 = kNB * 128;        // S^T accumulator, head_dim columns

__device__ __forceinline__ void tmem_st_x16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

template <int D>
struct BuildCfg {
  static constexpr int BOXES = D / 64;
  static constexpr int BOX = kBT * 128;                    // bytes of one 64-dim column block of a tile
  static constexpr int TILE = BOXES * BOX;                 // 32 KB (d = 128) or 16 KB (d = 64)
  static constexpr int NS = D == 128 ? 5 : 10;             // slots of the key/value ring (2 NS + 4 kNB + 2 barriers <= 40)
  static constexpr size_t whi = 0;                         // W_k hi / lo operand tiles: 128 feature rows x D dims, swizzled
  static constexpr size_t wlo = whi + TILE;
  static constexpr size_t ring = wlo + TILE;
  static constexpr size_t small = ring + (size_t)NS * TILE;
  // small: barriers (<= 40), snorm[kNB][128], misc; the per-group feature sums reuse the ring at the end
  static constexpr size_t total = small + 40 * 8 + 4 * (kNB * 128 + 16);
};

// MODE 0: features computed; 1: computed and also stored to the feature cache; 2: read from the
// feature cache (no key tiles, no GEMM 1): for feature maps evaluated elsewhere (mlp_features.cu).
template <int D, int MODE>
__global__ void __launch_bounds__(kBuildThreads, 1)
build_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
             const BuildProblem p) {
  using C = BuildCfg<D>;
  constexpr int NS = C::NS, BOXES = C::BOXES;
  constexpr int LPT = MODE == 2 ? 1 : 2;       // ring loads per tile
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* whi = smem + C::whi;
  unsigned char* wlo = smem + C::wlo;
  unsigned char* ring = smem + C::ring;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::small);
  uint64_t* full = bars;                   // [NS] tile landed
  uint64_t* empty = full + NS;             // [NS] the MMAs that read the slot are complete (and, for a key tile, its norms taken)
  uint64_t* d1_full = empty + NS;          // [kNB]  GEMM 1 accumulator complete
  uint64_t* buf_free = d1_full + kNB;      // [kNB]  GEMM 2 of the tile is complete: its buffer may take the next accumulator
  uint64_t* p_ready = buf_free + kNB;      // [kNB]  feature operand of the tile stored to tensor memory
  uint64_t* n_ready = p_ready + kNB;       // [kNB]  key norms of the tile in shared memory
  uint64_t* d2_full = n_ready + kNB;       // [1]  last GEMM 2 complete
  uint64_t* w_ready = d2_full + 1;         // [1]  W_k operand tiles converted
  float* snorm = reinterpret_cast<float*>(bars + 40);        // [kNB][128]  -gamma log2e |k_t|^2, -inf if masked
  float* ucomb = reinterpret_cast<float*>(ring);             // [kNG][128], written after the last MMA has read the ring
  int* misc = reinterpret_cast<int*>(snorm + kNB * 128);
  volatile int* s_abort = misc;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc + 1);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.z, kvh = blockIdx.y, chunk = blockIdx.x;
  const int R = p.n_feat;
  const int unit = b * p.n_kv_heads + kvh;
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, tail_of(p, b));
  float* S_out = p.S + (size_t)unit * D * R;
  float* u_out = p.u + (size_t)unit * R;
  pdl_launch_next();                       // the reduction kernel may be scheduled; it waits for this grid's completion
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
  // Ring loads are issued in the order in which the tensor pipe consumes the tiles: K0, K1, V0, K2, V1, ...,
  // V(last) (GEMM 1 of tile i+1 runs before GEMM 2 of tile i), so that no landed tile waits in a slot while a
  // later one is consumed.  Sequence numbers of the key and the value tile of tile i:
  auto seq_k = [&](int i) { return MODE == 2 ? 0 : (i == 0 ? 0 : 2 * i - 1); };
  auto seq_v = [&](int i) { return MODE == 2 ? i : (2 * i + 2 < 2 * n_my - 1 ? 2 * i + 2 : 2 * n_my - 1); };

  // ---- set-up: barriers and tensor memory first, so that the producer can start the key/value
  // stream while the other warps convert the W_k operand tiles (scaled by log2 e, hi + lo)
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int s = 0; s < kNB; ++s) {
      mbar_init(&p_ready[s], kFWarps); mbar_init(&n_ready[s], 4); mbar_init(&d1_full[s], 1); mbar_init(&buf_free[s], 1);
    }
    mbar_init(d2_full, 1);
    mbar_init(w_ready, kBuildThreads / 32 - 1);
    mbar_fence_init();
    *s_abort = 0;
  }
  if (warp == 1) tmem_alloc(s_tmem, kBuildTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  if (MODE != 2 && warp != 0) {
    const float* W = p.w_k + (size_t)kvh * R * D;
    constexpr int CPR = D / 8;
    for (int i = tid - 32; i < 128 * CPR; i += kBuildThreads - 32) {
      const int row = i / CPR, c = i % CPR;
      unsigned hw[4] = {0, 0, 0, 0}, lw[4] = {0, 0, 0, 0};
      if (row < R) {
        const float4 w0 = __ldg(reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8));
        const float4 w1 = __ldg(reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8 + 4));
        const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float a0 = w[2 * e] * kLog2e, a1 = w[2 * e + 1] * kLog2e;
          const __nv_bfloat162 hp = __floats2bfloat162_rn(a0, a1);
          const __nv_bfloat162 lp = __floats2bfloat162_rn(a0 - __bfloat162float(hp.x), a1 - __bfloat162float(hp.y));
          hw[e] = *reinterpret_cast<const uint32_t*>(&hp);
          lw[e] = *reinterpret_cast<const uint32_t*>(&lp);
        }
      }
      const uint32_t off = (c >> 3) * C::BOX + swz128(row, c & 7);
      *reinterpret_cast<uint4*>(whi + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      *reinterpret_cast<uint4*>(wlo + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(w_ready);
  }

  if (warp == 0) {
    // ================================================================ TMA producer
    if (lane == 0) {
      bool ok = true;
      int last_n[NS];                                      // last load issued into each slot
#pragma unroll
      for (int s = 0; s < NS; ++s) last_n[s] = -1;
      const uint64_t pol = l2_policy_evict_first();        // K and V are read once
      for (int n = 0; n < LPT * n_my && ok; ++n) {
        const int slot = n % NS;
        const bool is_key = MODE != 2 && n != 2 * n_my - 1 && (n == 0 || (n & 1) != 0);
        const int it = MODE == 2 ? n : (n == 0 ? 0 : n == 2 * n_my - 1 ? n_my - 1 : is_key ? (n + 1) / 2 : n / 2 - 1);
        const int row = row0 + (t0 + it) * kBT;
        ok = mbar_wait(&empty[slot], ((uint32_t)(n / NS) & 1u) ^ 1u, s_abort);
        if (!ok) break;
#pragma unroll
        for (int s = 0; s < NS; ++s)
          if (s == slot) last_n[s] = n;
        mbar_expect_tx(&full[slot], C::TILE);
#pragma unroll
        for (int x = 0; x < BOXES; ++x)
          tma_load_3d(ring + slot * C::TILE + x * C::BOX, is_key ? &tmap_k : &tmap_v, &full[slot], x * 64, row, kvh, pol);
      }
      if (!ok) {
        // every copy that was issued must land before shared memory is released
#pragma unroll
        for (int s = 0; s < NS; ++s)
          for (uint32_t w = 0; last_n[s] >= 0 && w < kWaitPolls; ++w) {
            if (mbar_try_wait(&full[s], (uint32_t)(last_n[s] / NS) & 1u)) break;
            __nanosleep(64);
          }
      }
    }
  } else if (warp == 1) {
    // ================================================================ GEMM-1 issuer
    if (MODE != 2 && lane == 0) {
      constexpr uint32_t idesc1 = umma_idesc_bf16(128, kBT, 0, 0);
      const uint64_t ring_k = umma_smem_desc(smem_u32(ring), 16, 1024);
      const uint64_t whi_d = umma_smem_desc(smem_u32(whi), 16, 1024);
      const uint64_t wlo_d = umma_smem_desc(smem_u32(wlo), 16, 1024);
      bool ok = mbar_wait(w_ready, 0, s_abort);
      tc_fence_after_sync();
      for (int it = 0; it < n_my && ok; ++it) {
        const int buf = it % kNB, nk = seq_k(it), ks = nk % NS;
        // the buffer is free once GEMM 2 of tile it - kNB has read its features
        ok = mbar_wait(&full[ks], (uint32_t)(nk / NS) & 1u, s_abort) &&
             (it < kNB || mbar_wait(&buf_free[buf], (uint32_t)(it / kNB - 1) & 1u, s_abort));
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t kd = ring_k + (uint64_t)((ks * C::TILE) >> 4);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint64_t wd = half == 0 ? whi_d : wlo_d;
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint64_t off = (uint64_t)(((k >> 2) * C::BOX + (k & 3) * 32) >> 4);
            umma_ss(tmem_base + kColBuf + buf * 128, wd + off, kd + off, idesc1, (half | k) ? 1u : 0u);
          }
        }
        tc_commit(&d1_full[buf]);
        // the slot is released once GEMM 1 is complete and the norm warps have read the tile
        ok = mbar_wait(&n_ready[buf], (uint32_t)(it / kNB) & 1u, s_abort);
        if (!ok) break;
        tc_commit(&empty[ks]);
      }
    }
  } else if (warp == kWarpG2) {
    // ================================================================ GEMM-2 issuer
    if (lane == 0) {
      constexpr uint32_t idesc2 = umma_idesc_bf16(128, D, 0, 1);
      // value tile as an MN-major operand: 64-dim column blocks BOX bytes apart, groups of
      // eight token rows 1024 bytes apart
      const uint64_t ring_v = umma_smem_desc(smem_u32(ring), C::BOX, 1024);
      bool ok = true;
      for (int j = 0; j < n_my && ok; ++j) {
        const int buf = j % kNB, nv = seq_v(j), vs = nv % NS;
        ok = mbar_wait(&p_ready[buf], (uint32_t)(j / kNB) & 1u, s_abort) &&
             mbar_wait(&full[vs], (uint32_t)(nv / NS) & 1u, s_abort);
        if (!ok) break;
        tc_fence_after_sync();
        const uint64_t vd = ring_v + (uint64_t)((vs * C::TILE) >> 4);
#pragma unroll
        for (int kk = 0; kk < kBT / 16; ++kk) {
          // tokens 16 kk .. 16 kk + 15: eight packed columns of Phi hi, then of Phi lo, against sixteen rows of the value tile
          const uint64_t bd = vd + (uint64_t)((kk * 16 * 128) >> 4);
          const uint32_t a_col = kColBuf + buf * 128 + (kk * 16 / kTPT) * kTPT + (kk * 16 % kTPT) / 2;
          umma_ts(tmem_base + kColD2, tmem_base + a_col, bd, idesc2, (j > 0 || kk > 0) ? 1u : 0u);
          umma_ts(tmem_base + kColD2, tmem_base + a_col + kTPT / 2, bd, idesc2, 1u);
        }
        tc_commit(&empty[vs]);
        tc_commit(&buf_free[buf]);
      }
      if (ok) tc_commit(d2_full);
    }
  } else if (warp < kWarpNorm) {
    // ================================================================ feature warps
    const int quad = warp & 3;                     // tensor-memory lane quadrant
    const int g = (warp - 2) >> 2;                 // which token group of the tile
    const int j = quad * 32 + lane;                // feature
    const float bj = (MODE != 2 && j < R) ? p.b_k[(size_t)kvh * R + j] * kLog2e : 0.f;
    float u_acc = 0.f;                             // sum of feature j over this thread's tokens
    // feature cache (written in mode 1, read in mode 2): row of mid token 0 of this head, column j
    float* cache_j = (MODE != 0 && j < R) ? p.phi_cache + ((size_t)kvh * p.total_tokens + (size_t)row0) * R + j : nullptr;
    bool ok = true;
    for (int it = 0; it < n_my && ok; ++it) {
      const int buf = it % kNB;
      const uint32_t ph = (uint32_t)(it / kNB) & 1u;
      // mode 2 has no GEMM 1 whose issuer would wait for the buffer
      ok = (MODE == 2 ? (it < kNB || mbar_wait(&buf_free[buf], (uint32_t)(it / kNB - 1) & 1u, s_abort))
                      : mbar_wait(&d1_full[buf], ph, s_abort)) &&
           mbar_wait(&n_ready[buf], ph, s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const float* sn = snorm + buf * 128 + g * kTPT;
      uint32_t hi[kTPT / 2], lo[kTPT / 2];         // this thread's tokens, packed in pairs
      float vv[kTPT / 32][32];
      if (MODE != 2) {
        // this thread's whole accumulator slice into registers: the features go over the same columns
#pragma unroll
        for (int c = 0; c < kTPT / 32; ++c)
          tmem_ld_x32(tmem_addr(tmem_base, quad * 32, kColBuf + buf * 128 + g * kTPT + c * 32), vv[c]);
        tc_wait_ld();
      }
#pragma unroll
      for (int c = 0; c < kTPT / 32; ++c) {
        float (&v)[32] = vv[c];
        if (MODE == 2) {
          // snorm says which tokens are in the mid-region
          const int tok0 = (t0 + it) * kBT + g * kTPT + c * 32;
#pragma unroll
          for (int e = 0; e < 32; ++e)
            v[e] = (cache_j != nullptr && sn[c * 32 + e] == 0.f) ? __ldcs(cache_j + (size_t)(tok0 + e) * R) : 0.f;
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float f0 = MODE == 2 ? v[2 * e] : ex2_approx(v[2 * e] + bj + sn[c * 32 + 2 * e]);
          const float f1 = MODE == 2 ? v[2 * e + 1] : ex2_approx(v[2 * e + 1] + bj + sn[c * 32 + 2 * e + 1]);
          u_acc += f0;
          u_acc += f1;
          const __nv_bfloat162 hp = __floats2bfloat162_rn(f0, f1);          // .x (low half) = even token
          const __nv_bfloat162 lp =
              __floats2bfloat162_rn(f0 - __bfloat162float(hp.x), f1 - __bfloat162float(hp.y));
          hi[c * 16 + e] = *reinterpret_cast<const uint32_t*>(&hp);
          lo[c * 16 + e] = *reinterpret_cast<const uint32_t*>(&lp);
          if (MODE == 1 && cache_j) {
            // one token per store: the 32 lanes of the warp write 32 consecutive features
            const int tok = (t0 + it) * kBT + g * kTPT + c * 32 + 2 * e;
            if (tok < n_mid) __stcs(cache_j + (size_t)tok * R, f0);
            if (tok + 1 < n_mid) __stcs(cache_j + (size_t)(tok + 1) * R, f1);
          }
        }
      }
      // over the columns this thread has read: packed columns hi (column c = tokens 2c, 2c + 1 of the group), then lo
#pragma unroll
      for (int c = 0; c < kTPT / 32; ++c) {
        tmem_st_x16(tmem_addr(tmem_base, quad * 32, kColBuf + buf * 128 + g * kTPT + c * 16), *reinterpret_cast<const uint32_t(*)[16]>(&hi[c * 16]));
        tmem_st_x16(tmem_addr(tmem_base, quad * 32, kColBuf + buf * 128 + g * kTPT + kTPT / 2 + c * 16), *reinterpret_cast<const uint32_t(*)[16]>(&lo[c * 16]));
      }
      tc_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_ready[buf]);
    }
    // ---- S^T of this CTA's tiles -> partial (thread = feature; the first two token groups' warps take half of the dims each)
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(d2_full, 0, s_abort));
    if (ok) {
      tc_fence_after_sync();
      float* part = p.partials + ((size_t)unit * p.chunks_per_unit + chunk) * ((size_t)D * R + R);
      constexpr int HALF = D / 2;
#pragma unroll
      for (int c = 0; c < HALF / 32; ++c) {
        if (g < 2) {                                 // warp-uniform
          float v[32];
          tmem_ld_x32(tmem_addr(tmem_base, quad * 32, kColD2 + g * HALF + c * 32), v);
          tc_wait_ld();
          if (j < R) {
#pragma unroll
            for (int e = 0; e < 32; ++e) part[(size_t)(g * HALF + c * 32 + e) * R + j] = v[e];
          }
        }
      }
      ucomb[g * 128 + j] = u_acc;
    }
  } else {
    // ================================================================ key norms and masking
    const int t = (warp - kWarpNorm) * 32 + lane;  // token of the tile
    const float g2 = p.gamma_k * kLog2e;
    bool ok = true;
    for (int it = 0; it < n_my && ok; ++it) {
      const int buf = it % kNB, nk = seq_k(it), ks = nk % NS;
      // snorm[buf] was last read by the feature warps for tile it - kNB: wait for their p_ready
      ok = (MODE == 2 || mbar_wait(&full[ks], (uint32_t)(nk / NS) & 1u, s_abort)) &&
           mbar_wait(&p_ready[buf], ((uint32_t)(it / kNB) & 1u) ^ 1u, s_abort);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const unsigned char* tile = ring + ks * C::TILE;
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
      if (lane == 0) mbar_arrive(&n_ready[buf]);             // the GEMM-1 issuer releases the key slot after this
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
  if (tid < R) {
    float us = 0.f;
#pragma unroll
    for (int g = 0; g < kNG; ++g) us += ucomb[g * 128 + tid];
    part[(size_t)D * R + tid] = us;
  }
}

// Adds the chunk partials of every unit in chunk order (fixed order: run-to-run identical).
// Launched as a programmatic dependent of the build kernel: waits for that grid first.
constexpr int kRedThreads = 256;
__global__ void __launch_bounds__(kRedThreads) build_reduce_kernel(const BuildProblem p) {
  pdl_wait();
  const int unit = blockIdx.y, b = unit / p.n_kv_heads;
  const int D = p.head_dim, R = p.n_feat, n_out = D * R + R;
  const long long len_b = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
  const int n_mid = mid_len(len_b, p.n_sink, tail_of(p, b));
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
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((n_out + kRedThreads - 1) / kRedThreads, p.n_kv_heads * p.batch, 1);
  cfg.blockDim = dim3(kRedThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, build_reduce_kernel, p);
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
