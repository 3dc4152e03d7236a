// Step (1) of the decode path: score every mid-region key against the G query
// heads of its KV-head group (s_i = q.k_i / sqrt(d_h), Sec. 3 Eq. full_attention)
// and select, per query head, the K highest-scoring mid-region indices with ties
// broken towards the lower index (exhaustive Top-K control selector, Sec. 5.1).
//
// Three kernels:
//   score_hist_kernel      streams the keys once (TMA-staged 128B-swizzled tiles, 4-stage
//                          mbarrier ring), writes fp32 scores and a 4096-bin histogram of the
//                          leading 12 bits of the order-preserving score key; the last
//                          CTA to finish a (sequence, KV head) unit turns the histogram
//                          into a threshold bin per query head.
//   partition_kernel       one pass over the (L2-resident) scores: bitmaps of positions
//                          above the threshold bin ("sure") and inside it ("candidates").
//   finalize_select_kernel one CTA per query head: radix-refines the remaining 20 key
//                          bits among the candidates, resolves exact ties in index
//                          order, and writes the ascending index list.
#include "common.cuh"

namespace tkphi {

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      " .reg .pred p;\n"
      " mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.b32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (each poll may itself suspend
// for a hardware-defined time), so a copy that never lands cannot hang the GPU.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 32) __nanosleep(64);
  }
  return false;
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* tm, uint64_t* bar, int c0, int c1,
                                            int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(smem_u32(dst)),
      "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// ------------------------------------------------------------------ score + histogram
constexpr int kScoreThreads = 256;
constexpr int kScoreStages = 4;
constexpr int kScoreTileBytes = 32768;

template <int D>
struct ScoreCfg {
  static constexpr int LPK = D / 32;                   // lanes sharing one key (32 dims each)
  static constexpr int KPP = kScoreThreads / LPK;      // keys per pass of the CTA
  static constexpr int TK = 2 * KPP;                   // keys per tile: two per thread
  static_assert(TK * D * 2 == kScoreTileBytes, "tile size");
};

struct TileCursor {
  int b, kvh, t, nt;   // sequence, KV head, tile in unit, tiles per unit of sequence b
};

// pre[b] = n_kv_heads * (tiles of sequences before b); tiles of b = (pre[b+1]-pre[b])/n_kv_heads
__device__ __forceinline__ void cursor_seek(TileCursor& c, const int* pre, int batch, int n_kv, int f) {
  int lo = 0, hi = batch - 1;       // largest b with pre[b] <= f
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (pre[mid] <= f) lo = mid; else hi = mid - 1;
  }
  // skip empty sequences that share the same prefix value
  while (lo < batch - 1 && pre[lo + 1] <= f) ++lo;
  c.b = lo;
  c.nt = (pre[lo + 1] - pre[lo]) / n_kv;
  int rem = f - pre[lo];
  c.kvh = c.nt ? rem / c.nt : 0;
  c.t = c.nt ? rem % c.nt : 0;
}
__device__ __forceinline__ void cursor_next(TileCursor& c, const int* pre, int batch, int n_kv) {
  if (++c.t < c.nt) return;
  c.t = 0;
  if (++c.kvh < n_kv) return;
  c.kvh = 0;
  do {
    ++c.b;
    c.nt = c.b < batch ? (pre[c.b + 1] - pre[c.b]) / n_kv : 1;
  } while (c.nt == 0);
}

template <int D, int G>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_hist_kernel(const __grid_constant__ CUtensorMap tmap_k, const Problem p, const int g0, const int pass) {
  using C = ScoreCfg<D>;
  constexpr int LPK = C::LPK, KPP = C::KPP, TK = C::TK;
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* tiles = smem;                                              // [stages][32 KB]
  unsigned* hist_s = reinterpret_cast<unsigned*>(smem + kScoreStages * kScoreTileBytes);  // [G][bins]
  int* pre = reinterpret_cast<int*>(hist_s + G * kHistBins);               // [batch+1]
  uint64_t* full = reinterpret_cast<uint64_t*>(pre + kMaxBatch + 1 + ((kMaxBatch + 1) & 1));
  int* scratch = reinterpret_cast<int*>(full + kScoreStages);              // [40]
  int* s_flag = scratch + 36;

  const int tid = threadIdx.x, lane = tid & 31;
  const int n_kv = p.n_kv_heads, batch = p.batch;

  // ---- tiles per sequence -> prefix in shared memory
  {
    const int per = (batch + kScoreThreads - 1) / kScoreThreads;
    const int b0 = tid * per;
    int local = 0;
    for (int i = 0; i < per; ++i) {
      int b = b0 + i;
      if (b < batch) {
        int nm = mid_len(p.cu_seqlens[b + 1] - p.cu_seqlens[b], p.n_sink, p.n_tail);
        int nt = (p.topk[b] > 0) ? (nm + TK - 1) / TK : 0;
        local += nt * n_kv;
      }
    }
    int total;
    int excl = block_exclusive_scan(local, scratch, &total);
    int run = excl;
    for (int i = 0; i < per; ++i) {
      int b = b0 + i;
      if (b < batch) {
        pre[b] = run;
        int nm = mid_len(p.cu_seqlens[b + 1] - p.cu_seqlens[b], p.n_sink, p.n_tail);
        int nt = (p.topk[b] > 0) ? (nm + TK - 1) / TK : 0;
        run += nt * n_kv;
      }
    }
    if (tid == 0) pre[batch] = total;
  }
  for (int i = tid; i < G * kHistBins; i += kScoreThreads) hist_s[i] = 0;
  if (tid == 0) {
    for (int s = 0; s < kScoreStages; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int F = pre[batch];
  const int f0 = (int)((long long)F * blockIdx.x / gridDim.x);
  const int f1 = (int)((long long)F * (blockIdx.x + 1) / gridDim.x);
  if (f0 >= f1) return;

  // ---- producer prologue (thread 0): fill the ring
  TileCursor pc;   // producer cursor (thread 0 only)
  int issued = 0;
  if (tid == 0) {
    cursor_seek(pc, pre, batch, n_kv, f0);
    for (; issued < kScoreStages && f0 + issued < f1; ++issued) {
      mbar_expect_tx(&full[issued], kScoreTileBytes);
      int row = (int)(p.cu_seqlens[pc.b] + p.n_sink) + pc.t * TK;
#pragma unroll
      for (int x = 0; x < D / 64; ++x)
        tma_load_3d(tiles + issued * kScoreTileBytes + x * (TK * 128), &tmap_k, &full[issued], x * 64, row, pc.kvh);
      cursor_next(pc, pre, batch, n_kv);
    }
  }

  // ---- per-thread geometry.  Tiles are stored with the 128-byte TMA swizzle: the
  // 16-byte chunk c of row r sits at chunk position c ^ (r & 7).  The eight lanes
  // of a shared-memory access phase read the same logical chunk of eight
  // consecutive rows, so they hit eight different positions: no bank conflicts,
  // and every key is accumulated in the same (natural) order wherever it sits.
  constexpr int KPW = 32 / LPK;             // keys per warp and pass
  const int s = lane / KPW;                 // 32-dim slice of the key handled by this lane
  const int kk = (tid >> 5) * KPW + (lane % KPW);   // key within a pass
  const int sub_off = (s >> 1) * (TK * 128);        // D = 128: second 64-dim half is a second box
  int coff[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) coff[c] = ((((s & 1) * 4 + c) ^ (kk & 7)) << 4);
  const int offA = sub_off + kk * 128, offB = sub_off + (kk + KPP) * 128;   // KPP % 8 == 0

  TileCursor cc;
  cursor_seek(cc, pre, batch, n_kv, f0);
  int cur_b = -1, cur_kvh = -1, tiles_done = 0, n_mid = 0;
  long long row_base0 = 0, len_b = 0;
  float qreg[G][32];
  bool timed_out = false;

  auto finish_unit = [&]() {
    // publish this CTA's share of the unit's histogram, then take a ticket
    const int row0 = cur_b * p.n_q_heads + cur_kvh * p.group + g0;
    for (int i = tid; i < G * kHistBins; i += kScoreThreads) {
      unsigned h = hist_s[i];
      if (h) {
        atomicAdd(&p.hist[(size_t)(row0 + i / kHistBins) * kHistBins + (i % kHistBins)], h);
        hist_s[i] = 0;
      }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const int unit = cur_b * n_kv + cur_kvh;
      const unsigned nt_unit = (unsigned)((pre[cur_b + 1] - pre[cur_b]) / n_kv);
      unsigned prev = atomicAdd(&p.unit_counter[(size_t)pass * batch * n_kv + unit], (unsigned)tiles_done);
      *s_flag = (prev + (unsigned)tiles_done == nt_unit) ? 1 : 0;
    }
    __syncthreads();
    if (*s_flag) {
      // last CTA of the unit: threshold bin per query head from the full histogram
      __threadfence();
      const int K = p.topk[cur_b];
      for (int g = 0; g < G; ++g) {
        const unsigned* h = p.hist + (size_t)(row0 + g) * kHistBins + tid * 16;
        unsigned loc[16];
        int lsum = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) { loc[i] = __ldcg(h + i); lsum += (int)loc[i]; }
        int total;
        int excl = block_exclusive_scan(lsum, scratch, &total);
        int above = total - excl - lsum;          // elements in bins above this thread's 16
        if (above < K && K <= above + lsum) {
          int cum = above;
#pragma unroll
          for (int i = 15; i >= 0; --i) {
            if (cum < K && K <= cum + (int)loc[i]) p.rowinfo[row0 + g] = make_int4(tid * 16 + i, cum, (int)loc[i], total);
            cum += (int)loc[i];
          }
        }
      }
    }
    __syncthreads();
    tiles_done = 0;
  };

  const int n_my = f1 - f0;
  for (int it = 0; it < n_my; ++it) {
    if (cc.b != cur_b || cc.kvh != cur_kvh) {
      if (cur_b >= 0) finish_unit();
      cur_b = cc.b; cur_kvh = cc.kvh;
      const long long cu_b = p.cu_seqlens[cur_b];
      len_b = p.cu_seqlens[cur_b + 1] - cu_b;
      n_mid = mid_len(len_b, p.n_sink, p.n_tail);
      row_base0 = score_row_base(p, cur_b, cur_kvh * p.group + g0, cu_b, len_b);
      // this lane's 32-dim slice of the G queries
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const __nv_bfloat16* qp = p.q + ((size_t)cur_b * p.n_q_heads + cur_kvh * p.group + g0 + g) * D + s * 32;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint4 raw = *reinterpret_cast<const uint4*>(qp + (c << 3));
          const unsigned w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            qreg[g][c * 8 + 2 * e] = bf16_lo(w[e]);
            qreg[g][c * 8 + 2 * e + 1] = bf16_hi(w[e]);
          }
        }
      }
    }
    const int slot = it % kScoreStages;
    const uint32_t parity = (uint32_t)(it / kScoreStages) & 1u;
    if (!mbar_wait_bounded(&full[slot], parity)) timed_out = true;

    const unsigned char* tile = tiles + slot * kScoreTileBytes;
    float acc[2][G];
#pragma unroll
    for (int g = 0; g < G; ++g) { acc[0][g] = 0.f; acc[1][g] = 0.f; }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint4 ra = *reinterpret_cast<const uint4*>(tile + offA + coff[c]);
      const uint4 rb = *reinterpret_cast<const uint4*>(tile + offB + coff[c]);
      const unsigned wa[4] = {ra.x, ra.y, ra.z, ra.w};
      const unsigned wb[4] = {rb.x, rb.y, rb.z, rb.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a0 = bf16_lo(wa[e]), a1 = bf16_hi(wa[e]);
        const float b0 = bf16_lo(wb[e]), b1 = bf16_hi(wb[e]);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          acc[0][g] = fmaf(a0, qreg[g][c * 8 + 2 * e], acc[0][g]);
          acc[0][g] = fmaf(a1, qreg[g][c * 8 + 2 * e + 1], acc[0][g]);
          acc[1][g] = fmaf(b0, qreg[g][c * 8 + 2 * e], acc[1][g]);
          acc[1][g] = fmaf(b1, qreg[g][c * 8 + 2 * e + 1], acc[1][g]);
        }
      }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
      for (int o = KPW; o < 32; o <<= 1) {
        acc[0][g] += __shfl_xor_sync(0xffffffffu, acc[0][g], o);
        acc[1][g] += __shfl_xor_sync(0xffffffffu, acc[1][g], o);
      }
    }
    // lane with slice s writes heads g == s (mod LPK)
    const int jA = cc.t * TK + kk, jB = jA + KPP;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      if ((g % LPK) == s) {
        float* srow = p.scores + row_base0 + (long long)g * len_b;
        if (jA < n_mid) {
          const float sc = acc[0][g] * p.scale;
          srow[jA] = sc;
          atomicAdd(&hist_s[g * kHistBins + (ordered_key(sc) >> kLowBits)], 1u);
        }
        if (jB < n_mid) {
          const float sc = acc[1][g] * p.scale;
          srow[jB] = sc;
          atomicAdd(&hist_s[g * kHistBins + (ordered_key(sc) >> kLowBits)], 1u);
        }
      }
    }
    ++tiles_done;
    cursor_next(cc, pre, batch, n_kv);
    // everyone is done with this slot: refill it, or bail out together on a timeout
    if (__syncthreads_or(timed_out ? 1 : 0)) {
      if (tid == 0) atomicExch(p.status, kStatusTimeout);
      // wait (bounded) for copies still in flight before giving the shared memory back
      if (tid == 0)
        for (int j = it + 1; j < issued; ++j)
          mbar_wait_bounded(&full[j % kScoreStages], (uint32_t)(j / kScoreStages) & 1u);
      __syncthreads();
      return;
    }
    if (tid == 0 && f0 + issued < f1) {
      mbar_expect_tx(&full[slot], kScoreTileBytes);
      int row = (int)(p.cu_seqlens[pc.b] + p.n_sink) + pc.t * TK;
#pragma unroll
      for (int x = 0; x < D / 64; ++x)
        tma_load_3d(tiles + slot * kScoreTileBytes + x * (TK * 128), &tmap_k, &full[slot], x * 64, row, pc.kvh);
      cursor_next(pc, pre, batch, n_kv);
      ++issued;
    }
  }
  finish_unit();
}

static size_t score_smem_bytes(int G) {
  return (size_t)kScoreStages * kScoreTileBytes + (size_t)G * kHistBins * 4 + (size_t)(kMaxBatch + 2) * 4 +
         kScoreStages * 8 + 40 * 4 + 64;
}

template <int D, int G>
static cudaError_t launch_score_t(const Problem& p, const CUtensorMap& tm, int g0, int pass, int n_sm,
                                  cudaStream_t st) {
  static bool configured = false;   // attribute is per function; cheap to set once
  const size_t smem = score_smem_bytes(G);
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(score_hist_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  score_hist_kernel<D, G><<<n_sm, kScoreThreads, smem, st>>>(tm, p, g0, pass);
  return cudaGetLastError();
}

cudaError_t launch_score_hist(const Problem& p, const CUtensorMap& tm, int pass, int n_sm, cudaStream_t st) {
  const int g0 = pass * 4;
  const int g = p.group - g0 < 4 ? p.group - g0 : 4;
#define TKPHI_DISPATCH(DD, GG) \
  if (p.head_dim == DD && g == GG) return launch_score_t<DD, GG>(p, tm, g0, pass, n_sm, st);
  TKPHI_DISPATCH(64, 1) TKPHI_DISPATCH(64, 2) TKPHI_DISPATCH(64, 3) TKPHI_DISPATCH(64, 4)
  TKPHI_DISPATCH(128, 1) TKPHI_DISPATCH(128, 2) TKPHI_DISPATCH(128, 3) TKPHI_DISPATCH(128, 4)
#undef TKPHI_DISPATCH
  return cudaErrorInvalidValue;
}

// ------------------------------------------------------------------ partition into bitmaps
constexpr int kPartThreads = 256;
constexpr int kPartChunk = kPartThreads * 32;      // scores per CTA: each warp 32 words

__global__ void __launch_bounds__(kPartThreads) partition_kernel(const Problem p) {
  const int b = blockIdx.z, hq = blockIdx.y;
  const int K = p.topk[b];
  if (K == 0) return;
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  const int chunk0 = blockIdx.x * kPartChunk;
  if (chunk0 >= n_mid) return;
  const int row = b * p.n_q_heads + hq;
  const unsigned tb = (unsigned)p.rowinfo[row].x;
  const float* srow = p.scores + score_row_base(p, b, hq, cu_b, len_b);
  const long long wbase = bitmap_row_base(p, b, hq, cu_b, len_b);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int base = chunk0 + warp * 1024;
  if (base >= n_mid) return;
  unsigned my_sure = 0, my_cand = 0;
#pragma unroll 4
  for (int it = 0; it < 32; ++it) {
    const int j = base + it * 32 + lane;
    bool sure = false, cand = false;
    if (j < n_mid) {
      const unsigned bin = ordered_key(srow[j]) >> kLowBits;
      sure = bin > tb;
      cand = bin == tb;
    }
    const unsigned ws = __ballot_sync(0xffffffffu, sure);
    const unsigned wc = __ballot_sync(0xffffffffu, cand);
    if (lane == it) { my_sure = ws; my_cand = wc; }
  }
  const int word = (base >> 5) + lane;
  if (word * 32 < n_mid) {
    p.bm_sure[wbase + word] = my_sure;
    p.bm_cand[wbase + word] = my_cand;
  }
}

cudaError_t launch_partition(const Problem& p, int max_mid, cudaStream_t st) {
  if (max_mid <= 0) return cudaSuccess;
  dim3 grid((max_mid + kPartChunk - 1) / kPartChunk, p.n_q_heads, p.batch);
  partition_kernel<<<grid, kPartThreads, 0, st>>>(p);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ finalize selection
constexpr int kFinThreads = 512;
constexpr int kRefBins = 1 << (kLowBits / 2);      // 1024: two refinement digits of 10 bits

// Walks a 1024-bin histogram from the top and returns the digit at which the
// cumulative count reaches `need`; *rem = how many are still needed inside it.
__device__ int find_digit(const unsigned* h, int need, int* rem, int* scratch) {
  __shared__ int s_digit, s_rem;
  const int tid = threadIdx.x;
  // thread t owns bins [2t, 2t+1] of 1024 with 512 threads
  const int c0 = (int)h[2 * tid], c1 = (int)h[2 * tid + 1];
  int total;
  const int excl = block_exclusive_scan(c0 + c1, scratch, &total);
  const int above = total - excl - (c0 + c1);
  if (above < need && need <= above + c1) { s_digit = 2 * tid + 1; s_rem = need - above; }
  else if (above + c1 < need && need <= above + c1 + c0) { s_digit = 2 * tid; s_rem = need - above - c1; }
  __syncthreads();
  *rem = s_rem;
  return s_digit;
}

__global__ void __launch_bounds__(kFinThreads) finalize_select_kernel(const Problem p) {
  __shared__ unsigned h[kRefBins];
  __shared__ int scratch[40];
  const int row = blockIdx.x, b = row / p.n_q_heads, hq = row % p.n_q_heads;
  const int tid = threadIdx.x;
  const int D = p.head_dim, r = p.n_feat;

  // ---- query-side log-features a_q = W_q q + b_q - gamma_q |q|^2 (Sec. 4.1), kept as
  // exp(a_q - m_q) and m_q so that tiny features cannot underflow the merge.
  if (p.with_phi) {
    float* aq = p.aq + (size_t)row * (r + 4);
    const __nv_bfloat16* qp = p.q + (size_t)row * D;
    const float* W = p.w_q + (size_t)hq * r * D;
    const int lane = tid & 31, warp = tid >> 5;
    float qn = 0.f;
    for (int c = lane; c < D; c += 32) { float x = __bfloat162float(qp[c]); qn = fmaf(x, x, qn); }
    qn = warp_sum(qn);
    for (int j = warp; j < r; j += kFinThreads / 32) {
      float a = 0.f;
      for (int c = lane; c < D; c += 32) a = fmaf(W[(size_t)j * D + c], __bfloat162float(qp[c]), a);
      a = warp_sum(a);
      if (lane == 0) aq[j] = a + p.b_q[(size_t)hq * r + j] - p.gamma_q * qn;
    }
    __syncthreads();
    if (tid < 32) {
      float m = -INFINITY;
      for (int j = tid; j < r; j += 32) m = fmaxf(m, aq[j]);
      m = warp_max(m);
      for (int j = tid; j < r; j += 32) aq[j] = expf(aq[j] - m);
      if (tid == 0) aq[r] = m;
    }
    __syncthreads();
  }

  const int K = p.topk[b];
  int* out = p.idx + (size_t)row * p.topk_max;
  int* out2 = p.idx_out ? p.idx_out + (size_t)row * p.topk_max : nullptr;
  if (out2)
    for (int i = K + tid; i < p.topk_max; i += kFinThreads) out2[i] = -1;
  if (K == 0) return;

  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  const int n_words = (n_mid + 31) >> 5;
  const float* srow = p.scores + score_row_base(p, b, hq, cu_b, len_b);
  unsigned* sure = p.bm_sure + bitmap_row_base(p, b, hq, cu_b, len_b);
  unsigned* cand = p.bm_cand + bitmap_row_base(p, b, hq, cu_b, len_b);
  const int4 info = p.rowinfo[row];
  const int need = K - info.y;                 // candidates to take, 1 <= need <= info.z
  const int n_cand = info.z;

  unsigned tau_low = 0;                        // low 20 bits of the threshold key
  int need_ties = n_cand;                      // ties to admit, in index order
  const bool refine = need < n_cand;
  if (refine) {
    // digit 1: bits 19..10 of the key among the candidates
    for (int i = tid; i < kRefBins; i += kFinThreads) h[i] = 0;
    __syncthreads();
    for (int w = tid; w < n_words; w += kFinThreads) {
      unsigned bits = cand[w];
      while (bits) {
        const int j = (w << 5) + __ffs(bits) - 1;
        bits &= bits - 1;
        atomicAdd(&h[(ordered_key(srow[j]) >> 10) & (kRefBins - 1)], 1u);
      }
    }
    __syncthreads();
    int rem1;
    const unsigned d1 = (unsigned)find_digit(h, need, &rem1, scratch);
    __syncthreads();
    // digit 2: bits 9..0 among candidates whose digit 1 matches
    for (int i = tid; i < kRefBins; i += kFinThreads) h[i] = 0;
    __syncthreads();
    for (int w = tid; w < n_words; w += kFinThreads) {
      unsigned bits = cand[w];
      while (bits) {
        const int j = (w << 5) + __ffs(bits) - 1;
        bits &= bits - 1;
        const unsigned key = ordered_key(srow[j]);
        if (((key >> 10) & (kRefBins - 1)) == d1) atomicAdd(&h[key & (kRefBins - 1)], 1u);
      }
    }
    __syncthreads();
    int rem2;
    const unsigned d2 = (unsigned)find_digit(h, rem1, &rem2, scratch);
    tau_low = (d1 << 10) | d2;
    need_ties = rem2;
  }

  // ---- final pass: thread t owns the contiguous words [w0, w1)
  const int wpt = (n_words + kFinThreads - 1) / kFinThreads;
  const int w0 = min(tid * wpt, n_words), w1 = min(w0 + wpt, n_words);
  const unsigned low_mask = (1u << kLowBits) - 1u;
  int my_ties = 0;
  if (refine) {
    for (int w = w0; w < w1; ++w) {
      unsigned bits = cand[w], def = sure[w], tie = 0;
      while (bits) {
        const int bit = __ffs(bits) - 1;
        bits &= bits - 1;
        const unsigned low = ordered_key(srow[(w << 5) + bit]) & low_mask;
        if (low > tau_low) def |= 1u << bit;
        else if (low == tau_low) tie |= 1u << bit;
      }
      sure[w] = def;
      cand[w] = tie;
      my_ties += __popc(tie);
    }
  } else {
    for (int w = w0; w < w1; ++w) my_ties += __popc(cand[w]);
  }
  int total_ties;
  int tie_rank = block_exclusive_scan(my_ties, scratch, &total_ties);
  int my_count = 0;
  for (int w = w0; w < w1; ++w) {
    unsigned tie = cand[w], fin = sure[w];
    while (tie && tie_rank < need_ties) {
      fin |= tie & (0u - tie);                 // lowest set bit: lowest index first
      tie &= tie - 1;
      ++tie_rank;
    }
    tie_rank += __popc(tie);
    sure[w] = fin;
    my_count += __popc(fin);
  }
  int total_sel;
  int off = block_exclusive_scan(my_count, scratch, &total_sel);
  for (int w = w0; w < w1; ++w) {
    unsigned fin = sure[w];
    while (fin) {
      const int bit = __ffs(fin) - 1;
      fin &= fin - 1;
      const int pos = p.n_sink + (w << 5) + bit;
      if (off < K) {
        out[off] = pos;
        if (out2) out2[off] = pos;
      }
      ++off;
    }
  }
}

cudaError_t launch_finalize_select(const Problem& p, cudaStream_t st) {
  finalize_select_kernel<<<p.batch * p.n_q_heads, kFinThreads, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace tkphi
