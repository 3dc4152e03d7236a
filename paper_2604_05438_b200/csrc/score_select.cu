// Step (1) of the decode path: score every mid-region key against the G query
// heads of its KV-head group (s_i = q.k_i / sqrt(d_h), Sec. 3 Eq. full_attention)
// and select, per query head, the K highest-scoring mid-region indices with ties
// broken towards the lower index (exhaustive Top-K control selector, Sec. 5.1).
//
// Three kernels:
//   score_hist_kernel      streams the keys once.  A producer thread issues TMA loads of
//                          128B-swizzled 32 KB key tiles into a 4-stage mbarrier ring; one
//                          thread issues tcgen05.mma with the key tile as the A operand
//                          straight from shared memory and the group's queries (zero padded
//                          to 16 rows) as B, so the dot products cost no issue slots of the
//                          CUDA cores; four warps read the 128 x 16 fp32 accumulators back
//                          from tensor memory, write the score rows and add to a 4096-bin
//                          histogram of the leading 12 bits of the order-preserving score
//                          key.  The last CTA to finish a (sequence, KV head) unit turns the
//                          histogram into a threshold bin per query head.
//   compact_kernel         one pass over the (L2-resident) scores: a bitmap of positions above
//                          the threshold bin and, per 4096-score chunk, the ordered list of
//                          positions inside it.  Spare CTAs evaluate the query-side
//                          log-features and split W_k into bf16 operand tiles for the
//                          retrieved-key feature recompute.
//   finalize_select_kernel one CTA per query head: radix-refines the remaining 20 key bits
//                          among the candidates (in shared memory), admits exact ties in index
//                          order, and expands the final bitmap into the ascending index list.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

// ------------------------------------------------------------------ score + histogram
constexpr int kScoreThreads = 192;        // warp 0: TMA producer, warp 1: MMA issuer, warps 2..5: read-back
constexpr int kScoreStages = 4;
constexpr int kScoreTileBytes = 32768;
constexpr int kAccStages = 4;             // accumulator buffers in tensor memory
constexpr int kScoreN = 16;               // MMA N: query heads of the group, zero padded
constexpr int kEpiThreads = 128;

template <int D>
struct ScoreCfg {
  static constexpr int TK = kScoreTileBytes / (2 * D);   // keys per TMA tile
  static constexpr int SUB = TK / 128;                   // 128-key MMA tiles per TMA tile
  static constexpr int BOXES = D / 64;                   // 64-dim (128-byte) column blocks
  static constexpr int BOX_BYTES = TK * 128;
  static constexpr int QBOX_BYTES = kScoreN * 128;
  static_assert(TK * D * 2 == kScoreTileBytes && SUB >= 1, "tile size");
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

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// True iff `x` holds on all 128 read-back threads (a barrier among them).
__device__ __forceinline__ bool epi_all(bool x) {
  uint32_t r;
  asm volatile(
      "{\n"
      " .reg .pred p, q;\n"
      " setp.ne.b32 q, %1, 0;\n"
      " bar.red.and.pred p, 1, 128, q;\n"
      " selp.b32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(r)
      : "r"(x ? 1u : 0u)
      : "memory");
  return r != 0;
}

// Exclusive prefix sum over the 128 read-back threads (et = 0..127); scratch >= 8 ints.
__device__ __forceinline__ int epi_exclusive_scan(int x, int et, int* scratch, int* total) {
  const int lane = et & 31, w = et >> 5;
  int incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  epi_sync();
  if (lane == 31) scratch[w] = incl;
  epi_sync();
  int base = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int s = scratch[i];
    if (i < w) base += s;
    tot += s;
  }
  *total = tot;
  return base + incl - x;
}

template <int D, int G>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_hist_kernel(const __grid_constant__ CUtensorMap tmap_k, const Problem p, const int g0, const int pass) {
  using C = ScoreCfg<D>;
  constexpr int TK = C::TK, SUB = C::SUB, BOXES = C::BOXES;
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* tiles = smem;                                              // [stages][32 KB]
  unsigned char* qtile = smem + kScoreStages * kScoreTileBytes;             // [BOXES][16 rows][128 B]
  unsigned* hist_s = reinterpret_cast<unsigned*>(qtile + BOXES * C::QBOX_BYTES);   // [G][bins]
  int* pre = reinterpret_cast<int*>(hist_s + G * kHistBins);               // [batch+1]
  uint64_t* bars = reinterpret_cast<uint64_t*>(pre + kMaxBatch + 2);
  uint64_t* full = bars;                          // TMA tile landed
  uint64_t* empty = full + kScoreStages;          // MMAs that read the tile are done
  uint64_t* acc_full = empty + kScoreStages;      // accumulator buffer holds a finished tile
  uint64_t* acc_empty = acc_full + kAccStages;    // accumulator buffer has been read back
  uint64_t* qbar = acc_empty + kAccStages;        // every MMA issued so far is done
  int* scratch = reinterpret_cast<int*>(qbar + 1);                         // [40]
  int* s_flag = scratch + 36;
  volatile int* s_abort = scratch + 37;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(scratch + 38);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    for (int s = 0; s < kScoreStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < kAccStages; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], kEpiThreads); }
    mbar_init(qbar, 1);
    mbar_fence_init();
    *s_abort = 0;
  }
  if (warp == 1) tmem_alloc(s_tmem, kAccStages * kScoreN);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  const int F = pre[batch];
  const int f0 = (int)((long long)F * blockIdx.x / gridDim.x);
  const int f1 = (int)((long long)F * (blockIdx.x + 1) / gridDim.x);
  const int n_my = f1 - f0;

  if (n_my > 0) {
    if (warp == 0) {
      // ================================================================ TMA producer
      if (lane == 0) {
        TileCursor pc;
        cursor_seek(pc, pre, batch, n_kv, f0);
        int it = 0;
        for (; it < n_my; ++it) {
          const int slot = it % kScoreStages;
          const uint32_t ph = (uint32_t)(it / kScoreStages) & 1u;
          if (!mbar_wait(&empty[slot], ph ^ 1u, s_abort)) break;
          mbar_expect_tx(&full[slot], kScoreTileBytes);
          const int row = (int)(p.cu_seqlens[pc.b] + p.n_sink) + pc.t * TK;
#pragma unroll
          for (int x = 0; x < BOXES; ++x)
            tma_load_3d(tiles + slot * kScoreTileBytes + x * C::BOX_BYTES, &tmap_k, &full[slot], x * 64, row,
                        pc.kvh);
          cursor_next(pc, pre, batch, n_kv);
        }
        if (it == n_my) {
          // the last tiles' "empty" arrivals must land before the shared memory is released
          for (int j = (n_my > kScoreStages ? n_my - kScoreStages : 0); j < n_my; ++j)
            if (!mbar_wait(&empty[j % kScoreStages], (uint32_t)(j / kScoreStages) & 1u, s_abort)) break;
        } else {
          // gave up: let the copies already issued land before the shared memory is released
          for (int j = (it > kScoreStages ? it - kScoreStages : 0); j < it; ++j)
            for (uint32_t w = 0; w < kWaitPolls; ++w) {
              if (mbar_try_wait(&full[j % kScoreStages], (uint32_t)(j / kScoreStages) & 1u)) break;
              __nanosleep(64);
            }
        }
      }
    } else if (warp == 1) {
      // ================================================================ MMA issuer
      constexpr uint32_t idesc = umma_idesc_bf16(128, kScoreN, 0, 0);
      TileCursor mc;
      cursor_seek(mc, pre, batch, n_kv, f0);
      int cur_b = -1, cur_kvh = -1, acc_it = 0;
      uint32_t qphase = 0;
      bool ok = true;
      for (int it = 0; it < n_my && ok; ++it) {
        if (mc.b != cur_b || mc.kvh != cur_kvh) {
          // the MMAs issued so far read the previous unit's queries: let them finish
          if (it > 0) {
            if (lane == 0) tc_commit(qbar);
            __syncwarp();
            ok = mbar_wait(qbar, qphase, s_abort);
            qphase ^= 1u;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          cur_b = mc.b; cur_kvh = mc.kvh;
          // rows 0..G-1: the group's queries, rows G..15 zero; 128B-swizzled like the key tiles
          const __nv_bfloat16* qp = p.q + ((size_t)cur_b * p.n_q_heads + cur_kvh * p.group + g0) * D;
          for (int i = lane; i < kScoreN * (D / 8); i += 32) {
            const int r = i / (D / 8), c = i % (D / 8);
            uint4 val = make_uint4(0, 0, 0, 0);
            if (r < G) val = *reinterpret_cast<const uint4*>(qp + (size_t)r * D + c * 8);
            *reinterpret_cast<uint4*>(qtile + (c >> 3) * C::QBOX_BYTES + swz128(r, c & 7)) = val;
          }
          fence_proxy_async_smem();
          __syncwarp();
        }
        const int slot = it % kScoreStages;
        const uint32_t ph = (uint32_t)(it / kScoreStages) & 1u;
        if (lane == 0) {
          ok = mbar_wait(&full[slot], ph, s_abort);
          tc_fence_after_sync();
          for (int sub = 0; sub < SUB && ok; ++sub, ++acc_it) {
            const int a = acc_it % kAccStages;
            const uint32_t aph = (uint32_t)(acc_it / kAccStages) & 1u;
            ok = mbar_wait(&acc_empty[a], aph ^ 1u, s_abort);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t tile_addr = smem_u32(tiles + slot * kScoreTileBytes) + sub * (128 * 128);
            const uint32_t q_addr = smem_u32(qtile);
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
              const uint64_t adesc = umma_smem_desc(tile_addr + (k >> 2) * C::BOX_BYTES + (k & 3) * 32, 16, 1024);
              const uint64_t bdesc = umma_smem_desc(q_addr + (k >> 2) * C::QBOX_BYTES + (k & 3) * 32, 16, 1024);
              umma_ss(tmem_base + a * kScoreN, adesc, bdesc, idesc, k > 0 ? 1u : 0u);
            }
            tc_commit(&acc_full[a]);
          }
          if (ok) tc_commit(&empty[slot]);
        }
        acc_it = __shfl_sync(0xffffffffu, acc_it, 0);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        cursor_next(mc, pre, batch, n_kv);
      }
    } else {
      // ================================================================ read-back, scores, histogram
      const int et = tid - 64;                  // 0..127
      const int quad = warp & 3;                // tensor-memory lane quadrant this warp may read
      const int krow = quad * 32 + lane;        // key row inside a 128-key MMA tile
      TileCursor cc;
      cursor_seek(cc, pre, batch, n_kv, f0);
      int cur_b = -1, cur_kvh = -1, tiles_done = 0, n_mid = 0, acc_it = 0;
      long long row_base0 = 0, len_b = 0;
      bool ok = true;

      auto finish_unit = [&]() {
        // publish this CTA's share of the unit's histogram, then take a ticket
        epi_sync();
        const int row0 = cur_b * p.n_q_heads + cur_kvh * p.group + g0;
        for (int i = et; i < G * kHistBins; i += kEpiThreads) {
          unsigned h = hist_s[i];
          if (h) {
            atomicAdd(&p.hist[(size_t)(row0 + i / kHistBins) * kHistBins + (i % kHistBins)], h);
            hist_s[i] = 0;
          }
        }
        __threadfence();
        epi_sync();
        if (et == 0) {
          const int unit = cur_b * n_kv + cur_kvh;
          const unsigned nt_unit = (unsigned)((pre[cur_b + 1] - pre[cur_b]) / n_kv);
          unsigned prev = atomicAdd(&p.unit_counter[(size_t)pass * batch * n_kv + unit], (unsigned)tiles_done);
          *s_flag = (prev + (unsigned)tiles_done == nt_unit) ? 1 : 0;
        }
        epi_sync();
        if (*s_flag) {
          // last CTA of the unit: threshold bin per query head from the full histogram
          __threadfence();
          const int K = p.topk[cur_b];
          constexpr int BPT = kHistBins / kEpiThreads;       // 32 bins per thread
          for (int g = 0; g < G; ++g) {
            const unsigned* h = p.hist + (size_t)(row0 + g) * kHistBins + et * BPT;
            unsigned loc[BPT];
            int lsum = 0;
#pragma unroll
            for (int i = 0; i < BPT; ++i) { loc[i] = __ldcg(h + i); lsum += (int)loc[i]; }
            int total;
            int excl = epi_exclusive_scan(lsum, et, scratch, &total);
            int above = total - excl - lsum;          // elements in bins above this thread's range
            if (above < K && K <= above + lsum) {
              int cum = above;
#pragma unroll
              for (int i = BPT - 1; i >= 0; --i) {
                if (cum < K && K <= cum + (int)loc[i])
                  p.rowinfo[row0 + g] = make_int4(et * BPT + i, cum, (int)loc[i], total);
                cum += (int)loc[i];
              }
            }
          }
        }
        epi_sync();
        tiles_done = 0;
      };

      for (int it = 0; it < n_my && ok; ++it) {
        if (cc.b != cur_b || cc.kvh != cur_kvh) {
          if (cur_b >= 0) finish_unit();
          cur_b = cc.b; cur_kvh = cc.kvh;
          const long long cu_b = p.cu_seqlens[cur_b];
          len_b = p.cu_seqlens[cur_b + 1] - cu_b;
          n_mid = mid_len(len_b, p.n_sink, p.n_tail);
          row_base0 = score_row_base(p, cur_b, cur_kvh * p.group + g0, cu_b, len_b);
        }
        for (int sub = 0; sub < SUB; ++sub, ++acc_it) {
          const int a = acc_it % kAccStages;
          const uint32_t aph = (uint32_t)(acc_it / kAccStages) & 1u;
          ok = epi_all(mbar_wait(&acc_full[a], aph, s_abort));   // all 128 threads go on, or none
          if (!ok) break;
          tc_fence_after_sync();
          float v[4];
          tmem_ld_x4(tmem_addr(tmem_base, quad * 32, a * kScoreN), v);
          tc_wait_ld();
          tc_fence_before_sync();
          mbar_arrive(&acc_empty[a]);
          const int j = cc.t * TK + sub * 128 + krow;
          if (j < n_mid) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
              const float sc = v[g] * p.scale;
              p.scores[row_base0 + (long long)g * len_b + j] = sc;
              atomicAdd(&hist_s[g * kHistBins + (ordered_key(sc) >> kLowBits)], 1u);
            }
          }
        }
        ++tiles_done;
        cursor_next(cc, pre, batch, n_kv);
      }
      // a CTA that gave up publishes nothing: the unit's ticket never completes and the
      // status word tells the host
      if (ok) finish_unit();
    }
  }

  // ---- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*s_abort && tid == 0) atomicExch(p.status, kStatusTimeout);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kAccStages * kScoreN);
  }
}

static size_t score_smem_bytes(int D, int G) {
  return (size_t)kScoreStages * kScoreTileBytes + (size_t)(D / 64) * kScoreN * 128 + (size_t)G * kHistBins * 4 +
         (size_t)(kMaxBatch + 2) * 4 + (2 * kScoreStages + 2 * kAccStages + 1) * 8 + 40 * 4 + 64;
}

template <int D, int G>
static cudaError_t launch_score_t(const Problem& p, const CUtensorMap& tm, int g0, int pass, int n_sm,
                                  cudaStream_t st) {
  static bool configured = false;   // attribute is per function; cheap to set once
  const size_t smem = score_smem_bytes(D, G);
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

// ------------------------------------------------------------------ compaction against the threshold bin
constexpr int kCompThreads = 256;
constexpr int kCompPerWarp = kCompactChunk / (kCompThreads / 32);   // 512 scores per warp
constexpr int kCompIters = kCompPerWarp / 32;                        // 16

// Query-side log-features a_q = W_q q + b_q - gamma_q |q|^2 (Sec. 4.1), kept as
// exp(a_q - m_q) and m_q so that tiny features cannot underflow the merge.
__device__ void phi_q_job(const Problem& p, int row, int hq) {
  __shared__ float s_a[128];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = p.head_dim, r = p.n_feat;
  float* aq = p.aq + (size_t)row * (r + 4);
  const __nv_bfloat16* qp = p.q + (size_t)row * D;
  const float* W = p.w_q + (size_t)hq * r * D;
  float qn = 0.f;
  for (int c = lane; c < D; c += 32) { float x = __bfloat162float(qp[c]); qn = fmaf(x, x, qn); }
  qn = warp_sum(qn);
  for (int j = warp; j < r; j += kCompThreads / 32) {
    float a = 0.f;
    for (int c = lane; c < D; c += 32) a = fmaf(W[(size_t)j * D + c], __bfloat162float(qp[c]), a);
    a = warp_sum(a);
    if (lane == 0) s_a[j] = a + p.b_q[(size_t)hq * r + j] - p.gamma_q * qn;
  }
  __syncthreads();
  if (tid < 32) {
    float m = -INFINITY;
    for (int j = tid; j < r; j += 32) m = fmaxf(m, s_a[j]);
    m = warp_max(m);
    for (int j = tid; j < r; j += 32) aq[j] = expf(s_a[j] - m);
    if (tid == 0) aq[r] = m;
  }
}

// W_k of one KV head (fp32 [r][d]) -> two bf16 images, hi = bf16(W) and lo = bf16(W - hi),
// each laid out as the K-major, 128B-swizzled B operand of the feature recompute MMA:
// [d/64 column blocks][r rows][128 bytes].
__device__ void wk_split_job(const Problem& p, int kvh) {
  const int D = p.head_dim, r = p.n_feat;
  const float* W = p.w_k + (size_t)kvh * r * D;
  unsigned char* hi = reinterpret_cast<unsigned char*>(p.wk_img + (size_t)kvh * 2 * r * D);
  unsigned char* lo = hi + (size_t)r * D * 2;
  const int cpr = D / 8;
  for (int i = threadIdx.x; i < r * cpr; i += kCompThreads) {
    const int row = i / cpr, c = i % cpr;
    const float4 w0 = *reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8);
    const float4 w1 = *reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8 + 4);
    const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
    unsigned hw[4], lw[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const __nv_bfloat16 h0 = __float2bfloat16_rn(w[2 * e]), h1 = __float2bfloat16_rn(w[2 * e + 1]);
      const __nv_bfloat16 l0 = __float2bfloat16_rn(w[2 * e] - __bfloat162float(h0));
      const __nv_bfloat16 l1 = __float2bfloat16_rn(w[2 * e + 1] - __bfloat162float(h1));
      hw[e] = (unsigned)__bfloat16_as_ushort(h0) | ((unsigned)__bfloat16_as_ushort(h1) << 16);
      lw[e] = (unsigned)__bfloat16_as_ushort(l0) | ((unsigned)__bfloat16_as_ushort(l1) << 16);
    }
    const size_t off = (size_t)(c >> 3) * r * 128 + swz128(row, c & 7);
    *reinterpret_cast<uint4*>(hi + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
    *reinterpret_cast<uint4*>(lo + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
  }
}

__global__ void __launch_bounds__(kCompThreads) compact_kernel(const Problem p, const int n_chunk_ctas) {
  const int b = blockIdx.z, hq = blockIdx.y;
  const int row = b * p.n_q_heads + hq;
  if ((int)blockIdx.x >= n_chunk_ctas) {
    // spare CTAs: feature-map work that does not depend on the scores
    if ((int)blockIdx.x == n_chunk_ctas) phi_q_job(p, row, hq);
    else if (b == 0 && hq % p.group == 0) wk_split_job(p, hq / p.group);
    return;
  }
  __shared__ int s_warp[kCompThreads / 32];
  const int K = p.topk[b];
  if (K == 0) return;
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  const int chunk0 = blockIdx.x * kCompactChunk;
  if (chunk0 >= n_mid) return;
  const unsigned tb = (unsigned)p.rowinfo[row].x;
  const long long rbase = score_row_base(p, b, hq, cu_b, len_b);
  const float* srow = p.scores + rbase;
  const long long wbase = bitmap_row_base(p, b, hq, cu_b, len_b);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int base = chunk0 + warp * kCompPerWarp;
  float sc[kCompIters];
#pragma unroll
  for (int it = 0; it < kCompIters; ++it) {
    const int j = base + it * 32 + lane;
    sc[it] = j < n_mid ? __ldcg(srow + j) : -INFINITY;
  }
  unsigned my_sure = 0, cand_words[kCompIters];
  int n_cand_w = 0;
#pragma unroll
  for (int it = 0; it < kCompIters; ++it) {
    const int j = base + it * 32 + lane;
    bool sure = false, cand = false;
    if (j < n_mid) {
      const unsigned bin = ordered_key(sc[it]) >> kLowBits;
      sure = bin > tb;
      cand = bin == tb;
    }
    const unsigned ws = __ballot_sync(0xffffffffu, sure);
    cand_words[it] = __ballot_sync(0xffffffffu, cand);
    if (lane == it) my_sure = ws;
    n_cand_w += __popc(cand_words[it]);
  }
  if (lane < kCompIters) {
    const int word = (base >> 5) + lane;
    if (word * 32 < n_mid) p.bm_sure[wbase + word] = my_sure;
  }
  if (lane == 0) s_warp[warp] = n_cand_w;
  __syncthreads();
  int off = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kCompThreads / 32; ++w) {
    const int c = s_warp[w];
    if (w < warp) off += c;
    total += c;
  }
  if (threadIdx.x == 0) p.chunk_ncand[(size_t)row * p.max_chunks + blockIdx.x] = total;
  // ordered write: (warp, iteration, lane)
  int* out = p.cand + rbase + chunk0;
  const unsigned lt = (1u << lane) - 1u;
#pragma unroll
  for (int it = 0; it < kCompIters; ++it) {
    const unsigned w = cand_words[it];
    if ((w >> lane) & 1u) out[off + __popc(w & lt)] = base + it * 32 + lane;
    off += __popc(w);
  }
}

cudaError_t launch_compact(const Problem& p, int max_mid, cudaStream_t st) {
  const int n_chunk_ctas = max_mid > 0 ? (max_mid + kCompactChunk - 1) / kCompactChunk : 0;
  const int extra = p.with_phi ? 2 : 0;
  if (n_chunk_ctas + extra == 0) return cudaSuccess;
  dim3 grid(n_chunk_ctas + extra, p.n_q_heads, p.batch);
  compact_kernel<<<grid, kCompThreads, 0, st>>>(p, n_chunk_ctas);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ finalize selection
constexpr int kFinThreads = 1024;
constexpr int kRefBins = 1 << (kLowBits / 2);      // 1024: two refinement digits of 10 bits
constexpr int kCandCap = 4096;                     // candidates cached in shared memory
static_assert(kRefBins == kFinThreads, "one refinement bin per thread");

// Walks the 1024-bin histogram from the top and returns the digit at which the
// cumulative count reaches `need`; *rem = how many are still needed inside it.
__device__ int find_digit(const unsigned* h, int need, int* rem, int* scratch, int* s_out) {
  const int tid = threadIdx.x;
  const int c = (int)h[tid];
  int total;
  const int excl = block_exclusive_scan(c, scratch, &total);
  const int above = total - excl - c;
  if (above < need && need <= above + c) { s_out[0] = tid; s_out[1] = need - above; }
  __syncthreads();
  *rem = s_out[1];
  return s_out[0];
}

__global__ void __launch_bounds__(kFinThreads) finalize_select_kernel(const Problem p) {
  __shared__ unsigned h[kRefBins];
  __shared__ int cpre[kMaxChunks + 1];
  __shared__ int s_pos[kCandCap];
  __shared__ unsigned s_low[kCandCap];
  __shared__ int scratch[40];
  __shared__ int s_out[2];
  const int row = blockIdx.x, b = row / p.n_q_heads, hq = row % p.n_q_heads;
  const int tid = threadIdx.x;

  const int K = p.topk[b];
  int* out = p.idx + (size_t)row * p.topk_max;
  int* out2 = p.idx_out ? p.idx_out + (size_t)row * p.topk_max : nullptr;
  if (out2)
    for (int i = K + tid; i < p.topk_max; i += kFinThreads) out2[i] = -1;
  if (K == 0) return;

  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  const int n_words = (n_mid + 31) >> 5;
  const int n_chunks = (n_mid + kCompactChunk - 1) / kCompactChunk;
  const long long rbase = score_row_base(p, b, hq, cu_b, len_b);
  const float* srow = p.scores + rbase;
  const int* cand = p.cand + rbase;
  unsigned* sure = p.bm_sure + bitmap_row_base(p, b, hq, cu_b, len_b);
  const int4 info = p.rowinfo[row];
  const int need = K - info.y;                 // candidates to take, 1 <= need <= info.z
  const int n_cand = info.z;
  const unsigned low_mask = (1u << kLowBits) - 1u;

  // ---- prefix of the per-chunk candidate counts (n_chunks <= kMaxChunks, checked on the host)
  {
    const int per = (n_chunks + kFinThreads - 1) / kFinThreads;     // 1 or 2
    int loc[2] = {0, 0}, lsum = 0;
    for (int i = 0; i < per; ++i) {
      const int c = tid * per + i;
      if (c < n_chunks) { loc[i] = p.chunk_ncand[(size_t)row * p.max_chunks + c]; lsum += loc[i]; }
    }
    int total;
    int run = block_exclusive_scan(lsum, scratch, &total);
    for (int i = 0; i < per; ++i) {
      const int c = tid * per + i;
      if (c < n_chunks) { cpre[c] = run; run += loc[i]; }
    }
    if (tid == 0) cpre[n_chunks] = total;
    __syncthreads();
  }
  // candidate i (in index order) -> its mid offset
  auto cand_pos = [&](int i) -> int {
    int lo = 0, hi = n_chunks - 1;             // largest c with cpre[c] <= i
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (cpre[mid] <= i) lo = mid; else hi = mid - 1;
    }
    return cand[(size_t)lo * kCompactChunk + (i - cpre[lo])];
  };
  const bool cached = n_cand <= kCandCap;
  if (cached) {
    for (int i = tid; i < n_cand; i += kFinThreads) {
      const int j = cand_pos(i);
      s_pos[i] = j;
      s_low[i] = ordered_key(__ldcg(srow + j)) & low_mask;
    }
    __syncthreads();
  }
  auto get = [&](int i, int* j, unsigned* low) {
    if (cached) { *j = s_pos[i]; *low = s_low[i]; }
    else { *j = cand_pos(i); *low = ordered_key(__ldcg(srow + *j)) & low_mask; }
  };

  unsigned tau_low = 0;                        // low 20 bits of the threshold key
  int need_ties = n_cand;                      // ties to admit, in index order
  const bool refine = need < n_cand;
  if (refine) {
    // digit 1: bits 19..10 of the key among the candidates
    h[tid] = 0;
    __syncthreads();
    for (int i = tid; i < n_cand; i += kFinThreads) {
      int j; unsigned low;
      get(i, &j, &low);
      atomicAdd(&h[low >> 10], 1u);
    }
    __syncthreads();
    int rem1;
    const unsigned d1 = (unsigned)find_digit(h, need, &rem1, scratch, s_out);
    __syncthreads();
    // digit 2: bits 9..0 among candidates whose digit 1 matches
    h[tid] = 0;
    __syncthreads();
    for (int i = tid; i < n_cand; i += kFinThreads) {
      int j; unsigned low;
      get(i, &j, &low);
      if ((low >> 10) == d1) atomicAdd(&h[low & (kRefBins - 1)], 1u);
    }
    __syncthreads();
    int rem2;
    const unsigned d2 = (unsigned)find_digit(h, rem1, &rem2, scratch, s_out);
    tau_low = (d1 << 10) | d2;
    need_ties = rem2;
  }

  // ---- admit candidates: above the threshold, or tied with it and early enough in index
  // order (thread t owns the contiguous candidates [i0, i1))
  {
    const int per = (n_cand + kFinThreads - 1) / kFinThreads;
    const int i0 = min(tid * per, n_cand), i1 = min(i0 + per, n_cand);
    int my_ties = 0;
    for (int i = i0; i < i1; ++i) {
      int j; unsigned low;
      get(i, &j, &low);
      if (low == tau_low || !refine) ++my_ties;
    }
    int total_ties;
    int tie_rank = block_exclusive_scan(my_ties, scratch, &total_ties);
    for (int i = i0; i < i1; ++i) {
      int j; unsigned low;
      get(i, &j, &low);
      bool take = refine && low > tau_low;
      if (low == tau_low || !refine) { take = take || tie_rank < need_ties; ++tie_rank; }
      if (take) atomicOr(&sure[j >> 5], 1u << (j & 31));
    }
  }
  __threadfence();
  __syncthreads();

  // ---- expand the final bitmap: thread t owns the contiguous words [w0, w1)
  const int wpt = (n_words + kFinThreads - 1) / kFinThreads;
  const int w0 = min(tid * wpt, n_words), w1 = min(w0 + wpt, n_words);
  int my_count = 0;
  for (int w = w0; w < w1; ++w) my_count += __popc(__ldcg(sure + w));
  int total_sel;
  int off = block_exclusive_scan(my_count, scratch, &total_sel);
  for (int w = w0; w < w1; ++w) {
    unsigned fin = __ldcg(sure + w);
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
