// Step (1) of the decode path, first half: score every mid-region key against the G
// query heads of its KV-head group (s_i = q.k_i / sqrt(d_h), Sec. 3 Eq. full_attention).
// The selection over the score rows is in select_cluster.cu.
//
//   score_kernel   streams the keys once.  A producer thread issues TMA loads of
//                  128B-swizzled 32 KB key tiles into a 3-stage mbarrier ring; one thread
//                  issues tcgen05.mma with the key tile as an operand straight from shared
//                  memory and the group's queries (zero padded) as the other, so the dot
//                  products cost no issue slots of the CUDA cores; two warps (even and odd
//                  tiles) read the fp32 accumulators back from tensor memory and write the
//                  score rows (with one warp that stage bounds the kernel at head_dim 64,
//                  where a tile holds 256 keys of four heads).  The
//                  CTAs also clear the workspace counters.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

// ------------------------------------------------------------------ scoring
constexpr int kScoreThreads = 160;        // warps 0 and 4: read-back (even / odd tiles; a warp reads tensor-memory lanes
                                          // 32 (w % 4) .. + 31 and the scores sit in lanes 0..15), warp 1: MMA issuer,
                                          // warp 2: TMA producer, warp 3 idle
constexpr int kScoreStages = 3;          // measured: 3-4 stages beat 6 (less queueing in the memory system)
constexpr int kScoreTileBytes = 32768;
constexpr int kScoreM = 64;               // MMA M: query heads of the group (<= 8), zero padded
constexpr int kTmemCols = 512;

template <int D>
struct ScoreCfg {
  static constexpr int TK = kScoreTileBytes / (2 * D);   // keys per TMA tile = MMA N (128 or 256)
  static constexpr int BOXES = D / 64;                   // 64-dim (128-byte) column blocks
  static constexpr int BOX_BYTES = TK * 128;
  static constexpr int QBOX_BYTES = kScoreM * 128;
  static constexpr int ACC_STAGES = kTmemCols / TK;      // accumulator buffers in tensor memory
  static_assert(TK * D * 2 == kScoreTileBytes && TK <= 256, "tile size");
  static_assert(ACC_STAGES % 2 == 0, "two read-back warps alternate over the accumulator buffers");
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

// The contraction is issued as scores^T = Q K^T: the group's queries (zero padded to 64
// rows) are the A operand and the key tile, exactly as TMA lands it, is the B operand
// (N = keys of the tile).  The tensor core fetches B rows twice as fast as A rows, which
// halves the time the key tile is being read out of shared memory compared with the
// transposed form; row g of the accumulator (tensor-memory lane g) holds head g's scores.
template <int D>
__global__ void __launch_bounds__(kScoreThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tmap_k, const Problem p) {
  using C = ScoreCfg<D>;
  constexpr int TK = C::TK, BOXES = C::BOXES, ACC = C::ACC_STAGES;
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* tiles = smem;                                              // [stages][32 KB]
  unsigned char* qtile = smem + kScoreStages * kScoreTileBytes;             // [BOXES][64 rows][128 B]
  int* pre = reinterpret_cast<int*>(qtile + BOXES * C::QBOX_BYTES);        // [batch+1]
  uint64_t* bars = reinterpret_cast<uint64_t*>(pre + kMaxBatch + 2);
  uint64_t* full = bars;                          // TMA tile landed
  uint64_t* empty = full + kScoreStages;          // MMAs that read the tile are done
  uint64_t* acc_full = empty + kScoreStages;      // accumulator buffer holds a finished tile
  uint64_t* acc_empty = acc_full + ACC;           // accumulator buffer has been read back
  uint64_t* qbar = acc_empty + ACC;               // every MMA issued so far is done
  int* scratch = reinterpret_cast<int*>(qbar + 1);                         // [40]
  volatile int* s_abort = scratch + 37;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(scratch + 38);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_kv = p.n_kv_heads, batch = p.batch, G = p.group;

  pdl_launch_next();
  // ---- tiles per sequence -> prefix in shared memory (reads only the call's inputs)
  {
    const int per = (batch + kScoreThreads - 1) / kScoreThreads;
    const int b0 = tid * per;
    int local = 0;
    for (int i = 0; i < per; ++i) {
      int b = b0 + i;
      if (b < batch) {
        int nm = mid_len(p.cu_seqlens[b + 1] - p.cu_seqlens[b], p.n_sink, tail_of(p, b));
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
        int nm = mid_len(p.cu_seqlens[b + 1] - p.cu_seqlens[b], p.n_sink, tail_of(p, b));
        int nt = (p.topk[b] > 0) ? (nm + TK - 1) / TK : 0;
        run += nt * n_kv;
      }
    }
    if (tid == 0) pre[batch] = total;
  }
  if (tid == 0) {
    for (int s = 0; s < kScoreStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < ACC; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 1); }
    mbar_init(qbar, 1);
    mbar_fence_init();
    *s_abort = 0;
  }
  // everything below touches the workspace, which kernels of the previous call may still use;
  // tensor memory is also taken only now, so that a CTA that started early never holds
  // columns a CTA of a predecessor kernel is waiting for
  pdl_wait();
  if (warp == 1) tmem_alloc(s_tmem, kTmemCols);
  // ---- clear this CTA's slice of the workspace head (counters, status word)
  {
    uint4* z = reinterpret_cast<uint4*>(p.status);
    const size_t n16 = p.zero_bytes / 16;
    for (size_t i = (size_t)blockIdx.x * kScoreThreads + tid; i < n16; i += (size_t)gridDim.x * kScoreThreads)
      z[i] = make_uint4(0, 0, 0, 0);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  const int F = pre[batch];
  const int f0 = (int)((long long)F * blockIdx.x / gridDim.x);
  const int f1 = (int)((long long)F * (blockIdx.x + 1) / gridDim.x);
  const int n_my = f1 - f0;

  if (n_my > 0) {
    if (warp == 2) {
      // ================================================================ TMA producer
      if (lane == 0) {
        TileCursor pc;
        cursor_seek(pc, pre, batch, n_kv, f0);
        int it = 0, row_b = -1, row0 = 0;
        const uint64_t pol = l2_policy_evict_first();      // the keys are read once
        for (; it < n_my; ++it) {
          const int slot = it % kScoreStages;
          const uint32_t ph = (uint32_t)(it / kScoreStages) & 1u;
          if (!mbar_wait(&empty[slot], ph ^ 1u, s_abort)) break;
          mbar_expect_tx(&full[slot], kScoreTileBytes);
          if (pc.b != row_b) { row_b = pc.b; row0 = (int)(p.cu_seqlens[pc.b] + p.n_sink); }
          const int row = row0 + pc.t * TK;
#pragma unroll
          for (int x = 0; x < BOXES; ++x)
            tma_load_3d(tiles + slot * kScoreTileBytes + x * C::BOX_BYTES, &tmap_k, &full[slot], x * 64, row,
                        pc.kvh, pol);
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
      constexpr uint32_t idesc = umma_idesc_bf16(kScoreM, TK, 0, 0);
      // operand descriptors: the address field counts 16-byte units, so moving to another
      // tile, column block or K step is one 64-bit add of a small constant
      const uint64_t adesc0 = umma_smem_desc(smem_u32(qtile), 16, 1024);
      const uint64_t bdesc0 = umma_smem_desc(smem_u32(tiles), 16, 1024);
      TileCursor mc;
      cursor_seek(mc, pre, batch, n_kv, f0);
      int cur_b = -1, cur_kvh = -1;
      uint32_t qphase = 0;
      bool ok = true;
      for (int it = 0; it < n_my && ok; ++it) {
        if (mc.b != cur_b || mc.kvh != cur_kvh) {
          // the MMAs issued so far read the previous unit's queries: let them finish
          if (it > 0) {
            if (lane == 0) tc_commit(qbar);
            __syncwarp();
            ok = __all_sync(0xffffffffu, mbar_wait(qbar, qphase, s_abort));
            qphase ^= 1u;
            if (!ok) break;
          }
          cur_b = mc.b; cur_kvh = mc.kvh;
          // rows 0..G-1: the group's queries, rows G..63 zero; 128B-swizzled like the key tiles
          const __nv_bfloat16* qp = p.q + ((size_t)cur_b * p.n_q_heads + cur_kvh * G) * D;
          for (int i = lane; i < kScoreM * (D / 8); i += 32) {
            const int r = i / (D / 8), c = i % (D / 8);
            uint4 val = make_uint4(0, 0, 0, 0);
            if (r < G) val = *reinterpret_cast<const uint4*>(qp + (size_t)r * D + c * 8);
            *reinterpret_cast<uint4*>(qtile + (c >> 3) * C::QBOX_BYTES + swz128(r, c & 7)) = val;
          }
          fence_proxy_async_smem();
          __syncwarp();
        }
        if (lane == 0) {
          const int slot = it % kScoreStages;
          const uint32_t ph = (uint32_t)(it / kScoreStages) & 1u;
          const int a = it % ACC;
          const uint32_t aph = (uint32_t)(it / ACC) & 1u;
          ok = mbar_wait(&full[slot], ph, s_abort) && mbar_wait(&acc_empty[a], aph ^ 1u, s_abort);
          if (ok) {
            tc_fence_after_sync();
            const uint64_t bdesc = bdesc0 + (uint64_t)((slot * kScoreTileBytes) >> 4);
#pragma unroll
            for (int k = 0; k < D / 16; ++k)
              umma_ss(tmem_base + a * TK, adesc0 + (uint64_t)(((k >> 2) * C::QBOX_BYTES + (k & 3) * 32) >> 4),
                      bdesc + (uint64_t)(((k >> 2) * C::BOX_BYTES + (k & 3) * 32) >> 4), idesc, k > 0 ? 1u : 0u);
            tc_commit(&acc_full[a]);
            tc_commit(&empty[slot]);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        cursor_next(mc, pre, batch, n_kv);
      }
    } else if (warp == 0 || warp == 4) {
      // ================================================================ read-back, score rows
      // warp 0 reads tensor-memory lanes 0..15: thread t holds head (t / 4), key columns
      // 8 i + 2 (t % 4) + {0, 1} of each 8-column block i (the second register pair of a
      // block belongs to rows 8..15, which are zero padding)
      TileCursor cc;
      cursor_seek(cc, pre, batch, n_kv, f0);
      int cur_b = -1, cur_kvh = -1, n_mid = 0;
      long long len_b = 0;
      float* my_row = nullptr;
      const int g = lane >> 2, cpair = 2 * (lane & 3);
      const uint64_t keep = l2_policy_evict_last();         // the score rows are read back right away
      bool ok = true;
      for (int it = 0; it < n_my && ok; ++it) {
        if (cc.b != cur_b || cc.kvh != cur_kvh) {
          cur_b = cc.b; cur_kvh = cc.kvh;
          const long long cu_b = p.cu_seqlens[cur_b];
          len_b = p.cu_seqlens[cur_b + 1] - cu_b;
          n_mid = mid_len(len_b, p.n_sink, tail_of(p, cur_b));
          my_row = p.scores + score_row_base(p, cur_b, cur_kvh * G, cu_b, len_b) + (long long)g * len_b;
        }
        // the other read-back warp's tile (every accumulator buffer belongs to one warp: their number is even)
        if ((it & 1) != (warp >> 2)) { cursor_next(cc, pre, batch, n_kv); continue; }
        const int a = it % ACC;
        const uint32_t aph = (uint32_t)(it / ACC) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[a], aph, s_abort));
        if (!ok) break;
        tc_fence_after_sync();
        const int j0 = cc.t * TK + cpair;
#pragma unroll
        for (int half = 0; half < TK / 64; ++half) {
          float v[32];
          tmem_ld_16x256b_x8(tmem_addr(tmem_base, 0, a * TK + half * 64), v);
          tc_wait_ld();
          if (g < G) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int j = j0 + half * 64 + i * 8;
              if (j < n_mid) st_global_f32(my_row + j, v[4 * i] * p.scale, keep);
              if (j + 1 < n_mid) st_global_f32(my_row + j + 1, v[4 * i + 1] * p.scale, keep);
            }
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[a]);
        cursor_next(cc, pre, batch, n_kv);
      }
    }
  }

  // ---- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*s_abort && tid == 0) atomicExch(p.status, kStatusTimeout);
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

static size_t score_smem_bytes(int D) {
  return (size_t)kScoreStages * kScoreTileBytes + (size_t)(D / 64) * kScoreM * 128 + (size_t)(kMaxBatch + 2) * 4 +
         (2 * kScoreStages + 2 * 4 + 1) * 8 + 40 * 4 + 64;
}

template <int D>
static cudaError_t launch_score_t(const Problem& p, const CUtensorMap& tm, int n_sm, cudaStream_t st) {
  static PerDeviceFlag configured;
  const size_t smem = score_smem_bytes(D);
  cudaError_t e = set_max_dynamic_smem(configured, reinterpret_cast<const void*>(score_kernel<D>), smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(score_kernel<D>, dim3(n_sm), dim3(kScoreThreads), smem, st, tm, p);
}

cudaError_t launch_score(const Problem& p, const CUtensorMap& tm, int n_sm, cudaStream_t st) {
  if (p.head_dim == 64) return launch_score_t<64>(p, tm, n_sm, st);
  if (p.head_dim == 128) return launch_score_t<128>(p, tm, n_sm, st);
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
