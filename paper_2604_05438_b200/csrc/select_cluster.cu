// Exact Top-K selection over the score rows (exhaustive Top-K control selector, Sec. 5.1;
// ties broken towards the lower index) in ONE kernel: a thread-block cluster of up to eight
// CTAs per query head (1, 2, 4 or 8, enough to hold the longest row of the call).
//
// Each CTA owns a contiguous eighth of the head's mid-region; each warp a contiguous
// 1024-score run of it, read coalesced (lane l, step i -> element 32 i + l), so that
// (CTA, round, warp, step, lane) order is index order.  For sequences of up to 131072
// mid-region keys every CTA keeps its 16384 order-preserving score keys in shared memory
// and the row is read from L2 exactly once (longer rows, up to 2,097,152 keys, are read twice
// and the shared memory holds per-round bit masks instead) (the loops over a thread's 32 keys stay rolled:
// straight-line code that runs once is bound by instruction fetch, not by its work).  The exact K-th largest key is found by radix
// selection over 12 + 10 + 10 bits: every CTA builds a local histogram in shared memory
// and adds its non-zero bins into the accumulator of every CTA through distributed shared
// memory; every CTA then walks its own copy of the accumulator.  Positions above the
// threshold, and as many threshold ties as are still needed in index order, are then
// written straight to their slot of the ascending index list: the per-thread bit masks
// are transposed inside each warp so that thread order is index order, and offsets come
// from one block scan and per-CTA totals exchanged through distributed shared memory.  CTAs of a cluster only meet at hardware cluster barriers
// (no flag spinning, no global scratch, nothing to clear between calls).
//
// Extra clusters of the same launch do the work that depends only on the call's inputs
// (query-side features, W_k operand split), off the critical path.
#include "common.cuh"
#include "sm100.cuh"
#include "feature_jobs.cuh"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace tkphi {

constexpr int kSelThreads = 512;
constexpr int kSelPer = 32;                              // scores per thread and round
constexpr int kSelChunk = kSelThreads * kSelPer;         // 16384 scores per CTA and round
constexpr int kSelCluster = 8;                            // largest cluster; the launch picks 1, 2, 4 or 8
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kRefBins = 1024;                           // two refinement digits of 10 bits

struct SelShared {
  unsigned hist[kHistBins];      // local 12-bit histogram
  unsigned acc[kHistBins];       // the cluster's 12-bit histogram (every CTA receives every CTA's bins)
  unsigned h1[kRefBins];         // local refinement histogram
  unsigned acc1[kRefBins];       // the cluster's histogram of refinement digit 1
  unsigned acc2[kRefBins];       // ... of refinement digit 2
  int scratch[40];
  int res[4];                    // result of a histogram walk: digit, count above it, count in it
  int tot[2 * kSelCluster];      // per CTA: selected-for-sure count, tie count
  int wdef[kSelWarps], wtie[kSelWarps];
};

// Walks an n-bin histogram (n = NB, a multiple of 512) from the top and finds the bin at
// which the cumulative count reaches `need`; res = {bin, count above it, count in it}.
// All 512 threads of the CTA call it.
template <int NB>
__device__ void walk_from_top(const unsigned* h, int need, int* res, int* scratch) {
  constexpr int BPT = NB / kSelThreads;
  const int tid = threadIdx.x;
  unsigned loc[BPT];
  int lsum = 0;
#pragma unroll
  for (int i = 0; i < BPT; ++i) { loc[i] = h[tid * BPT + i]; lsum += (int)loc[i]; }
  int total;
  const int excl = block_exclusive_scan(lsum, scratch, &total);
  const int above = total - excl - lsum;                   // elements in bins above this thread's range
  if (above < need && need <= above + lsum) {
    int cum = above;
#pragma unroll
    for (int i = BPT - 1; i >= 0; --i) {
      if (cum < need && need <= cum + (int)loc[i]) { res[0] = tid * BPT + i; res[1] = cum; res[2] = (int)loc[i]; }
      cum += (int)loc[i];
    }
  }
  __syncthreads();
}

// Transposes the 32 x 32 bit matrix whose row l is the word of lane l: afterwards bit j of
// lane t is what bit t of lane j was.
__device__ __forceinline__ unsigned warp_transpose32(unsigned x, int lane) {
  unsigned m = 0x0000ffffu;
#pragma unroll
  for (int j = 16; j; j >>= 1) {
    const unsigned y = __shfl_xor_sync(0xffffffffu, x, j);
    if ((lane & j) == 0) x ^= (((x >> j) ^ y) & m) << j;
    else x ^= ((y >> j) ^ x) & m;
    m ^= m << (j >> 1);
  }
  return x;
}

__global__ void __launch_bounds__(kSelThreads, 2)
select_kernel(const Problem p, const int n_rows, const int csize) {
  __shared__ SelShared sm;
  extern __shared__ __align__(16) unsigned keys_s[];       // [kSelPer][kSelThreads]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_next();
  if ((int)blockIdx.y >= n_rows) {
    // ---- feature clusters: one task per CTA (query rows first, then KV heads)
    pdl_wait();                                            // the workspace is free once the predecessors are done
    const int task = ((int)blockIdx.y - n_rows) * csize + (int)blockIdx.x;
    if (task < n_rows) {
      phi_q_stage1<kSelThreads>(p, task);
      __threadfence_block();
      __syncthreads();
      phi_q_stage2<kSelThreads>(p, task);
    } else if (task < n_rows + p.n_kv_heads && !(p.flags & 1u) && !p.zbuf) {   // (cached features need no W_k tiles)
      wk_split_job<kSelThreads>(p, task - n_rows);
    }
    return;
  }
  // Everything up to the wait reads only the call's inputs (sequence lengths, budgets) and this
  // CTA's shared memory, so it overlaps the scoring kernel's run: the first loads of the score
  // row are issued 1.5 us earlier than with the wait at the top.
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int row = blockIdx.y, b = row / p.n_q_heads, hq = row % p.n_q_heads;
  const int K = p.topk[b];
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, tail_of(p, b));
  const float* srow = p.scores + score_row_base(p, b, hq, cu_b, len_b);
  const int n_chunks = (n_mid + kSelChunk - 1) / kSelChunk;
  const int rounds = (n_chunks + csize - 1) / csize;       // per CTA
  const bool resident = rounds == 1;                       // the keys stay in shared memory
  const unsigned low_mask = (1u << kLowBits) - 1u;
  for (int i = tid; i < kHistBins; i += kSelThreads) { sm.hist[i] = 0; sm.acc[i] = 0; }
  for (int i = tid; i < kRefBins; i += kSelThreads) { sm.h1[i] = 0; sm.acc1[i] = 0; sm.acc2[i] = 0; }
  pdl_wait();                                              // score rows and workspace of the predecessors
  int* out = p.idx + (size_t)row * p.topk_max;
  int* out2 = p.idx_out ? p.idx_out + (size_t)row * p.topk_max : nullptr;
  if (out2 && rank == 0)
    for (int i = K + tid; i < p.topk_max; i += kSelThreads) out2[i] = -1;
  if (K == 0) return;                                      // the same for all CTAs of the cluster

  // Resident mode (one round per CTA): the order-preserving keys of this thread's 32 scores
  // stay in shared memory (element i at keys[i * 512]) and its bit masks in registers.
  // Otherwise (2..16 rounds) the keys are recomputed from the L2-resident row where needed and
  // the shared-memory array holds the per-round bit masks instead.
  unsigned* keys = keys_s + tid;
  const int base_w = warp * (32 * kSelPer) + lane;
  auto round_base = [&](int k) { return (rank * rounds + k) * kSelChunk + base_w; };
  auto load_regs = [&](int k, unsigned (&kr)[kSelPer]) -> unsigned {      // returns the validity mask
    const int base = round_base(k);
    float sc[kSelPer];
#pragma unroll
    for (int i = 0; i < kSelPer; ++i) sc[i] = (base + i * 32 < n_mid) ? __ldcg(srow + base + i * 32) : 0.f;
    unsigned vm = 0;
#pragma unroll
    for (int i = 0; i < kSelPer; ++i) {
      kr[i] = ordered_key(sc[i]);
      if (base + i * 32 < n_mid) vm |= 1u << i;
    }
    return vm;
  };
  auto key_at = [&](int k, int i) -> unsigned {            // key i of round k (valid positions only)
    return resident ? keys[i * kSelThreads] : ordered_key(__ldcg(srow + round_base(k) + i * 32));
  };
  // adds the non-zero bins of a local histogram into the accumulator of every CTA
  auto push_all = [&](unsigned* local, unsigned* accum, int n_bins, bool clear) {
    for (int i = tid; i < n_bins; i += kSelThreads) {
      const unsigned c = local[i];
      if (c) {
        for (int r = 0; r < csize; ++r) atomicAdd(cluster.map_shared_rank(accum, r) + i, c);
        if (clear) local[i] = 0;
      }
    }
  };

  // ---- 12-bit histogram of the row, replicated in every CTA (the histograms were cleared before the wait)
  __syncthreads();
  cluster.barrier_arrive();                                // "my accumulators are cleared"; waited for below
  unsigned vmask0 = 0;                                     // validity mask of the resident round
  for (int k = 0; k < rounds; ++k) {
    unsigned kr[kSelPer];
    const unsigned vm = load_regs(k, kr);
#pragma unroll
    for (int i = 0; i < kSelPer; ++i) {
      if (resident) keys[i * kSelThreads] = kr[i];
      if ((vm >> i) & 1u) atomicAdd(&sm.hist[kr[i] >> kLowBits], 1u);
    }
    vmask0 = vm;
  }
  __syncthreads();
  cluster.barrier_wait();                                  // every accumulator of the cluster is cleared
  push_all(sm.hist, sm.acc, kHistBins, false);
  cluster.sync();
  walk_from_top<kHistBins>(sm.acc, K, sm.res, sm.scratch);
  const unsigned tb = (unsigned)sm.res[0];                 // threshold bin
  const int need = K - sm.res[1];                          // keys to take inside it, 1 <= need <= n_cand
  const int n_cand = sm.res[2];
  const bool refine = need < n_cand;                       // the same in every CTA

  // bit i of a "sure" mask: key i lies above the threshold bin; of a "cand" mask: inside it
  unsigned smask = 0, cmask = 0;                           // resident mode
  auto get_masks = [&](int k, unsigned* s_, unsigned* c_) {
    if (resident) { *s_ = smask; *c_ = cmask; }
    else { *s_ = keys_s[(2 * k) * kSelThreads + tid]; *c_ = keys_s[(2 * k + 1) * kSelThreads + tid]; }
  };
  auto put_masks = [&](int k, unsigned s_, unsigned c_) {
    if (resident) { smask = s_; cmask = c_; }
    else { keys_s[(2 * k) * kSelThreads + tid] = s_; keys_s[(2 * k + 1) * kSelThreads + tid] = c_; }
  };
  if (resident) {
    unsigned s_ = 0, c_ = 0;
#pragma unroll 4
    for (int i = 0; i < kSelPer; ++i) {
      const unsigned bin = keys[i * kSelThreads] >> kLowBits;
      s_ |= (bin > tb ? 1u : 0u) << i;
      c_ |= (bin == tb ? 1u : 0u) << i;
    }
    smask = s_ & vmask0; cmask = c_ & vmask0;
  } else {
    for (int k = 0; k < rounds; ++k) {
      unsigned kr[kSelPer];
      const unsigned vm = load_regs(k, kr);
      unsigned s_ = 0, c_ = 0;
#pragma unroll
      for (int i = 0; i < kSelPer; ++i) {
        const unsigned bin = kr[i] >> kLowBits;
        s_ |= (bin > tb ? 1u : 0u) << i;
        c_ |= (bin == tb ? 1u : 0u) << i;
      }
      put_masks(k, s_ & vm, c_ & vm);
    }
  }

  unsigned tau_low = 0;
  int need_ties = n_cand;
  if (refine) {
    // ---- digit 1: bits 19..10 of the key among the keys of the threshold bin
    for (int k = 0; k < rounds; ++k) {
      unsigned s_, c_;
      get_masks(k, &s_, &c_);
      for (unsigned m = c_; m; m &= m - 1) atomicAdd(&sm.h1[(key_at(k, __ffs(m) - 1) & low_mask) >> 10], 1u);
    }
    __syncthreads();
    push_all(sm.h1, sm.acc1, kRefBins, true);
    cluster.sync();
    walk_from_top<kRefBins>(sm.acc1, need, sm.res, sm.scratch);
    const unsigned d1 = (unsigned)sm.res[0];
    const int rem1 = need - sm.res[1];
    __syncthreads();
    // ---- digit 2: bits 9..0 among the keys whose digit 1 matches
    for (int k = 0; k < rounds; ++k) {
      unsigned s_, c_;
      get_masks(k, &s_, &c_);
      for (unsigned m = c_; m; m &= m - 1) {
        const unsigned low = key_at(k, __ffs(m) - 1) & low_mask;
        if ((low >> 10) == d1) atomicAdd(&sm.h1[low & (kRefBins - 1)], 1u);
      }
    }
    __syncthreads();
    push_all(sm.h1, sm.acc2, kRefBins, false);
    cluster.sync();
    walk_from_top<kRefBins>(sm.acc2, rem1, sm.res, sm.scratch);
    tau_low = (d1 << 10) | (unsigned)sm.res[0];
    need_ties = rem1 - sm.res[1];
  }

  // after this, "sure": keys above the exact threshold; "cand": keys equal to it (without
  // refinement the whole threshold bin counts as tied: all of it is taken)
  if (refine) {
    for (int k = 0; k < rounds; ++k) {
      unsigned s_, c_, tie = 0;
      get_masks(k, &s_, &c_);
      for (unsigned m = c_; m; m &= m - 1) {
        const int i = __ffs(m) - 1;
        const unsigned low = key_at(k, i) & low_mask;
        if (low > tau_low) s_ |= 1u << i;
        else if (low == tau_low) tie |= 1u << i;
      }
      put_masks(k, s_, tie);
    }
  }

  // ---- per-CTA totals, exchanged so that every CTA knows what the CTAs before it contribute
  {
    int n_sure = 0, n_tie = 0;
    for (int k = 0; k < rounds; ++k) {
      unsigned s_, c_;
      get_masks(k, &s_, &c_);
      n_sure += __popc(s_);
      n_tie += __popc(c_);
    }
    n_sure = warp_sum_int(n_sure);
    n_tie = warp_sum_int(n_tie);
    if (lane == 0) { sm.wdef[warp] = n_sure; sm.wtie[warp] = n_tie; }
    __syncthreads();
    if (tid < csize) {
      int a = 0, c = 0;
      for (int w = 0; w < kSelWarps; ++w) { a += sm.wdef[w]; c += sm.wtie[w]; }
      int* r = cluster.map_shared_rank(sm.tot, tid);
      r[2 * rank] = a;
      r[2 * rank + 1] = c;
    }
  }
  cluster.sync();                                          // also the last access to another CTA's memory
  int tie_base = 0, out_base = 0;                          // ties / selected positions before this CTA
  for (int r = 0; r < rank; ++r) {
    const int t = sm.tot[2 * r + 1];
    int take = need_ties - tie_base;
    take = take < 0 ? 0 : (take > t ? t : take);
    out_base += sm.tot[2 * r] + take;
    tie_base += t;
  }

  // ---- write the selected positions of this CTA in index order.  The masks are transposed
  // inside each warp first, so that lane t holds the bits of the 32 consecutive positions
  // 32 t .. 32 t + 31 of the warp's run and thread order is index order; one block scan of
  // the packed (tie, sure) counts then gives every thread its first output slot.
  for (int k = 0; k < rounds; ++k) {
    unsigned s_, c_;
    get_masks(k, &s_, &c_);
    s_ = warp_transpose32(s_, lane);
    c_ = warp_transpose32(c_, lane);
    const int nt = __popc(c_);
    int total;
    const int excl = block_exclusive_scan((nt << 16) | __popc(s_), sm.scratch, &total);   // counts <= 16384 each
    const int admit = max(need_ties - tie_base, 0);        // ties of this round that are still admitted
    const int ties_before = excl >> 16;
    int off = out_base + (excl & 0xffff) + min(ties_before, admit);
    int take = min(max(admit - ties_before, 0), nt);       // admitted ties of this thread, in index order
    const int pos0 = p.n_sink + (rank * rounds + k) * kSelChunk + warp * (32 * kSelPer) + lane * kSelPer;
    for (unsigned m = s_ | c_; m; m &= m - 1) {
      const int i = __ffs(m) - 1;
      bool sel = (s_ >> i) & 1u;
      if (!sel) { sel = take > 0; --take; }
      if (sel) {
        if (off < K) {
          out[off] = pos0 + i;
          if (out2) out2[off] = pos0 + i;
        }
        ++off;
      }
    }
    out_base += (total & 0xffff) + min(total >> 16, admit);
    tie_base += total >> 16;
  }
}

cudaError_t launch_select(const Problem& p, int max_mid, int n_sm, cudaStream_t st) {
  const int rows = p.batch * p.n_q_heads;
  // cluster size: enough CTAs to keep the longest row in shared memory, at most 8 ...
  int csize = 1;
  while (csize < kSelCluster && (long long)csize * kSelChunk < max_mid) csize *= 2;
  // ... but with many rows the grid fills the GPU several times over anyway, and smaller
  // clusters (down to one CTA per row, which then reads its row twice) save the cluster
  // barriers; a CTA handles at most 16 rounds
  const int n_chunks = (max_mid + kSelChunk - 1) / kSelChunk;
  while (csize > 1 && (long long)rows * csize > 4LL * n_sm && (n_chunks + csize / 2 - 1) / (csize / 2) <= 16)
    csize /= 2;
  const int n_tasks = p.with_phi ? rows + p.n_kv_heads : 0;
  const int feat_clusters = (n_tasks + csize - 1) / csize;
  static PerDeviceFlag configured;
  constexpr size_t smem = sizeof(unsigned) * kSelChunk;
  cudaError_t e = set_max_dynamic_smem(configured, reinterpret_cast<const void*>(select_kernel), smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(csize, rows + feat_clusters, 1);
  cfg.blockDim = dim3(kSelThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = csize; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, select_kernel, p, rows, csize);
}

}  // namespace tkphi
