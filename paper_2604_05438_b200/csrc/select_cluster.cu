// Exact Top-K selection over the score rows (exhaustive Top-K control selector, Sec. 5.1;
// ties broken towards the lower index) in ONE kernel: a thread-block cluster of up to eight
// CTAs per query head (1, 2, 4 or 8, enough to hold the longest row of the call).
//
// Each CTA owns a contiguous eighth of the head's mid-region; each warp a contiguous
// 1024-score run of it, read coalesced (lane l, step i -> element 32 i + l), so that
// (CTA, round, warp, step, lane) order is index order.  For sequences of up to 131072
// mid-region keys every CTA keeps its 16384 order-preserving score keys in shared memory
// and the row is read from L2 exactly once (longer rows, up to 2,097,152 keys, are read twice
// and the shared memory holds per-round bit masks instead).
//
// The exact K-th largest key is found by histogram selection over WINDOWS of the 32-bit
// order-preserving key: a window (lo, shift) maps a key >= lo to bin min((key - lo) >> shift,
// 4095), which is monotone in the key, so counting from the top bin down to the bin where
// the count reaches K brackets the threshold exactly whatever the window is.  The first
// window is placed by a sample: every CTA of the cluster reads the same 2048 strided scores of
// the row and takes, from a coarse histogram of them, a lower edge that lies below the K-th
// largest score with high probability and an upper edge at the sample's maximum.  Keys below
// the window (about 97% of a row at a 1% budget) cost no shared-memory atomic, and the bins
// that are hit spread evenly, so the atomics neither collide nor leave a crowded threshold
// bin: it holds a handful of keys instead of thousands.  When the sample misleads (the
// threshold lies below the window, or in the clamped top bin) the count says so and the next
// window covers exactly the range that is left; windows shrink by a factor of at least 2048
// per level, so a few levels resolve any input, exact ties included.
//
// Every CTA builds a local histogram in shared memory and adds its non-zero bins into the
// accumulator of every CTA through distributed shared memory; every CTA then walks its own copy.
// A threshold bin of at most 512 keys is resolved directly: its (key, position) pairs are
// gathered into every CTA and each thread ranks one of them (higher key first, lower position
// first among equal keys).  Positions above the threshold, and as many threshold ties as are
// still needed in index order, are then written straight to their slot of the ascending index
// list: the per-thread bit masks are transposed inside each warp so that thread order is index
// order, and offsets come from one block scan and per-CTA totals exchanged through distributed
// shared memory.  CTAs of a cluster only meet at hardware cluster barriers (no flag spinning,
// no global scratch, nothing to clear between calls).
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
constexpr int kSamplePer = 4;                            // sampled scores per thread
constexpr int kSampleMax = kSelThreads * kSamplePer;     // scores of a row that place the first window
constexpr int kCandCap = kSelThreads;                    // a threshold bin of up to this many keys is ranked directly
constexpr int kSelLevels = 8;                            // windows per row, at most (five suffice for any input)

struct SelShared {
  unsigned hist[kHistBins];      // local histogram of the current window
  unsigned acc[kHistBins];       // the cluster's histogram (every CTA receives every CTA's bins)
  unsigned cand_key[kCandCap];   // keys of the threshold bin, gathered from the whole cluster
  int cand_pos[kCandCap];        // their mid-region positions
  unsigned selw[kSelThreads];    // resident mode: selection bits that the direct ranking decided
  unsigned cand_n;               // entries of the candidate list
  unsigned wmax[kSelWarps];
  int scratch[40];
  int res[4];                    // result of a histogram walk: bin (-1: not reached), count above it, count in it, total
  int tot[2 * kSelCluster];      // per CTA: selected-for-sure count, tie count
  int wdef[kSelWarps], wtie[kSelWarps];
};

// Walks the kHistBins-bin histogram h from the top and finds the bin at which the cumulative
// count reaches `need`; res = {bin, count above it, count in it, count of all bins}, bin = -1
// when the histogram holds fewer than `need` entries.  All 512 threads of the CTA call it.
__device__ void walk_from_top(const unsigned* h, int need, int* res, int* scratch) {
  constexpr int BPT = kHistBins / kSelThreads;
  const int tid = threadIdx.x;
  unsigned loc[BPT];
  int lsum = 0;
#pragma unroll
  for (int i = 0; i < BPT; ++i) { loc[i] = h[tid * BPT + i]; lsum += (int)loc[i]; }
  if (tid == 0) res[0] = -1;                               // (ordered before the finder's write by the scan's barriers)
  int total;
  const int excl = block_exclusive_scan(lsum, scratch, &total);
  const int above = total - excl - lsum;                   // elements in bins above this thread's range
  if (tid == 0) res[3] = total;
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

// smallest s with 2^s >= x (x >= 1)
__device__ __forceinline__ int ceil_log2_u64(unsigned long long x) {
  return x <= 1 ? 0 : 64 - __clzll((long long)(x - 1));
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
    } else if (task < n_rows + p.n_kv_heads && !(p.flags & 1u)) {
      wk_split_job<kSelThreads>(p, task - n_rows);
    }
    return;
  }
  // Everything up to the wait reads only the call's inputs (sequence lengths, budgets) and
  // this CTA's shared memory, so it overlaps the scoring kernel's run.
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  const int row = blockIdx.y, b = row / p.n_q_heads, hq = row % p.n_q_heads;
  const int K = p.topk[b];
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int n_mid = mid_len(len_b, p.n_sink, p.n_tail);
  const float* srow = p.scores + score_row_base(p, b, hq, cu_b, len_b);
  const int n_chunks = (n_mid + kSelChunk - 1) / kSelChunk;
  const int rounds = (n_chunks + csize - 1) / csize;       // per CTA
  const bool resident = rounds == 1;                       // the keys stay in shared memory
  for (int i = tid; i < kHistBins; i += kSelThreads) { sm.hist[i] = 0; sm.acc[i] = 0; }
  sm.selw[tid] = 0;
  if (tid == 0) sm.cand_n = 0;
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
  // adds the non-zero bins of the local histogram into the accumulator of every CTA
  auto push_all = [&]() {
    for (int i = tid; i < kHistBins; i += kSelThreads) {
      const unsigned c = sm.hist[i];
      if (c)
        for (int r = 0; r < csize; ++r) atomicAdd(cluster.map_shared_rank(sm.acc, r) + i, c);
    }
  };

  // ---- the row's sample (the same positions in every CTA of the cluster) and, in resident
  // mode, this thread's 32 scores: all loads are issued before the first one is used
  const int m_s = n_mid < kSampleMax ? n_mid : kSampleMax;
  int r_s;                                                 // rank, in the sample, of the first window's lower edge
  {
    const float mp = (float)m_s * (float)K / (float)n_mid;
    r_s = (int)ceilf(mp + 4.f * sqrtf(mp) + 4.f);          // the expected rank of the threshold plus four deviations
  }
  const bool sampled = r_s < m_s;                          // otherwise the first window is the whole key range
  unsigned skey[kSamplePer];
#pragma unroll
  for (int e = 0; e < kSamplePer; ++e) {
    const int j = tid + e * kSelThreads;
    skey[e] = (sampled && j < m_s) ? ordered_key(__ldcg(srow + (long long)j * n_mid / m_s)) : 0u;
  }
  unsigned kr0[kSelPer];
  unsigned vmask0 = 0;                                     // validity mask of the resident round
  if (resident) vmask0 = load_regs(0, kr0);
  __syncthreads();

  unsigned win_lo = 0;                                     // first window: keys >= win_lo, bins of 2^win_shift keys
  int win_shift = kLowBits;
  if (sampled) {
    unsigned smax = 0;
#pragma unroll
    for (int e = 0; e < kSamplePer; ++e)
      if (tid + e * kSelThreads < m_s) {
        atomicAdd(&sm.acc[skey[e] >> kLowBits], 1u);
        smax = max(smax, skey[e]);
      }
    smax = __reduce_max_sync(0xffffffffu, smax);
    if (lane == 0) sm.wmax[warp] = smax;
    __syncthreads();
    walk_from_top(sm.acc, r_s, sm.res, sm.scratch);        // r_s <= m_s: always found
    const unsigned cb = (unsigned)sm.res[0];
    unsigned cbmax = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) cbmax = max(cbmax, sm.wmax[w]);
    cbmax >>= kLowBits;
    win_lo = cb << kLowBits;
    win_shift = kLowBits - kHistBits + ceil_log2_u64((unsigned long long)(cbmax - cb + 1));
#pragma unroll
    for (int e = 0; e < kSamplePer; ++e)
      if (tid + e * kSelThreads < m_s) sm.acc[skey[e] >> kLowBits] = 0;   // the accumulator is clean again
    __syncthreads();
  }
  cluster.barrier_arrive();                                // "my accumulator is cleared"; waited for below

  // ---- histogram of the first window
  for (int k = 0; k < rounds; ++k) {
    unsigned vm = vmask0;
    if (!resident) vm = load_regs(k, kr0);
#pragma unroll
    for (int i = 0; i < kSelPer; ++i) {
      if (resident) keys[i * kSelThreads] = kr0[i];
      if (((vm >> i) & 1u) && kr0[i] >= win_lo)
        atomicAdd(&sm.hist[min((kr0[i] - win_lo) >> win_shift, (unsigned)(kHistBins - 1))], 1u);
    }
  }
  __syncthreads();
  cluster.barrier_wait();                                  // every accumulator of the cluster is cleared
  push_all();
  cluster.sync();
  walk_from_top(sm.acc, K, sm.res, sm.scratch);

  // The threshold lies in the key range [r_lo, r_hi]: keys above it are selected for sure,
  // `need` of the n_cand keys inside it are still to be taken.
  unsigned r_lo, r_hi;
  int need, n_cand;
  if (sm.res[0] >= 0) {
    const unsigned long long lo64 = (unsigned long long)win_lo + ((unsigned long long)sm.res[0] << win_shift);
    const unsigned long long hi64 = sm.res[0] == kHistBins - 1 ? 0xffffffffull : lo64 + (1ull << win_shift) - 1;
    r_lo = (unsigned)lo64;
    r_hi = (unsigned)(hi64 < 0xffffffffull ? hi64 : 0xffffffffull);
    need = K - sm.res[1];
    n_cand = sm.res[2];
  } else {                                                 // fewer than K keys in the window: the threshold lies below it
    r_lo = 0;
    r_hi = win_lo - 1;                                     // (win_lo > 0: a whole-range window holds every key)
    need = K - sm.res[3];
    n_cand = n_mid - sm.res[3];
  }

  // bit i of a "sure" mask: key i lies above the range; of a "cand" mask: inside it
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
      const unsigned key = keys[i * kSelThreads];
      s_ |= (key > r_hi ? 1u : 0u) << i;
      c_ |= ((key >= r_lo && key <= r_hi) ? 1u : 0u) << i;
    }
    smask = s_ & vmask0; cmask = c_ & vmask0;
  } else {
    for (int k = 0; k < rounds; ++k) {
      const unsigned vm = load_regs(k, kr0);
      unsigned s_ = 0, c_ = 0;
#pragma unroll
      for (int i = 0; i < kSelPer; ++i) {
        s_ |= (kr0[i] > r_hi ? 1u : 0u) << i;
        c_ |= ((kr0[i] >= r_lo && kr0[i] <= r_hi) ? 1u : 0u) << i;
      }
      put_masks(k, s_ & vm, c_ & vm);
    }
  }

  // ---- resolve the threshold range.  Every decision below depends only on the cluster's
  // histogram, so all CTAs of the cluster take the same path and meet at the same barriers.
  int need_ties = n_cand;                                  // need == n_cand: the whole range is taken
  for (int level = 0; level < kSelLevels && need < n_cand; ++level) {
    if (n_cand <= kCandCap) {
      // ---- direct ranking: every CTA gets every (key, position) of the range
      for (int k = 0; k < rounds; ++k) {
        unsigned s_, c_;
        get_masks(k, &s_, &c_);
        for (unsigned m = c_; m; m &= m - 1) {
          const int i = __ffs(m) - 1;
          const unsigned key = key_at(k, i);
          const int pos = round_base(k) + i * 32;
          for (int r = 0; r < csize; ++r) {
            const unsigned slot = atomicAdd(cluster.map_shared_rank(&sm.cand_n, r), 1u);
            if (slot < (unsigned)kCandCap) {
              cluster.map_shared_rank(sm.cand_key, r)[slot] = key;
              cluster.map_shared_rank(sm.cand_pos, r)[slot] = pos;
            }
          }
        }
      }
      cluster.sync();
      if (tid < n_cand) {
        const unsigned mykey = sm.cand_key[tid];
        const int mypos = sm.cand_pos[tid];
        int better = 0;                                    // keys of the range that come before this one
        for (int j = 0; j < n_cand; ++j) {
          const unsigned kj = sm.cand_key[j];
          better += (kj > mykey || (kj == mykey && sm.cand_pos[j] < mypos)) ? 1 : 0;
        }
        const int local = mypos - rank * rounds * kSelChunk;
        if (better < need && local >= 0 && local < rounds * kSelChunk) {
          const int k = local / kSelChunk, in = local % kSelChunk;
          const int t = (in >> 10) * 32 + (in & 31), i = (in >> 5) & 31;
          if (resident) atomicOr(&sm.selw[t], 1u << i);
          else atomicOr(&keys_s[(2 * k) * kSelThreads + t], 1u << i);
        }
      }
      __syncthreads();
      if (resident) { smask |= sm.selw[tid]; cmask = 0; }
      else
        for (int k = 0; k < rounds; ++k) keys_s[(2 * k + 1) * kSelThreads + tid] = 0;
      need_ties = 0;
      break;
    }
    if (r_lo == r_hi) { need_ties = need; break; }         // one key value: exact ties, admitted in index order
    // ---- next window: the whole range that is left, in 4096 bins
    const int z_shift = max(0, ceil_log2_u64((unsigned long long)r_hi - r_lo + 1) - kHistBits);
    for (int i = tid; i < kHistBins; i += kSelThreads) { sm.hist[i] = 0; sm.acc[i] = 0; }
    __syncthreads();
    cluster.sync();                                        // every accumulator of the cluster is cleared
    for (int k = 0; k < rounds; ++k) {
      unsigned s_, c_;
      get_masks(k, &s_, &c_);
      for (unsigned m = c_; m; m &= m - 1) atomicAdd(&sm.hist[(key_at(k, __ffs(m) - 1) - r_lo) >> z_shift], 1u);
    }
    __syncthreads();
    push_all();
    cluster.sync();
    walk_from_top(sm.acc, need, sm.res, sm.scratch);       // need <= n_cand: always found
    const unsigned long long lo64 = (unsigned long long)r_lo + ((unsigned long long)sm.res[0] << z_shift);
    const unsigned long long hi64 = lo64 + (1ull << z_shift) - 1;
    const unsigned n_lo = (unsigned)lo64, n_hi = hi64 < (unsigned long long)r_hi ? (unsigned)hi64 : r_hi;
    for (int k = 0; k < rounds; ++k) {
      unsigned s_, c_, keep = 0;
      get_masks(k, &s_, &c_);
      for (unsigned m = c_; m; m &= m - 1) {
        const int i = __ffs(m) - 1;
        const unsigned key = key_at(k, i);
        if (key > n_hi) s_ |= 1u << i;
        else if (key >= n_lo) keep |= 1u << i;
      }
      put_masks(k, s_, keep);
    }
    need -= sm.res[1];
    n_cand = sm.res[2];
    r_lo = n_lo;
    r_hi = n_hi;
    need_ties = n_cand;                                    // (if the loop ends here, need == n_cand)
    __syncthreads();                                       // sm.res is rewritten by the next walk
  }

  // after this, "sure": keys above the exact threshold; "cand": keys equal to it, of which the
  // first need_ties in index order are taken

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
