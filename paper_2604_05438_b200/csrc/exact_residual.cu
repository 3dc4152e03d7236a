// Steps (2)-(5) of the decode path for one query head per CTA column:
//   (2) exact branch over E = A U K(q): m_E, Z_E = sum exp(s_i - m_E),
//       nu_E = sum exp(s_i - m_E) v_i                      (Sec. 3, Eq. exact_terms)
//   (3) retrieved-token subtraction                         (Sec. 4.2, Eq. subtraction)
//   (4) residual estimate nu_hat_R = S_R phi_q, Z_hat_R = phi_q . u_R   (Sec. 4.3)
//   (5) single-normalisation merge                          (Sec. 4.3, Eq. hybrid_merge)
//
// Steps (3)-(4) are evaluated in the reassociated form
//   nu_hat_R = S_M phi_q - sum_{i in K(q)} z_i v_i,  Z_hat_R = phi_q . u_M - sum z_i,
//   z_i = <phi_q(q), phi_k(k_i)>,
// which equals contracting S_R = S_M - sum v_i phi_k(k_i)^T with phi_q but needs
// 2K(r+d) instead of 2Kdr flops after the feature recompute, and lets each
// retrieved token contribute to both branches while its v row is in shared memory.
// phi_q is carried as exp(a_q - m_q) with the log-scale m_q separate.
//
// The support list of a query head is cut into slices of 128 tokens; a CTA takes two
// adjacent slices, one per group of 128 threads, which share the W_k operand tiles (so a
// decode call at a 1% budget of a 128K context is a single wave of one CTA per SM).
// The k and v rows of a slice are gathered into 128B-swizzled shared-memory tiles.
// The feature recompute of the retrieved keys, W_k k_i for 128 tokens x r features, is
// a dense [128 x d] x [d x r] contraction: it runs as tcgen05.mma with the gathered key
// tile as A and W_k, split into bf16 hi + lo parts (error ~2^-18 |W|) that are stacked
// into one B operand of 2r rows (an MMA with M = 128 takes the same time for N = 2r as
// for N = r), as B; the 128 x 2r fp32 result stays in tensor memory and each thread reads
// the row of its own token and adds the hi and lo halves, so <phi_q, phi_k(k_i)> needs no
// cross-thread reduction.  Each CTA writes partial sums; the last CTA of a head (one atomic
// ticket, no spinning) combines them in slice order, so results are run-to-run
// identical.
//
// With cached key features (Sec. 4.2 mentions a cached implementation; cached_features.cu) the z_i of
// the retrieved tokens come from a buffer instead: no key rows of retrieved tokens, no W_k tiles, no
// tensor-core work; everything else is the same.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr int kExGroups = 2;                        // slices per CTA
constexpr int kExThreads = kExGroups * kSlice;      // one thread per token of a slice = per tensor-memory lane

template <int D, int R>
struct ExSmem {
  static constexpr int BOXES = D / 64;
  static constexpr int KV_BOX = kSlice * 128;                 // bytes of one 64-dim column block of k or v
  static constexpr int W_BOX = 2 * R * 128;                   // hi rows, then lo rows
  static constexpr size_t kv_tile = (size_t)BOXES * KV_BOX;   // one k or v tile [BOXES][128][128 B]
  static constexpr size_t kt = 0;                             // bf16 k tiles, one per group
  static constexpr size_t whi = kt + kExGroups * kv_tile;     // bf16 W_k hi|lo  [BOXES][2R][128 B]
  // the v tiles take over the W_k region once the MMAs have read it (the v rows wait in
  // registers until then)
  static constexpr size_t vt = whi;
  static constexpr size_t w_bytes = (size_t)BOXES * W_BOX, v_bytes = kExGroups * kv_tile;
  static constexpr size_t small = whi + (w_bytes > v_bytes ? w_bytes : v_bytes);
  // small: bars[4] (32 B), tok[T] int, isret[T] int, wgt[T], zt[T] (T threads), qf[D], cj[R], spare[R],
  //        red[groups][4*D], misc[32]
  static constexpr size_t total = small + 32 + 4 * (4 * kExThreads + D + 2 * R + kExGroups * 4 * D + 32);
};

// ------------------------------------------------------------------ per-slice arithmetic shared by both kernels
// Thread = token `gt` of a 128-token slice whose k rows sit in the 128B-swizzled tile `kt`:
// returns q . k_t / sqrt(d) (*dot_scaled) and |k_t|^2 (*kn).
template <int D>
__device__ __forceinline__ void token_dot_and_norm(const unsigned char* kt, int gt, const float* qf, float scale,
                                                   float* dot_scaled, float* kn_out) {
  using L = ExSmem<D, 64>;                                  // (tile geometry does not depend on R)
  float dot = 0.f, kn = 0.f;
#pragma unroll
  for (int c = 0; c < D / 8; ++c) {
    const uint4 raw = *reinterpret_cast<const uint4*>(kt + (c >> 3) * L::KV_BOX + swz128(gt, c & 7));
    const unsigned w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float x0 = bf16_lo(w[e]), x1 = bf16_hi(w[e]);
      dot = fmaf(x0, qf[c * 8 + 2 * e], dot);
      dot = fmaf(x1, qf[c * 8 + 2 * e + 1], dot);
      kn = fmaf(x0, x0, kn);
      kn = fmaf(x1, x1, kn);
    }
  }
  *dot_scaled = dot * scale;
  *kn_out = kn;
}

// z_t = <phi_q, phi_k(k_t)> / exp(m_q) from this token's row of the feature-recompute accumulator
// (columns [0, R): W_hi k_t, [R, 2R): W_lo k_t, both scaled by log2 e; lane of tensor memory = token):
// z = 2^(-gamma log2e |k|^2) * sum_j 2^(hi_j + lo_j + c_j), c_j = log2 w_j + b_k[j] log2 e; four partial
// sums in a fixed order.  Called by whole warps (gwarp = warp index inside the slice's group).
template <int R>
__device__ __forceinline__ float z_from_accumulator(uint32_t tmem_d, int gwarp, const float* cj, float gamma_k, float kn) {
  float zp[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int c4 = 0; c4 < R / 32; ++c4) {
    float v[32], vl[32];
    tmem_ld_x32(tmem_addr(tmem_d, gwarp * 32, c4 * 32), v);
    tmem_ld_x32(tmem_addr(tmem_d, gwarp * 32, R + c4 * 32), vl);
    tc_wait_ld();
#pragma unroll
    for (int j = 0; j < 32; ++j) zp[j & 3] += ex2_approx((v[j] + vl[j]) + cj[c4 * 32 + j]);
  }
  return ((zp[0] + zp[1]) + (zp[2] + zp[3])) * ex2_approx(-gamma_k * kLog2e * kn);
}

// Value pass of one slice (thread gt of its group): nu[dv] = sum_t w_t v_t[dv], zv[dv] = sum_t z_t v_t[dv]
// over the thread's token group, even / odd tokens added in a fixed order, into red[tg][2 D].
template <int D>
__device__ __forceinline__ void slice_value_pass(const unsigned char* vt, const float* wgt, const float* zt, int gt,
                                                 float* red) {
  using L = ExSmem<D, 64>;
  constexpr int NGV = kSlice / D;            // token groups for the value pass (1 or 2)
  constexpr int TPV = kSlice / NGV;
  const int dv = gt % D, tg = gt / D;
  const unsigned char* vcol = vt + (dv >> 6) * L::KV_BOX + (dv & 7) * 2;
  const uint32_t ch = (dv & 63) >> 3;
  float nu0 = 0.f, nu1 = 0.f, zv0 = 0.f, zv1 = 0.f;
#pragma unroll 4
  for (int t = tg * TPV; t < (tg + 1) * TPV; t += 2) {
    const unsigned short r0 = *reinterpret_cast<const unsigned short*>(vcol + swz128(t, ch));
    const unsigned short r1 = *reinterpret_cast<const unsigned short*>(vcol + swz128(t + 1, ch));
    const float x0 = __uint_as_float((unsigned)r0 << 16), x1 = __uint_as_float((unsigned)r1 << 16);
    nu0 = fmaf(wgt[t], x0, nu0);
    zv0 = fmaf(zt[t], x0, zv0);
    nu1 = fmaf(wgt[t + 1], x1, nu1);
    zv1 = fmaf(zt[t + 1], x1, zv1);
  }
  red[tg * 2 * D + dv] = nu0 + nu1;
  red[tg * 2 * D + D + dv] = zv0 + zv1;
}

// Writes a slice's partial sums: part[0..3] = m_slice, Z = sum w_t, zs = sum z_t, 0; part[4..] = nu, zv.
// Called by the 128 threads of the slice's group after slice_value_pass and a barrier.
template <int D>
__device__ __forceinline__ void slice_write_partials(float* part, const float* red, const float* wgt, const float* zt,
                                                     int gt, int gwarp, int lane, float m_slice) {
  constexpr int NGV = kSlice / D;
  for (int i = gt; i < 2 * D; i += kSlice) {
    float x = red[i];
    if (NGV == 2) x += red[2 * D + i];       // second token group, fixed order
    part[4 + i] = x;
  }
  if (gwarp == 0) {
    float Z = 0.f, zs = 0.f;
#pragma unroll
    for (int i = 0; i < kSlice / 32; ++i) { Z += wgt[lane + 32 * i]; zs += zt[lane + 32 * i]; }
    Z = warp_sum(Z);
    zs = warp_sum(zs);
    if (lane == 0) { part[0] = m_slice; part[1] = Z; part[2] = zs; part[3] = 0.f; }
  }
}

// The last CTA of a head combines the slice partials in slice order, by a fixed assignment
// of slices to lanes and of output columns to threads, so the result does not depend on
// timing; then the residual estimate and the merge under one normalisation (Sec. 4.3,
// Eq. hybrid_merge).  Called by all kExThreads threads of the CTA; misc: >= 18 floats of
// shared memory.  BAR 0: the CTA has exactly these threads (__syncthreads); BAR 1: they are
// the first kExThreads of a larger CTA and meet at named barrier 1.
template <int BAR>
__device__ __forceinline__ void ex_sync() {
  if (BAR == 0) __syncthreads();
  else asm volatile("bar.sync 1, %0;" ::"n"(kExThreads) : "memory");
}
template <int BAR>
__device__ __forceinline__ bool ex_sync_and(bool x) {
  if (BAR == 0) return __syncthreads_and(x ? 1 : 0) != 0;
  uint32_t r;
  asm volatile(
      "{\n"
      " .reg .pred p, q;\n"
      " setp.ne.u32 q, %1, 0;\n"
      " bar.red.and.pred p, 1, %2, q;\n"
      " selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(r)
      : "r"(x ? 1u : 0u), "n"(kExThreads)
      : "memory");
  return r != 0;
}

template <int D, int R, int BAR>
__device__ __forceinline__ void merge_head(const Problem& p, int row, int n_slices, int nE, float* misc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // slice partials are combined in slice order by a fixed assignment of slices to
  // lanes and of output columns to threads, so the result does not depend on timing
  const float* parts = p.partials + (size_t)row * p.max_slices * p.partial_stride;
  constexpr int kFast = 16;                  // up to this many slices every load is issued at once
  float m_E = -INFINITY, Z_E = 0.f, zs = 0.f, nu_E = 0.f, zv = 0.f;
  const float* aqr = p.aq + (size_t)row * aq_stride(R, D);
  float aq_m = 0.f, aq_u = 0.f, aq_s = 0.f;   // m_q, w . u_M, (S_M w)[tid]
  if (p.with_phi) { aq_m = __ldcg(aqr + R); aq_u = __ldcg(aqr + R + 1); if (tid < D) aq_s = __ldcg(aqr + R + 4 + tid); }
  if (n_slices <= kFast) {
    // every thread combines the slice scalars itself (same order everywhere, no barrier)
    float ms[kFast], Zs[kFast], zz[kFast], nus[kFast], zvs[kFast];
    const int dv = tid < D ? tid : 0;
#pragma unroll
    for (int s = 0; s < kFast; ++s) {
      const float* ps = parts + (size_t)(s < n_slices ? s : 0) * p.partial_stride;
      ms[s] = __ldcg(ps); Zs[s] = __ldcg(ps + 1); zz[s] = __ldcg(ps + 2);
      nus[s] = __ldcg(ps + 4 + dv); zvs[s] = __ldcg(ps + 4 + D + dv);
    }
    if (nE > 0) {
#pragma unroll
      for (int s = 0; s < kFast; ++s) if (s < n_slices) m_E = fmaxf(m_E, ms[s]);
    }
#pragma unroll
    for (int s = 0; s < kFast; ++s) {
      if (s < n_slices) {
        const float f = nE > 0 ? expf(ms[s] - m_E) : 0.f;
        Z_E = fmaf(f, Zs[s], Z_E);
        zs += zz[s];
        nu_E = fmaf(f, nus[s], nu_E);
        zv += zvs[s];
      }
    }
  } else {
    float m_loc = -INFINITY;
    if (nE > 0)
      for (int s = tid; s < n_slices; s += kExThreads) m_loc = fmaxf(m_loc, __ldcg(parts + (size_t)s * p.partial_stride));
    m_loc = warp_max(m_loc);
    if (lane == 0) misc[warp] = m_loc;
    ex_sync<BAR>();
#pragma unroll
    for (int w = 0; w < kExThreads / 32; ++w) m_E = fmaxf(m_E, misc[w]);
    if (warp == 0) {
      float Zp = 0.f, zp = 0.f;
      for (int s = lane; s < n_slices; s += 32) {
        const float* ps = parts + (size_t)s * p.partial_stride;
        const float f = nE > 0 ? expf(__ldcg(ps) - m_E) : 0.f;
        Zp = fmaf(f, __ldcg(ps + 1), Zp);
        zp += __ldcg(ps + 2);
      }
      Zp = warp_sum(Zp);
      zp = warp_sum(zp);
      if (lane == 0) { misc[16] = Zp; misc[17] = zp; }
    }
    if (tid < D) {
#pragma unroll 8
      for (int s = 0; s < n_slices; ++s) {
        const float* ps = parts + (size_t)s * p.partial_stride;
        const float f = nE > 0 ? expf(__ldcg(ps) - m_E) : 0.f;
        nu_E = fmaf(f, __ldcg(ps + 4 + tid), nu_E);
        zv += __ldcg(ps + 4 + D + tid);
      }
    }
    ex_sync<BAR>();
    Z_E = misc[16]; zs = misc[17];
  }
  float y = 0.f, yR = 0.f, logZR = -INFINITY, Mx = m_E;
  if (p.with_phi) {
    // S_M phi_q and phi_q . u_M (in units of exp(m_q)) were prepared alongside phi_q
    const float m_q = aq_m;
    const float Zt = aq_u - zs;                            // Z_hat_R / exp(m_q)
    if (Zt > 0.f) {
      logZR = m_q + logf(Zt);
      Mx = fmaxf(m_E, logZR);
      const float cE = nE > 0 ? expf(m_E - Mx) : 0.f, cR = expf(logZR - Mx);
      if (tid < D) {
        yR = (aq_s - zv) / Zt;
        y = (cE * nu_E + cR * yR) / (cE * Z_E + cR);
      }
    } else if (tid < D) {
      y = nE > 0 ? nu_E / Z_E : 0.f;
    }
  } else if (tid < D) {
    y = nE > 0 ? nu_E / Z_E : 0.f;
  }
  if (tid < D) p.y_out[(size_t)row * D + tid] = y;
  if (p.dbg_out) {
    float* dbg = p.dbg_out + (size_t)row * (4 + D);
    if (tid < D) dbg[4 + tid] = yR;
    if (tid == 0) { dbg[0] = m_E; dbg[1] = Z_E; dbg[2] = logZR; dbg[3] = Mx; }
  }
}

template <int D, int R>
__global__ void __launch_bounds__(kExThreads) exact_residual_kernel(const Problem p) {
  using L = ExSmem<D, R>;
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = tid / kSlice, gt = tid % kSlice, gwarp = warp & 3;   // group, token (= tensor-memory lane), warp of the group
  unsigned char* kt = smem + L::kt + grp * L::kv_tile;      // this group's tiles
  unsigned char* vt = smem + L::vt + grp * L::kv_tile;
  unsigned char* whi = smem + L::whi;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::small);   // [0]: W tiles landed, [1 + g]: MMAs of group g done
  int* tok = reinterpret_cast<int*>(bars + 4) + grp * kSlice;        // per-token arrays: this group's part
  int* isret = reinterpret_cast<int*>(bars + 4) + kExThreads + grp * kSlice;
  float* wgt = reinterpret_cast<float*>(bars + 4) + 2 * kExThreads + grp * kSlice;
  float* zt = reinterpret_cast<float*>(bars + 4) + 3 * kExThreads + grp * kSlice;
  float* qf = reinterpret_cast<float*>(bars + 4) + 4 * kExThreads;
  float* cj = qf + D;               // log2 w_j + b_k[j] log2 e
  float* red = cj + 2 * R + grp * 4 * D;
  float* misc = cj + 2 * R + kExGroups * 4 * D;
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 28);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc + 29);

  const int b = blockIdx.z, hq = blockIdx.y, slice0 = blockIdx.x * kExGroups, slice = slice0 + grp;
  pdl_launch_next();
  const int row = b * p.n_q_heads + hq, kvh = hq / p.group;
  const int K = p.topk[b];
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int nA1 = (int)(len_b < p.n_sink ? len_b : p.n_sink);
  long long ts = len_b - tail_of(p, b);
  if (ts < p.n_sink) ts = p.n_sink;
  if (ts > len_b) ts = len_b;
  const int tail_start = (int)ts, n_tail_eff = (int)(len_b - ts);
  const int nE = nA1 + K + n_tail_eff;
  const int n_slices = nE > 0 ? (nE + kSlice - 1) / kSlice : 1;
  if (slice0 >= n_slices) return;
  const int n_ctas = (n_slices + kExGroups - 1) / kExGroups;
  const bool live = slice < n_slices;            // the last CTA of a head may hold one empty group
  const bool do_phi = p.with_phi && !(p.flags & 1u) && !p.zbuf;   // recompute the retrieved keys' features here
  // does a slice hold retrieved tokens (positions nA1 .. nA1+K-1 of the support list) whose features are recomputed?
  auto slice_has_ret = [&](int s) { return do_phi && s < n_slices && s * kSlice < nA1 + K && (s + 1) * kSlice > nA1; };
  const bool has_ret = slice_has_ret(slice);
  bool any_ret = false;
#pragma unroll
  for (int g = 0; g < kExGroups; ++g) any_ret = any_ret || slice_has_ret(slice0 + g);

  const __nv_bfloat16* kbase = p.k + (long long)kvh * p.stride_head + cu_b * p.stride_token;
  const __nv_bfloat16* vbase = p.v + (long long)kvh * p.stride_head + cu_b * p.stride_token;
  const float* srow = p.scores + score_row_base(p, b, hq, cu_b, len_b);

  // ---- 0. barriers, tensor memory, W_k operand tiles
  if (tid == 0) {
    mbar_init(&bars[0], 1);
#pragma unroll
    for (int g = 0; g < kExGroups; ++g) mbar_init(&bars[1 + g], 1);
    mbar_fence_init();
    *s_abort = 0;
  }
  pdl_wait();                                  // the index lists, features and score rows of the predecessors
  if (any_ret && warp == 0) tmem_alloc(s_tmem, kExGroups * 2 * R);   // after the wait: never hold columns a predecessor needs
  // ---- 1. token list of this slice
  float z_cached = 0.f;                        // cached features: z of this thread's token
  {
    const int pi = slice * kSlice + gt;
    int t = -1, ret = 0;
    if (live && pi < nE) {
      if (pi < nA1) t = pi;
      else if (pi < nA1 + K) { t = p.idx[(size_t)row * p.topk_max + (pi - nA1)]; ret = 1; }
      else t = tail_start + (pi - nA1 - K);
    }
    tok[gt] = t;
    isret[gt] = ret;
    if (ret && p.zbuf) z_cached = __ldcg(p.zbuf + (size_t)row * p.topk_max + (pi - nA1));   // used in step 5
  }
  for (int c = tid; c < D; c += kExThreads) qf[c] = __bfloat162float(p.q[(size_t)row * D + c]);
  if (do_phi) {
    for (int j = tid; j < R; j += kExThreads)
      cj[j] = p.aq[(size_t)row * aq_stride(R, D) + R + 4 + D + j] + p.b_k[(size_t)kvh * R + j] * kLog2e;
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (any_ret && tid == 0) {
    const unsigned char* img = reinterpret_cast<const unsigned char*>(p.wk_img + (size_t)kvh * 2 * R * D);
    mbar_expect_tx(&bars[0], 2u * R * D * 2u);
    bulk_load(whi, img, 2 * R * D * 2, &bars[0]);
  }

  // ---- 2. gather rows into swizzled tiles: v always; k for anchors (scores) and, with phi,
  // retrieved rows.  Sixteen-byte copies, all in flight at once: k asynchronously into its tile,
  // v into registers (its tile reuses the W_k region later).
  constexpr int CPR = D / 8;                 // 16-byte chunks per row = copies per thread
  uint4 vreg[CPR];
  const uint64_t pol = l2_policy_evict_first();   // support rows are read once per head
#pragma unroll
  for (int n = 0; n < CPR; ++n) {
    const int i = gt + n * kSlice;
    const int t = i / CPR, c = i % CPR;
    const int ti = tok[t];
    const uint32_t off = (c >> 3) * L::KV_BOX + swz128(t, c & 7);
    vreg[n] = make_uint4(0, 0, 0, 0);
    if (ti >= 0) {
      vreg[n] = ld_global_16(vbase + (long long)ti * p.stride_token + c * 8, pol);
      if (!isret[t] || do_phi) cp_async_16(kt + off, kbase + (long long)ti * p.stride_token + c * 8, pol);
      else *reinterpret_cast<uint4*>(kt + off) = make_uint4(0, 0, 0, 0);
    } else {
      *reinterpret_cast<uint4*>(kt + off) = make_uint4(0, 0, 0, 0);
    }
  }
  cp_async_wait_all();
  fence_proxy_async_smem();
  __syncthreads();

  // ---- 3. feature recompute on the tensor core: acc[t][j] = sum_c k_t[c] (W_hi + W_lo)[j][c]
  bool ok = true;
  if (any_ret && tid == 0) {
    ok = mbar_wait(&bars[0], 0, s_abort);
    if (ok) {
      tc_fence_after_sync();
      constexpr uint32_t idesc = umma_idesc_bf16(128, 2 * R, 0, 0);
      const uint64_t bdesc0 = umma_smem_desc(smem_u32(whi), 16, 1024);
#pragma unroll
      for (int g = 0; g < kExGroups; ++g) {
        if (!slice_has_ret(slice0 + g)) continue;
        const uint32_t tmem_d = *s_tmem + g * 2 * R;         // group g: hi part in columns [2gR, 2gR+R), lo part after it
        const uint64_t adesc0 = umma_smem_desc(smem_u32(smem + L::kt + g * L::kv_tile), 16, 1024);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          umma_ss(tmem_d, adesc0 + (uint64_t)(((k >> 2) * L::KV_BOX + (k & 3) * 32) >> 4),
                  bdesc0 + (uint64_t)(((k >> 2) * L::W_BOX + (k & 3) * 32) >> 4), idesc, k ? 1u : 0u);
        tc_commit(&bars[1 + g]);
      }
    }
  }

  // ---- 4. per token (thread = token): |k|^2, anchor score, softmax weight
  const int ti = tok[gt];
  float s_val = -INFINITY, kn = 0.f;
  if (ti >= 0) {
    float dot;
    token_dot_and_norm<D>(kt, gt, qf, p.scale, &dot, &kn);
    s_val = isret[gt] ? srow[ti - p.n_sink] : dot;
  }
  {
    const float m = warp_max(s_val);
    if (lane == 0) misc[warp] = m;
  }
  __syncthreads();
  const float m_slice = fmaxf(fmaxf(misc[4 * grp], misc[4 * grp + 1]), fmaxf(misc[4 * grp + 2], misc[4 * grp + 3]));
  const float w_t = ti >= 0 ? expf(s_val - m_slice) : 0.f;
  wgt[gt] = w_t;

  // ---- 5. z_t = <phi_q, phi_k(k_t)> from the accumulator row of this token
  float z_t = 0.f;
  if (has_ret) ok = mbar_wait(&bars[1 + grp], 0, s_abort);
  ok = __syncthreads_and(ok ? 1 : 0) != 0;         // every group's MMAs are done: the W_k tiles are free
  // the v rows move from registers into their tile (over the W_k region)
#pragma unroll
  for (int n = 0; n < CPR; ++n) {
    const int i = gt + n * kSlice;
    const int t = i / CPR, c = i % CPR;
    *reinterpret_cast<uint4*>(vt + (c >> 3) * L::KV_BOX + swz128(t, c & 7)) = vreg[n];
  }
  if (has_ret && ok) {
    tc_fence_after_sync();
    z_t = z_from_accumulator<R>(*s_tmem + grp * 2 * R, gwarp, cj, p.gamma_k, kn);
    if (!isret[gt]) z_t = 0.f;
  }
  if (p.zbuf) z_t = z_cached;                  // (zero for anchors)
  zt[gt] = z_t;
  __syncthreads();

  // ---- 6. slice partials: nu = sum w_t v_t, zv = sum z_t v_t, Z = sum w_t, zs = sum z_t
  slice_value_pass<D>(vt, wgt, zt, gt, red);
  __syncthreads();
  if (live)
    slice_write_partials<D>(p.partials + ((size_t)row * p.max_slices + slice) * p.partial_stride, red, wgt, zt, gt, gwarp,
                            lane, m_slice);

  // ---- tensor memory is no longer needed
  tc_fence_before_sync();
  __syncthreads();
  if (any_ret && warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(*s_tmem, kExGroups * 2 * R);
  }
  if (*s_abort) {
    if (tid == 0) atomicExch(p.status, kStatusTimeout);
    return;
  }

  // ---- ticket: the last CTA of this head merges
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned prev = atomicAdd(&p.row_counter[row], 1u);
    misc[8] = (prev == (unsigned)(n_ctas - 1)) ? 1.f : 0.f;
  }
  __syncthreads();
  if (misc[8] == 0.f) return;
  __threadfence();

  merge_head<D, R, 0>(p, row, n_slices, nE, misc);
}

// ---------------------------------------------------------------------------------------
// Streaming variant for calls whose slice pairs do not fit one wave of CTAs (budgets of 2%
// and more at 128K, million-token contexts): a persistent grid of one CTA per SM, every CTA
// a contiguous range of (query head, slice pair) items.  The W_k tiles stay in shared memory
// across items of a KV head, the k and v tiles have regions of their own, and the gathers of
// item i+1 are issued while item i is being computed: the k rows as soon as the MMAs and the
// token phase of item i are done with the k tiles, the v rows as soon as its value pass is
// done with the v tiles.  The gathers are TMA row gathers issued by two producer warps of
// their own (warp 8: k rows, warp 9: v rows; a warp issues its 128 gathers of an item in
// about 4.5 us), which the eight compute warps tell through mbarriers when a tile region is
// free; the compute warps meet at a named barrier, so they never wait for the issue of a
// gather.  Per item the arithmetic and its order are those of exact_residual_kernel.
// Needs a cache whose rows form a 2-D tensor.
template <int D, int R>
struct ExStreamSmem {
  using B = ExSmem<D, R>;
  static constexpr size_t kt = 0;
  static constexpr size_t w = kt + kExGroups * B::kv_tile;
  static constexpr size_t vt = w + B::w_bytes;
  static constexpr size_t small = vt + kExGroups * B::kv_tile;
  // small: bars[8], tok[2][T] int, isret[2][T] int, wgt[T], zt[T], qf[2][D], cj[2][R], red[groups][4*D],
  //        misc[32], pre[kMaxBatch + 2] int, zc[2][T]
  static constexpr size_t total =
      small + 64 + 4 * (8 * kExThreads + 2 * D + 2 * R + kExGroups * 4 * D + 32 + kMaxBatch + 2);
};

constexpr int kExStreamThreads = kExThreads + 64;   // compute warps 0..7, producer warps 8 (k rows) and 9 (v rows)

struct ExItem {
  int b, hq, row, kvh, K, nA1, tail_start, nE, n_slices, n_ctas, slice0;
  long long cu_b, len_b;
};

template <int D, int R>
__global__ void __launch_bounds__(kExStreamThreads, 1)
exact_residual_stream_kernel(const __grid_constant__ CUtensorMap gmap_k, const __grid_constant__ CUtensorMap gmap_v,
                             const Problem p) {
  using L = ExStreamSmem<D, R>;
  using LB = ExSmem<D, R>;
  extern __shared__ __align__(1024) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = tid / kSlice, gt = tid % kSlice, gwarp = warp & 3;
  unsigned char* kt = smem + L::kt + grp * LB::kv_tile;
  unsigned char* vt = smem + L::vt + grp * LB::kv_tile;
  unsigned char* wt = smem + L::w;
  // bars [0]: W tiles landed, [1 + g]: MMAs of group g done, [3]: k tiles landed, [4]: v tiles landed,
  //      [5]: k tiles free and the next item's token list staged, [6]: v tiles free
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::small);
  const bool producer = warp >= kExThreads / 32;
  int* tok_all = reinterpret_cast<int*>(bars + 8);                  // [2 buffers][T]
  int* isret_all = tok_all + 2 * kExThreads;
  float* wgt = reinterpret_cast<float*>(isret_all + 2 * kExThreads) + grp * kSlice;
  float* zt = reinterpret_cast<float*>(isret_all + 2 * kExThreads) + kExThreads + grp * kSlice;
  float* qf_all = reinterpret_cast<float*>(isret_all + 2 * kExThreads) + 2 * kExThreads;   // [2][D]
  float* cj_all = qf_all + 2 * D;                                                          // [2][R]
  float* red = cj_all + 2 * R + grp * 4 * D;
  float* misc = cj_all + 2 * R + kExGroups * 4 * D;
  volatile int* s_abort = reinterpret_cast<volatile int*>(misc + 28);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(misc + 29);
  int* pre = reinterpret_cast<int*>(misc + 32);                     // [batch + 1] items before sequence b
  float* zc_all = reinterpret_cast<float*>(pre + kMaxBatch + 2);    // [2 buffers][T] cached z of the tokens

  pdl_launch_next();
  const bool do_phi = p.with_phi && !(p.flags & 1u) && !p.zbuf;     // recompute the retrieved keys' features here
  const int batch = p.batch, Hq = p.n_q_heads;

  // ---- items per sequence -> prefix (reads only the call's inputs)
  auto pairs_of = [&](int b) {
    const long long len_b = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
    const int nA1 = (int)(len_b < p.n_sink ? len_b : p.n_sink);
    long long ts = len_b - tail_of(p, b);
    if (ts < p.n_sink) ts = p.n_sink;
    if (ts > len_b) ts = len_b;
    const int nE = nA1 + p.topk[b] + (int)(len_b - ts);
    const int n_slices = nE > 0 ? (nE + kSlice - 1) / kSlice : 1;
    return (n_slices + kExGroups - 1) / kExGroups;
  };
  {
    const int per = (batch + kExStreamThreads - 1) / kExStreamThreads;
    const int b0 = tid * per;
    int local = 0;
    for (int i = 0; i < per; ++i)
      if (b0 + i < batch) local += Hq * pairs_of(b0 + i);
    int total;
    int run = block_exclusive_scan(local, tok_all, &total);   // (the token buffers are not in use yet)
    for (int i = 0; i < per; ++i)
      if (b0 + i < batch) { pre[b0 + i] = run; run += Hq * pairs_of(b0 + i); }
    if (tid == 0) pre[batch] = total;
  }
  if (tid == 0) {
    mbar_init(&bars[0], 1);
#pragma unroll
    for (int g = 0; g < kExGroups; ++g) mbar_init(&bars[1 + g], 1);
    mbar_init(&bars[3], 1);
    mbar_init(&bars[4], 1);
    mbar_init(&bars[5], 1);
    mbar_init(&bars[6], 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (tid == 0) *s_abort = 0;
  const int n_items = pre[batch];
  const int i0 = (int)((long long)n_items * blockIdx.x / gridDim.x);
  const int i1 = (int)((long long)n_items * (blockIdx.x + 1) / gridDim.x);

  auto item_of = [&](int i, const ExItem* prev) {
    ExItem it;
    if (prev && i >= pre[prev->b] && i < pre[prev->b + 1]) {   // same sequence as the previous item: no loads
      it = *prev;
      const int rem = i - pre[it.b];
      it.hq = rem / it.n_ctas;
      it.slice0 = (rem % it.n_ctas) * kExGroups;
      it.row = it.b * Hq + it.hq;
      it.kvh = it.hq / p.group;
      return it;
    }
    int lo = 0, hi = batch - 1;                // largest b with pre[b] <= i
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (pre[mid] <= i) lo = mid; else hi = mid - 1;
    }
    while (lo < batch - 1 && pre[lo + 1] <= i) ++lo;
    it.b = lo;
    it.cu_b = p.cu_seqlens[lo];
    it.len_b = p.cu_seqlens[lo + 1] - it.cu_b;
    it.K = p.topk[lo];
    it.nA1 = (int)(it.len_b < p.n_sink ? it.len_b : p.n_sink);
    long long ts = it.len_b - tail_of(p, lo);
    if (ts < p.n_sink) ts = p.n_sink;
    if (ts > it.len_b) ts = it.len_b;
    it.tail_start = (int)ts;
    it.nE = it.nA1 + it.K + (int)(it.len_b - ts);
    it.n_slices = it.nE > 0 ? (it.nE + kSlice - 1) / kSlice : 1;
    it.n_ctas = (it.n_slices + kExGroups - 1) / kExGroups;
    const int rem = i - pre[lo];
    it.hq = rem / it.n_ctas;
    it.slice0 = (rem % it.n_ctas) * kExGroups;
    it.row = lo * Hq + it.hq;
    it.kvh = it.hq / p.group;
    return it;
  };
  auto slice_has_ret = [&](const ExItem& it, int sl) {
    return do_phi && sl < it.n_slices && sl * kSlice < it.nA1 + it.K && (sl + 1) * kSlice > it.nA1;
  };
  // token list, queries and query-side feature terms of an item: loaded into registers first
  // (stage_load) and written to buffer `buf` later (stage_store), so that the loads of the next
  // item are in flight while the current one is computed.  D, R <= kExThreads: one value each.
  struct Staged { int t, ret; float qv, cv, zc; };
  auto stage_load = [&](const ExItem& it) {
    Staged sg;
    const int sl = it.slice0 + grp;
    const int pi = sl * kSlice + gt;
    sg.t = -1; sg.ret = 0; sg.zc = 0.f;
    if (sl < it.n_slices && pi < it.nE) {
      if (pi < it.nA1) sg.t = pi;
      else if (pi < it.nA1 + it.K) {
        sg.t = __ldcg(p.idx + (size_t)it.row * p.topk_max + (pi - it.nA1));
        sg.ret = 1;
        if (p.zbuf) sg.zc = __ldcg(p.zbuf + (size_t)it.row * p.topk_max + (pi - it.nA1));
      }
      else sg.t = it.tail_start + (pi - it.nA1 - it.K);
    }
    sg.qv = tid < D ? __bfloat162float(p.q[(size_t)it.row * D + tid]) : 0.f;
    sg.cv = (do_phi && tid < R) ? __ldcg(p.aq + (size_t)it.row * aq_stride(R, D) + R + 4 + D + tid) +
                                      p.b_k[(size_t)it.kvh * R + tid] * kLog2e
                                : 0.f;
    return sg;
  };
  auto stage_store = [&](const Staged& sg, int buf) {
    tok_all[buf * kExThreads + tid] = sg.t;
    isret_all[buf * kExThreads + tid] = sg.ret;
    zc_all[buf * kExThreads + tid] = sg.zc;
    if (tid < D) qf_all[buf * D + tid] = sg.qv;
    if (tid < R) cj_all[buf * R + tid] = sg.cv;
  };
  constexpr int CPR = D / 8;                   // 16-byte chunks per row
  const uint64_t pol = l2_policy_evict_first();
  // Row gathers of one tile kind (k or v) for both groups of an item, by the 32 lanes of the
  // calling warp: a lane issues rows 4l .. 4l+3 of each group, one instruction per 64-dim
  // column block; rows without a source get an out-of-range index and arrive as zeros.
  auto issue_rows = [&](const ExItem& it, int buf, bool keys) {
    uint64_t* bar = &bars[keys ? 3 : 4];
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)(kExGroups * LB::kv_tile));
    __syncwarp();
#pragma unroll
    for (int g = 0; g < kExGroups; ++g) {
      const int* tk = tok_all + buf * kExThreads + g * kSlice;
      const int* ir = isret_all + buf * kExThreads + g * kSlice;
      int r[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int t = 4 * lane + j;
        const int ti = tk[t];
        const bool want = ti >= 0 && (!keys || !ir[t] || do_phi);
        const long long cache_row = it.cu_b + ti;
        const long long gr = p.gather_mode == 0 ? (long long)it.kvh * p.gather_ratio + cache_row
                                                : cache_row * p.gather_ratio + it.kvh;
        r[j] = want ? (int)gr : (int)p.gather_rows;
      }
      unsigned char* tile = smem + (keys ? L::kt : L::vt) + g * LB::kv_tile + 4 * lane * 128;
#pragma unroll
      for (int x = 0; x < LB::BOXES; ++x)
        tma_gather4_2d(tile + x * LB::KV_BOX, keys ? &gmap_k : &gmap_v, bar, x * 64, r[0], r[1], r[2], r[3], pol);
    }
  };

  pdl_wait();                                  // the index lists, features and score rows of the predecessors
  if (i0 >= i1) return;                        // (more CTAs than items: nothing allocated yet)
  if (do_phi && warp == 0) tmem_alloc(s_tmem, kExGroups * 2 * R);
  ExItem cur = item_of(i0, nullptr);
  if (!producer) stage_store(stage_load(cur), 0);
  if (tid == 0) {                              // the first item's tiles: announced here, issued by all compute warps below
    mbar_expect_tx(&bars[3], (uint32_t)(kExGroups * LB::kv_tile));
    mbar_expect_tx(&bars[4], (uint32_t)(kExGroups * LB::kv_tile));
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  // The gathers of the first item are on every CTA's critical path, and one warp needs about
  // 4.5 us to issue the 128 gathers of a tile pair: here each of the eight compute warps
  // issues one (k or v, group, column block) combination, one gather per lane.
  if (!producer) {
    static_assert(kExGroups * LB::BOXES * 2 == kExThreads / 32, "one (kind, group, column block) per compute warp");
    const bool keys = warp < kExThreads / 64;
    const int g = (warp / LB::BOXES) % kExGroups, x = warp % LB::BOXES;
    const int* tk = tok_all + g * kSlice;
    const int* ir = isret_all + g * kSlice;
    int r[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int t = 4 * lane + j;
      const int ti = tk[t];
      const bool want = ti >= 0 && (!keys || !ir[t] || do_phi);
      const long long cache_row = cur.cu_b + ti;
      const long long gr = p.gather_mode == 0 ? (long long)cur.kvh * p.gather_ratio + cache_row
                                              : cache_row * p.gather_ratio + cur.kvh;
      r[j] = want ? (int)gr : (int)p.gather_rows;
    }
    tma_gather4_2d(smem + (keys ? L::kt : L::vt) + g * LB::kv_tile + x * LB::KV_BOX + 4 * lane * 128,
                   keys ? &gmap_k : &gmap_v, &bars[keys ? 3 : 4], x * 64, r[0], r[1], r[2], r[3], pol);
  }

  if (producer) {
    // ================================================================ row-gather producers
    const bool keys = warp == kExThreads / 32;
    uint64_t* free_bar = &bars[keys ? 5 : 6];
    int issued = 1;                            // (the first item's gathers were issued by the compute warps)
    for (int i = i0; i + 1 < i1; ++i) {
      const ExItem nx = item_of(i + 1, &cur);
      // the compute warps are done with the tiles of item i (and have staged item i+1's token list)
      if (!mbar_wait(free_bar, (uint32_t)(i - i0) & 1u, s_abort)) break;
      issue_rows(nx, (i + 1 - i0) & 1, keys);
      ++issued;
      cur = nx;
    }
    // after a wait gave up somewhere, the last gather may still be in flight
    if (*s_abort && lane == 0)
      for (uint32_t w = 0; w < kWaitPolls; ++w) {
        if (mbar_try_wait(&bars[keys ? 3 : 4], (uint32_t)(issued - 1) & 1u)) break;
        __nanosleep(64);
      }
  } else {
  // ================================================================ compute warps

  int w_kvh = -1;                              // KV head whose W_k tiles are in shared memory
  uint32_t w_phase = 0, mma_phase = 0;         // mbarrier parities (mma_phase: this thread's group)
  uint32_t kv_phase = 0;                       // parity of the k and v tile barriers (one completion per item each)
  bool ok = true;
  for (int i = i0; i < i1; ++i) {
    const int buf = (i - i0) & 1;
    const int slice = cur.slice0 + grp;
    const bool live = slice < cur.n_slices;
    const bool has_ret = slice_has_ret(cur, slice);
    bool any_ret = false;
#pragma unroll
    for (int g = 0; g < kExGroups; ++g) any_ret = any_ret || slice_has_ret(cur, cur.slice0 + g);
    const int* tok = tok_all + buf * kExThreads + grp * kSlice;
    const int* isret = isret_all + buf * kExThreads + grp * kSlice;
    const float* qf = qf_all + buf * D;
    const float* cj = cj_all + buf * R;
    const float* srow = p.scores + score_row_base(p, cur.b, cur.hq, cur.cu_b, cur.len_b);

    // ---- W_k tiles of this KV head (every MMA that read the previous ones has completed)
    bool w_new = false;
    if (any_ret && (cur.kvh != w_kvh)) {
      w_new = true;
      w_kvh = cur.kvh;
      if (tid == 0) {
        const unsigned char* img = reinterpret_cast<const unsigned char*>(p.wk_img + (size_t)cur.kvh * 2 * R * D);
        mbar_expect_tx(&bars[0], 2u * R * D * 2u);
        bulk_load(wt, img, 2 * R * D * 2, &bars[0]);
      }
    }
    // ---- next item: token list and query terms into the other buffer
    ExItem nxt = cur;
    const bool has_next = i + 1 < i1;
    Staged sg_next{-1, 0, 0.f, 0.f, 0.f};
    if (has_next) { nxt = item_of(i + 1, &cur); sg_next = stage_load(nxt); }

    // ---- k tiles of this item have landed (the v tiles may still be in flight)
    ok = mbar_wait(&bars[3], kv_phase, s_abort);
    ok = ex_sync_and<1>(ok);
    if (!ok) break;

    // ---- feature recompute on the tensor core
    if (any_ret && tid == 0) {
      if (w_new) ok = mbar_wait(&bars[0], w_phase, s_abort);
      if (ok) {
        tc_fence_after_sync();
        constexpr uint32_t idesc = umma_idesc_bf16(128, 2 * R, 0, 0);
        const uint64_t bdesc0 = umma_smem_desc(smem_u32(wt), 16, 1024);
#pragma unroll
        for (int g = 0; g < kExGroups; ++g) {
          if (!slice_has_ret(cur, cur.slice0 + g)) continue;
          const uint32_t tmem_d = *s_tmem + g * 2 * R;
          const uint64_t adesc0 = umma_smem_desc(smem_u32(smem + L::kt + g * LB::kv_tile), 16, 1024);
#pragma unroll
          for (int k = 0; k < D / 16; ++k)
            umma_ss(tmem_d, adesc0 + (uint64_t)(((k >> 2) * LB::KV_BOX + (k & 3) * 32) >> 4),
                    bdesc0 + (uint64_t)(((k >> 2) * LB::W_BOX + (k & 3) * 32) >> 4), idesc, k ? 1u : 0u);
          tc_commit(&bars[1 + g]);
        }
      }
    }
    if (w_new) w_phase ^= 1u;

    // ---- per token: |k|^2, anchor score, softmax weight
    const int ti = tok[gt];
    float s_val = -INFINITY, kn = 0.f;
    if (ti >= 0) {
      float dot;
      token_dot_and_norm<D>(kt, gt, qf, p.scale, &dot, &kn);
      s_val = isret[gt] ? srow[ti - p.n_sink] : dot;
    }
    {
      const float m = warp_max(s_val);
      if (lane == 0) misc[warp] = m;
    }
    ex_sync<1>();
    const float m_slice = fmaxf(fmaxf(misc[4 * grp], misc[4 * grp + 1]), fmaxf(misc[4 * grp + 2], misc[4 * grp + 3]));
    const float w_t = ti >= 0 ? expf(s_val - m_slice) : 0.f;
    wgt[gt] = w_t;
    if (has_next) stage_store(sg_next, buf ^ 1);   // (the loads were issued at the top of the iteration)

    // ---- the MMAs are done: the k tiles are free for the next item
    if (has_ret) { ok = mbar_wait(&bars[1 + grp], mma_phase, s_abort); mma_phase ^= 1u; }
    ok = ex_sync_and<1>(ok);
    if (tid == 0) mbar_arrive(&bars[5]);       // the k producer may refill the k tiles

    // ---- v tiles of this item have landed
    if (ok) ok = mbar_wait(&bars[4], kv_phase, s_abort);
    kv_phase ^= 1u;
    float z_t = 0.f;
    if (has_ret && ok) {
      tc_fence_after_sync();
      z_t = z_from_accumulator<R>(*s_tmem + grp * 2 * R, gwarp, cj, p.gamma_k, kn);
      if (!isret[gt]) z_t = 0.f;
    }
    if (p.zbuf) z_t = zc_all[buf * kExThreads + tid];
    zt[gt] = z_t;
    tc_fence_before_sync();                    // the accumulator reads precede the next item's MMAs
    ex_sync<1>();

    // ---- slice partials
    slice_value_pass<D>(vt, wgt, zt, gt, red);
    ok = ex_sync_and<1>(ok);                   // the v tiles are free for the next item
    if (tid == 0) mbar_arrive(&bars[6]);
    if (live)
      slice_write_partials<D>(p.partials + ((size_t)cur.row * p.max_slices + slice) * p.partial_stride, red, wgt, zt, gt,
                              gwarp, lane, m_slice);
    if (!ok) break;                            // a wait gave up (the same for every thread)

    // ---- ticket: the last CTA of this head merges
    __threadfence();
    ex_sync<1>();
    if (tid == 0) {
      const unsigned prev = atomicAdd(&p.row_counter[cur.row], 1u);
      misc[8] = (prev == (unsigned)(cur.n_ctas - 1)) ? 1.f : 0.f;
    }
    ex_sync<1>();
    if (misc[8] != 0.f) {
      __threadfence();
      merge_head<D, R, 1>(p, cur.row, cur.n_slices, cur.nE, misc);
      ex_sync<1>();                            // misc is reused by the next item
    }
    cur = nxt;
  }
  }  // compute warps

  // ---- teardown: nothing may be in flight when the shared memory is released
  tc_fence_before_sync();
  __syncthreads();
  if (do_phi && warp == 0) {
    tc_fence_after_sync();
    tmem_dealloc(*s_tmem, kExGroups * 2 * R);
  }
  if (*s_abort && tid == 0) atomicExch(p.status, kStatusTimeout);
}

template <int D, int R>
static cudaError_t launch_ex_t(const Problem& p, const CUtensorMap& gk, const CUtensorMap& gv, cudaStream_t st) {
  static PerDeviceFlag configured;
  const size_t smem = ExSmem<D, R>::total;
  cudaError_t e = set_max_dynamic_smem(configured, reinterpret_cast<const void*>(exact_residual_kernel<D, R>), smem);
  if (e != cudaSuccess) return e;
  dim3 grid((p.max_slices + kExGroups - 1) / kExGroups, p.n_q_heads, p.batch);
  return launch_pdl(exact_residual_kernel<D, R>, grid, dim3(kExThreads), smem, st, p);
}

template <int D, int R>
static cudaError_t launch_ex_stream_t(const Problem& p, const CUtensorMap& gk, const CUtensorMap& gv, int n_ctas,
                                      cudaStream_t st) {
  static PerDeviceFlag configured;
  const size_t smem = ExStreamSmem<D, R>::total;
  cudaError_t e =
      set_max_dynamic_smem(configured, reinterpret_cast<const void*>(exact_residual_stream_kernel<D, R>), smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(exact_residual_stream_kernel<D, R>, dim3(n_ctas), dim3(kExStreamThreads), smem, st, gk, gv, p);
}

cudaError_t launch_exact_residual(const Problem& p, const CUtensorMap& gk, const CUtensorMap& gv, long long n_pairs,
                                  int n_sm, cudaStream_t st) {
  // n_pairs: slice pairs of the whole call.  More than one wave of CTAs: persistent streaming kernel.
  // (with head_dim 64 several one-shot CTAs fit an SM and overlap by themselves)
  if (n_pairs > n_sm && p.head_dim == 128 && p.gather_mode >= 0) {
    if (p.n_feat == 64) return launch_ex_stream_t<128, 64>(p, gk, gv, n_sm, st);
    if (p.n_feat == 128) return launch_ex_stream_t<128, 128>(p, gk, gv, n_sm, st);
    return cudaErrorInvalidValue;
  }
  if (p.head_dim == 64 && p.n_feat == 64) return launch_ex_t<64, 64>(p, gk, gv, st);
  if (p.head_dim == 64 && p.n_feat == 128) return launch_ex_t<64, 128>(p, gk, gv, st);
  if (p.head_dim == 128 && p.n_feat == 64) return launch_ex_t<128, 64>(p, gk, gv, st);
  if (p.head_dim == 128 && p.n_feat == 128) return launch_ex_t<128, 128>(p, gk, gv, st);
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
