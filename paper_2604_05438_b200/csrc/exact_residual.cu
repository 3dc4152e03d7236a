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
// The support list of a query head is cut into slices of kSlice tokens; one CTA
// per slice writes partial sums, and the last CTA of a head (one atomic ticket, no
// spinning) combines them in slice order, so results are run-to-run identical.
#include "common.cuh"

namespace tkphi {

constexpr int kExThreads = 256;

template <int D, int R>
struct ExSmem {
  static constexpr int WT_LD = R + 1;                       // padded leading dim of W^T
  static constexpr size_t wt = 0;                           // float [D][R+1]   (phi only)
  static constexpr size_t kf = wt + sizeof(float) * D * WT_LD;     // float [D][kSlice]
  static constexpr size_t vs = kf + sizeof(float) * D * kSlice;    // bf16  [kSlice][D]
  static constexpr size_t red = vs + 2 * kSlice * D;               // float [4][2*D]
  static constexpr size_t zpart = red + sizeof(float) * 4 * 2 * D; // float [8][kSlice]
  static constexpr size_t small = zpart + sizeof(float) * 8 * kSlice;
  // small: tok[kSlice] int, isret[kSlice] int, sc[kSlice], wgt[kSlice], zt[kSlice], knorm[kSlice], qf[D], phiq[R], misc[16]
  static constexpr size_t total = small + 4 * (6 * kSlice + D + R + 16);
};

template <int D, int R>
__global__ void __launch_bounds__(kExThreads) exact_residual_kernel(const Problem p) {
  using L = ExSmem<D, R>;
  extern __shared__ __align__(16) unsigned char smem[];
  float* Wt = reinterpret_cast<float*>(smem + L::wt);
  float* kf = reinterpret_cast<float*>(smem + L::kf);
  __nv_bfloat16* vs = reinterpret_cast<__nv_bfloat16*>(smem + L::vs);
  float* red = reinterpret_cast<float*>(smem + L::red);
  float* zpart = reinterpret_cast<float*>(smem + L::zpart);
  int* tok = reinterpret_cast<int*>(smem + L::small);
  int* isret = tok + kSlice;
  float* sc = reinterpret_cast<float*>(isret + kSlice);
  float* wgt = sc + kSlice;
  float* zt = wgt + kSlice;
  float* knorm = zt + kSlice;
  float* qf = knorm + kSlice;
  float* phiq = qf + D;
  float* misc = phiq + R;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.z, hq = blockIdx.y, slice = blockIdx.x;
  const int row = b * p.n_q_heads + hq, kvh = hq / p.group;
  const int K = p.topk[b];
  const long long cu_b = p.cu_seqlens[b], len_b = p.cu_seqlens[b + 1] - cu_b;
  const int nA1 = (int)(len_b < p.n_sink ? len_b : p.n_sink);
  long long ts = len_b - p.n_tail;
  if (ts < p.n_sink) ts = p.n_sink;
  if (ts > len_b) ts = len_b;
  const int tail_start = (int)ts, n_tail_eff = (int)(len_b - ts);
  const int nE = nA1 + K + n_tail_eff;
  const int n_slices = nE > 0 ? (nE + kSlice - 1) / kSlice : 1;
  if (slice >= n_slices) return;
  const bool do_phi = p.with_phi && !(p.flags & 1u);

  const __nv_bfloat16* kbase = p.k + (long long)kvh * p.stride_head + cu_b * p.stride_token;
  const __nv_bfloat16* vbase = p.v + (long long)kvh * p.stride_head + cu_b * p.stride_token;
  const float* srow = p.scores + score_row_base(p, b, hq, cu_b, len_b);

  // ---- 1. token list of this slice
  if (tid < kSlice) {
    const int pi = slice * kSlice + tid;
    int t = -1, ret = 0;
    if (pi < nE) {
      if (pi < nA1) t = pi;
      else if (pi < nA1 + K) { t = p.idx[(size_t)row * p.topk_max + (pi - nA1)]; ret = 1; }
      else t = tail_start + (pi - nA1 - K);
    }
    tok[tid] = t;
    isret[tid] = ret;
  }
  for (int c = tid; c < D; c += kExThreads) qf[c] = __bfloat162float(p.q[(size_t)row * D + c]);
  if (do_phi) {
    for (int j = tid; j < R; j += kExThreads) phiq[j] = p.aq[(size_t)row * (R + 4) + j];
    // W_k^T into shared memory: global reads run along a row of W_k, the padded
    // leading dimension keeps the transposed stores conflict-free
    const float* W = p.w_k + (size_t)kvh * R * D;
    for (int i = tid; i < R * D; i += kExThreads) {
      const int j = i / D, c = i % D;
      Wt[c * L::WT_LD + j] = W[i];
    }
  }
  __syncthreads();

  // ---- 2. gather rows: v always; k for anchors (scores) and, with phi, retrieved rows
  constexpr int CPR = D / 8;                 // 16-byte chunks per row
  for (int i = tid; i < kSlice * CPR; i += kExThreads) {
    const int t = i / CPR, c = i % CPR;
    const int ti = tok[t];
    uint4 vraw = make_uint4(0, 0, 0, 0), kraw = make_uint4(0, 0, 0, 0);
    if (ti >= 0) {
      vraw = *reinterpret_cast<const uint4*>(vbase + (long long)ti * p.stride_token + c * 8);
      if (!isret[t] || do_phi)
        kraw = *reinterpret_cast<const uint4*>(kbase + (long long)ti * p.stride_token + c * 8);
    }
    *reinterpret_cast<uint4*>(vs + t * D + c * 8) = vraw;
    const unsigned w[4] = {kraw.x, kraw.y, kraw.z, kraw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      kf[(c * 8 + 2 * e) * kSlice + t] = bf16_lo(w[e]);
      kf[(c * 8 + 2 * e + 1) * kSlice + t] = bf16_hi(w[e]);
    }
  }
  __syncthreads();

  // ---- 3. scores, slice max, softmax weights
  if (tid < kSlice) {
    const int ti = tok[tid];
    float s_val = -INFINITY, kn = 0.f;
    if (ti >= 0) {
      float dot = 0.f;
      for (int c = 0; c < D; ++c) {
        const float x = kf[c * kSlice + tid];
        dot = fmaf(x, qf[c], dot);
        kn = fmaf(x, x, kn);
      }
      s_val = isret[tid] ? srow[ti - p.n_sink] : dot * p.scale;
    }
    sc[tid] = s_val;
    knorm[tid] = kn;
    float m = warp_max(s_val);
    if (lane == 0) misc[warp] = m;
  }
  __syncthreads();
  const float m_slice = fmaxf(misc[0], misc[1]);
  if (tid < kSlice) {
    const float w = tok[tid] >= 0 ? expf(sc[tid] - m_slice) : 0.f;
    wgt[tid] = w;
    zt[tid] = 0.f;
  }

  // ---- 4. z_i = <phi_q, phi_k(k_i)> for the retrieved rows of the slice
  if (do_phi) {
    constexpr int NG = kExThreads / R;       // token groups
    constexpr int TPG = kSlice / NG;         // tokens per group
    const int j = tid % R, tg = tid / R, t0 = tg * TPG;
    float acc[TPG];
#pragma unroll
    for (int t = 0; t < TPG; ++t) acc[t] = 0.f;
    for (int c = 0; c < D; ++c) {
      const float w = Wt[c * L::WT_LD + j];
      const float4* kp = reinterpret_cast<const float4*>(kf + c * kSlice + t0);
#pragma unroll
      for (int t4 = 0; t4 < TPG / 4; ++t4) {
        const float4 kv = kp[t4];
        acc[4 * t4 + 0] = fmaf(w, kv.x, acc[4 * t4 + 0]);
        acc[4 * t4 + 1] = fmaf(w, kv.y, acc[4 * t4 + 1]);
        acc[4 * t4 + 2] = fmaf(w, kv.z, acc[4 * t4 + 2]);
        acc[4 * t4 + 3] = fmaf(w, kv.w, acc[4 * t4 + 3]);
      }
    }
    const float bj = p.b_k[(size_t)kvh * R + j], pq = phiq[j];
    // warp w of the group covers features 32*(w in group)..; sum over the warp,
    // then over the group's warps in fixed order
    const int wg = (tid % R) >> 5;           // warp within the group
#pragma unroll
    for (int t = 0; t < TPG; ++t) {
      float z = 0.f;
      if (isret[t0 + t]) z = pq * expf(acc[t] + bj - p.gamma_k * knorm[t0 + t]);
      z = warp_sum(z);
      if (lane == 0) zpart[wg * kSlice + t0 + t] = z;
    }
    __syncthreads();
    if (tid < kSlice) {
      float z = 0.f;
#pragma unroll
      for (int w = 0; w < R / 32; ++w) z += zpart[w * kSlice + tid];
      zt[tid] = z;
    }
  }
  __syncthreads();

  // ---- 5. slice partials: nu = sum w_t v_t, zv = sum z_t v_t, Z = sum w_t, zs = sum z_t
  {
    constexpr int NGV = kExThreads / D;      // token groups for the value pass (2 or 4)
    constexpr int TPV = kSlice / NGV;
    const int dv = tid % D, tg = tid / D;
    float nu = 0.f, zv = 0.f;
    for (int t = tg * TPV; t < (tg + 1) * TPV; ++t) {
      const float x = __bfloat162float(vs[t * D + dv]);
      nu = fmaf(wgt[t], x, nu);
      zv = fmaf(zt[t], x, zv);
    }
    red[tg * 2 * D + dv] = nu;
    red[tg * 2 * D + D + dv] = zv;
  }
  __syncthreads();
  float* part = p.partials + ((size_t)row * p.max_slices + slice) * p.partial_stride;
  if (tid < 2 * D) {
    constexpr int NGV = kExThreads / D;
    float x = 0.f;
#pragma unroll
    for (int g = 0; g < NGV; ++g) x += red[g * 2 * D + tid];
    part[4 + tid] = x;
  }
  if (tid < 32) {
    float Z = wgt[tid] + wgt[tid + 32], zs = zt[tid] + zt[tid + 32];
    Z = warp_sum(Z);
    zs = warp_sum(zs);
    if (tid == 0) { part[0] = m_slice; part[1] = Z; part[2] = zs; part[3] = 0.f; }
  }

  // ---- ticket: the last slice CTA of this head merges
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned prev = atomicAdd(&p.row_counter[row], 1u);
    misc[8] = (prev == (unsigned)(n_slices - 1)) ? 1.f : 0.f;
  }
  __syncthreads();
  if (misc[8] == 0.f) return;
  __threadfence();

  const float* parts = p.partials + (size_t)row * p.max_slices * p.partial_stride;
  float m_E = -INFINITY;
  if (nE > 0)
    for (int s = 0; s < n_slices; ++s) m_E = fmaxf(m_E, __ldcg(parts + (size_t)s * p.partial_stride));
  float Z_E = 0.f, zs = 0.f;
  for (int s = 0; s < n_slices; ++s) {
    const float* ps = parts + (size_t)s * p.partial_stride;
    const float f = nE > 0 ? expf(__ldcg(ps) - m_E) : 0.f;
    Z_E = fmaf(f, __ldcg(ps + 1), Z_E);
    zs += __ldcg(ps + 2);
  }
  float nu_E = 0.f, zv = 0.f;
  if (tid < D) {
    for (int s = 0; s < n_slices; ++s) {
      const float* ps = parts + (size_t)s * p.partial_stride;
      const float f = nE > 0 ? expf(__ldcg(ps) - m_E) : 0.f;
      nu_E = fmaf(f, __ldcg(ps + 4 + tid), nu_E);
      zv += __ldcg(ps + 4 + D + tid);
    }
  }
  float y = 0.f, yR = 0.f, logZR = -INFINITY, Mx = m_E;
  if (p.with_phi) {
    // S_M phi_q and phi_q . u_M, both in units of exp(m_q)
    for (int j = tid; j < R; j += kExThreads) phiq[j] = p.aq[(size_t)row * (R + 4) + j];
    __syncthreads();
    const float m_q = p.aq[(size_t)row * (R + 4) + R];
    const float* Sg = p.S + ((size_t)b * p.n_kv_heads + kvh) * D * R;
    const float* ug = p.u + ((size_t)b * p.n_kv_heads + kvh) * R;
    // one warp per row of S: lanes run along the features
    for (int dv = warp; dv < D; dv += kExThreads / 32) {
      float a = 0.f;
      for (int j = lane; j < R; j += 32) a = fmaf(Sg[(size_t)dv * R + j], phiq[j], a);
      a = warp_sum(a);
      if (lane == 0) red[dv] = a;
    }
    if (warp == 0) {
      float a = 0.f;
      for (int j = lane; j < R; j += 32) a = fmaf(ug[j], phiq[j], a);
      a = warp_sum(a);
      if (lane == 0) misc[9] = a;
    }
    __syncthreads();
    const float Zt = misc[9] - zs;                         // Z_hat_R / exp(m_q)
    if (Zt > 0.f) {
      logZR = m_q + logf(Zt);
      Mx = fmaxf(m_E, logZR);
      const float cE = nE > 0 ? expf(m_E - Mx) : 0.f, cR = expf(logZR - Mx);
      if (tid < D) {
        yR = (red[tid] - zv) / Zt;
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
static cudaError_t launch_ex_t(const Problem& p, cudaStream_t st) {
  static bool configured = false;
  const size_t smem = ExSmem<D, R>::total;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(exact_residual_kernel<D, R>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(p.max_slices, p.n_q_heads, p.batch);
  exact_residual_kernel<D, R><<<grid, kExThreads, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_exact_residual(const Problem& p, cudaStream_t st) {
  if (p.head_dim == 64 && p.n_feat == 64) return launch_ex_t<64, 64>(p, st);
  if (p.head_dim == 64 && p.n_feat == 128) return launch_ex_t<64, 128>(p, st);
  if (p.head_dim == 128 && p.n_feat == 64) return launch_ex_t<128, 64>(p, st);
  if (p.head_dim == 128 && p.n_feat == 128) return launch_ex_t<128, 128>(p, st);
  return cudaErrorInvalidValue;
}

}  // namespace tkphi
