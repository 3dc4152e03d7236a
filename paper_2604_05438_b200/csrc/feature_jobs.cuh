// Query-side feature work and the W_k operand split, shared by the selection kernels.
#pragma once
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

// ------------------------------------------------------------------ query-side feature work
// Work that depends only on the call's inputs is done by spare CTAs of the selection
// kernel, where it is off the critical path and the memory system is not saturated.
//
// Query-side quantities (Sec. 4.1, Sec. 4.3): a_q = W_q q + b_q - gamma_q |q|^2, kept as
// w = exp(a_q - m_q) and m_q so that tiny features cannot underflow the merge, and the
// unsubtracted residual terms S_M w (d values) and w . u_M.  Row layout of p.aq:
// [0, r) w, [r] m_q, [r+1] w . u_M, [r+4, r+4+d) S_M w, [r+4+d, 2r+4+d) log2 w.

// Stage 1, by all NT threads of a CTA: w and m_q of query row `row`.  With the MLP feature map on the
// query side the exponents log phi_q(q) come from the layer kernels that ran before (mlp_query.cu).
template <int NT>
__device__ void phi_q_stage1(const Problem& p, int row) {
  __shared__ float s_q[128];
  __shared__ float s_a[128];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = p.head_dim, r = p.n_feat;
  const int hq = row % p.n_q_heads;
  float* aq = p.aq + (size_t)row * aq_stride(r, D);
  const __nv_bfloat16* qp = p.q + (size_t)row * D;
  const float* W = p.w_q + (size_t)hq * r * D;
  for (int c = tid; c < D; c += NT) s_q[c] = __bfloat162float(qp[c]);
  if (p.mlp_q.w_s != nullptr) {
    const float* a = p.mlp_vec + (size_t)row * (3 * p.mlp_q.d_emb + r) + 3 * p.mlp_q.d_emb;
    if (tid < r) s_a[tid] = __ldcg(a + tid);
    __syncthreads();
    float m = -INFINITY;
    for (int j = lane; j < r; j += 32) m = fmaxf(m, s_a[j]);
    m = warp_max(m);
    if (tid < r) {
      aq[tid] = expf(s_a[tid] - m);
      aq[r + 4 + D + tid] = (s_a[tid] - m) * kLog2e;
    }
    if (tid == 0) aq[r] = m;
    return;
  }
  // each warp owns r/NW feature rows: every lane loads its float4 of every row first (all
  // loads in flight), then the dot products are reduced across the warp
  constexpr int NW = NT / 32;
  constexpr int MAXR = 128 / NW;                      // rows per warp at r = 128
  const int rows_w = r / NW;
  float4 w4[MAXR];
  float bq[MAXR];
  const bool active = lane * 4 < D;
#pragma unroll
  for (int i = 0; i < MAXR; ++i) {
    w4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    bq[i] = 0.f;
    if (i < rows_w) {
      if (active) w4[i] = __ldg(reinterpret_cast<const float4*>(W + (size_t)(warp * rows_w + i) * D + lane * 4));
      bq[i] = __ldg(p.b_q + (size_t)hq * r + warp * rows_w + i);
    }
  }
  __syncthreads();
  float qn = 0.f;
  for (int c = lane; c < D; c += 32) qn = fmaf(s_q[c], s_q[c], qn);
  qn = warp_sum(qn);
  const float q0 = active ? s_q[lane * 4] : 0.f, q1 = active ? s_q[lane * 4 + 1] : 0.f;
  const float q2 = active ? s_q[lane * 4 + 2] : 0.f, q3 = active ? s_q[lane * 4 + 3] : 0.f;
#pragma unroll
  for (int i = 0; i < MAXR; ++i) {
    const float a = warp_sum(w4[i].x * q0 + w4[i].y * q1 + w4[i].z * q2 + w4[i].w * q3);
    if (i < rows_w && lane == 0) s_a[warp * rows_w + i] = a + bq[i] - p.gamma_q * qn;
  }
  __syncthreads();
  float m = -INFINITY;
  for (int j = lane; j < r; j += 32) m = fmaxf(m, s_a[j]);
  m = warp_max(m);                                    // every warp computes the same maximum
  if (tid < r) {
    aq[tid] = expf(s_a[tid] - m);
    aq[r + 4 + D + tid] = (s_a[tid] - m) * kLog2e;     // the same weight in the log2 domain
  }
  if (tid == 0) aq[r] = m;
}

// Stage 2, by all NT threads of a CTA of a later kernel: S_M w and w . u_M of query row `row`.
template <int NT>
__device__ void phi_q_stage2(const Problem& p, int row) {
  __shared__ float s_w[128];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = p.head_dim, r = p.n_feat;
  const int b = row / p.n_q_heads, hq = row % p.n_q_heads, kvh = hq / p.group;
  float* aq = p.aq + (size_t)row * aq_stride(r, D);
  const float* Sg = p.S + ((size_t)b * p.n_kv_heads + kvh) * D * r;
  const float* ug = p.u + ((size_t)b * p.n_kv_heads + kvh) * r;
  constexpr int NW = NT / 32;
  constexpr int MAXR = 128 / NW;
  const int rows_d = D / NW;
  const bool act_r = lane * 4 < r;
  float4 s4[MAXR];
#pragma unroll
  for (int i = 0; i < MAXR; ++i) {
    s4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < rows_d && act_r)
      s4[i] = __ldg(reinterpret_cast<const float4*>(Sg + (size_t)(warp * rows_d + i) * r + lane * 4));
  }
  if (tid < r) s_w[tid] = __ldcg(aq + tid);            // written by stage 1 in an earlier kernel
  __syncthreads();
  const float w0 = act_r ? s_w[lane * 4] : 0.f, w1 = act_r ? s_w[lane * 4 + 1] : 0.f;
  const float w2 = act_r ? s_w[lane * 4 + 2] : 0.f, w3 = act_r ? s_w[lane * 4 + 3] : 0.f;
#pragma unroll
  for (int i = 0; i < MAXR; ++i) {
    const float a = warp_sum(s4[i].x * w0 + s4[i].y * w1 + s4[i].z * w2 + s4[i].w * w3);
    if (i < rows_d && lane == 0) aq[r + 4 + warp * rows_d + i] = a;
  }
  if (warp == 0) {
    float a = 0.f;
    for (int j = lane; j < r; j += 32) a = fmaf(__ldg(ug + j), s_w[j], a);
    a = warp_sum(a);
    if (lane == 0) aq[r + 1] = a;
  }
}

// W_k of one KV head (fp32 [r][d]), scaled by log2 e so that the recomputed exponents feed
// exp2 directly -> hi = bf16(W) and lo = bf16(W - hi), stacked into ONE K-major,
// 128B-swizzled B operand of 2r rows for the feature recompute MMA (rows 0..r-1 hi,
// rows r..2r-1 lo): [d/64 column blocks][2r rows][128 bytes].  By all NT threads of a CTA.
template <int NT>
__device__ void wk_split_job(const Problem& p, int kvh) {
  const int D = p.head_dim, r = p.n_feat;
  const float* W = p.w_k + (size_t)kvh * r * D;
  unsigned char* hi = reinterpret_cast<unsigned char*>(p.wk_img + (size_t)kvh * 2 * r * D);
  unsigned char* lo = hi + (size_t)r * 128;          // r is a multiple of 8: the swizzle phase of a row is kept
  const int cpr = D / 8;
#pragma unroll 4
  for (int i = threadIdx.x; i < r * cpr; i += NT) {
    const int row = i / cpr, c = i % cpr;
    const float4 w0 = __ldg(reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8));
    const float4 w1 = __ldg(reinterpret_cast<const float4*>(W + (size_t)row * D + c * 8 + 4));
    const float w[8] = {w0.x * kLog2e, w0.y * kLog2e, w0.z * kLog2e, w0.w * kLog2e,
                        w1.x * kLog2e, w1.y * kLog2e, w1.z * kLog2e, w1.w * kLog2e};
    unsigned hw[4], lw[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const __nv_bfloat16 h0 = __float2bfloat16_rn(w[2 * e]), h1 = __float2bfloat16_rn(w[2 * e + 1]);
      const __nv_bfloat16 l0 = __float2bfloat16_rn(w[2 * e] - __bfloat162float(h0));
      const __nv_bfloat16 l1 = __float2bfloat16_rn(w[2 * e + 1] - __bfloat162float(h1));
      hw[e] = (unsigned)__bfloat16_as_ushort(h0) | ((unsigned)__bfloat16_as_ushort(h1) << 16);
      lw[e] = (unsigned)__bfloat16_as_ushort(l0) | ((unsigned)__bfloat16_as_ushort(l1) << 16);
    }
    const size_t off = (size_t)(c >> 3) * (2 * r) * 128 + swz128(row, c & 7);
    *reinterpret_cast<uint4*>(hi + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
    *reinterpret_cast<uint4*>(lo + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
  }
}

}  // namespace tkphi
