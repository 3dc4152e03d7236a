// Query side of the one-block ReZero-MLP feature map (App. C.2), log phi_q(q) for every query head of a
// decode call:  g0 = W_s q + b_s;  h = GeLU(W_1 g0 + b_1);  g1 = g0 + alpha (W_2 h + b_2);  a = W_o g1 + b_o.
// One vector per head and step: matrix-vector work on fp32 weights (2.5 MB per head at d_emb = 512), bound
// by reading them.  Each layer is its own launch over (output-row blocks, query rows), so that a layer's
// weights are read by a few hundred CTAs at once instead of by the one CTA that owns the head; the four
// launches are chained as programmatic dependents.  The selection kernel's feature CTAs pick up `a`.
#include "common.cuh"
#include "sm100.cuh"

namespace tkphi {

constexpr int kMqThreads = 256;
constexpr int kMqRows = 32;            // output rows per CTA (four per warp)

// Layout of the per-row vectors in the workspace: [g0 (E) | h (E) | g1 (E) | a (r)], stride 3 E + r.
template <int STAGE>
__global__ void __launch_bounds__(kMqThreads) mlp_q_layer_kernel(const Problem p) {
  __shared__ __align__(16) float x[512];
  const MlpParams& m = p.mlp_q;
  const int E = m.d_emb, D = p.head_dim, r = p.n_feat;
  const int row = blockIdx.y, hq = row % p.n_q_heads;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_in = STAGE == 0 ? D : E, n_out = STAGE == 3 ? r : E;
  float* vec = p.mlp_vec + (size_t)row * (3 * E + r);
  pdl_launch_next();
  const float* W = (STAGE == 0 ? m.w_s : STAGE == 1 ? m.w_1 : STAGE == 2 ? m.w_2 : m.w_o) + (size_t)hq * n_out * n_in;
  const float* bias = (STAGE == 0 ? m.b_s : STAGE == 1 ? m.b_1 : STAGE == 2 ? m.b_2 : m.b_o) + (size_t)hq * n_out;
  const float al = STAGE == 2 ? __ldg(m.alpha + hq) : 0.f;
  pdl_wait();                           // the layer before (stage 0: whatever wrote q, and the workspace's readers)
  if (STAGE == 0) {
    for (int c = threadIdx.x; c < D; c += kMqThreads) x[c] = __bfloat162float(p.q[(size_t)row * D + c]);
  } else {
    const float* in = vec + (STAGE - 1) * E;         // stage 1 reads g0, 2 reads h, 3 reads g1
    for (int c = threadIdx.x; c < E; c += kMqThreads) x[c] = __ldcg(in + c);
  }
  __syncthreads();
  const int i0 = blockIdx.x * kMqRows;
  for (int i = i0 + warp; i < i0 + kMqRows && i < n_out; i += kMqThreads / 32) {
    const float* wr = W + (size_t)i * n_in;
    float acc = 0.f;
    for (int c = 4 * lane; c < n_in; c += 128) {
      const float4 w4 = __ldg(reinterpret_cast<const float4*>(wr + c));
      acc = fmaf(w4.x, x[c], fmaf(w4.y, x[c + 1], fmaf(w4.z, x[c + 2], fmaf(w4.w, x[c + 3], acc))));
    }
    acc = warp_sum(acc);
    if (lane == 0) {
      const float t = acc + __ldg(bias + i);
      if (STAGE == 0) vec[i] = t;
      else if (STAGE == 1) vec[E + i] = 0.5f * t * (1.f + erff(t * 0.70710678118654752f));
      else if (STAGE == 2) vec[2 * E + i] = fmaf(al, t, __ldcg(vec + i));
      else vec[3 * E + i] = t;
    }
  }
}

cudaError_t launch_mlp_query(const Problem& p, cudaStream_t st) {
  const int rows = p.batch * p.n_q_heads, E = p.mlp_q.d_emb;
  const dim3 g_e((E + kMqRows - 1) / kMqRows, rows), g_r((p.n_feat + kMqRows - 1) / kMqRows, rows);
  cudaError_t e = launch_pdl(mlp_q_layer_kernel<0>, g_e, dim3(kMqThreads), 0, st, p);
  if (e == cudaSuccess) e = launch_pdl(mlp_q_layer_kernel<1>, g_e, dim3(kMqThreads), 0, st, p);
  if (e == cudaSuccess) e = launch_pdl(mlp_q_layer_kernel<2>, g_e, dim3(kMqThreads), 0, st, p);
  if (e == cudaSuccess) e = launch_pdl(mlp_q_layer_kernel<3>, g_r, dim3(kMqThreads), 0, st, p);
  return e;
}

}  // namespace tkphi
