// C ABI of libtkphi: argument validation, workspace layout, launches.
#include "../../include/tkphi.h"
#include "common.cuh"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <vector>

using namespace tkphi;

namespace {

thread_local char g_err[512] = "";

tkphi_status fail(tkphi_status st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return st;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Shape {
  long long total_tokens;
  int max_len, max_mid, rows, units;
  long long score_tiles;          // tiles of the scoring kernel (all units)
};

// Tail-anchor count of sequence b: the per-sequence array when given, else n_tail.
inline int64_t tail_host(const tkphi_kv_desc* kv, int b) {
  return kv->n_tail_seq_host ? kv->n_tail_seq_host[b] : kv->n_tail;
}

tkphi_status validate_kv(const tkphi_kv_desc* kv, Shape* sh, bool need_data) {
  if (!kv) return fail(TKPHI_ERR_INVALID_ARG, "kv descriptor is NULL");
  if (kv->batch < 1 || kv->batch > kMaxBatch)
    return fail(TKPHI_ERR_INVALID_ARG, "batch must be in [1, %d], got %d", kMaxBatch, kv->batch);
  if (kv->head_dim != 64 && kv->head_dim != 128)
    return fail(TKPHI_ERR_UNSUPPORTED, "head_dim must be 64 or 128, got %d", kv->head_dim);
  if (kv->n_feat != 64 && kv->n_feat != 128)
    return fail(TKPHI_ERR_UNSUPPORTED, "n_feat must be 64 or 128, got %d", kv->n_feat);
  if (kv->n_kv_heads < 1 || kv->n_q_heads < 1 || kv->n_q_heads % kv->n_kv_heads != 0)
    return fail(TKPHI_ERR_INVALID_ARG, "n_q_heads (%d) must be a positive multiple of n_kv_heads (%d)",
                kv->n_q_heads, kv->n_kv_heads);
  if (kv->n_q_heads / kv->n_kv_heads > 8)
    return fail(TKPHI_ERR_UNSUPPORTED, "group size %d > 8", kv->n_q_heads / kv->n_kv_heads);
  if (kv->n_sink < 0 || kv->n_tail < 0) return fail(TKPHI_ERR_INVALID_ARG, "negative anchor count");
  if ((kv->n_tail_seq_host == nullptr) != (kv->n_tail_seq_dev == nullptr))
    return fail(TKPHI_ERR_INVALID_ARG, "n_tail_seq_host and n_tail_seq_dev must both be NULL or both be given");
  if (kv->n_tail_seq_host)
    for (int b = 0; b < kv->batch; ++b)
      if (kv->n_tail_seq_host[b] < 0) return fail(TKPHI_ERR_INVALID_ARG, "n_tail_seq[%d] = %d is negative", b, kv->n_tail_seq_host[b]);
  if (!kv->cu_seqlens_host) return fail(TKPHI_ERR_INVALID_ARG, "cu_seqlens_host is NULL");
  const int64_t* cu = kv->cu_seqlens_host;
  if (cu[0] != 0) return fail(TKPHI_ERR_INVALID_ARG, "cu_seqlens[0] must be 0");
  sh->max_len = 0; sh->max_mid = 0;
  for (int b = 0; b < kv->batch; ++b) {
    const int64_t len = cu[b + 1] - cu[b];
    if (len < 1) return fail(TKPHI_ERR_INVALID_ARG, "sequence %d has length %lld (< 1)", b, (long long)len);
    if (cu[b + 1] >= (1ll << 31)) return fail(TKPHI_ERR_INVALID_ARG, "more than 2^31-1 cache rows");
    if (len > sh->max_len) sh->max_len = (int)len;
    const int64_t mid = len - kv->n_sink - tail_host(kv, b);
    if (mid > sh->max_mid) sh->max_mid = (int)mid;
  }
  sh->total_tokens = cu[kv->batch];
  sh->rows = kv->batch * kv->n_q_heads;
  if ((long long)sh->rows + sh->rows + kv->n_kv_heads > 65535)
    return fail(TKPHI_ERR_UNSUPPORTED, "batch * n_q_heads = %d is too large for one call", sh->rows);
  sh->units = kv->batch * kv->n_kv_heads;
  if (need_data) {
    if (!kv->cu_seqlens_dev) return fail(TKPHI_ERR_INVALID_ARG, "cu_seqlens_dev is NULL");
    if (!kv->k || !kv->v) return fail(TKPHI_ERR_INVALID_ARG, "k or v is NULL");
    if (!aligned16(kv->k) || !aligned16(kv->v)) return fail(TKPHI_ERR_INVALID_ARG, "k and v must be 16-byte aligned");
    if (kv->kv_stride_token < kv->head_dim || kv->kv_stride_token % 8 != 0 || kv->kv_stride_head % 8 != 0 ||
        kv->kv_stride_head < 0)
      return fail(TKPHI_ERR_INVALID_ARG, "strides must be multiples of 8 elements, token stride >= head_dim");
    if (kv->n_kv_heads > 1) {
      // rows of different heads must not share memory: head-major (a head's rows come before the
      // next head's) or token-major (the heads of one token come before the next token's)
      const long long sth = kv->kv_stride_head, stt = kv->kv_stride_token;
      const bool head_major = sth >= sh->total_tokens * stt;
      const bool token_major = sth >= kv->head_dim && stt >= (long long)(kv->n_kv_heads - 1) * sth + kv->head_dim;
      if (!head_major && !token_major)
        return fail(TKPHI_ERR_INVALID_ARG,
                    "kv_stride_head = %lld with %d KV heads: the heads overlap (need kv_stride_head >= rows * "
                    "kv_stride_token, or kv_stride_head >= head_dim and kv_stride_token >= (n_kv_heads - 1) * "
                    "kv_stride_head + head_dim)", sth, kv->n_kv_heads);
    }
  }
  return TKPHI_OK;
}

tkphi_status validate_topk(const tkphi_kv_desc* kv, const int32_t* topk_host, int32_t topk_max, Shape* sh,
                           bool allow_empty_support) {
  if (!topk_host) return fail(TKPHI_ERR_INVALID_ARG, "topk_host is NULL");
  if (topk_max < 0) return fail(TKPHI_ERR_INVALID_ARG, "topk_max < 0");
  const int64_t* cu = kv->cu_seqlens_host;
  const int tk = score_tile_keys(kv->head_dim);
  sh->score_tiles = 0;
  for (int b = 0; b < kv->batch; ++b) {
    const int64_t len = cu[b + 1] - cu[b];
    int64_t mid = len - kv->n_sink - tail_host(kv, b);
    if (mid < 0) mid = 0;
    if (topk_host[b] < 0 || topk_host[b] > mid)
      return fail(TKPHI_ERR_INVALID_ARG, "topk[%d] = %d outside [0, |M| = %lld]", b, topk_host[b], (long long)mid);
    if (topk_host[b] > topk_max)
      return fail(TKPHI_ERR_INVALID_ARG, "topk[%d] = %d exceeds topk_max = %d", b, topk_host[b], topk_max);
    if (!allow_empty_support && topk_host[b] == 0 && kv->n_sink == 0 && tail_host(kv, b) == 0)
      return fail(TKPHI_ERR_INVALID_ARG, "sequence %d has an empty exact support (no anchors, topk = 0)", b);
    if (topk_host[b] > 0) sh->score_tiles += (int64_t)kv->n_kv_heads * ((mid + tk - 1) / tk);
    if (mid > 2097152)
      return fail(TKPHI_ERR_UNSUPPORTED, "sequence %d: mid-region of %lld tokens exceeds 2097152", b, (long long)mid);
  }
  if (sh->score_tiles >= (1ll << 31)) return fail(TKPHI_ERR_UNSUPPORTED, "too many key tiles");
  return TKPHI_OK;
}

int n_sm_cached() { return sm_count_current_device(); }

void decode_layout(const tkphi_kv_desc* kv, const Shape& sh, int32_t topk_max, WsLayout* L) {
  size_t o = 0;
  L->status = o;        o += 256;
  L->row_counter = o;   o = align_up(o + sizeof(unsigned) * sh.rows, 256);
  L->zero_end = o;
  L->scores = o;        o = align_up(o + sizeof(float) * (size_t)kv->n_q_heads * sh.total_tokens, 256);
  L->wk_img = o;        o = align_up(o + (size_t)kv->n_kv_heads * 2 * kv->n_feat * kv->head_dim * 2, 1024);
  L->idx = o;           o = align_up(o + sizeof(int) * (size_t)sh.rows * (topk_max > 0 ? topk_max : 1), 256);
  L->aq = o;            o = align_up(o + sizeof(float) * (size_t)sh.rows * aq_stride(kv->n_feat, kv->head_dim), 256);
  int64_t max_tail = kv->n_tail;
  if (kv->n_tail_seq_host) {
    max_tail = 0;
    for (int b = 0; b < kv->batch; ++b)
      if (kv->n_tail_seq_host[b] > max_tail) max_tail = kv->n_tail_seq_host[b];
  }
  int64_t max_support = (int64_t)kv->n_sink + max_tail + topk_max;
  if (max_support > sh.max_len) max_support = sh.max_len;
  L->max_slices = (int)((max_support + kSlice - 1) / kSlice);
  if (L->max_slices < 1) L->max_slices = 1;
  L->partial_stride = 4 + 2 * kv->head_dim;
  L->partials = o;      o = align_up(o + sizeof(float) * (size_t)sh.rows * L->max_slices * L->partial_stride, 256);
  L->zbuf = o;          o = align_up(o + sizeof(float) * (size_t)sh.rows * (topk_max > 0 ? topk_max : 1), 256);
  // layer outputs of the query-side MLP feature map at its largest hidden width (three vectors and the exponents per row)
  L->mlp_vec = o;       o = align_up(o + sizeof(float) * (size_t)sh.rows * (3 * 512 + kv->n_feat), 256);
  L->total = o;
}

void build_layout(const tkphi_kv_desc* kv, const Shape& sh, WsLayout* L) {
  size_t o = 0;
  L->status = o;        o += 256;
  L->zero_end = o;
  // One CTA per SM over all units, and no chunk longer than 256 tiles of 128 tokens: long units are cut into
  // more chunks than that (several CTAs per SM in turn), which balances the SMs when units x chunks does not
  // divide by the SM count and bounds the length of a tensor-memory accumulation chain (every MMA rounds its
  // fp32 accumulator once; over 2048 tiles the bias reached 6.5e-4 of max |S|).  Never more chunks than tiles.
  const int64_t max_tiles = sh.max_mid > 0 ? ((int64_t)sh.max_mid + 127) / 128 : 1;
  int64_t cpu = n_sm_cached() / sh.units;
  if (cpu < (max_tiles + 255) / 256) cpu = (max_tiles + 255) / 256;
  if (cpu < 1) cpu = 1;
  if (cpu > max_tiles) cpu = max_tiles;
  L->chunks_per_unit = (int)cpu;
  L->b_partials = o;
  o = align_up(o + sizeof(float) * (size_t)sh.units * L->chunks_per_unit *
                       ((size_t)kv->head_dim * kv->n_feat + kv->n_feat), 256);
  L->total = o;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// 3-D view [head][row][dim] of a K or V cache; box = 64 dims x box_rows rows of one head,
// stored with the 128-byte swizzle (head_dim 128 takes two boxes per tile).
tkphi_status make_tensor_map(const tkphi_kv_desc* kv, const void* base, int box_rows, long long total_tokens,
                             CUtensorMap* tm) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return fail(TKPHI_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  const cuuint64_t dims[3] = {(cuuint64_t)kv->head_dim, (cuuint64_t)total_tokens, (cuuint64_t)kv->n_kv_heads};
  const cuuint64_t strides[2] = {(cuuint64_t)kv->kv_stride_token * 2, (cuuint64_t)kv->kv_stride_head * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};   // 128-byte rows
  const cuuint32_t estr[3] = {1, 1, 1};
  // a single head (any stride is legal for the caller, the encoder rejects 0): give the unused
  // dimension a legal stride
  cuuint64_t st[2] = {strides[0], strides[1]};
  if (kv->n_kv_heads == 1) st[1] = st[0] * (cuuint64_t)total_tokens;
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, st, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(TKPHI_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return TKPHI_OK;
}

// 2-D view [row][dim] of a K or V cache for TMA row gathers: box = one row of 64 dims, 128-byte
// swizzle.  Possible when the rows of all heads lie on one pitch: head-major caches
// (stride_head a multiple of stride_token: row = head * ratio + token) or token-major ones
// (stride_token a multiple of stride_head: row = token * ratio + head).  Returns the mode
// (-1: not expressible; the kernel then gathers with 16-byte copies).
int make_gather_map(const tkphi_kv_desc* kv, const void* base, long long total_tokens, CUtensorMap* tm,
                    long long* ratio, long long* rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return -1;
  const long long sh = kv->kv_stride_head, stt = kv->kv_stride_token, H = kv->n_kv_heads;
  int mode;
  long long pitch;
  if (H == 1) { mode = 0; *ratio = total_tokens; pitch = stt; *rows = total_tokens; }
  else if (sh % stt == 0 && sh / stt >= total_tokens) { mode = 0; *ratio = sh / stt; pitch = stt; *rows = (H - 1) * *ratio + total_tokens; }
  else if (stt % sh == 0 && stt / sh >= H) { mode = 1; *ratio = stt / sh; pitch = sh; *rows = (total_tokens - 1) * *ratio + H; }
  else return -1;
  if (pitch < kv->head_dim || (pitch * 2) % 16 != 0 || *rows >= (1LL << 31) - 1 || *rows < 1) return -1;
  const cuuint64_t dims[2] = {(cuuint64_t)kv->head_dim, (cuuint64_t)*rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  const cuuint32_t box[2] = {64, 1};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? mode : -1;
}

// ---- optional per-kernel timing (off by default): CUDA events around every launch
struct TimedSpan { cudaEvent_t a, b; int kind; };
bool g_timing = false;
std::vector<TimedSpan> g_spans;

struct ScopedSpan {
  cudaStream_t st; int kind; cudaEvent_t a = nullptr, b = nullptr;
  ScopedSpan(cudaStream_t s, int k) : st(s), kind(k) {
    if (!g_timing) return;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { a = b = nullptr; return; }
    cudaEventRecord(a, st);
  }
  ~ScopedSpan() {
    if (!a) return;
    cudaEventRecord(b, st);
    g_spans.push_back({a, b, kind});
  }
};

tkphi_status check_ws(void* ws, size_t have, size_t need) {
  if (!ws) return fail(TKPHI_ERR_WORKSPACE, "workspace is NULL");
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return fail(TKPHI_ERR_WORKSPACE, "workspace must be 256-byte aligned");
  if (have < need) return fail(TKPHI_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", have, need);
  return TKPHI_OK;
}

tkphi_status cuda_fail(cudaError_t e, const char* what) {
  return fail(TKPHI_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// Workspace of tkphi_mlp_key_features: status word, bf16 copies of the weights, three bf16 activation
// buffers [n_kv_heads][T_total][d_emb] (g0, GeLU output, g1).
struct MlpLayout { size_t status, w_s, w_1, w_2, w_o, g0, h, g1, total; };
MlpLayout mlp_layout(const tkphi_kv_desc* kv, const Shape& sh, int E) {
  MlpLayout L{};
  const size_t H = kv->n_kv_heads, T = (size_t)sh.total_tokens;
  size_t o = 0;
  L.status = o; o += 1024;
  L.w_s = o;    o = align_up(o + H * E * kv->head_dim * 2, 1024);
  L.w_1 = o;    o = align_up(o + H * E * E * 2, 1024);
  L.w_2 = o;    o = align_up(o + H * E * E * 2, 1024);
  L.w_o = o;    o = align_up(o + H * kv->n_feat * E * 2, 1024);
  L.g0 = o;     o = align_up(o + H * T * E * 2, 1024);
  L.h = o;      o = align_up(o + H * T * E * 2, 1024);
  L.g1 = o;     o = align_up(o + H * T * E * 2, 1024);
  L.total = o;
  return L;
}

// 3-D view [head][row][k] of a bf16 matrix set for the MLP layers: box = 64 k x box_rows rows of one head,
// 128-byte swizzle.  Strides in elements.
tkphi_status make_gemm_map(const void* base, long long k, long long rows, long long heads, long long stride_row,
                           long long stride_head, int box_rows, CUtensorMap* tm) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return fail(TKPHI_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  const cuuint64_t dims[3] = {(cuuint64_t)k, (cuuint64_t)rows, (cuuint64_t)heads};
  cuuint64_t st[2] = {(cuuint64_t)stride_row * 2, (cuuint64_t)stride_head * 2};
  if (heads == 1) st[1] = st[0] * (cuuint64_t)rows;
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, st, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(TKPHI_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return TKPHI_OK;
}

tkphi_status validate_mlp(const tkphi_mlp_desc* m, int n_heads, const char* what) {
  if (!m) return fail(TKPHI_ERR_INVALID_ARG, "%s is NULL", what);
  if (m->d_emb < 128 || m->d_emb > 512 || m->d_emb % 128 != 0)
    return fail(TKPHI_ERR_UNSUPPORTED, "%s: d_emb must be 128, 256, 384 or 512, got %d", what, m->d_emb);
  if (m->n_heads != n_heads) return fail(TKPHI_ERR_INVALID_ARG, "%s: n_heads = %d, expected %d", what, m->n_heads, n_heads);
  const void* ptrs[9] = {m->w_s, m->b_s, m->w_1, m->b_1, m->w_2, m->b_2, m->alpha, m->w_o, m->b_o};
  for (const void* q : ptrs)
    if (!q || !aligned16(q)) return fail(TKPHI_ERR_INVALID_ARG, "%s: a parameter pointer is NULL or not 16-byte aligned", what);
  return TKPHI_OK;
}

MlpParams mlp_params(const tkphi_mlp_desc* m) {
  MlpParams o{};
  o.d_emb = m->d_emb;
  o.w_s = m->w_s; o.b_s = m->b_s; o.w_1 = m->w_1; o.b_1 = m->b_1; o.w_2 = m->w_2; o.b_2 = m->b_2;
  o.alpha = m->alpha; o.w_o = m->w_o; o.b_o = m->b_o;
  return o;
}

tkphi_status decode_common(const tkphi_kv_desc* kv, const tkphi_phi_desc* phi, const void* q,
                           const int32_t* topk_host, const int32_t* topk_dev, int32_t topk_max, const float* S,
                           const float* u, int32_t* idx_out, float* y_out, float* dbg_out, uint32_t flags,
                           void* ws, size_t ws_bytes, void* stream, bool with_phi,
                           const tkphi_mlp_desc* mlp_q = nullptr, const float* mlp_cache = nullptr) {
  g_err[0] = 0;
  Shape sh{};
  tkphi_status st = validate_kv(kv, &sh, true);
  if (st != TKPHI_OK) return st;
  st = validate_topk(kv, topk_host, topk_max, &sh, with_phi);
  if (st != TKPHI_OK) return st;
  if (!topk_dev) return fail(TKPHI_ERR_INVALID_ARG, "topk_dev is NULL");
  if (!q || !aligned16(q)) return fail(TKPHI_ERR_INVALID_ARG, "q is NULL or not 16-byte aligned");
  if (!y_out) return fail(TKPHI_ERR_INVALID_ARG, "y_out is NULL");
  if (flags & ~1u) return fail(TKPHI_ERR_INVALID_ARG, "unknown flag bits 0x%x", flags);
  if (with_phi && mlp_q) {
    st = validate_mlp(mlp_q, kv->n_q_heads, "mlp_q");
    if (st != TKPHI_OK) return st;
    if (!S || !u || !aligned16(S) || !aligned16(u)) return fail(TKPHI_ERR_INVALID_ARG, "S or u is NULL or not 16-byte aligned");
    if (!(flags & TKPHI_FLAG_NOSUB) && (!mlp_cache || !aligned16(mlp_cache)))
      return fail(TKPHI_ERR_INVALID_ARG, "phi_k_cache is NULL or not 16-byte aligned");
  } else if (with_phi) {
    if (!phi || !phi->w_q || !phi->b_q || !phi->w_k || !phi->b_k)
      return fail(TKPHI_ERR_INVALID_ARG, "phi descriptor or one of its pointers is NULL");
    if (!S || !u) return fail(TKPHI_ERR_INVALID_ARG, "S or u is NULL");
    if (!aligned16(phi->w_q) || !aligned16(phi->w_k) || !aligned16(S) || !aligned16(u))
      return fail(TKPHI_ERR_INVALID_ARG, "w_q, w_k, S and u must be 16-byte aligned");
    if (!std::isfinite(phi->gamma_q) || !std::isfinite(phi->gamma_k))
      return fail(TKPHI_ERR_INVALID_ARG, "gamma must be finite");
    if (phi->phi_k_cache && !aligned16(phi->phi_k_cache))
      return fail(TKPHI_ERR_INVALID_ARG, "phi_k_cache must be 16-byte aligned");
  }
  WsLayout L{};
  decode_layout(kv, sh, topk_max, &L);
  st = check_ws(ws, ws_bytes, L.total);
  if (st != TKPHI_OK) return st;

  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(ws);
  Problem p{};
  p.batch = kv->batch; p.n_q_heads = kv->n_q_heads; p.n_kv_heads = kv->n_kv_heads;
  p.head_dim = kv->head_dim; p.n_feat = kv->n_feat; p.n_sink = kv->n_sink; p.n_tail = kv->n_tail;
  p.n_tail_seq = kv->n_tail_seq_dev;
  p.group = kv->n_q_heads / kv->n_kv_heads;
  p.cu_seqlens = reinterpret_cast<const long long*>(kv->cu_seqlens_dev);
  p.topk = topk_dev; p.topk_max = topk_max > 0 ? topk_max : 1;
  p.k = static_cast<const __nv_bfloat16*>(kv->k); p.v = static_cast<const __nv_bfloat16*>(kv->v);
  p.stride_head = kv->kv_stride_head; p.stride_token = kv->kv_stride_token;
  p.q = static_cast<const __nv_bfloat16*>(q);
  if (with_phi && mlp_q) {
    p.mlp_q = mlp_params(mlp_q);
    p.mlp_vec = reinterpret_cast<float*>(w + L.mlp_vec);
    p.S = S; p.u = u;
    if (!(flags & TKPHI_FLAG_NOSUB)) {
      p.phi_cache = mlp_cache;
      p.zbuf = reinterpret_cast<float*>(w + L.zbuf);
    }
  } else if (with_phi) {
    p.w_q = phi->w_q; p.b_q = phi->b_q; p.w_k = phi->w_k; p.b_k = phi->b_k;
    p.gamma_q = phi->gamma_q; p.gamma_k = phi->gamma_k; p.S = S; p.u = u;
    if (phi->phi_k_cache && !(flags & TKPHI_FLAG_NOSUB)) {
      p.phi_cache = phi->phi_k_cache;
      p.zbuf = reinterpret_cast<float*>(w + L.zbuf);
    }
  }
  p.total_tokens = sh.total_tokens;
  p.idx_out = idx_out; p.y_out = y_out; p.dbg_out = dbg_out; p.flags = flags; p.with_phi = with_phi ? 1 : 0;
  p.status = reinterpret_cast<int*>(w + L.status);
  p.row_counter = reinterpret_cast<unsigned*>(w + L.row_counter);
  p.scores = reinterpret_cast<float*>(w + L.scores);
  p.wk_img = reinterpret_cast<__nv_bfloat16*>(w + L.wk_img);
  p.idx = reinterpret_cast<int*>(w + L.idx);
  p.aq = reinterpret_cast<float*>(w + L.aq);
  p.partials = reinterpret_cast<float*>(w + L.partials);
  p.max_slices = L.max_slices; p.partial_stride = L.partial_stride;
  p.scale = 1.0f / sqrtf((float)kv->head_dim);
  // idx_out uses the caller's topk_max as its row length; the internal list uses p.topk_max
  if (topk_max == 0) p.idx_out = nullptr;

  p.zero_bytes = L.zero_end;
  cudaError_t e;
  if (p.mlp_q.w_s) {      // the four layers of the query-side MLP, before the key stream
    ScopedSpan sp(cs, TKPHI_KERNEL_MLP);
    e = launch_mlp_query(p, cs);
    if (e != cudaSuccess) return cuda_fail(e, "query-side MLP launch");
  }
  // The scoring kernel also clears the workspace counters; without keys to score a plain
  // memset does.  The selection kernel carries the query-side feature work on extra clusters.
  if (sh.score_tiles > 0) {
    CUtensorMap tm;
    st = make_tensor_map(kv, kv->k, score_tile_keys(kv->head_dim), sh.total_tokens, &tm);
    if (st != TKPHI_OK) return st;
    {
      ScopedSpan sp(cs, TKPHI_KERNEL_SCORE);
      e = launch_score(p, tm, n_sm_cached(), cs);
    }
    if (e != cudaSuccess) return cuda_fail(e, "score launch");
  } else {
    ScopedSpan sp(cs, TKPHI_KERNEL_MEMSET);
    e = cudaMemsetAsync(w, 0, L.zero_end, cs);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(workspace)");
  }
  {
    ScopedSpan sp(cs, TKPHI_KERNEL_SELECT);
    e = launch_select(p, sh.score_tiles > 0 ? sh.max_mid : 0, n_sm_cached(), cs);
  }
  if (e != cudaSuccess) return cuda_fail(e, "select launch");
  if (p.zbuf) {
    ScopedSpan sp(cs, TKPHI_KERNEL_CACHED_Z);
    e = launch_cached_z(p, cs);
    if (e != cudaSuccess) return cuda_fail(e, "cached-feature launch");
  }
  {
    ScopedSpan sp(cs, TKPHI_KERNEL_EXACT_RESIDUAL);
    // slice pairs of the whole call (two 128-token slices of a support list per CTA)
    long long n_pairs = 0;
    for (int b = 0; b < kv->batch; ++b) {
      const long long len_b = kv->cu_seqlens_host[b + 1] - kv->cu_seqlens_host[b];
      const long long n_a1 = len_b < kv->n_sink ? len_b : kv->n_sink;
      long long ts = len_b - tail_host(kv, b);
      if (ts < kv->n_sink) ts = kv->n_sink;
      if (ts > len_b) ts = len_b;
      const long long n_e = n_a1 + topk_host[b] + (len_b - ts);
      const long long n_slices = n_e > 0 ? (n_e + kSlice - 1) / kSlice : 1;
      n_pairs += (long long)kv->n_q_heads * ((n_slices + 1) / 2);
    }
    CUtensorMap gk, gv;
    memset(&gk, 0, sizeof(gk));
    memset(&gv, 0, sizeof(gv));
    long long ratio_v = 0, rows_v = 0;
    // the row-gather maps are needed (and encoded) only where the streaming kernel can be chosen
    p.gather_mode = -1;
    if (n_pairs > n_sm_cached() && kv->head_dim == 128) {
      p.gather_mode = make_gather_map(kv, kv->k, sh.total_tokens, &gk, &p.gather_ratio, &p.gather_rows);
      if (p.gather_mode >= 0 && make_gather_map(kv, kv->v, sh.total_tokens, &gv, &ratio_v, &rows_v) != p.gather_mode)
        p.gather_mode = -1;
    }
    e = launch_exact_residual(p, gk, gv, n_pairs, n_sm_cached(), cs);
  }
  if (e != cudaSuccess) return cuda_fail(e, "exact_residual launch");
  return TKPHI_OK;
}

tkphi_status build_common(const tkphi_kv_desc* kv, const float* w_k, const float* b_k, float gamma_k, float* cache,
                          bool from_cache, float* S, float* u, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  Shape sh{};
  tkphi_status st = validate_kv(kv, &sh, true);
  if (st != TKPHI_OK) return st;
  if (!S || !u) return fail(TKPHI_ERR_INVALID_ARG, "S or u is NULL");
  if (cache && !aligned16(cache)) return fail(TKPHI_ERR_INVALID_ARG, "phi_k_cache must be 16-byte aligned");
  WsLayout L{};
  build_layout(kv, sh, &L);
  st = check_ws(workspace, workspace_bytes, L.total);
  if (st != TKPHI_OK) return st;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* w = static_cast<char*>(workspace);
  BuildProblem p{};
  p.batch = kv->batch; p.n_kv_heads = kv->n_kv_heads; p.head_dim = kv->head_dim; p.n_feat = kv->n_feat;
  p.n_sink = kv->n_sink; p.n_tail = kv->n_tail; p.n_tail_seq = kv->n_tail_seq_dev;
  p.cu_seqlens = reinterpret_cast<const long long*>(kv->cu_seqlens_dev);
  p.k = static_cast<const __nv_bfloat16*>(kv->k); p.v = static_cast<const __nv_bfloat16*>(kv->v);
  p.stride_head = kv->kv_stride_head; p.stride_token = kv->kv_stride_token;
  p.w_k = w_k; p.b_k = b_k; p.gamma_k = gamma_k;
  p.phi_cache = cache; p.from_cache = from_cache ? 1 : 0; p.total_tokens = sh.total_tokens;
  p.S = S; p.u = u;
  p.status = reinterpret_cast<int*>(w + L.status);
  p.partials = reinterpret_cast<float*>(w + L.b_partials);
  p.chunks_per_unit = L.chunks_per_unit;
  CUtensorMap tk, tv;
  st = make_tensor_map(kv, kv->k, 128, sh.total_tokens, &tk);
  if (st != TKPHI_OK) return st;
  st = make_tensor_map(kv, kv->v, 128, sh.total_tokens, &tv);
  if (st != TKPHI_OK) return st;
  cudaError_t e;
  {
    ScopedSpan sp(cs, TKPHI_KERNEL_BUILD);
    e = launch_build(p, tk, tv, cs);      // clears the status word itself; needs no zeroed counters
  }
  if (e != cudaSuccess) return cuda_fail(e, "build launch");
  return TKPHI_OK;
}

}  // namespace

namespace tkphi {

int sm_count_current_device() {
  static int n_sm[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  if (n_sm[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    n_sm[dev] = n;
  }
  return n_sm[dev];
}

cudaError_t set_max_dynamic_smem(PerDeviceFlag& flag, const void* kernel, size_t bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < kMaxDevices;
  if (tracked && flag.done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess && tracked) flag.done[dev] = true;
  return e;
}

}  // namespace tkphi

extern "C" {

const char* tkphi_last_error(void) { return g_err; }
int32_t tkphi_version(void) { return 100; }

size_t tkphi_workspace_bytes(const tkphi_kv_desc* kv, const int32_t* topk_host, int32_t topk_max, int which) {
  g_err[0] = 0;
  Shape sh{};
  if (validate_kv(kv, &sh, false) != TKPHI_OK) return 0;
  WsLayout L{};
  if (which == TKPHI_WS_BUILD) {
    build_layout(kv, sh, &L);
    return L.total;
  }
  if (which == TKPHI_WS_MLP_KEY_FEATURES) return mlp_layout(kv, sh, 512).total;
  if (which != TKPHI_WS_TOPK_DECODE && which != TKPHI_WS_DECODE_STEP) {
    fail(TKPHI_ERR_INVALID_ARG, "unknown workspace kind %d", which);
    return 0;
  }
  if (validate_topk(kv, topk_host, topk_max, &sh, true) != TKPHI_OK) return 0;
  decode_layout(kv, sh, topk_max, &L);
  return L.total;
}

tkphi_status tkphi_build_summaries(const tkphi_kv_desc* kv, const tkphi_phi_desc* phi, float* S, float* u,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  g_err[0] = 0;
  if (!phi || !phi->w_k || !phi->b_k) return fail(TKPHI_ERR_INVALID_ARG, "phi->w_k or phi->b_k is NULL");
  if (!std::isfinite(phi->gamma_k)) return fail(TKPHI_ERR_INVALID_ARG, "gamma_k must be finite");
  if (!aligned16(phi->w_k)) return fail(TKPHI_ERR_INVALID_ARG, "w_k must be 16-byte aligned");
  return build_common(kv, phi->w_k, phi->b_k, phi->gamma_k, phi->phi_k_cache, false, S, u, workspace, workspace_bytes,
                      cuda_stream);
}

tkphi_status tkphi_build_summaries_cached(const tkphi_kv_desc* kv, const float* phi_k_cache, float* S, float* u,
                                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
  g_err[0] = 0;
  if (!phi_k_cache) return fail(TKPHI_ERR_INVALID_ARG, "phi_k_cache is NULL");
  return build_common(kv, nullptr, nullptr, 0.f, const_cast<float*>(phi_k_cache), true, S, u, workspace, workspace_bytes,
                      cuda_stream);
}

tkphi_status tkphi_mlp_key_features(const tkphi_kv_desc* kv, const tkphi_mlp_desc* mlp_k, float* phi_k_cache,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  g_err[0] = 0;
  Shape sh{};
  tkphi_status st = validate_kv(kv, &sh, true);
  if (st != TKPHI_OK) return st;
  st = validate_mlp(mlp_k, kv->n_kv_heads, "mlp_k");
  if (st != TKPHI_OK) return st;
  if (!phi_k_cache || !aligned16(phi_k_cache)) return fail(TKPHI_ERR_INVALID_ARG, "phi_k_cache is NULL or not 16-byte aligned");
  const int E = mlp_k->d_emb, D = kv->head_dim, R = kv->n_feat, H = kv->n_kv_heads;
  const long long T = sh.total_tokens;
  const MlpLayout L = mlp_layout(kv, sh, E);
  st = check_ws(workspace, workspace_bytes, L.total);
  if (st != TKPHI_OK) return st;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* w = static_cast<char*>(workspace);
  int* status = reinterpret_cast<int*>(w + L.status);
  __nv_bfloat16* ws_ = reinterpret_cast<__nv_bfloat16*>(w + L.w_s);
  __nv_bfloat16* w1_ = reinterpret_cast<__nv_bfloat16*>(w + L.w_1);
  __nv_bfloat16* w2_ = reinterpret_cast<__nv_bfloat16*>(w + L.w_2);
  __nv_bfloat16* wo_ = reinterpret_cast<__nv_bfloat16*>(w + L.w_o);
  __nv_bfloat16* g0 = reinterpret_cast<__nv_bfloat16*>(w + L.g0);
  __nv_bfloat16* hb = reinterpret_cast<__nv_bfloat16*>(w + L.h);
  __nv_bfloat16* g1 = reinterpret_cast<__nv_bfloat16*>(w + L.g1);
  ScopedSpan sp(cs, TKPHI_KERNEL_MLP);
  cudaError_t e = cudaMemsetAsync(status, 0, 256, cs);
  if (e == cudaSuccess) e = launch_f32_to_bf16(mlp_k->w_s, ws_, (size_t)H * E * D, cs);
  if (e == cudaSuccess) e = launch_f32_to_bf16(mlp_k->w_1, w1_, (size_t)H * E * E, cs);
  if (e == cudaSuccess) e = launch_f32_to_bf16(mlp_k->w_2, w2_, (size_t)H * E * E, cs);
  if (e == cudaSuccess) e = launch_f32_to_bf16(mlp_k->w_o, wo_, (size_t)H * R * E, cs);
  if (e != cudaSuccess) return cuda_fail(e, "weight conversion launch");
  // tensor maps: activations [head][token][k] (the keys through the cache's own strides), weights [head][n][k]
  CUtensorMap a_k, a_g0, a_h, a_g1, m_ws, m_w1, m_w2, m_wo;
  const int bn_e = mlp_gemm_bn(E), bn_o = mlp_gemm_bn(R);
  if ((st = make_tensor_map(kv, kv->k, 128, T, &a_k)) != TKPHI_OK) return st;
  if ((st = make_gemm_map(g0, E, T, H, E, T * E, 128, &a_g0)) != TKPHI_OK) return st;
  if ((st = make_gemm_map(hb, E, T, H, E, T * E, 128, &a_h)) != TKPHI_OK) return st;
  if ((st = make_gemm_map(g1, E, T, H, E, T * E, 128, &a_g1)) != TKPHI_OK) return st;
  if ((st = make_gemm_map(ws_, D, E, H, D, (long long)E * D, bn_e, &m_ws)) != TKPHI_OK) return st;
  if ((st = make_gemm_map(w1_, E, E, H, E, (long long)E * E, bn_e, &m_w1)) != TKPHI_OK) return st;
  if ((st = make_gemm_map(w2_, E, E, H, E, (long long)E * E, bn_e, &m_w2)) != TKPHI_OK) return st;
  if ((st = make_gemm_map(wo_, E, R, H, E, (long long)R * E, bn_o, &m_wo)) != TKPHI_OK) return st;
  GemmArgs g{};
  g.M = (int)T; g.heads = H; g.status = status;
  // g0 = W_s x + b_s
  g.N = E; g.K = D; g.epi = kEpiBias; g.bias = mlp_k->b_s; g.out = g0; g.out_head_stride = T * E;
  if ((e = launch_mlp_gemm(a_k, m_ws, g, cs)) != cudaSuccess) return cuda_fail(e, "MLP stem launch");
  // h = GeLU(W_1 g0 + b_1)
  g.K = E; g.epi = kEpiGelu; g.bias = mlp_k->b_1; g.out = hb;
  if ((e = launch_mlp_gemm(a_g0, m_w1, g, cs)) != cudaSuccess) return cuda_fail(e, "MLP layer 1 launch");
  // g1 = g0 + alpha (W_2 h + b_2)
  g.epi = kEpiResidual; g.bias = mlp_k->b_2; g.alpha = mlp_k->alpha; g.resid = g0; g.out = g1;
  if ((e = launch_mlp_gemm(a_h, m_w2, g, cs)) != cudaSuccess) return cuda_fail(e, "MLP layer 2 launch");
  // phi = exp(W_o g1 + b_o)
  g.N = R; g.epi = kEpiExp; g.bias = mlp_k->b_o; g.out = phi_k_cache; g.out_head_stride = T * R;
  if ((e = launch_mlp_gemm(a_g1, m_wo, g, cs)) != cudaSuccess) return cuda_fail(e, "MLP output layer launch");
  return TKPHI_OK;
}

tkphi_status tkphi_topk_decode(const tkphi_kv_desc* kv, const void* q, const int32_t* topk_host,
                               const int32_t* topk_dev, int32_t topk_max, int32_t* idx_out, float* y_out,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return decode_common(kv, nullptr, q, topk_host, topk_dev, topk_max, nullptr, nullptr, idx_out, y_out, nullptr, 0,
                       workspace, workspace_bytes, cuda_stream, false);
}

tkphi_status tkphi_decode_step(const tkphi_kv_desc* kv, const tkphi_phi_desc* phi, const void* q,
                               const int32_t* topk_host, const int32_t* topk_dev, int32_t topk_max, const float* S,
                               const float* u, int32_t* idx_out, float* y_out, float* dbg_out, uint32_t flags,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return decode_common(kv, phi, q, topk_host, topk_dev, topk_max, S, u, idx_out, y_out, dbg_out, flags, workspace,
                       workspace_bytes, cuda_stream, true);
}

tkphi_status tkphi_decode_step_mlp(const tkphi_kv_desc* kv, const tkphi_mlp_desc* mlp_q, const float* phi_k_cache,
                                   const void* q, const int32_t* topk_host, const int32_t* topk_dev, int32_t topk_max,
                                   const float* S, const float* u, int32_t* idx_out, float* y_out, float* dbg_out,
                                   uint32_t flags, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!mlp_q) { g_err[0] = 0; return fail(TKPHI_ERR_INVALID_ARG, "mlp_q is NULL"); }
  return decode_common(kv, nullptr, q, topk_host, topk_dev, topk_max, S, u, idx_out, y_out, dbg_out, flags, workspace,
                       workspace_bytes, cuda_stream, true, mlp_q, phi_k_cache);
}

tkphi_status tkphi_device_status(const void* workspace, void* cuda_stream, int32_t* status_out) {
  g_err[0] = 0;
  if (!workspace || !status_out) return fail(TKPHI_ERR_INVALID_ARG, "NULL argument");
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaMemcpyAsync(status_out, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, cs);
  if (e == cudaSuccess) e = cudaStreamSynchronize(cs);
  if (e != cudaSuccess) return cuda_fail(e, "reading the device status word");
  return TKPHI_OK;
}

void tkphi_kernel_timing_enable(int32_t on) {
  g_timing = on != 0;
  if (!g_timing) {
    for (auto& sp : g_spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    g_spans.clear();
  }
}

tkphi_status tkphi_kernel_timing_read(float* ms_out, int32_t* count_out) {
  g_err[0] = 0;
  if (!ms_out || !count_out) return fail(TKPHI_ERR_INVALID_ARG, "NULL argument");
  for (int i = 0; i < TKPHI_KERNEL_KINDS; ++i) { ms_out[i] = 0.f; count_out[i] = 0; }
  tkphi_status st = TKPHI_OK;
  for (auto& sp : g_spans) {
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(sp.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, sp.a, sp.b);
    if (e != cudaSuccess) st = cuda_fail(e, "reading a timing event");
    else { ms_out[sp.kind] += ms; count_out[sp.kind] += 1; }
    cudaEventDestroy(sp.a);
    cudaEventDestroy(sp.b);
  }
  g_spans.clear();
  return st;
}

}  // extern "C"
