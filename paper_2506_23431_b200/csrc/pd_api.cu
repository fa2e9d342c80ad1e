// Host side of the C ABI: configuration checks, workspace carving, the per-step launch
// sequence (own kernels + cuBLAS projections) and its CUDA-graph replay, result readers.
#include <cublasLt.h>
#include <cublas_v2.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

#include "pd_internal.h"

using namespace pd;

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kCublasWs = 64u << 20;

struct Region { size_t off = 0, bytes = 0; };

struct Layout {
  // integer state (offsets in int32 words from the start of the state block)
  size_t w_hdr, w_stats, w_k, w_done, w_steps, w_nact, w_ctx, w_ticket, w_start, w_len, w_state, w_flag, w_last,
      w_forced, w_row, w_prow, w_rtok, w_ptab, w_tokens, w_chosen, w_trace, w_plist_n, w_xtick, w_crow, w_t0, w_plan, state_words;
  Region state, plist, row_meta, bias_tab, ctx_len_in, forced_in, teacher, dist_bucket, rope_tab, x, hbuf, qkv, qbuf, self_out, cq, cross_out,
      ffn, logits, vpart_val, vpart_idx, vterm, part_o, part_ml, kv_c, kv_scale, kv_pool, enc_stage, proj_stage, cublas_ws;
  size_t total = 0;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Limits of this build on otherwise valid configurations, with the text pd_config_check returns.
const char *unsupported_reason(const pd_config &c) {
  if (c.pos_mode == PD_POS_T5_BIAS && c.time_max + c.sub_max + 2 > 512)
    return "T5-bias mode keeps one bias value per distance in shared memory: time_max + sub_max + 2 must not exceed 512";
  if (c.kv_c_dtype == PD_KV_E4M3 && (c.dtype != PD_DTYPE_BF16 || (c.max_ctx % 16) != 0))
    return "8-bit context keys/values need dtype = bf16 and max_ctx a multiple of 16";
  if (c.kv_c_dtype == PD_KV_E4M3 && c.delta_t >= 1 && (c.max_sub_len / c.delta_t + 1 < c.sub_max ? c.max_sub_len / c.delta_t + 1 : c.sub_max) > 32)
    return "8-bit context keys/values are read by the tensor-core kernel only: at most 32 rows per sequence";
  return nullptr;
}

bool make_dims(const pd_config &c, Dims &dm, int &max_splits) {
  if (c.n_layers < 1 || c.d_model < 64 || c.d_model > 4096 || c.n_heads < 1 || c.d_head != kDh || c.n_heads * c.d_head != c.d_model) return false;
  if (c.d_ff < 8 || c.vocab < 4 || (c.d_model % 8) || (c.d_ff % 8)) return false;
  if (c.dtype != PD_DTYPE_FP32 && c.dtype != PD_DTYPE_BF16) return false;
  if (c.max_batch < 1 || c.max_ctx < 1 || c.sub_max < 1 || c.sub_max > 64 || c.delta_t < 1 || c.time_max < 1) return false;
  if (c.max_sub_len < 1 || (c.page_tokens != 16 && c.page_tokens != 32)) return false;
  if (c.pos_mode != PD_POS_T5_BIAS && c.pos_mode != PD_POS_ROPE) return false;
  if (c.pos_mode == PD_POS_T5_BIAS && (c.rel_buckets < 2 || c.rel_buckets > 256 || (c.rel_buckets & 1) || c.rel_max_dist <= c.rel_buckets / 2)) return false;
  const int ids[3] = {c.bos_id, c.eos_id, c.sep_id};
  for (int v : ids) if (v < 0 || v >= c.vocab) return false;
  if (c.self_splits < 0 || c.self_splits > 32 || c.cross_splits < 0 || c.cross_splits > 32) return false;
  if (c.store_logits != 0 && c.store_logits != 1) return false;
  if (c.kv_c_dtype != PD_KV_SAME && c.kv_c_dtype != PD_KV_E4M3) return false;
  if (unsupported_reason(c) != nullptr) return false;
  if (!(c.attn_scale > 0.f) || !(c.norm_eps >= 0.f)) return false;
  dm.L = c.n_layers; dm.d = c.d_model; dm.H = c.n_heads; dm.ff = c.d_ff; dm.V = c.vocab;
  dm.B = c.max_batch; dm.ctx = c.max_ctx; dm.SM = c.sub_max; dm.dt = c.delta_t; dm.T = c.time_max;
  dm.MSL = c.max_sub_len;
  int conc = c.max_sub_len / c.delta_t + 1;   // subsequences that can be open at the same step
  dm.C = conc < c.sub_max ? conc : c.sub_max;
  dm.P = c.page_tokens;
  dm.PPS = (c.max_sub_len + 1 + dm.P - 1) / dm.P;
  long long worst = (long long)c.max_batch * c.sub_max * dm.PPS;
  dm.pool = c.pool_pages > 0 ? c.pool_pages : (int)worst;
  dm.pool_static = c.pool_pages == 0 ? 1 : 0;
  if (c.pool_pages < 0 || worst > 0x7fffffffLL) return false;
  if ((long long)c.n_layers * c.max_batch * c.n_heads * 2 * c.max_ctx > 0x7fffffffLL) return false;   // rows of the context K/V tensor map
  dm.bos = c.bos_id; dm.eos = c.eos_id; dm.sep = c.sep_id;
  dm.pos_mode = c.pos_mode;
  dm.n_dist = c.time_max + c.sub_max + 2;

  dm.scale_log2e = c.attn_scale * 1.4426950408889634f;
  dm.eps = c.norm_eps;
  max_splits = 32;
  return true;
}

void make_layout(const pd_config &c, const Dims &dm, int max_splits, Layout &L) {
  const size_t B = dm.B, SM = dm.SM, C = dm.C;
  size_t w = 0;
  auto take = [&](size_t n) { size_t o = w; w += n; return o; };
  L.w_hdr = take(HDR_WORDS);
  L.w_stats = take(2 * PD_STAT_COUNT);            // 64-bit counters, 8-byte aligned (HDR_WORDS is even)
  L.w_trace = take(2 * (size_t)dm.T * B);         // 64-bit masks
  L.w_plist_n = take(B);
  L.w_xtick = take(B * dm.H);
  L.w_crow = take(B);
  L.w_t0 = take(B);
  L.w_k = take(B); L.w_done = take(B); L.w_steps = take(B); L.w_nact = take(B); L.w_ctx = take(B); L.w_ticket = take(B);
  L.w_start = take(B * SM); L.w_len = take(B * SM); L.w_state = take(B * SM); L.w_flag = take(B * SM);
  L.w_last = take(B * SM); L.w_forced = take(B * SM); L.w_plan = take(B * SM);
  L.w_row = take(B * C); L.w_prow = take(B * C); L.w_rtok = take(B * C);
  L.w_ptab = take(B * SM * dm.PPS);
  L.w_tokens = take(B * SM * dm.MSL);
  L.w_chosen = take(B * SM * (dm.MSL + 1));
  L.state_words = w;

  size_t off = 0;
  auto reg = [&](Region &r, size_t bytes) { r.off = off; r.bytes = bytes; off = align_up(off + bytes, kAlign); };
  const size_t e = c.dtype == PD_DTYPE_BF16 ? 2 : 4;
  const size_t M = B * C;
  reg(L.state, L.state_words * 4);
  reg(L.plist, B * SM * dm.PPS * sizeof(int4));
  reg(L.row_meta, B * C * sizeof(int4));
  reg(L.bias_tab, (size_t)dm.H * dm.n_dist * 4);
  reg(L.ctx_len_in, B * 4);
  reg(L.forced_in, B * SM * 4);
  reg(L.teacher, B * SM * 4);
  reg(L.dist_bucket, (size_t)dm.n_dist * 4);
  reg(L.rope_tab, (size_t)dm.n_dist * (kDh / 2) * sizeof(float2));
  reg(L.x, M * dm.d * 4);
  reg(L.hbuf, M * dm.d * e);
  reg(L.qkv, M * 3 * dm.d * 4);
  reg(L.qbuf, M * dm.d * e);
  reg(L.self_out, M * dm.d * e);
  reg(L.cq, M * dm.d * e);
  reg(L.cross_out, M * dm.d * e);
  reg(L.ffn, M * dm.ff * e);
  reg(L.logits, M * (size_t)dm.V * 4);
  {
    const size_t tiles = (size_t)vocab_tc_tiles(dm.V);      // per-slice candidates of the vocabulary projection
    reg(L.vpart_val, tiles * M * 4);
    reg(L.vpart_idx, tiles * M * 4);
    reg(L.vterm, M * 2 * 4);
  }
  {
    size_t split_bytes = M * dm.H * max_splits * kDh * 4, flat_bytes = cross_attn_tma_partial_bytes(kMaxCrossCtas, dm.C);
    reg(L.part_o, split_bytes > flat_bytes ? split_bytes : flat_bytes);
  }
  reg(L.part_ml, M * dm.H * max_splits * 2 * 4);
  if (c.kv_c_dtype == PD_KV_E4M3) {
    reg(L.kv_c, (size_t)dm.L * B * dm.ctx * 2 * dm.d);                       // one byte per value
    reg(L.kv_scale, (size_t)dm.L * B * dm.H * 2 * sizeof(float) * 2);        // scales, then the maxima they come from
  } else {
    reg(L.kv_c, (size_t)dm.L * B * dm.ctx * 2 * dm.d * e);
    reg(L.kv_scale, 0);
  }
  reg(L.kv_pool, (size_t)dm.L * dm.pool * 2 * dm.H * dm.P * kDh * e);
  reg(L.enc_stage, B * dm.ctx * dm.d * e);
  reg(L.proj_stage, B * dm.ctx * 2 * dm.d * e);
  reg(L.cublas_ws, kCublasWs);
  L.total = off;
}

struct ProfRec { int kind; cudaEvent_t a, b; };

}  // namespace

struct pd_handle {
  pd_config cfg;
  Dims dm;
  Layout lay;
  int max_splits = 32;
  uint8_t *ws = nullptr;
  cudaStream_t stream = nullptr;
  cublasHandle_t blas = nullptr;
  cublasLtHandle_t lt = nullptr;
  // feed-forward up-projection with the ReLU in the GEMM epilogue (plan cached per row count)
  cublasLtMatmulDesc_t ff_desc = nullptr;
  cublasLtMatrixLayout_t ff_w = nullptr, ff_a = nullptr, ff_c = nullptr;
  cublasLtMatmulAlgo_t ff_algo;
  int ff_rows = -1;          // rows the plan was made for; -2 = cuBLASLt path unavailable
  DecState st;
  std::vector<const void *> layer_w;
  pd_weights w;
  CUtensorMap tmap_kvc, tmap_kvc_v;   // context keys/values (8-bit storage: the keys' lines and the transposed values)
  bool have_tmap = false;
  bool kv8 = false;
  VocabMaps vmaps;                 // hidden rows and lm_head for the tcgen05 vocabulary projection
  bool vocab_tc = false;
  // pd_generate_host: host-to-device copies of the encoder memory run on a stream of their own, in
  // chunks of sequences, so that the context projection of one chunk overlaps the copy of the next
  static constexpr int kMaxChunks = 8;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_entry = nullptr, ev_chunk[kMaxChunks] = {};
  // pd_run: a snapshot of the header after every step travels to pinned memory on the copy stream, so
  // that the host can follow the decode a couple of steps behind without ever draining the stream
  static constexpr int kRunSlots = 4;
  cudaEvent_t ev_step[kRunSlots] = {}, ev_snap[kRunSlots] = {};
  int batch = 0;
  bool encoded = false;
  int self_splits = 1, cross_splits = 1;
  int cross_ctas = 296;
  int steps_enqueued = 0;
  bool teacher_clear = false;
  // graph
  cudaGraphExec_t graph_exec = nullptr;
  int graph_batch = -1;
  long long graph_own = 0, graph_gemm = 0;
  // counters / profiling
  long long own_launches = 0, gemm_calls = 0;
  bool profiling = false;
  std::vector<ProfRec> prof;
  std::vector<cudaEvent_t> ev_pool;
  int32_t *pinned_flag = nullptr;
  std::string err;
  template <typename T> T *ptr(const Region &r) const { return reinterpret_cast<T *>(ws + r.off); }
};

namespace {

pd_status fail(pd_handle *h, pd_status s, const std::string &msg) {
  if (h) h->err = msg;
  return s;
}
#define CU_TRY(h, expr)                                                                                   \
  do {                                                                                                    \
    cudaError_t e__ = (expr);                                                                             \
    if (e__ != cudaSuccess) return fail(h, PD_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e__)); \
  } while (0)
#define PD_TRY(expr)                         \
  do {                                       \
    pd_status s__ = (expr);                  \
    if (s__ != PD_OK) return s__;            \
  } while (0)

cudaEvent_t get_event(pd_handle *h) {
  if (!h->ev_pool.empty()) { cudaEvent_t e = h->ev_pool.back(); h->ev_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

struct ProfScope {
  pd_handle *h; int kind; cudaEvent_t a = nullptr;
  ProfScope(pd_handle *h_, int k) : h(h_), kind(k) {
    if (h->profiling) { a = get_event(h); cudaEventRecord(a, h->stream); }
  }
  ~ProfScope() {
    if (h->profiling) { cudaEvent_t b = get_event(h); cudaEventRecord(b, h->stream); h->prof.push_back({kind, a, b}); }
  }
};

// row-major C[M,N] (+)= A[M,K] * W, with W row-major [K,N] (w_is_nk = false) or [N,K] (true)
pd_status gemm(pd_handle *h, bool w_is_nk, int M, int N, int K, const void *A, const void *W, void *Cmat,
               bool c_is_f32, float beta) {
  ProfScope ps(h, PD_PROF_GEMM);
  const bool bf = h->cfg.dtype == PD_DTYPE_BF16;
  cudaDataType in_t = bf ? CUDA_R_16BF : CUDA_R_32F;
  cudaDataType c_t = (c_is_f32 || !bf) ? CUDA_R_32F : CUDA_R_16BF;
  cublasComputeType_t comp = bf ? CUBLAS_COMPUTE_32F : CUBLAS_COMPUTE_32F_PEDANTIC;
  float alpha = 1.f;
  cublasStatus_t s = cublasGemmEx(h->blas, w_is_nk ? CUBLAS_OP_T : CUBLAS_OP_N, CUBLAS_OP_N, N, M, K, &alpha, W, in_t,
                                  w_is_nk ? K : N, A, in_t, K, &beta, Cmat, c_t, N, comp, CUBLAS_GEMM_DEFAULT);
  if (s != CUBLAS_STATUS_SUCCESS) return fail(h, PD_ERR_CUDA, "cublasGemmEx failed with status " + std::to_string((int)s));
  h->gemm_calls++;
  return PD_OK;
}

void drop_ff_plan(pd_handle *h) {
  if (h->ff_w) cublasLtMatrixLayoutDestroy(h->ff_w);
  if (h->ff_a) cublasLtMatrixLayoutDestroy(h->ff_a);
  if (h->ff_c) cublasLtMatrixLayoutDestroy(h->ff_c);
  if (h->ff_desc) cublasLtMatmulDescDestroy(h->ff_desc);
  h->ff_w = h->ff_a = h->ff_c = nullptr; h->ff_desc = nullptr;
}

// relu(A[M,K] * W[K,N]) -> C[M,N] (row-major, bf16 in and out, fp32 accumulate) in one cuBLASLt
// call.  Returns false when no plan could be made (the caller then runs GEMM + ReLU kernel).
bool make_ff_plan(pd_handle *h, int M, int N, int K) {
  if (h->ff_rows == M) return true;
  if (h->ff_rows == -2 || h->cfg.dtype != PD_DTYPE_BF16 || !h->lt) return false;
  drop_ff_plan(h);
  h->ff_rows = -2;
  cublasLtEpilogue_t epi = CUBLASLT_EPILOGUE_RELU;
  cublasOperation_t opn = CUBLAS_OP_N;
  if (cublasLtMatmulDescCreate(&h->ff_desc, CUBLAS_COMPUTE_32F, CUDA_R_32F) != CUBLAS_STATUS_SUCCESS) return false;
  if (cublasLtMatmulDescSetAttribute(h->ff_desc, CUBLASLT_MATMUL_DESC_TRANSA, &opn, sizeof(opn)) != CUBLAS_STATUS_SUCCESS ||
      cublasLtMatmulDescSetAttribute(h->ff_desc, CUBLASLT_MATMUL_DESC_TRANSB, &opn, sizeof(opn)) != CUBLAS_STATUS_SUCCESS ||
      cublasLtMatmulDescSetAttribute(h->ff_desc, CUBLASLT_MATMUL_DESC_EPILOGUE, &epi, sizeof(epi)) != CUBLAS_STATUS_SUCCESS)
    return false;
  // column-major view: C^T[N,M] = W^T[N,K] * A^T[K,M]
  if (cublasLtMatrixLayoutCreate(&h->ff_w, CUDA_R_16BF, N, K, N) != CUBLAS_STATUS_SUCCESS ||
      cublasLtMatrixLayoutCreate(&h->ff_a, CUDA_R_16BF, K, M, K) != CUBLAS_STATUS_SUCCESS ||
      cublasLtMatrixLayoutCreate(&h->ff_c, CUDA_R_16BF, N, M, N) != CUBLAS_STATUS_SUCCESS)
    return false;
  cublasLtMatmulPreference_t pref = nullptr;
  if (cublasLtMatmulPreferenceCreate(&pref) != CUBLAS_STATUS_SUCCESS) return false;
  size_t ws = kCublasWs;
  cublasLtMatmulPreferenceSetAttribute(pref, CUBLASLT_MATMUL_PREF_MAX_WORKSPACE_BYTES, &ws, sizeof(ws));
  cublasLtMatmulHeuristicResult_t res;
  int found = 0;
  cublasStatus_t st = cublasLtMatmulAlgoGetHeuristic(h->lt, h->ff_desc, h->ff_w, h->ff_a, h->ff_c, h->ff_c, pref, 1, &res, &found);
  cublasLtMatmulPreferenceDestroy(pref);
  if (st != CUBLAS_STATUS_SUCCESS || found < 1) return false;
  h->ff_algo = res.algo;
  h->ff_rows = M;
  return true;
}

#define OWN(h, kind, expr)                          \
  do {                                              \
    ProfScope ps__(h, kind);                        \
    CU_TRY(h, expr);                                \
    h->own_launches++;                              \
  } while (0)

bool self_tc(const pd_handle *h) { return h->cfg.dtype == PD_DTYPE_BF16 && self_attn_tc_supported(h->dm); }
// The tensor-core attention kernel places the new cache entries itself: from the projection's bf16 output when
// nothing is rotated (1), from its fp32 output, rotating queries and keys first, in rotary mode (2).
// In rotary mode the fused form pays one more dependent fetch for every page that receives a new entry, which is
// most pages when a subsequence fits one page (measured on the keyphrase shape: 20.6 us against 16.7 + 2.0 us for the
// append launch); there the append kernel stays.
int fused_append(const pd_handle *h) {
  if (!self_tc(h)) return 0;
  if (h->dm.pos_mode != PD_POS_ROPE) return 1;
  return h->dm.PPS >= 2 ? 2 : 0;
}

AttnArgs attn_args(pd_handle *h, int layer, bool self) {
  AttnArgs a;
  a.dm = h->dm; a.st = h->st; a.layer = layer; a.batch = h->batch;
  a.splits = self ? h->self_splits : h->cross_splits;
  a.q = self ? h->ptr<void>(h->lay.qbuf) : h->ptr<void>(h->lay.cq);
  a.kv = self ? h->ptr<void>(h->lay.kv_pool) : h->ptr<void>(h->lay.kv_c);
  a.out = self ? h->ptr<void>(h->lay.self_out) : h->ptr<void>(h->lay.cross_out);
  a.part_o = h->ptr<float>(h->lay.part_o);
  a.part_ml = h->ptr<float>(h->lay.part_ml);
  a.dist_bucket = h->ptr<int32_t>(h->lay.dist_bucket);
  a.rel_bias = h->w.rel_bias;
  a.rel_buckets = h->cfg.rel_buckets;
  a.tickets = h->ptr<int32_t>(h->lay.state) + h->lay.w_xtick;
  a.bias_tab = h->cfg.pos_mode == PD_POS_T5_BIAS ? h->ptr<float>(h->lay.bias_tab) : nullptr;
  a.qkv = h->ptr<void>(h->lay.qkv);
  a.fused_append = self ? fused_append(h) : 0;
  a.rope_tab = h->ptr<float2>(h->lay.rope_tab);
  a.kv_scale = (!self && h->kv8) ? h->ptr<float>(h->lay.kv_scale) : nullptr;
  a.kv_seq = nullptr; a.row_base = nullptr;
  return a;
}

// Pipelined self-attention of one layer.  The tensor-core kernel appends the step's keys/values itself and
// merges its splits in the same launch; the plain-ALU kernel follows the append kernel and, when split,
// is followed by the merge kernel.
pd_status enqueue_self_attention(pd_handle *h, int layer) {
  const int dt = h->cfg.dtype;
  AttnArgs a = attn_args(h, layer, true);
  if (self_tc(h)) {
    CU_TRY(h, launch_self_attn_tc(a, h->stream));
    h->own_launches++;
    return PD_OK;
  }
  CU_TRY(h, launch_attn_core(a, dt, true, h->stream));
  h->own_launches++;
  if (a.splits > 1) { CU_TRY(h, launch_attn_merge(a, dt, h->stream)); h->own_launches++; }
  return PD_OK;
}

// Batched cross-attention of one layer.
pd_status enqueue_cross_attention(pd_handle *h, int layer) {
  const int dt = h->cfg.dtype;
  AttnArgs a = attn_args(h, layer, false);
  if (dt == PD_DTYPE_BF16 && h->have_tmap && cross_attn_tma_supported(h->dm, h->batch)) {
    CU_TRY(h, launch_cross_attn_tma(a, h->tmap_kvc, h->kv8 ? h->tmap_kvc_v : h->tmap_kvc, h->cross_ctas, h->stream));   // merges its own partials
    h->own_launches++;
    return PD_OK;
  }
  CU_TRY(h, launch_attn_core(a, dt, false, h->stream));
  h->own_launches++;
  if (a.splits > 1) { CU_TRY(h, launch_attn_merge(a, dt, h->stream)); h->own_launches++; }
  return PD_OK;
}

// The launch sequence of one decode step (one pass of Eq. 3 for all active rows + Algorithm 1's bookkeeping).
pd_status enqueue_step(pd_handle *h) {
  const Dims &dm = h->dm;
  const int dt = h->cfg.dtype;
  const int M = h->batch * dm.C;
  cudaStream_t s = h->stream;
  float *x = h->ptr<float>(h->lay.x);
  void *hb = h->ptr<void>(h->lay.hbuf);
  float *qkv = h->ptr<float>(h->lay.qkv);
  void *ffn = h->ptr<void>(h->lay.ffn);
  float *logits = h->ptr<float>(h->lay.logits);

  OWN(h, PD_PROF_OTHER, launch_embed(dm, h->st, h->batch, dt, h->w.embed, x, h->layer_w[0], hb, s));   // with the first layer's norm
  for (int l = 0; l < dm.L; ++l) {
    const void *const *lw = &h->layer_w[(size_t)l * kLayerTensors];
    if (l > 0) OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, dt, x, lw[0], hb, s));
    if (fused_append(h) != 0) {
      // the attention kernel takes queries, keys and values straight from the projection's output (bf16, or fp32
      // where it has to rotate them) and appends the new cache entries itself
      PD_TRY(gemm(h, false, M, 3 * dm.d, dm.d, hb, lw[1], qkv, fused_append(h) == 2, 0.f));
    } else if (dt == PD_DTYPE_BF16 && dm.pos_mode != PD_POS_ROPE) {
      // nothing to rotate: the projection rounds to bf16 itself and the append only places the rows
      PD_TRY(gemm(h, false, M, 3 * dm.d, dm.d, hb, lw[1], qkv, false, 0.f));
      OWN(h, PD_PROF_APPEND, launch_append_copy_bf16(dm, h->st, h->batch, l, qkv, h->ptr<void>(h->lay.qbuf),
                                                     h->ptr<void>(h->lay.kv_pool), s));
    } else {
      PD_TRY(gemm(h, false, M, 3 * dm.d, dm.d, hb, lw[1], qkv, true, 0.f));
      OWN(h, PD_PROF_APPEND, launch_append(dm, h->st, h->batch, l, dt, qkv, h->ptr<void>(h->lay.qbuf),
                                           h->ptr<void>(h->lay.kv_pool), h->ptr<float2>(h->lay.rope_tab), s));
    }
    {
      ProfScope ps(h, PD_PROF_SELF_ATTN);
      PD_TRY(enqueue_self_attention(h, l));
    }
    PD_TRY(gemm(h, false, M, dm.d, dm.d, h->ptr<void>(h->lay.self_out), lw[2], x, true, 1.f));
    OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, dt, x, lw[3], hb, s));
    PD_TRY(gemm(h, false, M, dm.d, dm.d, hb, lw[4], h->ptr<void>(h->lay.cq), false, 0.f));
    {
      ProfScope ps(h, PD_PROF_CROSS_ATTN);
      PD_TRY(enqueue_cross_attention(h, l));
    }
    PD_TRY(gemm(h, false, M, dm.d, dm.d, h->ptr<void>(h->lay.cross_out), lw[6], x, true, 1.f));
    OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, dt, x, lw[7], hb, s));
    if (make_ff_plan(h, M, dm.ff, dm.d)) {
      ProfScope ps(h, PD_PROF_GEMM);
      const float one = 1.f, zero = 0.f;
      if (cublasLtMatmul(h->lt, h->ff_desc, &one, lw[8], h->ff_w, hb, h->ff_a, &zero, ffn, h->ff_c, ffn, h->ff_c, &h->ff_algo,
                         h->ptr<void>(h->lay.cublas_ws), kCublasWs, s) != CUBLAS_STATUS_SUCCESS)
        return fail(h, PD_ERR_CUDA, "cublasLtMatmul (feed-forward up-projection with ReLU) failed");
      h->gemm_calls++;
    } else {
      PD_TRY(gemm(h, false, M, dm.ff, dm.d, hb, lw[8], ffn, false, 0.f));
      OWN(h, PD_PROF_OTHER, launch_relu(dt, ffn, (size_t)M * dm.ff, s));
    }
    PD_TRY(gemm(h, false, M, dm.d, dm.ff, ffn, lw[9], x, true, 1.f));
  }
  if (h->vocab_tc) {
    // active rows only, packed; logits stay in tensor memory unless they were asked for
    VocabArgs va;
    va.n_active = h->st.n_active; va.batch = h->batch; va.m_fixed = 0; va.V = dm.V; va.K = dm.d; va.rows_cap = M;
    va.eos = dm.eos; va.sep = dm.sep;
    va.part_val = h->ptr<float>(h->lay.vpart_val); va.part_idx = h->ptr<int32_t>(h->lay.vpart_idx);
    va.term_val = h->ptr<float>(h->lay.vterm);
    va.logits = h->cfg.store_logits ? logits : nullptr;
    va.status = h->st.hdr + HDR_STATUS;
    OWN(h, PD_PROF_OTHER, launch_rmsnorm_packed(dm, h->st, h->batch, dt, x, h->w.final_norm, hb, s));
    OWN(h, PD_PROF_VOCAB, launch_vocab_tc(h->vmaps, va, s));
    OWN(h, PD_PROF_ARGMAX_SCHED, launch_pick_sched(dm, h->st, h->batch, vocab_tc_tiles(dm.V), va.part_val, va.part_idx, va.term_val,
                                                   h->ptr<int32_t>(h->lay.teacher), s));
    return PD_OK;
  }
  OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, dt, x, h->w.final_norm, hb, s));
  PD_TRY(gemm(h, true, M, dm.V, dm.d, hb, h->w.lm_head, logits, true, 0.f));
  OWN(h, PD_PROF_ARGMAX_SCHED, launch_argmax_sched(dm, h->st, h->batch, logits, h->ptr<int32_t>(h->lay.teacher), s));
  return PD_OK;
}

int t5_bucket(int dist, int num_buckets, int max_dist) {
  int exact = num_buckets / 2;
  if (dist < exact) return dist;
  int b = exact + (int)floor(log((double)dist / exact) / log((double)max_dist / exact) * (num_buckets - exact));
  return b < num_buckets - 1 ? b : num_buckets - 1;
}

pd_status make_tensor_map(pd_handle *h) {
  const Dims &dm = h->dm;
  int code = 0;
  cudaError_t e = h->kv8 ? encode_ctx_kv8_tensor_maps(&h->tmap_kvc, &h->tmap_kvc_v, h->ptr<void>(h->lay.kv_c), (uint64_t)dm.L * dm.B * dm.H,
                                                      (uint64_t)dm.ctx, &code)
                         : encode_ctx_kv_tensor_map(&h->tmap_kvc, h->ptr<void>(h->lay.kv_c), (uint64_t)dm.L * dm.B * dm.H * 2 * dm.ctx, &code);
  if (e != cudaSuccess) return fail(h, PD_ERR_CUDA, std::string("tensor map for the context keys/values: ") + cudaGetErrorString(e) +
                                                    " (driver code " + std::to_string(code) + ")");
  h->have_tmap = true;
  return PD_OK;
}

void drop_graph(pd_handle *h) {
  if (h->graph_exec) { cudaGraphExecDestroy(h->graph_exec); h->graph_exec = nullptr; }
  h->graph_batch = -1;
}

pd_status device_status(pd_handle *h) {
  int32_t hdr[HDR_WORDS];
  CU_TRY(h, cudaMemcpyAsync(hdr, h->st.hdr, sizeof(hdr), cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  if (hdr[HDR_STATUS] != 0) return fail(h, (pd_status)hdr[HDR_STATUS], "device-side error " + std::to_string(hdr[HDR_STATUS]));
  return PD_OK;
}

pd_status encode_prepare(pd_handle *h, const int32_t *ctx_len, int32_t batch, const int32_t *forced_len);
pd_status encode_project(pd_handle *h, const void *enc_mem, int b0, int nb);

// Chunks of whole sequences the encoder memory is projected in: at least 32 MiB each (many small
// GEMMs cost pd_encode_context more than the overlap with the host copy returns to
// pd_generate_host), at most kMaxChunks.
int encode_chunks(const pd_handle *h, int batch) {
  const size_t seq_bytes = (size_t)h->dm.ctx * h->dm.d * (h->cfg.dtype == PD_DTYPE_BF16 ? 2 : 4);
  int n = (int)((size_t)batch * seq_bytes / ((size_t)32 << 20));
  if (n > pd_handle::kMaxChunks) n = pd_handle::kMaxChunks;
  if (n > batch) n = batch;
  return n < 1 ? 1 : n;
}

}  // namespace

extern "C" {

pd_status pd_config_check(const pd_config *cfg, const char **reason) {
  if (reason) *reason = "";
  if (!cfg) { if (reason) *reason = "null configuration"; return PD_ERR_ARG; }
  Dims dm; int ms;
  if (make_dims(*cfg, dm, ms)) return PD_OK;
  const char *why = unsupported_reason(*cfg);
  if (why) { if (reason) *reason = why; return PD_ERR_UNSUPPORTED; }
  if (reason) *reason = "a field is out of range (see pd_config in pd.h)";
  return PD_ERR_ARG;
}

size_t pd_workspace_bytes(const pd_config *cfg) {
  if (!cfg) return 0;
  Dims dm; int ms; Layout L;
  if (!make_dims(*cfg, dm, ms)) return 0;
  make_layout(*cfg, dm, ms, L);
  return L.total;
}

pd_status pd_init(const pd_config *cfg, const pd_weights *weights, void *workspace, size_t workspace_bytes,
                  void *cuda_stream, pd_handle **out) {
  if (!cfg || !weights || !workspace || !out) return PD_ERR_ARG;
  *out = nullptr;
  Dims dm; int ms;
  if (!make_dims(*cfg, dm, ms)) return pd_config_check(cfg, nullptr);
  if (!weights->embed || !weights->layer || !weights->final_norm || !weights->lm_head) return PD_ERR_ARG;
  if (cfg->pos_mode == PD_POS_T5_BIAS && !weights->rel_bias) return PD_ERR_ARG;
  for (int i = 0; i < cfg->n_layers * kLayerTensors; ++i) if (!weights->layer[i]) return PD_ERR_ARG;
  pd_handle *h = new pd_handle();
  h->cfg = *cfg; h->dm = dm; h->max_splits = ms;
  make_layout(*cfg, dm, ms, h->lay);
  if (workspace_bytes < h->lay.total || (reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0) { delete h; return PD_ERR_WORKSPACE; }
  h->ws = reinterpret_cast<uint8_t *>(workspace);
  h->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  h->w = *weights;
  h->layer_w.assign(weights->layer, weights->layer + (size_t)cfg->n_layers * kLayerTensors);
  h->w.layer = h->layer_w.data();
  auto bail = [&](pd_status s) { pd_destroy(h); return s; };
  if (cudaSetDevice(cfg->device) != cudaSuccess) return bail(PD_ERR_CUDA);
  if (cublasCreate(&h->blas) != CUBLAS_STATUS_SUCCESS) return bail(PD_ERR_CUDA);
  if (cublasSetStream(h->blas, h->stream) != CUBLAS_STATUS_SUCCESS) return bail(PD_ERR_CUDA);
  if (cublasLtCreate(&h->lt) != CUBLAS_STATUS_SUCCESS) h->lt = nullptr;     // optional: the ReLU then runs as its own kernel
  if (cublasSetWorkspace(h->blas, h->ptr<void>(h->lay.cublas_ws), kCublasWs) != CUBLAS_STATUS_SUCCESS) return bail(PD_ERR_CUDA);
  if (cublasSetMathMode(h->blas, CUBLAS_DEFAULT_MATH) != CUBLAS_STATUS_SUCCESS) return bail(PD_ERR_CUDA);
  if (cudaHostAlloc((void **)&h->pinned_flag, 64 * (1 + pd_handle::kRunSlots), cudaHostAllocDefault) != cudaSuccess) return bail(PD_ERR_CUDA);
  if (cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&h->ev_entry, cudaEventDisableTiming) != cudaSuccess) return bail(PD_ERR_CUDA);
  for (int c = 0; c < pd_handle::kMaxChunks; ++c)
    if (cudaEventCreateWithFlags(&h->ev_chunk[c], cudaEventDisableTiming) != cudaSuccess) return bail(PD_ERR_CUDA);
  for (int c = 0; c < pd_handle::kRunSlots; ++c)
    if (cudaEventCreateWithFlags(&h->ev_step[c], cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_snap[c], cudaEventDisableTiming) != cudaSuccess) return bail(PD_ERR_CUDA);

  int32_t *sb = h->ptr<int32_t>(h->lay.state);
  const Layout &L = h->lay;
  DecState &st = h->st;
  st.hdr = sb + L.w_hdr; st.stats = reinterpret_cast<unsigned long long *>(sb + L.w_stats);
  st.trace = reinterpret_cast<unsigned long long *>(sb + L.w_trace);
  st.k = sb + L.w_k; st.done = sb + L.w_done; st.steps = sb + L.w_steps; st.n_active = sb + L.w_nact;
  st.ctx_len = sb + L.w_ctx; st.seq_ticket = sb + L.w_ticket; st.crow = sb + L.w_crow; st.t0 = sb + L.w_t0;
  st.plist_n = sb + L.w_plist_n; st.plist = h->ptr<int4>(L.plist); st.row_meta = h->ptr<int4>(L.row_meta);
  st.start = sb + L.w_start; st.len = sb + L.w_len; st.state = sb + L.w_state; st.flag = sb + L.w_flag;
  st.last_tok = sb + L.w_last; st.forced_len = sb + L.w_forced; st.plan = sb + L.w_plan;
  st.row_sub = sb + L.w_row; st.prev_row_sub = sb + L.w_prow; st.row_tok = sb + L.w_rtok;
  st.page_table = sb + L.w_ptab; st.tokens = sb + L.w_tokens; st.chosen = sb + L.w_chosen;

  // tables: distance -> bucket (T5 causal bucketing) and (cos, sin) per position and frequency
  std::vector<int32_t> lut(dm.n_dist, 0);
  if (cfg->pos_mode == PD_POS_T5_BIAS)
    for (int d0 = 0; d0 < dm.n_dist; ++d0) lut[d0] = t5_bucket(d0, cfg->rel_buckets, cfg->rel_max_dist);
  std::vector<float2> rope((size_t)dm.n_dist * (kDh / 2));
  for (int p = 0; p < dm.n_dist; ++p)
    for (int j = 0; j < kDh / 2; ++j) {
      double ang = (double)p * pow((double)cfg->rope_theta, -2.0 * j / kDh);
      rope[(size_t)p * (kDh / 2) + j] = make_float2((float)cos(ang), (float)sin(ang));
    }
  if (cudaMemcpyAsync(h->ptr<void>(L.dist_bucket), lut.data(), lut.size() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
      cudaMemcpyAsync(h->ptr<void>(L.rope_tab), rope.data(), rope.size() * sizeof(float2), cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
      cudaMemsetAsync(h->ptr<void>(L.state), 0, L.state.bytes, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return bail(PD_ERR_CUDA);
  if (cfg->pos_mode == PD_POS_T5_BIAS &&
      (launch_build_bias_table(dm, weights->rel_bias, cfg->rel_buckets, h->ptr<int32_t>(L.dist_bucket), h->ptr<float>(L.bias_tab),
                               h->stream) != cudaSuccess || cudaStreamSynchronize(h->stream) != cudaSuccess))
    return bail(PD_ERR_CUDA);
  h->kv8 = cfg->kv_c_dtype == PD_KV_E4M3;
  if (cfg->dtype == PD_DTYPE_BF16 && dm.C <= 32) {
    pd_status s = make_tensor_map(h);
    if (s != PD_OK) return bail(s);
    if (cross_attn_tma_prepare() != cudaSuccess) return bail(PD_ERR_CUDA);
    h->cross_ctas = cross_attn_ctas();
  }
  if (cfg->dtype == PD_DTYPE_BF16 && self_attn_tc_supported(dm) && self_attn_tc_prepare() != cudaSuccess) return bail(PD_ERR_CUDA);
  if (cfg->dtype == PD_DTYPE_BF16 && vocab_tc_supported(dm.d, dm.V) && reinterpret_cast<uintptr_t>(weights->lm_head) % 16 == 0) {
    int code = 0;
    if (encode_vocab_maps(&h->vmaps, h->ptr<void>(L.hbuf), (uint64_t)dm.B * dm.C, weights->lm_head, (uint64_t)dm.V,
                          (uint64_t)dm.d, &code) != cudaSuccess)
      return bail(PD_ERR_CUDA);
    if (vocab_tc_prepare() != cudaSuccess) return bail(PD_ERR_CUDA);
    h->vocab_tc = true;
  }
  *out = h;
  return PD_OK;
}

pd_status pd_encode_context(pd_handle *h, const void *enc_mem, const int32_t *ctx_len, int32_t batch,
                            const int32_t *forced_len) {
  if (!h) return PD_ERR_ARG;
  if (!enc_mem) return fail(h, PD_ERR_ARG, "pd_encode_context: bad argument");
  PD_TRY(encode_prepare(h, ctx_len, batch, forced_len));
  // the same chunks of sequences as pd_generate_host, so that both project with the same GEMM shapes
  // and give bit-identical keys/values
  const size_t seq_bytes = (size_t)h->dm.ctx * h->dm.d * (h->cfg.dtype == PD_DTYPE_BF16 ? 2 : 4);
  const int n_chunks = encode_chunks(h, batch);
  for (int c = 0; c < n_chunks; ++c) {
    const int b0 = (int)((long long)batch * c / n_chunks), b1 = (int)((long long)batch * (c + 1) / n_chunks);
    PD_TRY(encode_project(h, static_cast<const uint8_t *>(enc_mem) + b0 * seq_bytes, b0, b1 - b0));
  }
  h->encoded = true;
  h->steps_enqueued = 0;
  return PD_OK;
}

}  // extern "C"

namespace {

// Everything of pd_encode_context but the projections: argument checks, split factors, state reset.
pd_status encode_prepare(pd_handle *h, const int32_t *ctx_len, int32_t batch, const int32_t *forced_len) {
  if (!ctx_len || batch < 1 || batch > h->dm.B) return fail(h, PD_ERR_ARG, "pd_encode_context: bad argument");
  const Dims &dm = h->dm;
  for (int b = 0; b < batch; ++b)
    if (ctx_len[b] < 1 || ctx_len[b] > dm.ctx) return fail(h, PD_ERR_ARG, "pd_encode_context: ctx_len out of range");
  if (forced_len)
    for (int i = 0; i < batch * dm.SM; ++i)
      if (forced_len[i] > dm.MSL) return fail(h, PD_ERR_ARG, "pd_encode_context: forced_len exceeds max_sub_len");
  CU_TRY(h, cudaSetDevice(h->cfg.device));
  cudaStream_t s = h->stream;
  const Layout &L = h->lay;
  CU_TRY(h, cudaMemcpyAsync(h->ptr<void>(L.ctx_len_in), ctx_len, (size_t)batch * 4, cudaMemcpyHostToDevice, s));
  if (forced_len)
    CU_TRY(h, cudaMemcpyAsync(h->ptr<void>(L.forced_in), forced_len, (size_t)batch * dm.SM * 4, cudaMemcpyHostToDevice, s));
  CU_TRY(h, cudaMemsetAsync(h->ptr<void>(L.teacher), 0xFF, L.teacher.bytes, s));
  h->teacher_clear = true;
  if (batch != h->batch) drop_graph(h);
  h->batch = batch;
  make_ff_plan(h, batch * dm.C, dm.ff, dm.d);   // host-side planning, kept out of any stream capture
  // split-K factors
  auto cdiv = [](int a, int b) { return (a + b - 1) / b; };
  const int bh = batch * dm.H;
  int ss = h->cfg.self_splits > 0 ? h->cfg.self_splits : cdiv(2 * 148, bh);
  if (ss > 8 && h->cfg.self_splits == 0) ss = 8;
  if (h->cfg.self_splits == 0 && self_tc(h)) ss = self_attn_tc_splits(dm, bh, h->cross_ctas / 2);   // the kernel uses as many of them as the lists need
  int cs = h->cfg.cross_splits;
  if (cs == 0) {
    int tiles = cdiv(dm.ctx, 128);
    cs = cdiv(4 * 148, bh);
    int cap = tiles / 2 > 1 ? tiles / 2 : 1;
    if (cs > cap) cs = cap;
  }
  if (ss > h->max_splits) ss = h->max_splits;
  if (cs > h->max_splits) cs = h->max_splits;
  if (ss != h->self_splits || cs != h->cross_splits) drop_graph(h);
  h->self_splits = ss < 1 ? 1 : ss;
  h->cross_splits = cs < 1 ? 1 : cs;

  OWN(h, PD_PROF_OTHER, launch_reset_state(dm, h->st, batch, h->ptr<int32_t>(L.ctx_len_in),
                                           forced_len ? h->ptr<int32_t>(L.forced_in) : nullptr, L.state_words,
                                           h->ptr<int32_t>(L.state), s));
  h->own_launches++;   // the reset is two launches
  return PD_OK;
}

// Cross-attention keys/values of every layer for sequences b0 .. b0 + nb - 1, whose encoder memory
// starts at enc_mem (device, [nb, max_ctx, d]).
pd_status encode_project(pd_handle *h, const void *enc_mem, int b0, int nb) {
  const Dims &dm = h->dm;
  const Layout &L = h->lay;
  for (int l = 0; l < dm.L; ++l) {
    PD_TRY(gemm(h, false, nb * dm.ctx, 2 * dm.d, dm.d, enc_mem, h->layer_w[(size_t)l * kLayerTensors + 5],
                h->ptr<void>(L.proj_stage), false, 0.f));
    if (h->kv8) {
      float *scale = h->ptr<float>(L.kv_scale);
      OWN(h, PD_PROF_OTHER, launch_ctx_kv_quantize(dm, b0, nb, l, h->ptr<void>(L.proj_stage), h->st.ctx_len, scale,
                                                   scale + (size_t)dm.L * dm.B * dm.H * 2, h->ptr<void>(L.kv_c), h->stream));
      h->own_launches++;   // two launches
    } else {
      OWN(h, PD_PROF_OTHER, launch_ctx_kv_relayout(dm, b0, nb, l, h->cfg.dtype, h->ptr<void>(L.proj_stage), h->ptr<void>(L.kv_c), h->stream));
    }
  }
  return PD_OK;
}

}  // namespace

extern "C" {


pd_status pd_step(pd_handle *h, const int32_t *teacher_tokens) {
  if (!h) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_step before pd_encode_context");
  CU_TRY(h, cudaSetDevice(h->cfg.device));
  const Layout &L = h->lay;
  if (teacher_tokens) {
    CU_TRY(h, cudaMemcpyAsync(h->ptr<void>(L.teacher), teacher_tokens, (size_t)h->batch * h->dm.SM * 4,
                              cudaMemcpyDeviceToDevice, h->stream));
    h->teacher_clear = false;
  } else if (!h->teacher_clear) {
    CU_TRY(h, cudaMemsetAsync(h->ptr<void>(L.teacher), 0xFF, L.teacher.bytes, h->stream));
    h->teacher_clear = true;
  }
  if (h->cfg.use_graph && !h->profiling) {
    if (!h->graph_exec) {
      cudaGraph_t g = nullptr;
      long long own0 = h->own_launches, gemm0 = h->gemm_calls;
      CU_TRY(h, cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal));
      pd_status s = enqueue_step(h);
      cudaError_t ce = cudaStreamEndCapture(h->stream, &g);
      h->graph_own = h->own_launches - own0; h->graph_gemm = h->gemm_calls - gemm0;
      h->own_launches = own0; h->gemm_calls = gemm0;
      if (s != PD_OK) { if (g) cudaGraphDestroy(g); return s; }
      CU_TRY(h, ce);
      cudaError_t ie = cudaGraphInstantiate(&h->graph_exec, g, 0);
      cudaGraphDestroy(g);
      CU_TRY(h, ie);
      h->graph_batch = h->batch;
    }
    CU_TRY(h, cudaGraphLaunch(h->graph_exec, h->stream));
    h->own_launches += h->graph_own; h->gemm_calls += h->graph_gemm;
  } else {
    PD_TRY(enqueue_step(h));
  }
  h->steps_enqueued++;
  return PD_OK;
}

pd_status pd_done(pd_handle *h, int32_t *all_done) {
  if (!h || !all_done) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_done before pd_encode_context");
  CU_TRY(h, cudaMemcpyAsync(h->pinned_flag, h->st.hdr, 8 * sizeof(int32_t), cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  *all_done = h->pinned_flag[HDR_ALL_DONE];
  if (h->pinned_flag[HDR_STATUS] != 0)
    return fail(h, (pd_status)h->pinned_flag[HDR_STATUS], "device-side error " + std::to_string(h->pinned_flag[HDR_STATUS]));
  return PD_OK;
}

pd_status pd_run(pd_handle *h, int32_t poll_every, int32_t *steps_run) {
  if (!h || poll_every < 1) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_run before pd_encode_context");
  // The host stays `lag` steps ahead of the device: before it enqueues step n + 1 it waits for the
  // header snapshot taken after step n + 1 - lag (the stream still holds lag - 1 steps of work then).
  const int lag = poll_every < 2 ? poll_every : 2;      // two is enough to keep the stream fed; more only adds steps past the end
  int n = 0;
  int32_t done = 0;
  while (h->steps_enqueued < h->dm.T && !done) {
    PD_TRY(pd_step(h, nullptr));
    const int slot = n % pd_handle::kRunSlots;
    int32_t *snap = h->pinned_flag + 16 * (1 + slot);
    CU_TRY(h, cudaEventRecord(h->ev_step[slot], h->stream));
    CU_TRY(h, cudaStreamWaitEvent(h->copy_stream, h->ev_step[slot], 0));
    CU_TRY(h, cudaMemcpyAsync(snap, h->st.hdr, 8 * sizeof(int32_t), cudaMemcpyDeviceToHost, h->copy_stream));
    CU_TRY(h, cudaEventRecord(h->ev_snap[slot], h->copy_stream));
    ++n;
    if (n >= lag) {
      const int old = (n - lag) % pd_handle::kRunSlots;
      CU_TRY(h, cudaEventSynchronize(h->ev_snap[old]));
      const int32_t *s_old = h->pinned_flag + 16 * (1 + old);
      if (s_old[HDR_STATUS] != 0) return fail(h, (pd_status)s_old[HDR_STATUS], "device-side error " + std::to_string(s_old[HDR_STATUS]));
      done = s_old[HDR_ALL_DONE];
    }
  }
  PD_TRY(pd_done(h, &done));
  if (steps_run) *steps_run = n;
  return PD_OK;
}

pd_status pd_collect(pd_handle *h, int32_t *tokens, int32_t *lens, int32_t *n_sub, int32_t *flags, int32_t *steps) {
  if (!h) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_collect before pd_encode_context");
  const Dims &dm = h->dm;
  const size_t nb = h->batch;
  cudaStream_t s = h->stream;
  if (tokens) CU_TRY(h, cudaMemcpyAsync(tokens, h->st.tokens, nb * dm.SM * dm.MSL * 4, cudaMemcpyDeviceToHost, s));
  if (lens) CU_TRY(h, cudaMemcpyAsync(lens, h->st.len, nb * dm.SM * 4, cudaMemcpyDeviceToHost, s));
  if (n_sub) CU_TRY(h, cudaMemcpyAsync(n_sub, h->st.k, nb * 4, cudaMemcpyDeviceToHost, s));
  if (flags) CU_TRY(h, cudaMemcpyAsync(flags, h->st.flag, nb * dm.SM * 4, cudaMemcpyDeviceToHost, s));
  if (steps) CU_TRY(h, cudaMemcpyAsync(steps, h->st.steps, nb * 4, cudaMemcpyDeviceToHost, s));
  return device_status(h);
}

pd_status pd_set_start_plan(pd_handle *h, const int32_t *plan) {
  if (!h || !plan) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_set_start_plan before pd_encode_context");
  if (h->steps_enqueued != 0) return fail(h, PD_ERR_STATE, "pd_set_start_plan after the first pd_step");
  const Dims &dm = h->dm;
  for (int b = 0; b < h->batch; ++b)
    for (int i = 0; i < dm.SM; ++i) {
      const int s_i = plan[b * dm.SM + i];
      if (i == 0 ? s_i != 1 : s_i - plan[b * dm.SM + i - 1] < dm.dt)
        return fail(h, PD_ERR_ARG, "pd_set_start_plan: a plan starts at step 1 and its start steps are at least delta_t apart");
    }
  CU_TRY(h, cudaSetDevice(h->cfg.device));
  CU_TRY(h, cudaMemcpyAsync(h->st.plan, plan, (size_t)h->batch * dm.SM * 4, cudaMemcpyHostToDevice, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));          // the host array may go
  return PD_OK;
}

pd_status pd_admit(pd_handle *h, int32_t row, const void *enc_mem, int32_t ctx_len, const int32_t *forced_len) {
  if (!h) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_admit before pd_encode_context");
  const Dims &dm = h->dm;
  if (!enc_mem || row < 0 || row >= h->batch || ctx_len < 1 || ctx_len > dm.ctx) return fail(h, PD_ERR_ARG, "pd_admit: bad argument");
  if (!dm.pool_static)
    return fail(h, PD_ERR_UNSUPPORTED, "pd_admit needs the default page pool (pool_pages = 0): a row's pages are then its own and start over with it");
  if (forced_len)
    for (int i = 0; i < dm.SM; ++i)
      if (forced_len[i] > dm.MSL) return fail(h, PD_ERR_ARG, "pd_admit: forced_len exceeds max_sub_len");
  CU_TRY(h, cudaSetDevice(h->cfg.device));
  const Layout &L = h->lay;
  int32_t *fl_dev = h->ptr<int32_t>(L.forced_in) + (size_t)row * dm.SM;
  if (forced_len) CU_TRY(h, cudaMemcpyAsync(fl_dev, forced_len, (size_t)dm.SM * 4, cudaMemcpyHostToDevice, h->stream));
  OWN(h, PD_PROF_OTHER, launch_admit_row(dm, h->st, row, ctx_len, forced_len ? fl_dev : nullptr, h->stream));
  return encode_project(h, enc_mem, row, 1);
}

pd_status pd_rows_done(pd_handle *h, int32_t *done, int32_t *steps) {
  if (!h || !done) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_rows_done before pd_encode_context");
  CU_TRY(h, cudaMemcpyAsync(done, h->st.done, (size_t)h->batch * 4, cudaMemcpyDeviceToHost, h->stream));
  if (steps) CU_TRY(h, cudaMemcpyAsync(steps, h->st.steps, (size_t)h->batch * 4, cudaMemcpyDeviceToHost, h->stream));
  return device_status(h);
}

pd_status pd_collect_row(pd_handle *h, int32_t row, int32_t *tokens, int32_t *lens, int32_t *n_sub, int32_t *flags, int32_t *steps) {
  if (!h) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_collect_row before pd_encode_context");
  if (row < 0 || row >= h->batch) return fail(h, PD_ERR_ARG, "pd_collect_row: bad row");
  const Dims &dm = h->dm;
  cudaStream_t s = h->stream;
  const size_t r = (size_t)row;
  if (tokens) CU_TRY(h, cudaMemcpyAsync(tokens, h->st.tokens + r * dm.SM * dm.MSL, (size_t)dm.SM * dm.MSL * 4, cudaMemcpyDeviceToHost, s));
  if (lens) CU_TRY(h, cudaMemcpyAsync(lens, h->st.len + r * dm.SM, (size_t)dm.SM * 4, cudaMemcpyDeviceToHost, s));
  if (n_sub) CU_TRY(h, cudaMemcpyAsync(n_sub, h->st.k + r, 4, cudaMemcpyDeviceToHost, s));
  if (flags) CU_TRY(h, cudaMemcpyAsync(flags, h->st.flag + r * dm.SM, (size_t)dm.SM * 4, cudaMemcpyDeviceToHost, s));
  if (steps) CU_TRY(h, cudaMemcpyAsync(steps, h->st.steps + r, 4, cudaMemcpyDeviceToHost, s));
  return device_status(h);
}

// ---- the teacher-forced forward of Eq. 6 -----------------------------------------------------------------
namespace {
constexpr int kTfGroup = 32;          // query rows per attention group
constexpr int kTfCrossBatch = 256;    // groups per cross-attention launch
struct TfLayout { size_t tables, x, hb, qkv, att, cq, co, ffn, logprob, part, tickets, logits, total; int logit_rows; };

TfLayout tf_layout(const Dims &dm, size_t rows, bool own_logits) {
  TfLayout L;
  size_t off = 0;
  auto reg = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, kAlign); return o; };
  const size_t groups = rows / 1 + (size_t)dm.B;                     // generous: every sequence may end with a short group
  L.tables = reg((4 * rows + 6 * groups) * sizeof(int32_t));
  L.x = reg(rows * dm.d * 4);
  L.hb = reg(rows * dm.d * 2);
  L.qkv = reg(rows * 3 * dm.d * 4);
  L.att = reg(rows * dm.d * 2);
  L.cq = reg(rows * dm.d * 2);
  L.co = reg(rows * dm.d * 2);
  L.ffn = reg(rows * dm.ff * 2);
  L.logprob = reg(rows * 4);
  L.part = reg(cross_attn_tma_partial_bytes(kMaxCrossCtas, kTfGroup));
  L.tickets = reg((size_t)kTfCrossBatch * dm.H * 4);
  L.logit_rows = 0;
  L.logits = off;
  if (own_logits) {
    size_t lr = ((size_t)256 << 20) / ((size_t)dm.V * 4);             // a logits chunk of about 256 MiB
    if (lr < 1) lr = 1;
    if (lr > rows) lr = rows;
    L.logit_rows = (int)lr;
    L.logits = reg(lr * dm.V * 4);
  }
  L.total = off;
  return L;
}
}  // namespace

size_t pd_teacher_forward_scratch_bytes(const pd_handle *h, int32_t max_rows, int32_t own_logits) {
  if (!h || max_rows < 1) return 0;
  return tf_layout(h->dm, (size_t)max_rows, own_logits != 0).total;
}

pd_status pd_teacher_forward(pd_handle *h, const int32_t *n_sub, const int32_t *lens, const int32_t *tokens,
                             const int32_t *terminators, void *scratch, size_t scratch_bytes, float *logprob, float *logits,
                             int32_t *rows_out, double *loss_out) {
  if (!h) return PD_ERR_ARG;
  if (!n_sub || !lens || !tokens || !scratch) return fail(h, PD_ERR_ARG, "pd_teacher_forward: null argument");
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_teacher_forward before pd_encode_context");
  const Dims &dm = h->dm;
  if (h->cfg.dtype != PD_DTYPE_BF16 || !h->have_tmap)
    return fail(h, PD_ERR_UNSUPPORTED, "pd_teacher_forward runs on the bf16 path (tensor-core cross-attention) only");
  if (reinterpret_cast<uintptr_t>(scratch) % kAlign != 0) return fail(h, PD_ERR_ARG, "pd_teacher_forward: misaligned scratch");
  // ---- rows in (sequence, subsequence, position) order; groups of up to 32 rows inside a sequence
  std::vector<int32_t> row_sub, row_tau, row_tok, row_tgt, g_row0, g_n, g_srow0, g_srows, g_seq, g_ctx;
  std::vector<int32_t> ctx_len(h->batch), plan((size_t)h->batch * dm.SM);
  CU_TRY(h, cudaMemcpyAsync(ctx_len.data(), h->st.ctx_len, (size_t)h->batch * 4, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaMemcpyAsync(plan.data(), h->st.plan, plan.size() * 4, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  for (int b = 0; b < h->batch; ++b) {
    if (n_sub[b] < 0 || n_sub[b] > dm.SM) return fail(h, PD_ERR_ARG, "pd_teacher_forward: n_sub out of range");
    const int srow0 = (int)row_sub.size();
    for (int i = 1; i <= n_sub[b]; ++i) {
      const int m = lens[b * dm.SM + i - 1];
      if (m < 0 || m > dm.MSL) return fail(h, PD_ERR_ARG, "pd_teacher_forward: subsequence length out of range");
      const int32_t *sub = tokens + ((size_t)b * dm.SM + i - 1) * dm.MSL;
      const int term = terminators ? terminators[b * dm.SM + i - 1] : dm.sep;
      for (int p = 0; p <= m; ++p) {
        const int tok = p == 0 ? dm.bos : sub[p - 1], tgt = p < m ? sub[p] : term;
        if (tok < 0 || tok >= dm.V || tgt < 0 || tgt >= dm.V) return fail(h, PD_ERR_ARG, "pd_teacher_forward: token id out of range");
        row_sub.push_back(i); row_tau.push_back(plan[(size_t)b * dm.SM + i - 1] - 1 + p); row_tok.push_back(tok); row_tgt.push_back(tgt);
      }
    }
    const int srows = (int)row_sub.size() - srow0;
    if (srows > 0 && plan[(size_t)b * dm.SM + n_sub[b] - 1] - 1 + dm.MSL + dm.SM >= dm.n_dist)
      return fail(h, PD_ERR_ARG, "pd_teacher_forward: positions beyond the tables");
    for (int r = 0; r < srows; r += kTfGroup) {
      g_row0.push_back(srow0 + r); g_n.push_back(std::min(kTfGroup, srows - r));
      g_srow0.push_back(srow0); g_srows.push_back(srows); g_seq.push_back(b); g_ctx.push_back(ctx_len[b]);
    }
  }
  const size_t R = row_sub.size(), G = g_row0.size();
  if (rows_out) *rows_out = (int32_t)R;
  if (loss_out) *loss_out = 0.0;
  if (R == 0) return PD_OK;
  const TfLayout L = tf_layout(dm, R, logits == nullptr);
  if (scratch_bytes < L.total) return fail(h, PD_ERR_WORKSPACE, "pd_teacher_forward: scratch too small (pd_teacher_forward_scratch_bytes)");
  CU_TRY(h, cudaSetDevice(h->cfg.device));
  cudaStream_t s = h->stream;
  uint8_t *base = reinterpret_cast<uint8_t *>(scratch);
  int32_t *tab = reinterpret_cast<int32_t *>(base + L.tables);
  int32_t *d_sub = tab, *d_tau = tab + R, *d_tok = tab + 2 * R, *d_tgt = tab + 3 * R, *d_g = tab + 4 * R;
  int32_t *d_grow0 = d_g, *d_gn = d_g + G, *d_gsrow0 = d_g + 2 * G, *d_gsrows = d_g + 3 * G, *d_gseq = d_g + 4 * G, *d_gctx = d_g + 5 * G;
  auto up = [&](int32_t *dst, const std::vector<int32_t> &v) { return cudaMemcpyAsync(dst, v.data(), v.size() * 4, cudaMemcpyHostToDevice, s); };
  CU_TRY(h, up(d_sub, row_sub)); CU_TRY(h, up(d_tau, row_tau)); CU_TRY(h, up(d_tok, row_tok)); CU_TRY(h, up(d_tgt, row_tgt));
  CU_TRY(h, up(d_grow0, g_row0)); CU_TRY(h, up(d_gn, g_n)); CU_TRY(h, up(d_gsrow0, g_srow0)); CU_TRY(h, up(d_gsrows, g_srows));
  CU_TRY(h, up(d_gseq, g_seq)); CU_TRY(h, up(d_gctx, g_ctx));
  CU_TRY(h, cudaMemsetAsync(base + L.tickets, 0, (size_t)kTfCrossBatch * dm.H * 4, s));
  CU_TRY(h, cudaStreamSynchronize(s));               // the host vectors may go

  float *x = reinterpret_cast<float *>(base + L.x);
  void *hb = base + L.hb, *qkv = base + L.qkv, *att = base + L.att, *cq = base + L.cq, *co = base + L.co, *ffn = base + L.ffn;
  const int M = (int)R;
  const bool rope = dm.pos_mode == PD_POS_ROPE;
  OWN(h, PD_PROF_OTHER, launch_gather_rows(M, dm.d, d_tok, h->w.embed, x, s));
  for (int l = 0; l < dm.L; ++l) {
    const void *const *lw = &h->layer_w[(size_t)l * kLayerTensors];
    OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, PD_DTYPE_BF16, x, lw[0], hb, s));
    PD_TRY(gemm(h, false, M, 3 * dm.d, dm.d, hb, lw[1], qkv, rope, 0.f));
    DenseAttnArgs da;
    da.H = dm.H; da.d = dm.d; da.n_groups = (int)G; da.scale_log2e = dm.scale_log2e;
    da.qkv = qkv; da.qkv_f32 = rope ? 1 : 0; da.out = reinterpret_cast<__nv_bfloat16 *>(att);
    da.row_sub = d_sub; da.row_tau = d_tau; da.grp_row0 = d_grow0; da.grp_n = d_gn; da.grp_seq_row0 = d_gsrow0; da.grp_seq_rows = d_gsrows;
    da.bias_tab = rope ? nullptr : h->ptr<float>(h->lay.bias_tab); da.n_dist = dm.n_dist;
    da.rope_tab = rope ? h->ptr<float2>(h->lay.rope_tab) : nullptr;
    OWN(h, PD_PROF_SELF_ATTN, launch_dense_self_attn(da, s));
    PD_TRY(gemm(h, false, M, dm.d, dm.d, att, lw[2], x, true, 1.f));
    OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, PD_DTYPE_BF16, x, lw[3], hb, s));
    PD_TRY(gemm(h, false, M, dm.d, dm.d, hb, lw[4], cq, false, 0.f));
    for (size_t g0 = 0; g0 < G; g0 += kTfCrossBatch) {              // groups as "sequences" of the batched kernel, 256 at a time
      AttnArgs a = attn_args(h, l, false);
      a.dm.C = kTfGroup;
      a.batch = (int)std::min<size_t>(kTfCrossBatch, G - g0);
      a.q = cq; a.out = co;
      a.st.n_active = d_gn + g0; a.st.ctx_len = d_gctx + g0;
      a.kv_seq = d_gseq + g0; a.row_base = d_grow0 + g0;
      a.part_o = reinterpret_cast<float *>(base + L.part);
      a.tickets = reinterpret_cast<int32_t *>(base + L.tickets);
      OWN(h, PD_PROF_CROSS_ATTN, launch_cross_attn_tma(a, h->tmap_kvc, h->kv8 ? h->tmap_kvc_v : h->tmap_kvc, h->cross_ctas, s));
    }
    PD_TRY(gemm(h, false, M, dm.d, dm.d, co, lw[6], x, true, 1.f));
    OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, PD_DTYPE_BF16, x, lw[7], hb, s));
    PD_TRY(gemm(h, false, M, dm.ff, dm.d, hb, lw[8], ffn, false, 0.f));
    OWN(h, PD_PROF_OTHER, launch_relu(PD_DTYPE_BF16, ffn, (size_t)M * dm.ff, s));
    PD_TRY(gemm(h, false, M, dm.d, dm.ff, ffn, lw[9], x, true, 1.f));
  }
  OWN(h, PD_PROF_OTHER, launch_rmsnorm(dm, M, PD_DTYPE_BF16, x, h->w.final_norm, hb, s));
  float *d_lp = reinterpret_cast<float *>(base + L.logprob);
  if (logits != nullptr) {
    PD_TRY(gemm(h, true, M, dm.V, dm.d, hb, h->w.lm_head, logits, true, 0.f));
    OWN(h, PD_PROF_OTHER, launch_target_logprob(M, dm.V, logits, d_tgt, d_lp, s));
  } else {
    float *chunk = reinterpret_cast<float *>(base + L.logits);
    for (int r0 = 0; r0 < M; r0 += L.logit_rows) {
      const int n = std::min(L.logit_rows, M - r0);
      PD_TRY(gemm(h, true, n, dm.V, dm.d, reinterpret_cast<uint8_t *>(hb) + (size_t)r0 * dm.d * 2, h->w.lm_head, chunk, true, 0.f));
      OWN(h, PD_PROF_OTHER, launch_target_logprob(n, dm.V, chunk, d_tgt + r0, d_lp + r0, s));
    }
  }
  std::vector<float> lp(R);
  CU_TRY(h, cudaMemcpyAsync(lp.data(), d_lp, R * 4, cudaMemcpyDeviceToHost, s));
  PD_TRY(device_status(h));
  double loss = 0.0;
  for (size_t r = 0; r < R; ++r) { loss -= (double)lp[r]; if (logprob) logprob[r] = lp[r]; }
  if (loss_out) *loss_out = loss;
  return PD_OK;
}

pd_status pd_generate_host(pd_handle *h, const void *enc_mem_host, const int32_t *ctx_len, int32_t batch,
                           const int32_t *forced_len, int32_t *tokens, int32_t *lens, int32_t *n_sub,
                           int32_t *flags, int32_t *steps) {
  if (!h || !enc_mem_host) return PD_ERR_ARG;
  if (batch < 1 || batch > h->dm.B) return fail(h, PD_ERR_ARG, "pd_generate_host: bad batch");
  const size_t e = h->cfg.dtype == PD_DTYPE_BF16 ? 2 : 4;
  CU_TRY(h, cudaSetDevice(h->cfg.device));
  // Chunks of whole sequences: chunk c is projected on the handle's stream while chunk c + 1 is still
  // crossing PCIe on the copy stream.
  const size_t seq_bytes = (size_t)h->dm.ctx * h->dm.d * e;
  const int n_chunks = encode_chunks(h, batch);
  CU_TRY(h, cudaEventRecord(h->ev_entry, h->stream));                  // the staging buffer is free once earlier work is done
  CU_TRY(h, cudaStreamWaitEvent(h->copy_stream, h->ev_entry, 0));
  uint8_t *stage = h->ptr<uint8_t>(h->lay.enc_stage);
  const uint8_t *src = static_cast<const uint8_t *>(enc_mem_host);
  for (int c = 0; c < n_chunks; ++c) {
    const int b0 = (int)((long long)batch * c / n_chunks), b1 = (int)((long long)batch * (c + 1) / n_chunks);
    CU_TRY(h, cudaMemcpyAsync(stage + b0 * seq_bytes, src + b0 * seq_bytes, (size_t)(b1 - b0) * seq_bytes, cudaMemcpyHostToDevice,
                              h->copy_stream));
    CU_TRY(h, cudaEventRecord(h->ev_chunk[c], h->copy_stream));
  }
  PD_TRY(encode_prepare(h, ctx_len, batch, forced_len));
  for (int c = 0; c < n_chunks; ++c) {
    const int b0 = (int)((long long)batch * c / n_chunks), b1 = (int)((long long)batch * (c + 1) / n_chunks);
    CU_TRY(h, cudaStreamWaitEvent(h->stream, h->ev_chunk[c], 0));
    PD_TRY(encode_project(h, stage + b0 * seq_bytes, b0, b1 - b0));
  }
  h->encoded = true;
  h->steps_enqueued = 0;
  int32_t n = 0;
  PD_TRY(pd_run(h, 8, &n));
  return pd_collect(h, tokens, lens, n_sub, flags, steps);
}

pd_status pd_get_trace(pd_handle *h, uint64_t *active_mask) {
  if (!h || !active_mask) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_get_trace before pd_encode_context");
  const Dims &dm = h->dm;
  std::vector<uint64_t> tmp((size_t)dm.T * dm.B);
  CU_TRY(h, cudaMemcpyAsync(tmp.data(), h->st.trace, tmp.size() * 8, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  for (int t = 0; t < dm.T; ++t)
    for (int b = 0; b < h->batch; ++b) active_mask[(size_t)t * h->batch + b] = tmp[(size_t)t * dm.B + b];
  return PD_OK;
}

pd_status pd_get_logits(pd_handle *h, float *logits, int32_t *row_sub) {
  if (!h) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_get_logits before pd_encode_context");
  const size_t rows = (size_t)h->batch * h->dm.C;
  if (h->vocab_tc && logits) {
    // The tensor-core projection stores the rows that were active, packed in (sequence, row) order.
    if (!h->cfg.store_logits) return fail(h, PD_ERR_STATE, "pd_get_logits: the handle was made with store_logits = 0");
    std::vector<int32_t> prs(rows);
    CU_TRY(h, cudaMemcpyAsync(prs.data(), h->st.prev_row_sub, rows * 4, cudaMemcpyDeviceToHost, h->stream));
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    const size_t row_bytes = (size_t)h->dm.V * 4;
    const uint8_t *src = h->ptr<uint8_t>(h->lay.logits);
    size_t packed = 0;
    for (size_t r = 0; r < rows; ++r) {
      if (prs[r] > 0) CU_TRY(h, cudaMemcpyAsync(logits + r * h->dm.V, src + packed++ * row_bytes, row_bytes, cudaMemcpyDeviceToHost, h->stream));
      else memset(logits + r * h->dm.V, 0, row_bytes);
    }
    if (row_sub) memcpy(row_sub, prs.data(), rows * 4);
    CU_TRY(h, cudaStreamSynchronize(h->stream));
    return PD_OK;
  }
  if (logits) CU_TRY(h, cudaMemcpyAsync(logits, h->ptr<void>(h->lay.logits), rows * h->dm.V * 4, cudaMemcpyDeviceToHost, h->stream));
  if (row_sub) CU_TRY(h, cudaMemcpyAsync(row_sub, h->st.prev_row_sub, rows * 4, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  return PD_OK;
}

pd_status pd_get_chosen(pd_handle *h, int32_t *chosen) {
  if (!h || !chosen) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_get_chosen before pd_encode_context");
  CU_TRY(h, cudaMemcpyAsync(chosen, h->st.chosen, (size_t)h->batch * h->dm.SM * (h->dm.MSL + 1) * 4, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  return PD_OK;
}

int32_t pd_rows_per_seq(const pd_handle *h) { return h ? h->dm.C : 0; }

pd_status pd_debug_read(pd_handle *h, int32_t which, void *dst_host, size_t max_bytes, size_t *bytes_out) {
  if (!h || !dst_host) return PD_ERR_ARG;
  const Layout &L = h->lay;
  const Region *r = nullptr;
  switch (which) {
    case PD_BUF_X: r = &L.x; break;
    case PD_BUF_QKV: r = &L.qkv; break;
    case PD_BUF_SELF_OUT: r = &L.self_out; break;
    case PD_BUF_CROSS_Q: r = &L.cq; break;
    case PD_BUF_CROSS_OUT: r = &L.cross_out; break;
    case PD_BUF_STATE: r = &L.state; break;
    default: return fail(h, PD_ERR_ARG, "pd_debug_read: unknown buffer");
  }
  size_t n = r->bytes < max_bytes ? r->bytes : max_bytes;
  CU_TRY(h, cudaMemcpyAsync(dst_host, h->ws + r->off, n, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  if (bytes_out) *bytes_out = n;
  return PD_OK;
}

pd_status pd_get_counters(const pd_handle *h, int64_t *own_kernel_launches, int64_t *gemm_calls) {
  if (!h) return PD_ERR_ARG;
  if (own_kernel_launches) *own_kernel_launches = h->own_launches;
  if (gemm_calls) *gemm_calls = h->gemm_calls;
  return PD_OK;
}

pd_status pd_reset_counters(pd_handle *h) {
  if (!h) return PD_ERR_ARG;
  h->own_launches = 0; h->gemm_calls = 0;
  return PD_OK;
}

pd_status pd_profile_enable(pd_handle *h, int32_t on) {
  if (!h) return PD_ERR_ARG;
  h->profiling = on != 0;
  return PD_OK;
}

pd_status pd_profile_read(pd_handle *h, double *ms, int64_t *launches) {
  if (!h || !ms || !launches) return PD_ERR_ARG;
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  for (int k = 0; k < PD_PROF_COUNT; ++k) { ms[k] = 0.0; launches[k] = 0; }
  for (const ProfRec &r : h->prof) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) { ms[r.kind] += t; launches[r.kind]++; }
    h->ev_pool.push_back(r.a); h->ev_pool.push_back(r.b);
  }
  h->prof.clear();
  return PD_OK;
}

pd_status pd_time_attention(pd_handle *h, int32_t which, int32_t reps, float *avg_us) {
  if (!h || !avg_us || reps < 1 || (which != PD_PROF_SELF_ATTN && which != PD_PROF_CROSS_ATTN)) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_time_attention before pd_encode_context");
  CU_TRY(h, cudaSetDevice(h->cfg.device));
  cudaEvent_t a = get_event(h), b = get_event(h);
  const long long own0 = h->own_launches;
  pd_status st = PD_OK;
  for (int rep = -1; rep < reps && st == PD_OK; ++rep) {       // rep -1 is a warm-up pass
    if (rep == 0) cudaEventRecord(a, h->stream);
    for (int l = 0; l < h->dm.L && st == PD_OK; ++l)
      st = which == PD_PROF_SELF_ATTN ? enqueue_self_attention(h, l) : enqueue_cross_attention(h, l);
  }
  cudaEventRecord(b, h->stream);
  cudaError_t e = cudaStreamSynchronize(h->stream);
  float ms = 0.f;
  if (st == PD_OK && e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
  h->ev_pool.push_back(a); h->ev_pool.push_back(b);
  h->own_launches = own0;
  if (st != PD_OK) return st;
  CU_TRY(h, e);
  *avg_us = 1e3f * ms / (float)((long long)reps * h->dm.L);
  return PD_OK;
}

pd_status pd_get_stats(pd_handle *h, int64_t *stats) {
  if (!h || !stats) return PD_ERR_ARG;
  if (!h->encoded) return fail(h, PD_ERR_STATE, "pd_get_stats before pd_encode_context");
  CU_TRY(h, cudaMemcpyAsync(stats, h->st.stats, PD_STAT_COUNT * 8, cudaMemcpyDeviceToHost, h->stream));
  CU_TRY(h, cudaStreamSynchronize(h->stream));
  return PD_OK;
}

const char *pd_last_error(const pd_handle *h) { return h ? h->err.c_str() : "null handle"; }
const char *pd_version(void) { return "pd-b200 0.1 (sm_100a)"; }

void pd_destroy(pd_handle *h) {
  if (!h) return;
  drop_graph(h);
  for (const ProfRec &r : h->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
  if (h->pinned_flag) cudaFreeHost(h->pinned_flag);
  for (cudaEvent_t e : h->ev_chunk) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_step) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_snap) if (e) cudaEventDestroy(e);
  if (h->ev_entry) cudaEventDestroy(h->ev_entry);
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  drop_ff_plan(h);
  if (h->lt) cublasLtDestroy(h->lt);
  if (h->blas) cublasDestroy(h->blas);
  delete h;
}

}  // extern "C"
