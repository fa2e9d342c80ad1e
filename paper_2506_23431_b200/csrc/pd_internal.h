// Internal declarations shared by the host API and the kernel translation units.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pd.h"

namespace pd {

constexpr int kDh = 64;          // head width the kernels are written for
constexpr int kMaxRows = 64;     // most subsequences active at once per sequence (sub_max <= 64)
constexpr int kLayerTensors = 10;
constexpr size_t kOpHeaderBytes = 256;   // header (HDR_* words) at the start of a stand-alone op's scratch

// KV pool layout: [layer][page][head][entry][K 64 | V 64].  One (page, head) block holds its
// entries one after the other, each the key row followed by the value row, so the first n entries
// of a block - all that exist in a partly filled page - are one contiguous run.  With 2-byte
// elements the eight 16-byte chunks of a row are stored swizzled (chunk c of entry e at chunk
// c ^ (e & 7)), so a linear copy of the run into shared memory is already in the layout ldmatrix
// reads without bank conflicts.  Offset of element (entry e, column c) of the key (is_v = 0) or
// value (is_v = 1) row inside a block:
template <typename T>
__host__ __device__ __forceinline__ size_t kv_entry_offset(int e, int c, int is_v) {
  const size_t row = ((size_t)e * 2 + is_v) * kDh;
  if (sizeof(T) == 2) return row + ((((c >> 3) ^ (e & 7)) << 3) | (c & 7));
  return row + c;
}
__host__ __device__ __forceinline__ size_t kv_block_offset(int layer, int pool, int page, int H, int h, int P) {
  return ((((size_t)layer * pool + page) * H + h) * 2) * P * kDh;
}

// Context keys/values layout: [layer][sequence][head][K | V][max_ctx][64] - all keys of one head
// of one sequence are contiguous (then its values), so a tile of consecutive positions is one
// contiguous block.  Element offset of (layer, b, h, K or V, position 0):
__host__ __device__ __forceinline__ size_t ctx_kv_offset(int layer, int B, int b, int H, int h, int is_v, int ctx) {
  return (((((size_t)layer * B + b) * H + h) * 2 + is_v) * ctx) * kDh;
}

// header words of the state block
enum { HDR_STEP_T = 0, HDR_ALL_DONE = 1, HDR_STATUS = 2, HDR_PAGE_BUMP = 3, HDR_BATCH = 4, HDR_N_DONE = 5,
       HDR_TICKET = 6, HDR_WORDS = 16 };
enum { SUB_NONE = 0, SUB_ACTIVE = 1, SUB_ENDED = 2 };

// Shapes and rule parameters every kernel may need; passed by value.
struct Dims {
  int L, d, H, ff, V;
  int B;        // max_batch
  int ctx;      // max_ctx
  int SM;       // sub_max
  int dt;       // delta_t
  int T;        // time_max
  int MSL;      // max_sub_len
  int C;        // rows per sequence
  int P;        // page_tokens
  int PPS;      // pages per subsequence
  int pool;     // pool pages
  int pool_static;  // the pool holds the worst case: page j of subsequence i of sequence b is page (b SM + i - 1) PPS + j, nothing is allocated
  int bos, eos, sep;
  int pos_mode;
  int n_dist;   // entries of the distance -> bucket table
  float scale_log2e;  // attn_scale * log2(e)
  float eps;
};

// Device pointers into the integer state block (all int32 unless noted).
struct DecState {
  int32_t *hdr;                 // [HDR_WORDS]
  unsigned long long *stats;    // [PD_STAT_COUNT]
  int32_t *k, *done, *steps, *n_active, *ctx_len, *seq_ticket;        // [B]
  int32_t *t0;                  // [B] the sequence's step origin: its own step t = header step - t0 (0 unless it was admitted later)
  int32_t *crow;                // [B] first row of the sequence among the step's active rows packed back to back
  int32_t *plist_n;             // [B] entries of the sequence's page list for the coming step
  int4 *row_meta;               // [B*C] per row: (page, slot in it, position tau + i) of the entry the coming step appends, subsequence i (0 = unused row)
  int4 *plist;                  // [B][SM*PPS] (page, entries in it, subsequence i', distance base t - (tau' + i') of entry 0)
  int32_t *start, *len, *state, *flag, *last_tok, *forced_len;        // [B*SM]
  int32_t *plan;                // [B*SM] step (of the sequence's own clock) at which subsequence i is to start; Eq. 2's (i-1) delta_t + 1 unless set
  int32_t *row_sub, *prev_row_sub, *row_tok;                          // [B*C]
  int32_t *page_table;          // [B*SM*PPS]
  int32_t *tokens;              // [B*SM*MSL]
  int32_t *chosen;              // [B*SM*(MSL+1)]
  unsigned long long *trace;    // [T*B]
};

// Arguments of the attention kernels (self and cross share the struct).
struct AttnArgs {
  Dims dm;
  DecState st;
  int layer, batch, splits;
  const void *q;            // [rows, d] dtype
  const void *kv;           // self: page pool base; cross: kv_c base [L][B*ctx][2d]
  void *out;                // [rows, d] dtype
  float *part_o;            // [rows, H, splits, 64]
  float *part_ml;           // [rows, H, splits, 2]
  const int32_t *dist_bucket;  // [n_dist]
  const float *rel_bias;       // [H, rel_buckets]
  int rel_buckets;
  const float *bias_tab;       // [H, n_dist]: rel_bias[h][bucket(dist)] * log2(e), or null
  int32_t *tickets;            // one arrival counter per (sequence, head), zero between launches
  // tensor-core self-attention with the step's KV-append inside it: the projection's output [rows][3 d] in
  // bf16 (fused_append = 1) or in fp32, to be rotated with rope_tab (fused_append = 2); 0 = the append kernel ran
  const void *qkv;
  int fused_append;
  const float2 *rope_tab;
  // cross-attention over 8-bit keys/values: [layer][sequence][head][keys | values] fp32 scales (else null)
  const float *kv_scale;
  // cross-attention over row groups that are not one per sequence (the teacher-forced forward: many rows per
  // sequence, in groups of up to 32): the sequence whose context group g reads, and the group's first row;
  // null = group g is sequence g with rows g * C ...
  const int32_t *kv_seq;
  const int32_t *row_base;
};

// ---- teacher-forced dense forward (teacher_kernels.cu) ------------------------------------------------
struct DenseAttnArgs {
  int H, d, n_groups;
  float scale_log2e;
  const void *qkv; int qkv_f32;          // [rows][3 d]: bf16, or fp32 (rotary mode: rotated here)
  __nv_bfloat16 *out;                    // [rows][d]
  const int32_t *row_sub, *row_tau;      // [rows] subsequence i and timestamp tau of every row
  const int32_t *grp_row0, *grp_n;       // [groups] first row and number of rows (<= 32) of a query group
  const int32_t *grp_seq_row0, *grp_seq_rows;   // [groups] first row and row count of the group's sequence (its keys)
  const float *bias_tab; int n_dist;     // T5 mode: [H][n_dist], log2(e)-scaled; else null
  const float2 *rope_tab;                // rotary mode: [n_dist][32] (cos, sin); else null
};
cudaError_t launch_dense_self_attn(const DenseAttnArgs &a, cudaStream_t s);
cudaError_t launch_gather_rows(int rows, int d, const int32_t *row_tok, const void *embed, float *x, cudaStream_t s);
cudaError_t launch_target_logprob(int rows, int V, const float *logits, const int32_t *targets, float *logprob, cudaStream_t s);

// ---- launchers (each enqueues on `s`; returns cudaGetLastError()) ------------------------
cudaError_t launch_reset_state(const Dims &dm, const DecState &st, int batch, const int32_t *ctx_len_dev,
                               const int32_t *forced_len_dev, size_t state_words, int32_t *state_base, cudaStream_t s);
cudaError_t launch_admit_row(const Dims &dm, const DecState &st, int row, int ctx_len, const int32_t *forced_len_dev, cudaStream_t s);
cudaError_t launch_embed(const Dims &dm, const DecState &st, int batch, int dtype, const void *embed, float *x, const void *gain,
                         void *h, cudaStream_t s);
cudaError_t launch_rmsnorm(const Dims &dm, int rows, int dtype, const float *x, const void *gain, void *out,
                           cudaStream_t s);
cudaError_t launch_rmsnorm_packed(const Dims &dm, const DecState &st, int batch, int dtype, const float *x, const void *gain,
                                  void *out, cudaStream_t s);
cudaError_t launch_relu(int dtype, void *buf, size_t n, cudaStream_t s);
cudaError_t launch_append(const Dims &dm, const DecState &st, int batch, int layer, int dtype, const float *qkv,
                          void *q_out, void *kv_pool, const float2 *rope_tab, cudaStream_t s);
cudaError_t launch_append_copy_bf16(const Dims &dm, const DecState &st, int batch, int layer, const void *qkv, void *q_out,
                                    void *kv_pool, cudaStream_t s);
cudaError_t launch_ctx_kv_relayout(const Dims &dm, int b0, int batch, int layer, int dtype, const void *proj, void *kv_c,
                                   cudaStream_t s);
cudaError_t launch_attn_core(const AttnArgs &a, int dtype, bool self, cudaStream_t s);
cudaError_t launch_attn_merge(const AttnArgs &a, int dtype, cudaStream_t s);
constexpr int kMaxCrossCtas = 320;      // persistent cross-attention CTAs (two per SM) the scratch is sized for
cudaError_t launch_cross_attn_tma(const AttnArgs &a, const CUtensorMap &tmap, const CUtensorMap &tmap_v, int n_ctas, cudaStream_t s);
cudaError_t encode_ctx_kv8_tensor_maps(CUtensorMap *map_k, CUtensorMap *map_v, const void *base, uint64_t n_blocks, uint64_t ctx,
                                       int *driver_code);
cudaError_t launch_ctx_kv_quantize(const Dims &dm, int b0, int batch, int layer, const void *proj, const int32_t *ctx_len_dev,
                                   float *scale, float *amax, void *kv8, cudaStream_t s);
size_t cross_attn_tma_partial_bytes(int n_ctas, int rows_per_seq);
bool cross_attn_tma_supported(const Dims &dm, int batch);
int cross_attn_ctas();                  // 2 x SM count of the current device, capped at kMaxCrossCtas
cudaError_t launch_build_bias_table(const Dims &dm, const float *rel_bias, int rel_buckets, const int32_t *dist_bucket,
                                    float *bias_tab, cudaStream_t s);
bool self_attn_tc_supported(const Dims &dm);
int self_attn_tc_splits(const Dims &dm, int pairs, int sms);
cudaError_t self_attn_tc_prepare();     // once per device, outside any stream capture
cudaError_t launch_self_attn_tc(const AttnArgs &a, cudaStream_t s);
cudaError_t launch_argmax_sched(const Dims &dm, const DecState &st, int batch, const float *logits,
                                const int32_t *teacher, cudaStream_t s);
cudaError_t launch_pick_sched(const Dims &dm, const DecState &st, int batch, int tiles, const float *part_val,
                              const int32_t *part_idx, const float *term_val, const int32_t *teacher, cudaStream_t s);
cudaError_t encode_ctx_kv_tensor_map(CUtensorMap *out, const void *base, uint64_t rows, int *driver_code);
int cross_attn_tma_smem_bytes();
cudaError_t cross_attn_tma_prepare();   // once per device, outside any stream capture


// ---- vocabulary projection + per-slice maxima on tcgen05 (vocab_tc.cu) -------------------------
struct VocabArgs {
  const int32_t *n_active;   // [batch] active rows per sequence (the rows of `hidden` are these, packed), or null
  int batch;
  int m_fixed;               // number of rows when n_active is null
  int V, K;                  // vocabulary size, model width (a multiple of 64)
  int rows_cap;              // row stride of the partial arrays (>= the largest row count)
  int wn;                    // vocabulary ids per CTA (set by the launcher: vocab_tc_slice(V))
  int eos, sep;              // ids kept out of the maxima (their logits go to term_val); -1 = none
  float *part_val;           // [tiles][rows_cap] maximum of the row over the tile's ids
  int32_t *part_idx;         // [tiles][rows_cap] the id that holds it (lowest on ties; INT_MAX = none)
  float *term_val;           // [rows_cap][2] logits of eos and sep
  float *logits;             // [rows][V] fp32, or null when nobody reads them
  int32_t *status;           // error word (PD_ERR_TIMEOUT on an expired wait)
};
struct VocabMaps { CUtensorMap a, a32, b; };   // hidden rows (128-row and 32-row boxes), lm_head (one slice per box)
int vocab_tc_slice(int V);
int vocab_tc_tiles(int V);
bool vocab_tc_supported(int K, int V);
cudaError_t vocab_tc_prepare();          // once per device, outside any stream capture
cudaError_t encode_vocab_maps(VocabMaps *m, const void *hidden, uint64_t rows, const void *lm_head, uint64_t vocab, uint64_t K,
                              int *driver_code);
cudaError_t launch_vocab_tc(const VocabMaps &m, const VocabArgs &a, cudaStream_t s);

// ---- skinny-M linear layers on tcgen05 (linear_tc.cu) --------------------------------------------
enum { LIN_EPI_STORE = 0,   // out = bf16(acc * row_scale)
       LIN_EPI_RELU = 1,    // out = bf16(max(acc * row_scale, 0))
       LIN_EPI_RESID = 2 }; // x += acc (fp32 residual stream); xg = bf16(x * gain_next); partial sums of x^2 per row
struct LinearArgs {
  int K, N;                  // the weight is [N][K] (K contiguous)
  int BN, ksplit;            // columns per CTA; CTAs (one cluster) along K
  const int32_t *rows_dev;   // device word holding the number of packed rows, or null
  int rows_fixed;            // number of rows when rows_dev is null
  int rows_cap;              // rows the row-indexed buffers are allocated for
  int rows_per_cta;          // rows per CTA along grid.z (a multiple of 32; CTAs beyond the row count leave at once)
  int epi;                   // LIN_EPI_*
  // row scale of the RMSNorm in front of the layer (null: none): rsqrt(sum_p ssq_in[p][m] * inv_width + eps)
  const float *ssq_in; int parts_in; float inv_width, eps;
  __nv_bfloat16 *out;        // STORE / RELU: [rows][N]
  float *x;                  // RESID: fp32 [rows][N], read and written
  __nv_bfloat16 *xg;         // RESID: bf16 [rows][N] = x * gain_next (input of the next layer's GEMM)
  const __nv_bfloat16 *gain_next;  // RESID: [N]
  float *ssq_out;            // RESID: [(N / BN) * ksplit][rows_cap] partial sums of squares of the new x, or null
  int32_t *status;           // error word (PD_ERR_TIMEOUT on an expired wait)
};
int linear_tc_smem_bytes();
bool linear_tc_plan(int N, int K, int sms, int *BN_out, int *ksplit_out);
cudaError_t linear_tc_prepare();         // once per device, outside any stream capture
struct LinearActMaps { CUtensorMap full, part; };   // boxes of 128 rows and of 32 rows over the same activations
cudaError_t encode_linear_act_maps(LinearActMaps *out, const void *act, uint64_t rows, uint64_t K, int *driver_code);
cudaError_t encode_linear_weight_map(CUtensorMap *out, const void *w_nk, uint64_t N, uint64_t K, int BN, int *driver_code);
cudaError_t launch_linear_tc(const LinearActMaps &map_a, const CUtensorMap &map_w, const LinearArgs &a, bool pdl, cudaStream_t s);
cudaError_t launch_transpose_bf16(int K, int N, const void *w, void *wt, cudaStream_t s);

// ---- stand-alone cross-attention (attn_ops.cu) ---------------------------------------------
size_t cross_attention_scratch_layout(int dtype, int batch, int rows_per_seq, int n_heads, int splits, size_t *off_tickets,
                                      size_t *off_part_o, size_t *off_part_ml);
bool cross_attention_args_ok(int dtype, int batch, int rows_per_seq, int n_heads, int max_ctx, float attn_scale, int splits);
pd_status cross_attention_enqueue(int dtype, int batch, int rows_per_seq, int n_heads, int max_ctx, float attn_scale,
                                  int splits, const void *q, const void *kv, const int32_t *n_rows, const int32_t *ctx_len,
                                  void *out, void *scratch, cudaStream_t s);

}  // namespace pd
