// Stand-alone entry point for the batched cross-attention step: the same kernels pd_step
// launches, on caller-supplied queries and context keys/values, without a decoder handle.
#include <string.h>

#include "pd_internal.h"

using namespace pd;

namespace pd {

// Scratch of the stand-alone op: header, arrival counters, partial results.  The flat partial records
// of the tensor-core kernel are only reserved where that kernel can run (bf16, at most 32 rows per
// sequence); the plain-ALU kernel needs the split-K records alone.
size_t cross_attention_scratch_layout(int dtype, int batch, int rows_per_seq, int n_heads, int splits, size_t *off_tickets,
                                      size_t *off_part_o, size_t *off_part_ml) {
  const size_t rows = (size_t)batch * rows_per_seq;
  size_t off = kOpHeaderBytes;
  if (off_tickets) *off_tickets = off;
  off += ((size_t)batch * n_heads * sizeof(int32_t) + 255) / 256 * 256;      // cleared with the header
  if (off_part_o) *off_part_o = off;
  const size_t split_bytes = rows * n_heads * splits * kDh * sizeof(float);
  const bool tensor_core = dtype == PD_DTYPE_BF16 && rows_per_seq <= 32;
  const size_t flat_bytes = tensor_core ? cross_attn_tma_partial_bytes(kMaxCrossCtas, rows_per_seq) : 0;
  off += ((split_bytes > flat_bytes ? split_bytes : flat_bytes) + 255) / 256 * 256;
  if (off_part_ml) *off_part_ml = off;
  off += (rows * n_heads * splits * 2 * sizeof(float) + 255) / 256 * 256;
  return off;
}

bool cross_attention_args_ok(int dtype, int batch, int rows_per_seq, int n_heads, int max_ctx, float attn_scale,
                             int splits) {
  if (dtype != PD_DTYPE_FP32 && dtype != PD_DTYPE_BF16) return false;
  if (batch < 1 || batch > 65535 || rows_per_seq < 1 || rows_per_seq > kMaxRows) return false;
  if (n_heads < 1 || n_heads > 65535 || max_ctx < 1) return false;
  if (splits < 1 || splits > 32 || !(attn_scale > 0.f)) return false;
  if ((unsigned long long)batch * n_heads * 2 * max_ctx > 0x7fffffffull) return false;
  return true;
}

// Enqueues the cross-attention kernels on `scratch` (already known to be large enough).
pd_status cross_attention_enqueue(int dtype, int batch, int rows_per_seq, int n_heads, int max_ctx, float attn_scale,
                                  int splits, const void *q, const void *kv, const int32_t *n_rows,
                                  const int32_t *ctx_len, void *out, void *scratch, cudaStream_t s) {
  size_t off_t = 0, off_o = 0, off_ml = 0;
  cross_attention_scratch_layout(dtype, batch, rows_per_seq, n_heads, splits, &off_t, &off_o, &off_ml);
  uint8_t *base = reinterpret_cast<uint8_t *>(scratch);
  if (cudaMemsetAsync(base, 0, off_o, s) != cudaSuccess) return PD_ERR_CUDA;      // header and arrival counters

  AttnArgs a;
  memset(&a, 0, sizeof(a));
  Dims &dm = a.dm;
  dm.L = 1; dm.H = n_heads; dm.d = n_heads * kDh; dm.B = batch; dm.ctx = max_ctx; dm.C = rows_per_seq;
  dm.SM = rows_per_seq; dm.pos_mode = PD_POS_ROPE;   // no positional term in cross-attention
  dm.scale_log2e = attn_scale * 1.4426950408889634f;
  a.st.hdr = reinterpret_cast<int32_t *>(base);
  a.st.n_active = const_cast<int32_t *>(n_rows);
  a.st.ctx_len = const_cast<int32_t *>(ctx_len);
  a.layer = 0; a.batch = batch; a.splits = splits;
  a.q = q; a.kv = kv; a.out = out;
  a.part_o = reinterpret_cast<float *>(base + off_o);
  a.part_ml = reinterpret_cast<float *>(base + off_ml);
  a.tickets = reinterpret_cast<int32_t *>(base + off_t);

  cudaError_t e;
  if (dtype == PD_DTYPE_BF16 && cross_attn_tma_supported(dm, batch)) {
    CUtensorMap tmap;
    if (encode_ctx_kv_tensor_map(&tmap, kv, (uint64_t)batch * n_heads * 2 * max_ctx, nullptr) != cudaSuccess) return PD_ERR_CUDA;
    if (cross_attn_tma_prepare() != cudaSuccess) return PD_ERR_CUDA;
    return launch_cross_attn_tma(a, tmap, tmap, cross_attn_ctas(), s) == cudaSuccess ? PD_OK : PD_ERR_CUDA;
  }
  e = launch_attn_core(a, dtype, false, s);
  if (e != cudaSuccess) return PD_ERR_CUDA;
  if (splits > 1 && launch_attn_merge(a, dtype, s) != cudaSuccess) return PD_ERR_CUDA;
  return PD_OK;
}

}  // namespace pd

extern "C" {

size_t pd_cross_attention_scratch_bytes(int32_t batch, int32_t rows_per_seq, int32_t n_heads, int32_t splits) {
  if (!cross_attention_args_ok(PD_DTYPE_BF16, batch, rows_per_seq, n_heads, 1, 1.f, splits)) return 0;
  return cross_attention_scratch_layout(PD_DTYPE_BF16, batch, rows_per_seq, n_heads, splits, nullptr, nullptr, nullptr);   // the larger of the two types
}

pd_status pd_cross_attention(int32_t dtype, int32_t batch, int32_t rows_per_seq, int32_t n_heads, int32_t max_ctx,
                             float attn_scale, int32_t splits, const void *q, const void *kv, const int32_t *n_rows,
                             const int32_t *ctx_len, void *out, void *scratch, size_t scratch_bytes, void *cuda_stream) {
  if (!q || !kv || !n_rows || !ctx_len || !out || !scratch) return PD_ERR_ARG;
  if (!cross_attention_args_ok(dtype, batch, rows_per_seq, n_heads, max_ctx, attn_scale, splits)) return PD_ERR_ARG;
  if (reinterpret_cast<uintptr_t>(kv) % 16 != 0 || reinterpret_cast<uintptr_t>(q) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(out) % 16 != 0 || reinterpret_cast<uintptr_t>(scratch) % 256 != 0) return PD_ERR_ARG;
  if (scratch_bytes < cross_attention_scratch_layout(dtype, batch, rows_per_seq, n_heads, splits, nullptr, nullptr, nullptr))
    return PD_ERR_WORKSPACE;
  return cross_attention_enqueue(dtype, batch, rows_per_seq, n_heads, max_ctx, attn_scale, splits, q, kv, n_rows, ctx_len,
                                 out, scratch, reinterpret_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
