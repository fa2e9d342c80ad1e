// Stand-alone entry point for the vocabulary projection + greedy choice: the tcgen05 kernel that
// pd_step uses for the last stage of a decode step, on caller-supplied hidden rows, without a
// decoder handle.
#include <limits.h>

#include "pd_internal.h"

using namespace pd;

namespace {

struct VocabScratch { size_t off_part_val, off_part_idx, off_term, total; };

VocabScratch vocab_scratch_layout(int rows, int vocab) {
  VocabScratch L;
  const size_t tiles = (size_t)vocab_tc_tiles(vocab);
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  size_t off = kOpHeaderBytes;
  L.off_part_val = off; off += up(tiles * rows * sizeof(float));
  L.off_part_idx = off; off += up(tiles * rows * sizeof(int32_t));
  L.off_term = off; off += up((size_t)rows * 2 * sizeof(float));
  L.total = off;
  return L;
}

// One warp per row: the maximum over the tiles' partial maxima, ties to the lowest id.
__global__ void vocab_reduce_kernel(int rows, int tiles, int rows_cap, const float *__restrict__ part_val,
                                    const int32_t *__restrict__ part_idx, int32_t *__restrict__ best_id,
                                    float *__restrict__ best_val) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  float bv = -INFINITY;
  int bi = INT_MAX;
  for (int t = lane; t < tiles; t += 32) {
    const float v = part_val[(size_t)t * rows_cap + row];
    const int i = part_idx[(size_t)t * rows_cap + row];
    if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
  }
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  if (lane == 0) { best_id[row] = bi == INT_MAX ? 0 : bi; if (best_val) best_val[row] = bv; }
}

bool vocab_args_ok(int rows, int d_model, int vocab) {
  return rows >= 1 && rows <= (1 << 20) && vocab >= 1 && vocab_tc_supported(d_model, vocab) &&
         (unsigned long long)rows * vocab <= 0x7fffffffffffull;
}

}  // namespace

extern "C" {

size_t pd_vocab_argmax_scratch_bytes(int32_t rows, int32_t vocab) {
  if (rows < 1 || vocab < 1) return 0;
  return vocab_scratch_layout(rows, vocab).total;
}

pd_status pd_vocab_argmax(int32_t rows, int32_t d_model, int32_t vocab, const void *hidden, const void *lm_head,
                          int32_t *best_id, float *best_val, float *logits, void *scratch, size_t scratch_bytes,
                          void *cuda_stream) {
  if (!hidden || !lm_head || !best_id || !scratch) return PD_ERR_ARG;
  if (!vocab_args_ok(rows, d_model, vocab)) return PD_ERR_ARG;
  if (reinterpret_cast<uintptr_t>(hidden) % 16 != 0 || reinterpret_cast<uintptr_t>(lm_head) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(scratch) % 256 != 0) return PD_ERR_ARG;
  const VocabScratch L = vocab_scratch_layout(rows, vocab);
  if (scratch_bytes < L.total) return PD_ERR_WORKSPACE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint8_t *base = reinterpret_cast<uint8_t *>(scratch);
  if (cudaMemsetAsync(base, 0, kOpHeaderBytes, s) != cudaSuccess) return PD_ERR_CUDA;    // status word

  VocabMaps maps;
  if (encode_vocab_maps(&maps, hidden, (uint64_t)rows, lm_head, (uint64_t)vocab, (uint64_t)d_model, nullptr) != cudaSuccess)
    return PD_ERR_CUDA;
  if (vocab_tc_prepare() != cudaSuccess) return PD_ERR_CUDA;
  VocabArgs a;
  a.n_active = nullptr; a.batch = 0; a.m_fixed = rows; a.V = vocab; a.K = d_model; a.rows_cap = rows;
  a.eos = -1; a.sep = -1;
  a.part_val = reinterpret_cast<float *>(base + L.off_part_val);
  a.part_idx = reinterpret_cast<int32_t *>(base + L.off_part_idx);
  a.term_val = reinterpret_cast<float *>(base + L.off_term);
  a.logits = logits;
  a.status = reinterpret_cast<int32_t *>(base) + HDR_STATUS;
  if (launch_vocab_tc(maps, a, s) != cudaSuccess) return PD_ERR_CUDA;
  const int warps = 8;
  vocab_reduce_kernel<<<(rows + warps - 1) / warps, warps * 32, 0, s>>>(rows, vocab_tc_tiles(vocab), rows, a.part_val, a.part_idx,
                                                                         best_id, best_val);
  return cudaGetLastError() == cudaSuccess ? PD_OK : PD_ERR_CUDA;
}

}  // extern "C"
