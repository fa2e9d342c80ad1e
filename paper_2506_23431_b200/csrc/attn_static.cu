// Cross-attention for callers that cannot allocate device memory: the split-K partials live in
// a fixed array that is part of the library image instead of a caller-supplied scratch buffer.
#include <stdio.h>

#include <mutex>

#include "pd_internal.h"

using namespace pd;

namespace {

constexpr size_t kStaticScratchBytes = (size_t)8 << 20;   // 8 MiB, resident on every device that loads the library
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// functions, never a device address: kernels get the address cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mu;
void *g_scratch_addr[kMaxDevices] = {nullptr};     // per device, filled on first use
thread_local char g_err[256] = "";

pd_status fail(pd_status s, const char *fmt, long long a = 0, long long b = 0) {
  snprintf(g_err, sizeof(g_err), fmt, a, b);
  return s;
}

// Looks up (once per device, with that device current) where the array lives on the device.
pd_status static_scratch(void **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(PD_ERR_CUDA, "cudaGetDevice failed (CUDA error %lld)", (long long)e);
  if (dev < 0 || dev >= kMaxDevices) return fail(PD_ERR_UNSUPPORTED, "device ordinal %lld is beyond the %lld supported", dev, kMaxDevices);
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) return fail(PD_ERR_CUDA, "cudaGetSymbolAddress for the built-in scratch failed (CUDA error %lld)", (long long)e);
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return PD_OK;
}

}  // namespace

extern "C" {

size_t pd_cross_attention_static_max_bytes(void) { return kStaticScratchBytes; }

const char *pd_static_last_error(void) { return g_err; }

pd_status pd_cross_attention_static(int32_t dtype, int32_t batch, int32_t rows_per_seq, int32_t n_heads, int32_t max_ctx,
                                    float attn_scale, int32_t splits, const void *q, const void *kv,
                                    const int32_t *n_rows, const int32_t *ctx_len, void *out, void *cuda_stream) {
  g_err[0] = 0;
  if (!q || !kv || !n_rows || !ctx_len || !out) return fail(PD_ERR_ARG, "null pointer argument");
  if (!cross_attention_args_ok(dtype, batch, rows_per_seq, n_heads, max_ctx, attn_scale, splits))
    return fail(PD_ERR_ARG, "a size or parameter is out of range");
  if (reinterpret_cast<uintptr_t>(kv) % 16 != 0 || reinterpret_cast<uintptr_t>(q) % 16 != 0 || reinterpret_cast<uintptr_t>(out) % 16 != 0)
    return fail(PD_ERR_ARG, "q, kv and out must be 16-byte aligned");
  const size_t need = cross_attention_scratch_layout(dtype, batch, rows_per_seq, n_heads, splits, nullptr, nullptr, nullptr);
  if (need > kStaticScratchBytes)
    return fail(PD_ERR_WORKSPACE, "these sizes need %lld bytes of scratch; the built-in scratch holds %lld "
                                  "(fewer splits, fewer sequences or rows per call, or pd_cross_attention with a buffer of your own)",
                (long long)need, (long long)kStaticScratchBytes);
  void *scratch = nullptr;
  pd_status s = static_scratch(&scratch);
  if (s != PD_OK) return s;
  // The header (status word) is cleared inside the enqueue; the partials of every active row are
  // rewritten before the merge reads them, so nothing else of the previous call's contents matters.
  s = cross_attention_enqueue(dtype, batch, rows_per_seq, n_heads, max_ctx, attn_scale, splits, q, kv, n_rows, ctx_len, out,
                              scratch, reinterpret_cast<cudaStream_t>(cuda_stream));
  if (s != PD_OK) return fail(s, "enqueueing the cross-attention kernels failed (pd_status %lld)", (long long)s);
  return PD_OK;
}

pd_status pd_cross_attention_static_status(void *cuda_stream, int32_t *status_out) {
  g_err[0] = 0;
  if (!status_out) return fail(PD_ERR_ARG, "null pointer argument");
  void *scratch = nullptr;
  pd_status s = static_scratch(&scratch);
  if (s != PD_OK) return s;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  int32_t word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, reinterpret_cast<const int32_t *>(scratch) + HDR_STATUS, sizeof(word), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return fail(PD_ERR_CUDA, "reading the status word failed (CUDA error %lld)", (long long)e);
  *status_out = word;
  return PD_OK;
}

}  // extern "C"
