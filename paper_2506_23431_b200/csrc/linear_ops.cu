// Stand-alone entry point for one linear layer of the decoder stack on the tcgen05 kernel that
// pd_step uses for its projections, on caller-supplied tensors and without a decoder handle.
#include <string.h>

#include "pd_internal.h"

using namespace pd;

extern "C" {

size_t pd_linear_scratch_bytes(int32_t d_in, int32_t d_out) {
  if (d_in < 64 || d_out < 16 || d_in % 64 || d_out % 16) return 0;
  return kOpHeaderBytes + ((size_t)d_in * d_out * 2 + 255) / 256 * 256;
}

int32_t pd_linear_sumsq_parts(int32_t d_in, int32_t d_out) {
  int dev = 0, sms = 148, BN = 0, ks = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (!linear_tc_plan(d_out, d_in, sms, &BN, &ks)) return 0;
  return (d_out / BN) * ks;
}

pd_status pd_linear(int32_t rows, int32_t d_in, int32_t d_out, int32_t mode, const void *a, const void *w, const float *row_sumsq,
                    float eps, void *out, float *x, const void *gain_next, void *xg, float *sumsq_out, int32_t *sumsq_parts,
                    void *scratch, size_t scratch_bytes, void *cuda_stream) {
  if (!a || !w || !scratch || rows < 1 || rows > (1 << 20)) return PD_ERR_ARG;
  if (mode != LIN_EPI_STORE && mode != LIN_EPI_RELU && mode != LIN_EPI_RESID) return PD_ERR_ARG;
  if (mode == LIN_EPI_RESID ? (!x || !gain_next || !xg) : !out) return PD_ERR_ARG;
  int dev = 0, sms = 148, BN = 0, ks = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (!linear_tc_plan(d_out, d_in, sms, &BN, &ks)) return PD_ERR_ARG;
  if (sumsq_parts) *sumsq_parts = (d_out / BN) * ks;
  const uintptr_t al = reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(out) |
                       reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(xg) | reinterpret_cast<uintptr_t>(gain_next);
  if (al % 16 != 0 || reinterpret_cast<uintptr_t>(scratch) % 256 != 0) return PD_ERR_ARG;
  if (scratch_bytes < pd_linear_scratch_bytes(d_in, d_out)) return PD_ERR_WORKSPACE;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint8_t *base = reinterpret_cast<uint8_t *>(scratch);
  void *wt = base + kOpHeaderBytes;
  if (cudaMemsetAsync(base, 0, kOpHeaderBytes, s) != cudaSuccess) return PD_ERR_CUDA;      // status word
  if (launch_transpose_bf16(d_in, d_out, w, wt, s) != cudaSuccess) return PD_ERR_CUDA;
  LinearActMaps map_a;
  CUtensorMap map_w;
  if (encode_linear_act_maps(&map_a, a, (uint64_t)rows, (uint64_t)d_in, nullptr) != cudaSuccess ||
      encode_linear_weight_map(&map_w, wt, (uint64_t)d_out, (uint64_t)d_in, BN, nullptr) != cudaSuccess)
    return PD_ERR_CUDA;
  if (linear_tc_prepare() != cudaSuccess) return PD_ERR_CUDA;
  LinearArgs la;
  memset(&la, 0, sizeof(la));
  la.K = d_in; la.N = d_out; la.BN = BN; la.ksplit = ks;
  la.rows_dev = nullptr; la.rows_fixed = rows; la.rows_cap = rows; la.rows_per_cta = (rows + 127) / 128 * 128;
  la.epi = mode;
  la.ssq_in = row_sumsq; la.parts_in = 1; la.inv_width = 1.f / (float)d_in; la.eps = eps;
  la.out = reinterpret_cast<__nv_bfloat16 *>(out);
  la.x = x; la.xg = reinterpret_cast<__nv_bfloat16 *>(xg); la.gain_next = reinterpret_cast<const __nv_bfloat16 *>(gain_next);
  la.ssq_out = sumsq_out;
  la.status = reinterpret_cast<int32_t *>(base) + HDR_STATUS;
  return launch_linear_tc(map_a, map_w, la, false, s) == cudaSuccess ? PD_OK : PD_ERR_CUDA;
}

}  // extern "C"
