// Vocabulary projection fused with the first stage of the greedy choice of Eq. 4 (bf16, sm_100a):
// logits[m][v] = sum_k hidden[m][k] * lm_head[v][k] on the 5th-generation tensor cores, and per row
// the maximum (lowest id on ties) over each CTA's slice of the vocabulary - the [rows x vocab] fp32
// logits never travel through HBM unless the caller asks for them.
//
// One CTA per slice of the vocabulary; the slice width (a multiple of 16, at most 224) is chosen so that the
// slices fill whole waves of 148 SMs (224 ids for 32128: 144 CTAs, one wave; 176 for 50265: 286 CTAs, two
// balanced rounds instead of one and a half of 224).  Rows are the M dimension of
// tcgen05.mma (128 per accumulator, two accumulators = up to 256 rows per pass over the CTA's slice
// of lm_head; more rows take more passes, which re-read the slice from L2).  The number of rows is
// read on the device (the sum of the sequences' active rows), so work follows the rows that exist,
// not the allocated maximum.  Warp 0 streams 64-column blocks of hidden and lm_head into a
// three-stage shared-memory ring with TMA (128-byte swizzle, mbarrier completion; of a ragged last row
// tile only the 32-row boxes that hold rows travel; the first lm_head blocks, which do not depend on the
// kernel before, are requested ahead of the programmatic-dependency wait); one lane of
// warp 1 issues tcgen05.mma (M 128, N 224, K 16, bf16 in, fp32 accumulators in tensor memory) and
// commits each stage back to the producer; warps 2-5 read the finished accumulators with
// tcgen05.ld (one row per thread, 32 columns at a time) and keep the running maximum in registers.
// Every mbarrier wait is bounded: on expiry the kernel records PD_ERR_TIMEOUT, stops waiting,
// falls through to the common exit and frees its tensor memory.
#include <limits.h>

#include "pd_internal.h"

namespace pd {

constexpr int VT_N = 224;                       // most vocabulary ids per CTA (the N of one tcgen05.mma; the slice in use is a.wn)
constexpr int VT_SMS = 148;                     // SMs the slice width is balanced for
constexpr int VT_M = 128;                       // rows per accumulator
constexpr int VT_BK = 64;                       // columns of K per stage (128 bytes: one swizzle span)
constexpr int VT_STAGES = 3;
constexpr int VT_THREADS = 192;                 // producer warp, MMA warp, four epilogue warps
constexpr int VT_A_BYTES = VT_M * VT_BK * 2;    // 16 KB
constexpr int VT_B_BYTES = VT_N * VT_BK * 2;    // 28 KB: room for the widest slice
constexpr int VT_BOX_M = 32;                    // rows per box of a ragged row tile
constexpr int VT_BOX_BYTES = VT_BOX_M * VT_BK * 2;
constexpr int VT_STAGE_BYTES = 2 * VT_A_BYTES + VT_B_BYTES;
constexpr int VT_SMEM = VT_STAGES * VT_STAGE_BYTES + 128 /*barriers*/ + 1024 /*alignment slack*/;
constexpr int VT_TMEM_COLS = 512;               // two accumulators at columns 0 and 256
constexpr uint32_t VT_SPIN_LIMIT = 1u << 24;
// instruction descriptor of kind::f16: D fp32, A and B bf16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24
__device__ __forceinline__ uint32_t v_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(VT_M >> 4) << 24);
}

// Slice width for a vocabulary of V ids: the narrowest multiple of 16 with which k * 148 slices cover V, k the
// number of rounds the widest slice (224) would need; at least 64 (narrower slices only multiply the
// re-reads of the hidden rows), and no wider than V needs.
int vocab_tc_slice(int V) {
  const int k = (V + VT_SMS * VT_N - 1) / (VT_SMS * VT_N);
  int wn = ((V + VT_SMS * k - 1) / (VT_SMS * k) + 15) / 16 * 16;
  if (wn < 64) wn = 64;
  if (wn > VT_N) wn = VT_N;
  const int need = (V + 15) / 16 * 16;
  return wn < need ? wn : need;
}
int vocab_tc_tiles(int V) { const int wn = vocab_tc_slice(V); return (V + wn - 1) / wn; }

__device__ __forceinline__ uint32_t v_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void v_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void v_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void v_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait: false when the phase did not complete within the spin limit.
__device__ __forceinline__ bool v_mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < VT_SPIN_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void v_tma_load_2d(uint32_t dst, const CUtensorMap *tmap, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tmap), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzle:
// start address >> 4, leading offset 16 B (unused by swizzled K-major), 1024 B between 8-row groups.
__device__ __forceinline__ uint64_t v_smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void v_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The barrier gets one arrival once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void v_mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void v_tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void v_tmem_ld16(uint32_t taddr, uint32_t (&r)[32]) {     // 16 columns into r[0..15]
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void v_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void v_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__global__ void __launch_bounds__(VT_THREADS, 1)
vocab_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a32,
                const __grid_constant__ CUtensorMap map_b, VocabArgs a) {
  extern __shared__ uint8_t v_smem_raw[];
  __shared__ uint32_t tmem_base_s;
  __shared__ int red_s[VT_THREADS / 32];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int vt = blockIdx.x;

  // ---- rows that exist this launch (the same value in every thread of every CTA).  The counts were written by
  // the scheduler of the previous time-step, several kernels back: visible without the dependency wait.
  const int wn = a.wn;
  int Mc = a.m_fixed;
  if (a.n_active != nullptr) {
    int s = 0;
    for (int b = tid; b < a.batch; b += VT_THREADS) s += a.n_active[b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) red_s[warp] = s;
    __syncthreads();
    Mc = 0;
#pragma unroll
    for (int w = 0; w < VT_THREADS / 32; ++w) Mc += red_s[w];
  }
  if (Mc <= 0) {                                         // nothing allocated yet, nothing to free
    asm volatile("griddepcontrol.wait;" ::: "memory");
    return;
  }
  const int n_tt = (Mc + VT_M - 1) / VT_M;               // 128-row tiles
  const int n_pass = (n_tt + 1) / 2;                     // two tiles (accumulators) per pass
  const int nkb = a.K / VT_BK;

  const uint32_t base = (v_smem_u32(v_smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_full = base + VT_STAGES * VT_STAGE_BYTES;
  const uint32_t bar_empty = bar_full + 8 * VT_STAGES;
  const uint32_t bar_acc_full = bar_empty + 8 * VT_STAGES;
  const uint32_t bar_acc_empty = bar_acc_full + 8;
  if (tid == 0) {
    for (int s = 0; s < VT_STAGES; ++s) { v_mbar_init(bar_full + 8 * s, 1); v_mbar_init(bar_empty + 8 * s, 1); }
    v_mbar_init(bar_acc_full, 1);
    v_mbar_init(bar_acc_empty, 4);                       // one arrival per epilogue warp
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {                                       // the MMA warp owns the tensor-memory allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(v_smem_u32(&tmem_base_s)), "r"(VT_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  v_fence_before();
  __syncthreads();
  v_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  bool ok = true;
  const uint32_t b_bytes = (uint32_t)(wn * VT_BK * 2);
  // bytes of the hidden-row tiles of pass p that travel: whole 128-row tiles, 32-row boxes of the ragged last one
  auto a_bytes = [&](int p) {
    uint32_t n = 0;
    for (int j = 0; j < min(2, n_tt - 2 * p); ++j) {
      const int rows_here = min(VT_M, Mc - (2 * p + j) * VT_M);
      n += rows_here == VT_M ? (uint32_t)VT_A_BYTES : (uint32_t)((rows_here + VT_BOX_M - 1) / VT_BOX_M * VT_BOX_BYTES);
    }
    return n;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (one lane)
    if (lane == 0) {
      // the first stages' lm_head blocks do not depend on the kernel before: on their way ahead of the wait
      const int ahead = min(VT_STAGES, nkb);
      for (int kb = 0; kb < ahead; ++kb) {
        v_mbar_expect_tx(bar_full + 8 * kb, b_bytes + a_bytes(0));
        v_tma_load_2d(base + kb * VT_STAGE_BYTES + 2 * VT_A_BYTES, &map_b, bar_full + 8 * kb, kb * VT_BK, vt * wn);
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      int it = 0;
      for (int p = 0; p < n_pass && ok; ++p) {
        const int tiles = min(2, n_tt - 2 * p);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % VT_STAGES;
          const uint32_t dst = base + s * VT_STAGE_BYTES;
          if (it >= ahead) {
            const uint32_t u = (uint32_t)(it / VT_STAGES);
            if (!v_mbar_wait(bar_empty + 8 * s, (u & 1u) ^ 1u)) { ok = false; break; }
            v_mbar_expect_tx(bar_full + 8 * s, b_bytes + a_bytes(p));
            v_tma_load_2d(dst + 2 * VT_A_BYTES, &map_b, bar_full + 8 * s, kb * VT_BK, vt * wn);
          }
          for (int j = 0; j < tiles; ++j) {
            const int row0 = (2 * p + j) * VT_M, rows_here = min(VT_M, Mc - row0);
            if (rows_here == VT_M) {
              v_tma_load_2d(dst + j * VT_A_BYTES, &map_a, bar_full + 8 * s, kb * VT_BK, row0);
            } else {
              // what the slot keeps beyond the boxes feeds accumulator rows nobody reads
              for (int bx = 0; bx * VT_BOX_M < rows_here; ++bx)
                v_tma_load_2d(dst + j * VT_A_BYTES + bx * VT_BOX_BYTES, &map_a32, bar_full + 8 * s, kb * VT_BK, row0 + bx * VT_BOX_M);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue (one lane)
    if (lane == 0) {
      int it = 0;
      const uint32_t idesc = v_idesc(wn);
      for (int p = 0; p < n_pass && ok; ++p) {
        const int tiles = min(2, n_tt - 2 * p);
        // the epilogue must be done with the previous pass's accumulators
        if (!v_mbar_wait(bar_acc_empty, ((uint32_t)p & 1u) ^ 1u)) { ok = false; break; }
        v_fence_after();
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % VT_STAGES;
          const uint32_t u = (uint32_t)(it / VT_STAGES);
          if (!v_mbar_wait(bar_full + 8 * s, u & 1u)) { ok = false; break; }
          v_fence_after();
          const uint32_t sa = base + s * VT_STAGE_BYTES, sb = sa + 2 * VT_A_BYTES;
          for (int j = 0; j < tiles; ++j)
#pragma unroll
            for (int k4 = 0; k4 < VT_BK / 16; ++k4)      // 16 columns of K = 32 bytes further inside the swizzle span
              v_mma_bf16(tmem_base + (uint32_t)j * 256u, v_smem_desc(sa + j * VT_A_BYTES + k4 * 32), v_smem_desc(sb + k4 * 32), idesc,
                         (kb > 0 || k4 > 0) ? 1u : 0u);
          v_mma_commit(bar_empty + 8 * s);               // frees the stage once these MMAs have read it
        }
        if (ok) v_mma_commit(bar_acc_full);              // the pass's accumulators are complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: one row per thread
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int quarter = warp & 3;                        // tensor-memory lanes 32 * quarter .. + 31 belong to this warp
    const int v_tile0 = vt * wn;
    for (int p = 0; p < n_pass; ++p) {
      const int tiles = min(2, n_tt - 2 * p);
      if (ok && !v_mbar_wait(bar_acc_full, (uint32_t)p & 1u)) ok = false;
      if (!ok) break;
      v_fence_after();
      for (int j = 0; j < tiles; ++j) {
        const int m = (2 * p + j) * VT_M + quarter * 32 + lane;
        float bv = -INFINITY, te = -INFINITY, ts = -INFINITY;
        int bi = INT_MAX;
#pragma unroll 1
        for (int c = 0; c * 32 < wn; ++c) {              // 32 columns at a time; a slice of an odd number of 16s ends with 16
          uint32_t r[32];
          const int ncol = min(32, wn - c * 32);
          if (ncol == 32) {
            v_tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(j * 256 + c * 32), r);
          } else {
            v_tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(j * 256 + c * 32), r);
#pragma unroll
            for (int i = 16; i < 32; ++i) r[i] = 0xff800000u;    // -inf: never a maximum, never stored (beyond the slice)
          }
          const int v0 = v_tile0 + c * 32;
          const bool special = ncol < 32 || v0 + 32 > a.V || (a.eos >= v0 && a.eos < v0 + 32) || (a.sep >= v0 && a.sep < v0 + 32);
          if (!special) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {               // ascending ids and a strict compare: ties keep the lowest id
              const float x = __uint_as_float(r[i]);
              if (x > bv) { bv = x; bi = v0 + i; }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float x = __uint_as_float(r[i]);
              const int v = v0 + i;
              if (v >= a.V || i >= ncol) continue;
              if (v == a.eos) te = x;
              else if (v == a.sep) ts = x;
              else if (x > bv) { bv = x; bi = v; }
            }
          }
          if (a.logits != nullptr && m < Mc) {
            float *row = a.logits + (size_t)m * a.V + v0;
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (v0 + i < a.V && i < ncol) row[i] = __uint_as_float(r[i]);
          }
        }
        if (m < Mc) {
          a.part_val[(size_t)vt * a.rows_cap + m] = bv;
          a.part_idx[(size_t)vt * a.rows_cap + m] = bi;
          if (a.eos >= v_tile0 && a.eos < v_tile0 + wn) a.term_val[2 * m] = te;
          if (a.sep >= v_tile0 && a.sep < v_tile0 + wn) a.term_val[2 * m + 1] = ts;
        }
      }
      v_fence_before();
      __syncwarp();
      if (lane == 0) v_mbar_arrive(bar_acc_empty);
    }
  }
  if (!ok && lane == 0) atomicExch(a.status, (int)PD_ERR_TIMEOUT);
  v_fence_before();
  __syncthreads();
  if (warp == 1) {
    v_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(VT_TMEM_COLS) : "memory");
  }
}

// Tensor map of a row-major bf16 matrix [rows, cols]: boxes of box_rows rows x 64 columns (128 bytes,
// one swizzle span), 128-byte swizzle, out-of-range rows read as zeros.
cudaError_t encode_rowmajor_bf16_map(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                                     int *driver_code) {
  typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                               const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  if (driver_code) *driver_code = 0;
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)VT_BK, box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = ((EncodeFn)fn)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { if (driver_code) *driver_code = (int)r; return cudaErrorInvalidValue; }
  return cudaSuccess;
}

// hidden rows: boxes of 128 rows (whole row tiles) and of 32 rows (the ragged last tile); lm_head: boxes of one slice
cudaError_t encode_vocab_maps(VocabMaps *m, const void *hidden, uint64_t rows, const void *lm_head, uint64_t vocab, uint64_t K,
                              int *driver_code) {
  cudaError_t e = encode_rowmajor_bf16_map(&m->a, hidden, rows, K, VT_M, driver_code);
  if (e == cudaSuccess) e = encode_rowmajor_bf16_map(&m->a32, hidden, rows, K, VT_BOX_M, driver_code);
  if (e == cudaSuccess) e = encode_rowmajor_bf16_map(&m->b, lm_head, vocab, K, (uint32_t)vocab_tc_slice((int)vocab), driver_code);
  return e;
}

bool vocab_tc_supported(int K, int V) { return K >= VT_BK && K % VT_BK == 0 && V >= 1; }

cudaError_t vocab_tc_prepare() {
  return cudaFuncSetAttribute(vocab_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, VT_SMEM);
}

// Launched as a programmatic dependent of the kernel before it in the stream (the packed final norm, which lets its
// dependents start early): set-up and the first lm_head blocks overlap that kernel's tail.
cudaError_t launch_vocab_tc(const VocabMaps &m, const VocabArgs &a_in, cudaStream_t s) {
  VocabArgs a = a_in;
  a.wn = vocab_tc_slice(a.V);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(vocab_tc_tiles(a.V), 1, 1);
  cfg.blockDim = dim3(VT_THREADS, 1, 1);
  cfg.dynamicSmemBytes = VT_SMEM;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, vocab_tc_kernel, m.a, m.a32, m.b, a);
}

}  // namespace pd
