// Batched cross-attention for the bf16 path (sm_100a): every active subsequence of a sequence
// is a query row against the shared encoder keys/values (all context positions < ctx_len
// visible, no positional term).  This is the one part of the step that is a dense S x L_ctx
// contraction, so it runs on tensor cores; it stays HBM-bound (about S flop per byte).
//
// One CTA = one (split of the context, head, sequence).  A producer warp streams 128-key K and
// V tiles (16 KB each) from global memory into a ring of shared-memory stages with TMA
// (cp.async.bulk.tensor.2d, 128-byte swizzle, completion on an mbarrier); four consumer warps
// each take 32 keys of every tile: S = Q K^T with mma.sync m16n8k16 (bf16 in, fp32 accumulate),
// online softmax in the log2 domain with quad shuffles, O += P V.  The warps' partial
// (m, l, O) are merged in shared memory, and the context splits by a separate merge kernel.
// Every mbarrier wait is bounded: on expiry the kernel records PD_ERR_TIMEOUT and leaves.
#include "pd_internal.h"

namespace pd {

constexpr int XK = 128;                   // keys per tile
constexpr int XSTAGES = 3;
constexpr int XCW = 4;                    // consumer warps
constexpr int XTHREADS = (XCW + 1) * 32;
constexpr int XTILE_BYTES = XK * kDh * 2; // 16 KB
constexpr int XSTAGE_BYTES = 2 * XTILE_BYTES;
constexpr int XSMEM = XSTAGES * XSTAGE_BYTES + 128 /*barriers*/ + 1024 /*alignment slack*/;
constexpr uint32_t XSPIN_LIMIT = 1u << 24;

int cross_attn_tma_smem_bytes() { return XSMEM; }

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < XSPIN_LIMIT; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tmap, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tmap), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(XCW * 32) : "memory"); }

// Byte offset of (row, 16-byte chunk) inside a 128-byte-swizzled tile whose rows are 128 bytes.
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

template <int MT>   // MT = 16-row query tiles (rows per sequence <= 16 * MT)
__global__ void __launch_bounds__(XTHREADS) cross_attn_tma_kernel(const __grid_constant__ CUtensorMap tmap, AttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const Dims &dm = a.dm;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int S = a.st.n_active[b];
  const int row0 = b * dm.C;
  __nv_bfloat16 *out = (__nv_bfloat16 *)a.out;

  if (S == 0) {
    if (split == 0)
      for (int idx = tid; idx < dm.C * kDh; idx += XTHREADS)
        out[(size_t)(row0 + idx / kDh) * dm.d + h * kDh + idx % kDh] = __float2bfloat16_rn(0.f);
    return;
  }

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_full = base + XSTAGES * XSTAGE_BYTES;
  const uint32_t bar_empty = bar_full + 8 * XSTAGES;
  uint8_t *smem_al = smem_raw + (base - smem_u32(smem_raw));

  const int ctx_len = a.st.ctx_len[b];
  const int n_tiles = (ctx_len + XK - 1) / XK;
  const int per = (n_tiles + a.splits - 1) / a.splits;
  const int t0 = split * per;
  const int my = max(0, min(n_tiles, t0 + per) - t0);

  if (tid == 0) {
    for (int s = 0; s < XSTAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, XCW); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == XCW) {
    // ------------------------------------------------------------------ producer (one lane)
    if (lane == 0) {
      const int y0 = (int)(ctx_kv_offset(a.layer, dm.B, b, dm.H, h, 0, dm.ctx) / kDh);   // row of this head's key 0
      for (int it = 0; it < my; ++it) {
        int s = it % XSTAGES;
        uint32_t u = (uint32_t)(it / XSTAGES);
        if (!mbar_wait(bar_empty + 8 * s, (u & 1u) ^ 1u)) { atomicExch(&a.st.hdr[HDR_STATUS], (int)PD_ERR_TIMEOUT); break; }
        mbar_expect_tx(bar_full + 8 * s, XSTAGE_BYTES);
        uint32_t dst = base + s * XSTAGE_BYTES;
        int y = y0 + (t0 + it) * XK;
        tma_load_2d(dst, &tmap, bar_full + 8 * s, 0, y);                         // K tile
        tma_load_2d(dst + XTILE_BYTES, &tmap, bar_full + 8 * s, 0, y + dm.ctx);  // V tile
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int g = lane >> 2, tig = lane & 3;
  const __nv_bfloat16 *qbuf = (const __nv_bfloat16 *)a.q;
  uint32_t qf[MT][4][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    int r_lo = mt * 16 + g, r_hi = r_lo + 8;
    const __nv_bfloat16 *q_lo = qbuf + (size_t)(row0 + r_lo) * dm.d + h * kDh + 2 * tig;
    const __nv_bfloat16 *q_hi = qbuf + (size_t)(row0 + r_hi) * dm.d + h * kDh + 2 * tig;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      qf[mt][kk][0] = r_lo < S ? *reinterpret_cast<const uint32_t *>(q_lo + kk * 16) : 0u;
      qf[mt][kk][1] = r_hi < S ? *reinterpret_cast<const uint32_t *>(q_hi + kk * 16) : 0u;
      qf[mt][kk][2] = r_lo < S ? *reinterpret_cast<const uint32_t *>(q_lo + kk * 16 + 8) : 0u;
      qf[mt][kk][3] = r_hi < S ? *reinterpret_cast<const uint32_t *>(q_hi + kk * 16 + 8) : 0u;
    }
  }
  float o[MT][8][4];
  float m_run[MT][2], l_run[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    m_run[mt][0] = m_run[mt][1] = -INFINITY;
    l_run[mt][0] = l_run[mt][1] = 0.f;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) o[mt][dn][0] = o[mt][dn][1] = o[mt][dn][2] = o[mt][dn][3] = 0.f;
  }
  const int kb = warp * 32;          // this warp's keys inside every tile
  const float sl2 = dm.scale_log2e;
  bool ok = true;

  for (int it = 0; it < my; ++it) {
    const int s = it % XSTAGES;
    const uint32_t u = (uint32_t)(it / XSTAGES);
    if (!mbar_wait(bar_full + 8 * s, u & 1u)) {
      ok = false;
      mbar_wait(bar_full + 8 * s, u & 1u);   // one more bounded wait for the copies in flight
      break;
    }
    const uint32_t kbase = base + s * XSTAGE_BYTES, vbase = kbase + XTILE_BYTES;
    const int key0 = (t0 + it) * XK + kb;          // context position of this warp's first key
    const bool ragged = key0 + 32 > ctx_len;
    if (ragged) {
      // Rows at or beyond ctx_len hold whatever follows in memory (or the fill value).  Their
      // weights are exactly 0 below; zero the value rows so that 0 never multiplies a non-finite.
      if (key0 + lane >= ctx_len) {
        uint4 *vrow = reinterpret_cast<uint4 *>(smem_al + (vbase - base) + (kb + lane) * 128);
#pragma unroll
        for (int c = 0; c < 8; ++c) vrow[c] = make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // before the stage's next bulk copy
      }
      __syncwarp();
    }

    // ---- scores: S[mt][nt] = Q (16 x 64) . K^T (64 x 8 keys)
    float sc[MT][4][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) sc[mt][nt][0] = sc[mt][nt][1] = sc[mt][nt][2] = sc[mt][nt][3] = 0.f;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const int key = kb + nt * 8 + (lane & 7);
#pragma unroll
      for (int kp = 0; kp < 2; ++kp) {      // two k16 steps per ldmatrix.x4
        uint32_t b0, b1, b2, b3;
        ldsm_x4(kbase + swz(key, kp * 4 + (lane >> 3)), b0, b1, b2, b3);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_bf16(sc[mt][nt], qf[mt][2 * kp][0], qf[mt][2 * kp][1], qf[mt][2 * kp][2], qf[mt][2 * kp][3], b0, b1);
          mma_bf16(sc[mt][nt], qf[mt][2 * kp + 1][0], qf[mt][2 * kp + 1][1], qf[mt][2 * kp + 1][2],
                   qf[mt][2 * kp + 1][3], b2, b3);
        }
      }
    }
    // ---- scale, mask the ragged end of the context, online softmax
    uint32_t pf[MT][2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = sc[mt][nt][e] * sl2;
          if (ragged && key0 + nt * 8 + 2 * tig + (e & 1) >= ctx_len) v = -INFINITY;
          sc[mt][nt][e] = v;
        }
        mx0 = fmaxf(mx0, fmaxf(sc[mt][nt][0], sc[mt][nt][1]));
        mx1 = fmaxf(mx1, fmaxf(sc[mt][nt][2], sc[mt][nt][3]));
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m_run[mt][0], mx0), mn1 = fmaxf(m_run[mt][1], mx1);
      const float ref0 = mn0 == -INFINITY ? 0.f : mn0, ref1 = mn1 == -INFINITY ? 0.f : mn1;
      const float c0 = exp2f(m_run[mt][0] - ref0), c1 = exp2f(m_run[mt][1] - ref1);
      m_run[mt][0] = mn0; m_run[mt][1] = mn1;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        float p0 = exp2f(sc[mt][nt][0] - ref0), p1 = exp2f(sc[mt][nt][1] - ref0);
        float p2 = exp2f(sc[mt][nt][2] - ref1), p3 = exp2f(sc[mt][nt][3] - ref1);
        s0 += p0 + p1; s1 += p2 + p3;
        pf[mt][nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
        pf[mt][nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      l_run[mt][0] = l_run[mt][0] * c0 + s0;
      l_run[mt][1] = l_run[mt][1] * c1 + s1;
#pragma unroll
      for (int dn = 0; dn < 8; ++dn) { o[mt][dn][0] *= c0; o[mt][dn][1] *= c0; o[mt][dn][2] *= c1; o[mt][dn][3] *= c1; }
    }
    // ---- O += P (16 x 32 keys) . V (32 keys x 64)
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
      const int key = kb + ks * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
      for (int dp = 0; dp < 4; ++dp) {      // two 8-wide slices of the head per ldmatrix.x4
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vbase + swz(key, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          mma_bf16(o[mt][2 * dp], pf[mt][ks][0], pf[mt][ks][1], pf[mt][ks][2], pf[mt][ks][3], b0, b1);
          mma_bf16(o[mt][2 * dp + 1], pf[mt][ks][0], pf[mt][ks][1], pf[mt][ks][2], pf[mt][ks][3], b2, b3);
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_empty + 8 * s);
  }
  if (!ok && lane == 0) atomicExch(&a.st.hdr[HDR_STATUS], (int)PD_ERR_TIMEOUT);

  // ---- row sums across the quad, then merge the four warps' partials through shared memory
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      l_run[mt][hh] += __shfl_xor_sync(0xffffffffu, l_run[mt][hh], 1);
      l_run[mt][hh] += __shfl_xor_sync(0xffffffffu, l_run[mt][hh], 2);
    }
  consumer_bar_sync();   // every warp is past its last tile: the stages can be reused
  constexpr int ROWS = 16 * MT;
  float *mo = reinterpret_cast<float *>(smem_al);            // [XCW][ROWS][64]
  float *mm = mo + XCW * ROWS * kDh;                          // [XCW][ROWS]
  float *ml = mm + XCW * ROWS;                                // [XCW][ROWS]
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    int r_lo = mt * 16 + g, r_hi = r_lo + 8;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) {
      int col = dn * 8 + 2 * tig;
      *reinterpret_cast<float2 *>(&mo[(warp * ROWS + r_lo) * kDh + col]) = make_float2(o[mt][dn][0], o[mt][dn][1]);
      *reinterpret_cast<float2 *>(&mo[(warp * ROWS + r_hi) * kDh + col]) = make_float2(o[mt][dn][2], o[mt][dn][3]);
    }
    if (tig == 0) {
      mm[warp * ROWS + r_lo] = m_run[mt][0]; ml[warp * ROWS + r_lo] = l_run[mt][0];
      mm[warp * ROWS + r_hi] = m_run[mt][1]; ml[warp * ROWS + r_hi] = l_run[mt][1];
    }
  }
  consumer_bar_sync();
  for (int idx = tid; idx < dm.C * kDh; idx += XCW * 32) {
    int r = idx / kDh, col = idx % kDh;
    size_t orow = (size_t)(row0 + r) * dm.d + h * kDh + col;
    if (r >= S) {
      if (split == 0) out[orow] = __float2bfloat16_rn(0.f);
      continue;
    }
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < XCW; ++w) M = fmaxf(M, mm[w * ROWS + r]);
    float L = 0.f, O = 0.f;
    if (M != -INFINITY) {
#pragma unroll
      for (int w = 0; w < XCW; ++w) {
        float wgt = exp2f(mm[w * ROWS + r] - M);
        L += ml[w * ROWS + r] * wgt;
        O += mo[(w * ROWS + r) * kDh + col] * wgt;
      }
    }
    if (a.splits == 1) {
      out[orow] = __float2bfloat16_rn(O / L);
    } else {
      size_t pi = ((size_t)(row0 + r) * dm.H + h) * a.splits + split;
      a.part_o[pi * kDh + col] = O;
      if (col == 0) { a.part_ml[pi * 2] = M; a.part_ml[pi * 2 + 1] = L; }
    }
  }
}

// Tensor map of the context keys/values seen as a 2-D bf16 array [rows, 64] (row = one context
// position of one (layer, sequence, head, K or V)): boxes of 128 rows x 64 columns (one head's
// keys or values of one tile, 16 KB contiguous), 128-byte swizzle.  *driver_code gets the CUresult
// when the encode itself fails.
cudaError_t encode_ctx_kv_tensor_map(CUtensorMap *out, const void *base, uint64_t rows, int *driver_code) {
  typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                               const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  if (driver_code) *driver_code = 0;
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
  cuuint64_t gdim[2] = {(cuuint64_t)kDh, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)kDh * 2};
  cuuint32_t box[2] = {(cuuint32_t)kDh, (cuuint32_t)XK};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = ((EncodeFn)fn)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { if (driver_code) *driver_code = (int)r; return cudaErrorInvalidValue; }
  return cudaSuccess;
}

cudaError_t cross_attn_tma_prepare() {
  cudaError_t e = cudaFuncSetAttribute(cross_attn_tma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, XSMEM);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(cross_attn_tma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, XSMEM);
}

cudaError_t launch_cross_attn_tma(const AttnArgs &a, const CUtensorMap &tmap, cudaStream_t s) {
  dim3 grid(a.splits, a.dm.H, a.batch);
  int mt = (a.dm.C + 15) / 16;
  if (mt == 1) cross_attn_tma_kernel<1><<<grid, XTHREADS, XSMEM, s>>>(tmap, a);
  else if (mt == 2) cross_attn_tma_kernel<2><<<grid, XTHREADS, XSMEM, s>>>(tmap, a);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace pd
