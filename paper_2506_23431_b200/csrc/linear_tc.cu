// Skinny-M linear layers of the decoder stack (Eq. 3: a stacked transformer decoder) on the
// 5th-generation tensor cores (bf16, sm_100a):  acc[m][n] = sum_k A[m][k] * W[n][k]  for the few
// hundred packed active rows m of a decode step against a weight matrix that is streamed from HBM
// exactly once, with the work that surrounds the product in the layer fused into the epilogue
// (row scale of the preceding RMSNorm, ReLU, residual add + the next norm's inputs).
//
// The products are tiny (a few MB of weights, a few hundred rows), so the kernel is built around
// latency, not flops:
//  * grid = (N / BN) x ksplit CTAs, the ksplit CTAs of one N-slice forming a thread-block cluster;
//    each CTA takes K / ksplit columns of the reduction, so that even a d x d matrix is spread
//    over more than a hundred SMs and no CTA has to pull more than a few tens of KB of the
//    activations through its shared-memory port.
//  * one lane streams the CTA's weight slice (BN x 64 tiles) and the activation tiles (128 x 64)
//    through two small TMA rings (128-byte swizzle, mbarrier completion); the weight tiles do not
//    depend on the previous kernel of the step, so they are requested BEFORE the programmatic
//    dependency wait and travel while that kernel is still finishing.
//  * one lane issues tcgen05.mma (M 128, N = BN, K 16) into tensor memory, one accumulator per
//    128-row tile (up to 256 columns, i.e. 2-8 row tiles per pass).
//  * four warps read the accumulators back with tcgen05.ld and PUSH every column to the CTA of the
//    cluster that owns it after the reduction (CTA r owns columns [r * BN / ksplit, ...)): plain
//    stores into the peer's shared memory, which nobody waits for.  After one cluster barrier every
//    CTA finds all ksplit partial sums of its columns in its own shared memory, adds them in rank
//    order (results do not depend on timing) and applies the epilogue.  No partial sum ever travels
//    through global memory, and no CTA ever reads a peer's memory.
// Every mbarrier wait is bounded: on expiry the CTA records PD_ERR_TIMEOUT, stops computing, still
// takes part in every cluster barrier (those are executed unconditionally by all threads), waits
// for its own bulk copies and frees its tensor memory.
#include "pd_internal.h"

namespace pd {

constexpr int LT_BK = 64;                        // K columns per tile (128 bytes: one swizzle span)
constexpr int LT_M = 128;                        // rows per accumulator
constexpr int LT_SLOT = LT_M * LT_BK * 2;        // 16 KB: one activation tile; a weight tile (BN <= 128 rows) fits too
constexpr int LT_BOX_M = 32;                     // rows per activation box: a row tile is loaded as the 1-4 boxes that hold rows
constexpr int LT_BOX_BYTES = LT_BOX_M * LT_BK * 2;
constexpr int LT_NW = 3;                         // ring slots for weight tiles (each BN x 64, rounded up to 1 KB)
constexpr int LT_RING_BYTES = 6 * LT_SLOT;       // both rings; the activation ring gets what the weight ring leaves (3-5 slots)
constexpr int LT_NA_MAX = 5;
constexpr int LT_MT_MAX = 8;                     // most row tiles per pass
constexpr int LT_THREADS = 192;                  // loader warp, MMA warp, four epilogue warps
constexpr int LT_TMEM_COLS = 256;                // half of tensor memory: two CTAs (of this or a neighbouring kernel) share an SM
constexpr int LT_BAR_BYTES = 256;
constexpr int LT_SMEM = LT_RING_BYTES + LT_BAR_BYTES + 1024 /*alignment slack*/;
constexpr uint32_t LT_SPIN_LIMIT = 1u << 22;

int linear_tc_smem_bytes() { return LT_SMEM; }

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t l_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void l_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void l_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool l_mbar_try(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool l_mbar_wait(uint32_t bar, uint32_t parity) {   // bounded
  for (uint32_t it = 0; it < LT_SPIN_LIMIT; ++it)
    if (l_mbar_try(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void l_tma_load_2d(uint32_t dst, const CUtensorMap *tmap, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tmap), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
// K-major tile with 128-byte rows, 128-byte swizzle, 1024 bytes between 8-row groups
__device__ __forceinline__ uint64_t l_smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24
__device__ __forceinline__ uint32_t l_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(LT_M >> 4) << 24);
}
__device__ __forceinline__ void l_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void l_mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void l_tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void l_tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void l_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void l_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ uint32_t l_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Hardware barrier over all threads of the cluster (release / acquire: shared-memory writes made
// before it are visible to the peers' distributed-shared-memory reads after it).
__device__ __forceinline__ void l_cluster_sync_all() {
  __syncwarp();                                      // the barrier instructions want the whole warp together
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t l_peer_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
__device__ __forceinline__ void l_st_peer_v4(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
// Programmatic dependent launch: let the next kernel of the stream start its preamble; wait for the
// previous kernel's results.
__device__ __forceinline__ void l_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void l_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint2 l_pack4(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  return make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
}

// ---- the epilogue of one (row, four columns) group --------------------------------------------------
// v = the four sums of columns n .. n + 3 of packed row m.  `ss` accumulates the squares of what the
// residual epilogue writes (the next RMSNorm's input).
__device__ __forceinline__ void l_epilogue4(const LinearArgs &a, int m, int n, float4 v, float inv, float &ss) {
  switch (a.epi) {
    case LIN_EPI_STORE:
    case LIN_EPI_RELU: {
      v.x *= inv; v.y *= inv; v.z *= inv; v.w *= inv;
      if (a.epi == LIN_EPI_RELU) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
      *reinterpret_cast<uint2 *>(a.out + (size_t)m * a.N + n) = l_pack4(v.x, v.y, v.z, v.w);
      break;
    }
    case LIN_EPI_RESID: {
      *reinterpret_cast<float4 *>(a.x + (size_t)m * a.N + n) = v;      // v = old x + product (the caller added x)
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      const uint2 gbits = *reinterpret_cast<const uint2 *>(a.gain_next + n);
      const __nv_bfloat162 g0 = *reinterpret_cast<const __nv_bfloat162 *>(&gbits.x), g1 = *reinterpret_cast<const __nv_bfloat162 *>(&gbits.y);
      *reinterpret_cast<uint2 *>(a.xg + (size_t)m * a.N + n) =
          l_pack4(v.x * __low2float(g0), v.y * __high2float(g0), v.z * __low2float(g1), v.w * __high2float(g1));
      break;
    }
  }
}

__global__ void __launch_bounds__(LT_THREADS, 2)
linear_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a32,
                 const __grid_constant__ CUtensorMap map_w, LinearArgs a) {
  extern __shared__ uint8_t l_smem_raw[];
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_tile = blockIdx.x;
  const int BN = a.BN, ks = a.ksplit;
  const uint32_t rank = ks > 1 ? l_cluster_rank() : 0u;

  const uint32_t base = (l_smem_u32(l_smem_raw) + 1023u) & ~1023u;
  const int w_bytes = BN * LT_BK * 2;                // one weight tile
  const int w_slot = (w_bytes + 1023) & ~1023;
  const int NA = min(LT_NA_MAX, (LT_RING_BYTES - LT_NW * w_slot) / LT_SLOT);
  const uint32_t ring_w = base, ring_a = base + LT_RING_BYTES - NA * LT_SLOT;
  const uint32_t bars = base + LT_RING_BYTES;
  const uint32_t full_a = bars, empty_a = full_a + 8 * LT_NA_MAX, full_w = empty_a + 8 * LT_NA_MAX, empty_w = full_w + 8 * LT_NW;
  const uint32_t acc_full = empty_w + 8 * LT_NW;
  if (tid == 0) {
    for (int s = 0; s < LT_NA_MAX; ++s) { l_mbar_init(full_a + 8 * s, 1); l_mbar_init(empty_a + 8 * s, 1); }
    for (int s = 0; s < LT_NW; ++s) { l_mbar_init(full_w + 8 * s, 1); l_mbar_init(empty_w + 8 * s, 1); }
    l_mbar_init(acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(l_smem_u32(&tmem_base_s)), "r"(LT_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  l_fence_before();
  __syncthreads();
  l_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  l_launch_dependents();

  const int nkb = a.K / LT_BK / ks;                  // K tiles of this CTA
  const int kb0 = (int)rank * nkb;
  const int mtpp = min(LT_TMEM_COLS / BN, LT_MT_MAX);   // row tiles per pass (accumulators that fit)
  bool ok = true;

  // The row count was written by the scheduler of the previous time-step, many kernels back; every kernel
  // since has passed its own dependency wait, so that write is visible here without waiting.
  const int rows_all = a.rows_dev != nullptr ? min(max(__ldcg(a.rows_dev), 0), a.rows_cap) : a.rows_fixed;
  // this CTA's rows: group blockIdx.z of rows_per_cta rows (the same for every CTA of a cluster)
  const int row_base = (int)blockIdx.z * a.rows_per_cta;
  const int rows = min(max(rows_all - row_base, 0), a.rows_per_cta);
  const int n_mt = (rows + LT_M - 1) / LT_M;
  const int n_pass = (n_mt + mtpp - 1) / mtpp;

  // Weight tiles of the first pass that fit the ring: requested before the dependency wait (a CTA
  // without rows requests nothing and leaves through the common exit).
  int w_issued = 0;
  if (warp == 0 && lane == 0 && n_mt > 0) {
    for (; w_issued < LT_NW && w_issued < nkb; ++w_issued) {
      l_mbar_expect_tx(full_w + 8 * w_issued, (uint32_t)w_bytes);
      l_tma_load_2d(ring_w + w_issued * w_slot, &map_w, full_w + 8 * w_issued, (kb0 + w_issued) * LT_BK, n_tile * BN);
    }
  }
  l_dependency_wait();

  // after the reduction this CTA owns columns c_first .. c_first + cpr - 1 of the slice, ng groups of four
  const int cpr = BN / ks, ng = cpr / 4, c_first = (int)rank * cpr;
  const int q = warp & 3;                            // tensor-memory lanes 32 q .. 32 q + 31 belong to this warp
  const int row = q * 32 + lane;                     // row within a 128-row tile (epilogue warps)
  const int tile_bytes = BN * LT_M * 4;              // one fp32 tile of partial sums: [ksplit][ng][128 rows][4]
  uint8_t *red = l_smem_raw + (base - l_smem_u32(l_smem_raw));

  int a_issued = 0, a_used = 0, w_used = 0;          // ring positions (loader: issued; MMA lane: used)
  for (int p = 0; p < n_pass; ++p) {
    const int mts = min(mtpp, n_mt - p * mtpp);      // row tiles of this pass
    float inv[LT_MT_MAX];                            // epilogue threads: RMSNorm scale of their row in every tile of the pass
    if (warp == 0) {
      // ---------------------------------------------------------------- loader (one lane): two rings, neither blocks the other
      if (lane == 0 && ok) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the rings served as reduction buffer in the previous pass
        const int w_end = (p + 1) * nkb, a_end = a_issued + nkb * mts;
        uint32_t spins = 0;
        while (w_issued < w_end || a_issued < a_end) {
          bool progress = false;
          if (w_issued < w_end) {
            const int s = w_issued % LT_NW;
            if (l_mbar_try(empty_w + 8 * s, (((uint32_t)(w_issued / LT_NW)) & 1u) ^ 1u)) {
              l_mbar_expect_tx(full_w + 8 * s, (uint32_t)w_bytes);
              l_tma_load_2d(ring_w + s * w_slot, &map_w, full_w + 8 * s, (kb0 + w_issued % nkb) * LT_BK, n_tile * BN);
              ++w_issued; progress = true;
            }
          }
          if (a_issued < a_end) {
            const int s = a_issued % NA;
            if (l_mbar_try(empty_a + 8 * s, (((uint32_t)(a_issued / NA)) & 1u) ^ 1u)) {
              const int local = a_issued - (a_end - nkb * mts);          // item within the pass: k tile outer, row tile inner
              const int kb = local / mts, mt = p * mtpp + local % mts;
              // only the 32-row boxes that hold rows travel; what the slot keeps beyond them feeds accumulator
              // rows nobody reads (a row of the product depends on its own row of the activations alone)
              const int boxes = (min(LT_M, rows - mt * LT_M) + LT_BOX_M - 1) / LT_BOX_M;
              l_mbar_expect_tx(full_a + 8 * s, (uint32_t)(boxes * LT_BOX_BYTES));
              if (boxes == LT_M / LT_BOX_M) {
                l_tma_load_2d(ring_a + s * LT_SLOT, &map_a, full_a + 8 * s, (kb0 + kb) * LT_BK, row_base + mt * LT_M);
              } else {
                for (int bx = 0; bx < boxes; ++bx)
                  l_tma_load_2d(ring_a + s * LT_SLOT + bx * LT_BOX_BYTES, &map_a32, full_a + 8 * s, (kb0 + kb) * LT_BK, row_base + mt * LT_M + bx * LT_BOX_M);
              }
              ++a_issued; progress = true;
            }
          }
          if (progress) spins = 0;
          else if (++spins > LT_SPIN_LIMIT) { ok = false; break; }
        }
      }
    } else if (warp == 1) {
      // ---------------------------------------------------------------- MMA issue (one lane)
      if (lane == 0 && ok) {
        const uint32_t idesc = l_idesc(BN);
        for (int kb = 0; kb < nkb && ok; ++kb, ++w_used) {
          const int sw = w_used % LT_NW;
          if (!l_mbar_wait(full_w + 8 * sw, ((uint32_t)(w_used / LT_NW)) & 1u)) { ok = false; break; }
          for (int j = 0; j < mts; ++j, ++a_used) {
            const int sa = a_used % NA;
            if (!l_mbar_wait(full_a + 8 * sa, ((uint32_t)(a_used / NA)) & 1u)) { ok = false; break; }
            l_fence_after();
#pragma unroll
            for (int k4 = 0; k4 < LT_BK / 16; ++k4)
              l_mma(tmem_base + (uint32_t)(j * BN), l_smem_desc(ring_a + sa * LT_SLOT + k4 * 32), l_smem_desc(ring_w + sw * w_slot + k4 * 32),
                    idesc, (kb > 0 || k4 > 0) ? 1u : 0u);
            l_mma_commit(empty_a + 8 * sa);
          }
          if (ok) l_mma_commit(empty_w + 8 * sw);
        }
        if (ok) l_mma_commit(acc_full);
      }
    } else {
      // ---------------------------------------------------------------- epilogue warps, while the product runs: the rows' norm scales
#pragma unroll
      for (int j = 0; j < LT_MT_MAX; ++j) {
        inv[j] = 1.f;
        const int m = row_base + (p * mtpp + j) * LT_M + row;
        if (a.ssq_in != nullptr && j < mts && m - row_base < rows) {
          float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;      // fixed summation order
          int pp = 0;
          for (; pp + 3 < a.parts_in; pp += 4) {
            s0 += __ldcg(a.ssq_in + (size_t)pp * a.rows_cap + m);
            s1 += __ldcg(a.ssq_in + (size_t)(pp + 1) * a.rows_cap + m);
            s2 += __ldcg(a.ssq_in + (size_t)(pp + 2) * a.rows_cap + m);
            s3 += __ldcg(a.ssq_in + (size_t)(pp + 3) * a.rows_cap + m);
          }
          for (; pp < a.parts_in; ++pp) s0 += __ldcg(a.ssq_in + (size_t)pp * a.rows_cap + m);
          inv[j] = rsqrtf(((s0 + s1) + (s2 + s3)) * a.inv_width + a.eps);
        }
      }
      if (ok && !l_mbar_wait(acc_full, (uint32_t)p & 1u)) ok = false;
      l_fence_after();
    }
    // ------------------------------------------------------------------ accumulators -> owners' shared memory -> sums -> epilogue
    // The rings take the partial sums, as many row tiles at a time as fit - once every CTA of the cluster
    // is through with them (its epilogue warps have seen its last MMA complete).
    if (ks > 1) l_cluster_sync_all();
    const int gm = min(mts, LT_RING_BYTES / tile_bytes);
    for (int j0 = 0; j0 < mts; j0 += gm) {
      const int jn = min(gm, mts - j0);
      float4 xpre[2][2];                             // residual epilogue: the first values of x, requested before the barrier
      if (warp >= 2 && ok) {
        if (a.epi == LIN_EPI_RESID) {
#pragma unroll
          for (int jj = 0; jj < 2; ++jj)
#pragma unroll
            for (int g = 0; g < 2; ++g) {
              const int m = row_base + (p * mtpp + j0 + jj) * LT_M + row;
              if (jj < jn && g < ng && m - row_base < rows) xpre[jj][g] = *reinterpret_cast<const float4 *>(a.x + (size_t)m * a.N + n_tile * BN + c_first + 4 * g);
            }
        }
        for (int j = j0; j < j0 + jn; ++j) {
          const bool mine = (p * mtpp + j) * LT_M + row < rows;     // rows beyond the last one are not pushed (nobody reads them)
#pragma unroll 1
          for (int c0 = 0; c0 < BN / 16; c0 += 2) {  // 32 columns per round trip to tensor memory
            uint32_t r[2][16];
            l_tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(j * BN + c0 * 16), r[0]);
            if (c0 + 1 < BN / 16) l_tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(j * BN + c0 * 16 + 16), r[1]);
            l_tmem_ld_wait();
            if (!mine) continue;
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              if (c0 + cc >= BN / 16) break;
#pragma unroll
              for (int g4 = 0; g4 < 4; ++g4) {
                const int col = (c0 + cc) * 16 + 4 * g4, owner = col / cpr, g = (col - owner * cpr) >> 2;
                const uint32_t off = (uint32_t)((j - j0) * tile_bytes + ((((int)rank * ng + g) * LT_M + row) << 4));
                l_st_peer_v4(l_peer_addr(base + off, (uint32_t)owner), __uint_as_float(r[cc][4 * g4]), __uint_as_float(r[cc][4 * g4 + 1]),
                             __uint_as_float(r[cc][4 * g4 + 2]), __uint_as_float(r[cc][4 * g4 + 3]));
              }
            }
          }
        }
        l_fence_before();
      }
      // every CTA's partial sums of this CTA's columns are in its shared memory (a lone CTA reads back, thread
      // by thread, what that thread wrote itself)
      if (ks > 1) l_cluster_sync_all();
      if (warp >= 2 && ok) {
        for (int j = j0; j < j0 + jn; ++j) {
          const int m = row_base + (p * mtpp + j) * LT_M + row;
          if (m - row_base >= rows) continue;
          float sc = 1.f;
#pragma unroll
          for (int jj = 0; jj < LT_MT_MAX; ++jj) if (jj == j) sc = inv[jj];
          float ss = 0.f;
          const float4 *buf = reinterpret_cast<const float4 *>(red + (size_t)(j - j0) * tile_bytes) + row;
          for (int g = 0; g < ng; ++g) {
            float4 v = buf[(size_t)g * LT_M];
            for (int pr = 1; pr < ks; ++pr) {        // rank order: the sum does not depend on which CTA finished first
              const float4 u = buf[(size_t)(pr * ng + g) * LT_M];
              v.x += u.x; v.y += u.y; v.z += u.z; v.w += u.w;
            }
            const int n = n_tile * BN + c_first + 4 * g;
            if (a.epi == LIN_EPI_RESID) {
              float4 x0;
              if (j - j0 < 2 && g < 2) {
                x0 = xpre[0][0];
#pragma unroll
                for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                  for (int gg = 0; gg < 2; ++gg) if (jj == j - j0 && gg == g) x0 = xpre[jj][gg];
              } else {
                x0 = *reinterpret_cast<const float4 *>(a.x + (size_t)m * a.N + n);
              }
              v.x += x0.x; v.y += x0.y; v.z += x0.z; v.w += x0.w;
            }
            l_epilogue4(a, m, n, v, sc, ss);
          }
          if (a.epi == LIN_EPI_RESID && a.ssq_out != nullptr) a.ssq_out[(size_t)(n_tile * ks + (int)rank) * a.rows_cap + m] = ss;
        }
      }
      // Another group or pass pushes into the same buffers: every CTA must be done reading first.  After
      // the last group nothing remote is outstanding (all pushes into this CTA preceded the barrier above).
      if (ks > 1 && (j0 + jn < mts || p + 1 < n_pass)) l_cluster_sync_all();
    }
  }
  if (!ok && lane == 0) atomicExch(a.status, (int)PD_ERR_TIMEOUT);
  l_fence_before();
  __syncthreads();
  if (warp == 1) {
    l_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(LT_TMEM_COLS) : "memory");
  }
}

// ---- host side ------------------------------------------------------------------------------------
// Tensor map of a row-major bf16 matrix [rows, cols] (cols a multiple of 64): boxes of box_rows rows x
// 64 columns, 128-byte swizzle, rows beyond the matrix read as zeros.
cudaError_t encode_linear_map(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, int *driver_code) {
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
  cuuint32_t box[2] = {(cuuint32_t)LT_BK, box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = ((EncodeFn)fn)(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { if (driver_code) *driver_code = (int)r; return cudaErrorInvalidValue; }
  return cudaSuccess;
}
// activations: one map with 128-row boxes (full row tiles), one with 32-row boxes (the ragged last tile)
cudaError_t encode_linear_act_maps(LinearActMaps *out, const void *act, uint64_t rows, uint64_t K, int *driver_code) {
  cudaError_t e = encode_linear_map(&out->full, act, rows, K, LT_M, driver_code);
  if (e != cudaSuccess) return e;
  return encode_linear_map(&out->part, act, rows, K, LT_BOX_M, driver_code);
}
cudaError_t encode_linear_weight_map(CUtensorMap *out, const void *w_nk, uint64_t N, uint64_t K, int BN, int *driver_code) {
  return encode_linear_map(out, w_nk, N, K, (uint32_t)BN, driver_code);
}

// (BN, ksplit) for an N x K weight: BN a multiple of 16 that divides N, a cluster of at most 8 CTAs
// along K, every CTA owning a multiple of four columns after the reduction.  Among those the plan
// with the fewest bytes through one SM's shared-memory port wins (what bounds these small products):
// per K tile a CTA pulls its weight tile and the activation tiles (taken as 1.5 row tiles), and an SM
// hosts ceil(CTAs / SMs) CTAs.
bool linear_tc_plan(int N, int K, int sms, int *BN_out, int *ksplit_out) {
  if (K < LT_BK || K % LT_BK != 0 || N < 16 || N % 16 != 0) return false;
  const int nkb = K / LT_BK;
  long best_cost = -1;
  int best_bn = 0, best_ks = 0;
  for (int ks = 1; ks <= 8; ++ks) {
    if (nkb % ks) continue;
    for (int bn = 16; bn <= 128; bn += 16) {
      if (N % bn || bn % (4 * ks)) continue;
      const int ctas = (N / bn) * ks;
      if (ctas > 2 * sms) continue;
      const long per_cta = (long)(nkb / ks) * (bn * LT_BK * 2 + LT_SLOT * 3 / 2);
      const long cost = ((ctas + sms - 1) / sms) * per_cta;
      if (best_cost < 0 || cost < best_cost || (cost == best_cost && bn > best_bn)) { best_cost = cost; best_bn = bn; best_ks = ks; }
    }
  }
  if (best_cost < 0) return false;
  *BN_out = best_bn; *ksplit_out = best_ks;
  return true;
}

cudaError_t linear_tc_prepare() {
  return cudaFuncSetAttribute(linear_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LT_SMEM);
}

// Launch with the cluster shape (1, ksplit, 1) and, when `pdl` is set, as a programmatic dependent
// of the previous kernel in the stream.
cudaError_t launch_linear_tc(const LinearActMaps &map_a, const CUtensorMap &map_w, const LinearArgs &a, bool pdl, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.N / a.BN, a.ksplit, (a.rows_cap + a.rows_per_cta - 1) / a.rows_per_cta);
  cfg.blockDim = dim3(LT_THREADS, 1, 1);
  cfg.dynamicSmemBytes = LT_SMEM;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeClusterDimension;
  attr[n].val.clusterDim.x = 1; attr[n].val.clusterDim.y = a.ksplit; attr[n].val.clusterDim.z = 1;
  ++n;
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr; cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, linear_tc_kernel, map_a.full, map_a.part, map_w, a);
}

// ---- W [K, N] row-major  ->  Wt [N, K] row-major (once, when a handle is made) ----------------------
__global__ void transpose_bf16_kernel(int K, int N, const __nv_bfloat16 *__restrict__ w, __nv_bfloat16 *__restrict__ wt) {
  __shared__ __nv_bfloat16 tile[32][33];
  const int n0 = blockIdx.x * 32, k0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int k = k0 + r, n = n0 + threadIdx.x;
    if (k < K && n < N) tile[r][threadIdx.x] = w[(size_t)k * N + n];
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int n = n0 + r, k = k0 + threadIdx.x;
    if (k < K && n < N) wt[(size_t)n * K + k] = tile[threadIdx.x][r];
  }
}

cudaError_t launch_transpose_bf16(int K, int N, const void *w, void *wt, cudaStream_t s) {
  dim3 grid((N + 31) / 32, (K + 31) / 32), block(32, 8);
  transpose_bf16_kernel<<<grid, block, 0, s>>>(K, N, (const __nv_bfloat16 *)w, (__nv_bfloat16 *)wt);
  return cudaGetLastError();
}

}  // namespace pd
