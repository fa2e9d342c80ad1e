// Pipelined self-attention for bf16 storage (sm_100a): decode attention of all active
// subsequences of a sequence over the paged per-subsequence KV cache, with the dependency rule
// of Section 3.2 (a query of subsequence i sees subsequences i' <= i as generated so far)
// evaluated per page from (subsequence, start step, entry) metadata - no mask is ever stored.
//
// All S active rows of a sequence share its cache, so one key/value block serves up to S
// queries: with S around 8-16 the scores are far too many flops for the plain ALUs to keep
// up with HBM, so scores and P.V run on tensor cores (mma.sync m16n8k16, bf16 in, fp32
// accumulate) with the visibility rule and the T5 bias applied to the accumulator fragment.
//
// One CTA = one (split, head, sequence); each of its warps is an independent worker that takes
// every W-th page block of the sequence (W = splits * warps), streams it into its private ring
// of shared-memory slots with 1-D bulk copies (cp.async.bulk, completion on an mbarrier; only
// the rows that exist are copied) and keeps its own online-softmax state.  Pages are stored
// pre-swizzled (16-byte chunk c of entry e at chunk c ^ (e & 7)), so a linear copy lands in the
// bank-conflict-free layout ldmatrix wants.  The warps' partials are merged through shared
// memory, the splits by the merge kernel.  Every mbarrier wait is bounded.
#include "pd_internal.h"

namespace pd {

constexpr int SW = 4;                      // worker warps per CTA
constexpr int STHREADS = SW * 32;
constexpr int SDEPTH = 3;                  // page blocks in flight per warp
constexpr int SMAXTAB = 512;               // page-table entries of one sequence held in shared memory
constexpr int SMAXDIST = 512;
constexpr uint32_t SSPIN_LIMIT = 1u << 24;

__device__ __forceinline__ uint32_t s_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void s_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void s_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool s_mbar_try_wait(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool s_mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < SSPIN_LIMIT; ++it)
    if (s_mbar_try_wait(bar, parity)) return true;
  return false;
}
// 1-D bulk copy global -> shared; size a multiple of 16 bytes, both addresses 16-byte aligned.
__device__ __forceinline__ void s_bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void s_ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void s_ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void s_mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                           uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t s_pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// Byte offset of (entry, 16-byte chunk) inside a swizzled block whose entries are 128 bytes.
__device__ __forceinline__ uint32_t s_swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// Position of a worker in the sequence's list of page blocks: list index -> (subsequence, page).
struct PageCursor {
  int idx;   // index in the list (subsequence-major, pages of a subsequence in order)
  int s0;    // subsequence index, 0-based
  __device__ __forceinline__ void seek(const int *pfx) { while (idx >= pfx[s0 + 1]) ++s0; }
};

template <int MT>   // MT = 16-row query tiles (rows per sequence <= 16 * MT)
__global__ void __launch_bounds__(STHREADS) self_attn_tc_kernel(AttnArgs a) {
  extern __shared__ __align__(128) uint8_t s_ring_raw[];
  __shared__ __align__(8) unsigned long long bars[SW * SDEPTH];
  __shared__ int len_s[kMaxRows];          // cache entries of subsequence i (bos + content), index i-1
  __shared__ int tau0_s[kMaxRows];         // timestamp of its entry 0
  __shared__ int pfx_s[SW][kMaxRows + 1];  // per warp: pages before subsequence i
  __shared__ int rsub_s[16 * MT];          // subsequence of row r (0 = unused row)
  __shared__ int ptab_s[SMAXTAB];
  __shared__ float bias_s[SMAXDIST];

  const Dims &dm = a.dm;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int S = a.st.n_active[b];
  const int row0 = b * dm.C;
  __nv_bfloat16 *out = (__nv_bfloat16 *)a.out;

  if (S == 0) {   // nothing active: keep the output rows of this head defined
    if (split == 0)
      for (int idx = tid; idx < dm.C * kDh; idx += STHREADS)
        out[(size_t)(row0 + idx / kDh) * dm.d + h * kDh + idx % kDh] = __float2bfloat16_rn(0.f);
    return;
  }

  const int P = dm.P, PPS = dm.PPS;
  const uint32_t slot_bytes = 2u * P * 128u;
  const uint32_t ring0 = s_smem_u32(s_ring_raw);
  const uint32_t my_ring = ring0 + warp * SDEPTH * slot_bytes;
  const uint32_t my_bars = s_smem_u32(&bars[warp * SDEPTH]);

  // ---- metadata of the sequence, one round of independent loads
  const int t = a.st.hdr[HDR_STEP_T];
  for (int i = tid; i < dm.SM; i += STHREADS) {
    len_s[i] = a.st.len[b * dm.SM + i] + 1;
    tau0_s[i] = a.st.start[b * dm.SM + i] - 1;
  }
  for (int r = tid; r < 16 * MT; r += STHREADS) rsub_s[r] = r < S ? a.st.row_sub[row0 + r] : 0;
  for (int i = tid; i < dm.SM * PPS; i += STHREADS) ptab_s[i] = a.st.page_table[(size_t)b * dm.SM * PPS + i];
  // the ring starts out zeroed: slot rows beyond a partial page's entries are multiplied by
  // weights of exactly 0 and must be finite
  {
    uint4 *mine = reinterpret_cast<uint4 *>(s_ring_raw + warp * SDEPTH * slot_bytes);
    for (uint32_t i = lane; i < SDEPTH * slot_bytes / 16; i += 32) mine[i] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (lane == 0) {
    for (int s = 0; s < SDEPTH; ++s) s_mbar_init(my_bars + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // ---- pages per subsequence and their prefix sums (every warp computes its own copy)
  const int i_max = rsub_s[S - 1];           // rows are in increasing subsequence order
  int *pfx = pfx_s[warp];
  {
    int n0 = lane < i_max ? (len_s[lane] + P - 1) / P : 0;
    int n1 = lane + 32 < i_max ? (len_s[lane + 32] + P - 1) / P : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int v0 = __shfl_up_sync(0xffffffffu, n0, o), v1 = __shfl_up_sync(0xffffffffu, n1, o);
      if (lane >= o) { n0 += v0; n1 += v1; }
    }
    int tot0 = __shfl_sync(0xffffffffu, n0, 31);
    pfx[lane + 1] = n0;
    pfx[lane + 33] = tot0 + n1;
    if (lane == 0) pfx[0] = 0;
    __syncwarp();
  }
  const int total = pfx[i_max];
  const int W = a.splits * SW, g0 = split * SW + warp;
  const int n_mine = total > g0 ? (total - g0 + W - 1) / W : 0;

  const __nv_bfloat16 *pool = (const __nv_bfloat16 *)a.kv;
  auto issue = [&](int n, PageCursor &pc) {          // lane 0 only
    pc.idx = g0 + n * W;
    pc.seek(pfx);
    const int j = pc.idx - pfx[pc.s0];
    const int nv = min(P, len_s[pc.s0] - j * P);
    const int page = ptab_s[pc.s0 * PPS + j];
    const __nv_bfloat16 *src = pool + kv_block_offset(a.layer, dm.pool, page, dm.H, h, P);
    const int s = n % SDEPTH;
    const uint32_t dst = my_ring + s * slot_bytes, bar = my_bars + 8 * s;
    s_mbar_expect_tx(bar, 2u * nv * 128u);
    s_bulk_load(dst, src, nv * 128u, bar);                                   // keys
    s_bulk_load(dst + P * 128u, src + (size_t)P * kDh, nv * 128u, bar);      // values
  };
  PageCursor pc_issue{0, 0}, pc_use{0, 0};
  if (lane == 0)
    for (int n = 0; n < SDEPTH && n < n_mine; ++n) issue(n, pc_issue);

  // ---- while the first blocks fly: bias table and query fragments
  const bool use_bias = dm.pos_mode == PD_POS_T5_BIAS;
  if (use_bias)
    for (int dd = tid; dd < dm.n_dist && dd < SMAXDIST; dd += STHREADS)
      bias_s[dd] = a.rel_bias[h * a.rel_buckets + a.dist_bucket[dd]] * 1.4426950408889634f;   // log2 domain
  const int g = lane >> 2, tig = lane & 3;
  const __nv_bfloat16 *qbuf = (const __nv_bfloat16 *)a.q;
  uint32_t qf[MT][4][4];
  int rs[MT][2];                              // subsequence of rows g and g + 8 of every tile
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    int r_lo = mt * 16 + g, r_hi = r_lo + 8;
    rs[mt][0] = rsub_s[r_lo];
    rs[mt][1] = rsub_s[r_hi];
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
  __syncthreads();   // bias table complete

  const float sl2 = dm.scale_log2e;
  bool ok = true;
  for (int n = 0; n < n_mine; ++n) {
    const int s = n % SDEPTH;
    const uint32_t par = (uint32_t)(n / SDEPTH) & 1u;
    if (!s_mbar_wait(my_bars + 8 * s, par)) {
      ok = false;
      s_mbar_wait(my_bars + 8 * s, par);   // one more bounded wait for the copies in flight
      break;
    }
    pc_use.idx = g0 + n * W;
    pc_use.seek(pfx);
    const int j = pc_use.idx - pfx[pc_use.s0];
    const int nv = min(P, len_s[pc_use.s0] - j * P);          // entries of this page that exist
    const int ksub = pc_use.s0 + 1;                            // subsequence the page belongs to
    const int kpos0 = tau0_s[pc_use.s0] + j * P + ksub;        // position tau' + i' of its first entry
    const uint32_t kbase = my_ring + s * slot_bytes, vbase = kbase + P * 128u;

    for (int c0 = 0; c0 < nv; c0 += 16) {                      // 16 keys at a time
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        // Dependency rule: a row of subsequence i sees this page iff i' <= i (every stored entry
        // was generated before the current step).  Rows are sorted, so test the tile's last row.
        const int tile_last = rsub_s[min(S, 16 * (mt + 1)) - 1];
        if (16 * mt >= S || tile_last < ksub) continue;
        // ---- scores: Q (16 x 64) . K^T (64 x 16 keys)
        float sc[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
          const int key = c0 + nt * 8 + (lane & 7);
#pragma unroll
          for (int kp = 0; kp < 2; ++kp) {
            uint32_t b0, b1, b2, b3;
            s_ldsm_x4(kbase + s_swz(key, kp * 4 + (lane >> 3)), b0, b1, b2, b3);
            s_mma_bf16(sc[nt], qf[mt][2 * kp][0], qf[mt][2 * kp][1], qf[mt][2 * kp][2], qf[mt][2 * kp][3], b0, b1);
            s_mma_bf16(sc[nt], qf[mt][2 * kp + 1][0], qf[mt][2 * kp + 1][1], qf[mt][2 * kp + 1][2],
                       qf[mt][2 * kp + 1][3], b2, b3);
          }
        }
        // ---- scale, positional bias on the Manhattan distance, visibility, online softmax
        const bool see0 = rs[mt][0] >= ksub, see1 = rs[mt][1] >= ksub;
        const int qpos0 = t - 1 + rs[mt][0], qpos1 = t - 1 + rs[mt][1];   // position tau + i of the two rows
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int key = c0 + nt * 8 + 2 * tig + (e & 1);
            const bool vis = key < nv && ((e & 2) ? see1 : see0);
            float v = -INFINITY;
            if (vis) {
              v = sc[nt][e] * sl2;
              if (use_bias) v += bias_s[((e & 2) ? qpos1 : qpos0) - (kpos0 + key)];
            }
            sc[nt][e] = v;
          }
          mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m_run[mt][0], mx0), mn1 = fmaxf(m_run[mt][1], mx1);
        const float ref0 = mn0 == -INFINITY ? 0.f : mn0, ref1 = mn1 == -INFINITY ? 0.f : mn1;
        const float cr0 = exp2f(m_run[mt][0] - ref0), cr1 = exp2f(m_run[mt][1] - ref1);
        m_run[mt][0] = mn0; m_run[mt][1] = mn1;
        float s0 = 0.f, s1 = 0.f;
        uint32_t pf[4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          float p0 = exp2f(sc[nt][0] - ref0), p1 = exp2f(sc[nt][1] - ref0);
          float p2 = exp2f(sc[nt][2] - ref1), p3 = exp2f(sc[nt][3] - ref1);
          s0 += p0 + p1; s1 += p2 + p3;
          pf[nt * 2 + 0] = s_pack_bf16(p0, p1);
          pf[nt * 2 + 1] = s_pack_bf16(p2, p3);
        }
        l_run[mt][0] = l_run[mt][0] * cr0 + s0;
        l_run[mt][1] = l_run[mt][1] * cr1 + s1;
#pragma unroll
        for (int dn = 0; dn < 8; ++dn) { o[mt][dn][0] *= cr0; o[mt][dn][1] *= cr0; o[mt][dn][2] *= cr1; o[mt][dn][3] *= cr1; }
        // ---- O += P (16 x 16 keys) . V (16 keys x 64)
        const int vkey = c0 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
        for (int dp = 0; dp < 4; ++dp) {
          uint32_t b0, b1, b2, b3;
          s_ldsm_x4_t(vbase + s_swz(vkey, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
          s_mma_bf16(o[mt][2 * dp], pf[0], pf[1], pf[2], pf[3], b0, b1);
          s_mma_bf16(o[mt][2 * dp + 1], pf[0], pf[1], pf[2], pf[3], b2, b3);
        }
      }
    }
    __syncwarp();   // every lane is done reading the slot
    if (lane == 0 && n + SDEPTH < n_mine) issue(n + SDEPTH, pc_issue);
  }
  if (!ok && lane == 0) atomicExch(&a.st.hdr[HDR_STATUS], (int)PD_ERR_TIMEOUT);

  // ---- row sums across the quad, then merge the warps' partials through shared memory
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      l_run[mt][hh] += __shfl_xor_sync(0xffffffffu, l_run[mt][hh], 1);
      l_run[mt][hh] += __shfl_xor_sync(0xffffffffu, l_run[mt][hh], 2);
    }
  __syncthreads();   // every warp has consumed all the copies it issued: the ring can be reused
  constexpr int ROWS = 16 * MT;
  float *mo = reinterpret_cast<float *>(s_ring_raw);          // [SW][ROWS][64]
  float *mm = mo + SW * ROWS * kDh;                           // [SW][ROWS]
  float *ml = mm + SW * ROWS;                                 // [SW][ROWS]
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
  __syncthreads();
  for (int idx = tid; idx < dm.C * kDh; idx += STHREADS) {
    int r = idx / kDh, col = idx % kDh;
    size_t orow = (size_t)(row0 + r) * dm.d + h * kDh + col;
    if (r >= S) {
      if (split == 0) out[orow] = __float2bfloat16_rn(0.f);
      continue;
    }
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < SW; ++w) M = fmaxf(M, mm[w * ROWS + r]);
    float L = 0.f, O = 0.f;
    if (M != -INFINITY) {
#pragma unroll
      for (int w = 0; w < SW; ++w) {
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

static int self_attn_tc_smem(int P, int mt) {
  int ring = SW * SDEPTH * 2 * P * 128;
  int merge = SW * 16 * mt * (kDh + 2) * 4;
  return ring > merge ? ring : merge;
}

bool self_attn_tc_supported(const Dims &dm) {
  return dm.C <= 32 && dm.SM * dm.PPS <= SMAXTAB && (dm.pos_mode != PD_POS_T5_BIAS || dm.n_dist <= SMAXDIST);
}

cudaError_t self_attn_tc_prepare() {
  const int worst = self_attn_tc_smem(32, 2);
  cudaError_t e = cudaFuncSetAttribute(self_attn_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, worst);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(self_attn_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, worst);
}

cudaError_t launch_self_attn_tc(const AttnArgs &a, cudaStream_t s) {
  dim3 grid(a.splits, a.dm.H, a.batch);
  const int mt = (a.dm.C + 15) / 16;
  const int smem = self_attn_tc_smem(a.dm.P, mt);
  if (mt == 1) self_attn_tc_kernel<1><<<grid, STHREADS, smem, s>>>(a);
  else if (mt == 2) self_attn_tc_kernel<2><<<grid, STHREADS, smem, s>>>(a);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace pd
