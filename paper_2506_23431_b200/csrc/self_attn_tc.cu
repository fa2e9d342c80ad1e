// Pipelined self-attention for bf16 storage (sm_100a): decode attention of all active
// subsequences of a sequence over the paged per-subsequence KV cache, with the dependency rule
// of Section 3.2 (a query of subsequence i sees subsequences i' <= i as generated so far)
// evaluated per page from (subsequence, first position) metadata - no mask is ever stored.
//
// All S active rows of a sequence share its cache, so one key/value block serves up to S
// queries: with S around 8-16 the scores are far too many flops for the plain ALUs to keep
// up with HBM, so scores and P.V run on tensor cores (mma.sync m16n8k16, bf16 in, fp32
// accumulate) with the visibility rule and the T5 bias applied to the accumulator fragment.
//
// The scheduler leaves, once per step, a list of the sequence's pages (page, entries, subsequence,
// first position) that every layer and head reuses.  One CTA = one (split, head, sequence); each of
// its warps is an independent worker that takes every W-th page of the list (W = splits * warps),
// copies exactly the entries that exist - one contiguous run, key row and value row per entry -
// into its private two-slot ring with 16-byte cp.async (these blocks are a few KB and scattered:
// per-lane async copies have no per-request engine cost and need no barrier object) and keeps its
// own online-softmax state over all keys of the page at once.  Pages are stored pre-swizzled
// (16-byte chunk c of a row of entry e at chunk c ^ (e & 7)), so a linear copy lands in the
// bank-conflict-free layout ldmatrix wants.  The warps' partials are
// merged through shared memory, the splits by the merge kernel.  Nothing in the kernel waits on
// another warp's progress except the two CTA barriers of prologue and epilogue.
#include "pd_internal.h"

namespace pd {

constexpr int SW = 4;                      // worker warps per CTA
constexpr int STHREADS = SW * 32;
constexpr int SDEPTH = 2;                  // ring slots per warp: the page in use and the next one
constexpr int SMAXLIST = 256;              // page-list entries of one sequence held in shared memory
constexpr int SMAXDIST = 512;
constexpr int SMROW = kDh + 8;               // row stride of the merge scratch in floats (spreads the eight fragment rows over the banks)

__device__ __forceinline__ uint32_t s_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// 16-byte asynchronous copy global -> shared
__device__ __forceinline__ void s_cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void s_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void s_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void s_ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void s_ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// (not volatile: a pure function of its registers, free to be scheduled around other work)
__device__ __forceinline__ void s_mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                           uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float s_ex2(float x) {   // 2^x, flushes denormals; ex2(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t s_pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// Byte offset of 16-byte chunk `chunk` of entry `row`'s key row inside a block (256 bytes per
// entry: swizzled key row, then swizzled value row at + 128).
__device__ __forceinline__ uint32_t s_swz(int row, int chunk) { return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4)); }

// All lanes: copy the nv existing entries of one (page, head) block - nv * 256 contiguous bytes,
// key row then value row per entry - into a ring slot.
template <int P>
__device__ __forceinline__ void s_fetch_page(uint32_t slot, const __nv_bfloat16 *blk, int nv, int lane) {
  const uint8_t *src = reinterpret_cast<const uint8_t *>(blk) + lane * 16;
  const uint32_t dst = slot + lane * 16;
  const int nchunks = nv * 16;                   // 16-byte chunks of the run
#pragma unroll
  for (int k = 0; k < P / 2; ++k)                // P * 16 chunks over 32 lanes
    if (k * 32 + lane < nchunks) s_cp_async16(dst + k * 512, src + k * 512);
}

template <int MT, int P>   // MT = 16-row query tiles (rows per sequence <= 16 * MT); P = page_tokens
__global__ void __launch_bounds__(STHREADS) self_attn_tc_kernel(AttnArgs a) {
  constexpr int NT = P / 8;                // 8-key score tiles per page
  constexpr int KS = P / 16;               // 16-key steps of P.V per page
  constexpr uint32_t SLOT = 2u * P * 128u; // keys + values of one page of one head
  extern __shared__ __align__(128) uint8_t s_ring_raw[];
  __shared__ int4 plist_s[SMAXLIST];       // (page, entries, subsequence i', distance base of entry 0)
  __shared__ int rsub_s[16 * MT];          // subsequence of row r
  __shared__ float bias_s[SMAXDIST];

  const Dims &dm = a.dm;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row0 = b * dm.C;
  __nv_bfloat16 *out = (__nv_bfloat16 *)a.out;
  const int g = lane >> 2, tig = lane & 3;

  // ---- ONE round of independent global loads, none waiting for another: active-row count, page
  // list (first STHREADS entries), row -> subsequence, bias row of this head, query fragments.
  // What turns out to be unused (rows beyond the active ones) is masked afterwards.
  const int S = a.st.n_active[b];
  const int n_list = a.st.plist_n[b];
  const int list_cap = dm.SM * dm.PPS;
  const int4 *pl = a.st.plist + (size_t)b * list_cap;
  int4 my_entry = make_int4(0, 0, 0, 0);
  if (tid < list_cap) my_entry = pl[tid];
  // this warp's first two pages (entries g0 and g0 + W of the list), so that their copies can start
  // before the CTA has assembled the list in shared memory
  const int W = a.splits * SW, g0 = split * SW + warp;
  const int4 first0 = g0 < list_cap ? pl[g0] : make_int4(0, 0, 0, 0);
  const int4 first1 = g0 + W < list_cap ? pl[g0 + W] : make_int4(0, 0, 0, 0);
  int my_rsub = 0;
  if (tid < dm.C) my_rsub = a.st.row_sub[row0 + tid];
  const bool use_bias = a.bias_tab != nullptr;
  float my_bias[SMAXDIST / STHREADS];
#pragma unroll
  for (int k = 0; k < SMAXDIST / STHREADS; ++k) {
    const int dd = k * STHREADS + tid;
    my_bias[k] = (use_bias && dd < dm.n_dist) ? a.bias_tab[h * dm.n_dist + dd] : 0.f;
  }
  const __nv_bfloat16 *qbuf = (const __nv_bfloat16 *)a.q;
  uint32_t qf[MT][4][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
    const __nv_bfloat16 *q_lo = qbuf + (size_t)(row0 + r_lo) * dm.d + h * kDh + 2 * tig;
    const __nv_bfloat16 *q_hi = qbuf + (size_t)(row0 + r_hi) * dm.d + h * kDh + 2 * tig;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      qf[mt][kk][0] = r_lo < dm.C ? *reinterpret_cast<const uint32_t *>(q_lo + kk * 16) : 0u;
      qf[mt][kk][1] = r_hi < dm.C ? *reinterpret_cast<const uint32_t *>(q_hi + kk * 16) : 0u;
      qf[mt][kk][2] = r_lo < dm.C ? *reinterpret_cast<const uint32_t *>(q_lo + kk * 16 + 8) : 0u;
      qf[mt][kk][3] = r_hi < dm.C ? *reinterpret_cast<const uint32_t *>(q_hi + kk * 16 + 8) : 0u;
    }
  }

  if (S == 0) {   // nothing active: keep the output rows of this head defined
    if (split == 0)
      for (int idx = tid; idx < dm.C * kDh; idx += STHREADS)
        out[(size_t)(row0 + idx / kDh) * dm.d + h * kDh + idx % kDh] = __float2bfloat16_rn(0.f);
    return;
  }
  const int n_mine = n_list > g0 ? (n_list - g0 + W - 1) / W : 0;
  const uint32_t my_ring = s_smem_u32(s_ring_raw) + warp * SDEPTH * SLOT;
  const __nv_bfloat16 *pool_lh = (const __nv_bfloat16 *)a.kv + kv_block_offset(a.layer, dm.pool, 0, dm.H, h, P);
  const size_t page_stride = (size_t)dm.H * 2 * P * kDh;      // elements from one page's block of this head to the next page's
  auto fetch = [&](int n, int4 e) { s_fetch_page<P>(my_ring + (n & 1) * SLOT, pool_lh + e.x * page_stride, e.y, lane); };
  {
    // The warp's ring starts out zeroed: value rows beyond a partly filled page's entries get weights
    // of exactly 0 in P.V and must be finite, whatever the slot held before (later: earlier pages' data).
    uint4 *ring = reinterpret_cast<uint4 *>(s_ring_raw + (size_t)warp * SDEPTH * SLOT);
#pragma unroll
    for (int i = 0; i < (int)(SDEPTH * SLOT / 16) / 32; ++i) ring[i * 32 + lane] = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();                      // the zeros are in place before any lane's copy lands on them
    if (n_mine > 0) fetch(0, first0);
    s_cp_async_commit();
    if (n_mine > 1) fetch(1, first1);
    s_cp_async_commit();
  }
  if (tid < SMAXLIST) plist_s[tid] = my_entry;
  for (int i = tid + STHREADS; i < n_list; i += STHREADS) plist_s[i] = pl[i];   // lists longer than one round
  if (tid < 16 * MT) rsub_s[tid] = my_rsub;
#pragma unroll
  for (int k = 0; k < SMAXDIST / STHREADS; ++k) bias_s[k * STHREADS + tid] = my_bias[k];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {   // rows at or beyond S carry no query
    const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      if (r_lo >= S) qf[mt][kk][0] = qf[mt][kk][2] = 0u;
      if (r_hi >= S) qf[mt][kk][1] = qf[mt][kk][3] = 0u;
    }
  }
  __syncthreads();

  // ---- this warp's share of the page list is entries g0, g0 + W, ...; its first two pages are already on their way

  int rs[MT][2];                     // subsequence of rows g and g + 8 of every query tile
  int tile_last[MT];                 // subsequence of the tile's last active row (rows are sorted)
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    rs[mt][0] = rsub_s[min(mt * 16 + g, S - 1)];           // unused rows repeat the last active one
    rs[mt][1] = rsub_s[min(mt * 16 + g + 8, S - 1)];
    tile_last[mt] = 16 * mt < S ? rsub_s[min(16 * mt + 15, S - 1)] : 0;
  }
  const int sub_first = rsub_s[0];   // the smallest active subsequence: a page it sees, every row sees
  float o[MT][8][4];
  float m_run[MT][2], l_run[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    m_run[mt][0] = m_run[mt][1] = -INFINITY;
    l_run[mt][0] = l_run[mt][1] = 0.f;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) o[mt][dn][0] = o[mt][dn][1] = o[mt][dn][2] = o[mt][dn][3] = 0.f;
  }
  const float sl2 = dm.scale_log2e;

  for (int n = 0; n < n_mine; ++n) {
    s_cp_async_wait<1>();              // everything but the newest group has landed: page n is in its slot
    __syncwarp();
    const int4 e = plist_s[g0 + n * W];
    const int nv = e.y;                // entries of this page that exist
    const int ksub = e.z;              // subsequence the page belongs to
    const int d0 = e.w;                // distance base of its first entry: distance = d0 + i - key offset
    const uint32_t kbase = my_ring + (n & 1) * SLOT, vbase = kbase + 128u;
    // Dependency rule: a row of subsequence i sees this page iff i' <= i (every stored entry was
    // generated before the current step).  A query tile none of whose rows sees it is skipped;
    // a full page that every row sees needs no masking at all.
    bool act[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) act[mt] = tile_last[mt] >= ksub;
    const bool plain = nv == P && sub_first >= ksub;

    // ---- scores: Q (16 x 64) . K^T (64 x P keys); two accumulators per tile halve the mma chain
    float sc[MT][NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      if (nt * 8 < nv) {
        const int key = nt * 8 + (lane & 7);
        uint32_t b0, b1, b2, b3, c0, c1, c2, c3;
        s_ldsm_x4(kbase + s_swz(key, (lane >> 3)), b0, b1, b2, b3);        // dims 0..31
        s_ldsm_x4(kbase + s_swz(key, 4 + (lane >> 3)), c0, c1, c2, c3);    // dims 32..63
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if (!act[mt]) continue;
          float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
          s_mma_bf16(sa, qf[mt][0][0], qf[mt][0][1], qf[mt][0][2], qf[mt][0][3], b0, b1);
          s_mma_bf16(sb, qf[mt][1][0], qf[mt][1][1], qf[mt][1][2], qf[mt][1][3], b2, b3);
          s_mma_bf16(sa, qf[mt][2][0], qf[mt][2][1], qf[mt][2][2], qf[mt][2][3], c0, c1);
          s_mma_bf16(sb, qf[mt][3][0], qf[mt][3][1], qf[mt][3][2], qf[mt][3][3], c2, c3);
#pragma unroll
          for (int x = 0; x < 4; ++x) sc[mt][nt][x] = sa[x] + sb[x];
        }
      } else {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int x = 0; x < 4; ++x) sc[mt][nt][x] = 0.f;
      }
    }
    // ---- scale, positional bias on the Manhattan distance, visibility, online softmax (log2 domain)
    uint32_t pf[MT][KS][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      if (!act[mt]) continue;
      // distance of rows g / g+8 to the page's entry 0, minus this thread's first key column
      const float *bp0 = bias_s + (d0 + rs[mt][0] - 2 * tig);
      const float *bp1 = bias_s + (d0 + rs[mt][1] - 2 * tig);
      float mx0 = -INFINITY, mx1 = -INFINITY;
      if (plain) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const float bias = use_bias ? ((x & 2) ? bp1 : bp0)[-(nt * 8 + (x & 1))] : 0.f;
            sc[mt][nt][x] = fmaf(sc[mt][nt][x], sl2, bias);
          }
          mx0 = fmaxf(mx0, fmaxf(sc[mt][nt][0], sc[mt][nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sc[mt][nt][2], sc[mt][nt][3]));
        }
      } else {
        const bool see0 = rs[mt][0] >= ksub, see1 = rs[mt][1] >= ksub;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const int key = nt * 8 + 2 * tig + (x & 1);
            const bool vis = key < nv && ((x & 2) ? see1 : see0);
            float v = -INFINITY;
            if (vis) {
              const float bias = use_bias ? ((x & 2) ? bp1 : bp0)[-(nt * 8 + (x & 1))] : 0.f;
              v = fmaf(sc[mt][nt][x], sl2, bias);
            }
            sc[mt][nt][x] = v;
          }
          mx0 = fmaxf(mx0, fmaxf(sc[mt][nt][0], sc[mt][nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sc[mt][nt][2], sc[mt][nt][3]));
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m_run[mt][0], mx0), mn1 = fmaxf(m_run[mt][1], mx1);
      const float ref0 = mn0 == -INFINITY ? 0.f : mn0, ref1 = mn1 == -INFINITY ? 0.f : mn1;
      const float cr0 = s_ex2(m_run[mt][0] - ref0), cr1 = s_ex2(m_run[mt][1] - ref1);
      m_run[mt][0] = mn0; m_run[mt][1] = mn1;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float p0 = s_ex2(sc[mt][nt][0] - ref0), p1 = s_ex2(sc[mt][nt][1] - ref0);
        float p2 = s_ex2(sc[mt][nt][2] - ref1), p3 = s_ex2(sc[mt][nt][3] - ref1);
        s0 += p0 + p1; s1 += p2 + p3;
        pf[mt][nt >> 1][(nt & 1) * 2 + 0] = s_pack_bf16(p0, p1);
        pf[mt][nt >> 1][(nt & 1) * 2 + 1] = s_pack_bf16(p2, p3);
      }
      l_run[mt][0] = l_run[mt][0] * cr0 + s0;
      l_run[mt][1] = l_run[mt][1] * cr1 + s1;
      if (__any_sync(0xffffffffu, cr0 != 1.f || cr1 != 1.f)) {   // some row's running maximum moved
#pragma unroll
        for (int dn = 0; dn < 8; ++dn) { o[mt][dn][0] *= cr0; o[mt][dn][1] *= cr0; o[mt][dn][2] *= cr1; o[mt][dn][3] *= cr1; }
      }
    }
    // ---- O += P (16 x P keys) . V (P keys x 64)
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      if (ks * 16 < nv) {
        const int vkey = ks * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
        for (int dp = 0; dp < 4; ++dp) {
          uint32_t b0, b1, b2, b3;
          s_ldsm_x4_t(vbase + s_swz(vkey, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            if (!act[mt]) continue;
            s_mma_bf16(o[mt][2 * dp], pf[mt][ks][0], pf[mt][ks][1], pf[mt][ks][2], pf[mt][ks][3], b0, b1);
            s_mma_bf16(o[mt][2 * dp + 1], pf[mt][ks][0], pf[mt][ks][1], pf[mt][ks][2], pf[mt][ks][3], b2, b3);
          }
        }
      }
    }
    __syncwarp();   // every lane is done reading the slot
    if (n + 2 < n_mine) fetch(n + 2, plist_s[g0 + (n + 2) * W]);
    s_cp_async_commit();
  }
  s_cp_async_wait<0>();

  // ---- row sums across the quad, then merge the warps' partials through shared memory
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      l_run[mt][hh] += __shfl_xor_sync(0xffffffffu, l_run[mt][hh], 1);
      l_run[mt][hh] += __shfl_xor_sync(0xffffffffu, l_run[mt][hh], 2);
    }
  __syncthreads();   // every warp is past its last page: the ring can be reused
  constexpr int ROWS = 16 * MT;
  float *mo = reinterpret_cast<float *>(s_ring_raw);          // [SW][ROWS][SMROW]
  float *mm = mo + SW * ROWS * SMROW;                           // [SW][ROWS]
  float *ml = mm + SW * ROWS;                                 // [SW][ROWS]
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    int r_lo = mt * 16 + g, r_hi = r_lo + 8;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) {
      int col = dn * 8 + 2 * tig;
      *reinterpret_cast<float2 *>(&mo[(warp * ROWS + r_lo) * SMROW + col]) = make_float2(o[mt][dn][0], o[mt][dn][1]);
      *reinterpret_cast<float2 *>(&mo[(warp * ROWS + r_hi) * SMROW + col]) = make_float2(o[mt][dn][2], o[mt][dn][3]);
    }
    if (tig == 0) {
      mm[warp * ROWS + r_lo] = m_run[mt][0]; ml[warp * ROWS + r_lo] = l_run[mt][0];
      mm[warp * ROWS + r_hi] = m_run[mt][1]; ml[warp * ROWS + r_hi] = l_run[mt][1];
    }
  }
  __syncthreads();
  // per row once: the common maximum, each warp's weight (turned into mm in place) and the row sum
  if (tid < ROWS && tid < S) {
    const int r = tid;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < SW; ++w) M = fmaxf(M, mm[w * ROWS + r]);
    float L = 0.f;
#pragma unroll
    for (int w = 0; w < SW; ++w) {
      const float wgt = M == -INFINITY ? 0.f : s_ex2(mm[w * ROWS + r] - M);
      L += ml[w * ROWS + r] * wgt;
      mm[w * ROWS + r] = wgt;
    }
    ml[r] = L;                     // warp 0's slots now hold the merged row sums ...
    ml[ROWS + r] = M;              // ... and warp 1's the merged maxima
  }
  __syncthreads();
  for (int idx = tid; idx < dm.C * (kDh / 2); idx += STHREADS) {          // two columns per thread
    const int r = idx / (kDh / 2), col = 2 * (idx % (kDh / 2));
    const size_t orow = (size_t)(row0 + r) * dm.d + h * kDh + col;
    if (r >= S) {
      if (split == 0) *reinterpret_cast<__nv_bfloat162 *>(out + orow) = __floats2bfloat162_rn(0.f, 0.f);
      continue;
    }
    float2 O = make_float2(0.f, 0.f);
#pragma unroll
    for (int w = 0; w < SW; ++w) {
      const float wgt = mm[w * ROWS + r];
      const float2 v = *reinterpret_cast<const float2 *>(&mo[(w * ROWS + r) * SMROW + col]);
      O.x += v.x * wgt; O.y += v.y * wgt;
    }
    if (a.splits == 1) {
      const float inv = 1.f / ml[r];
      *reinterpret_cast<__nv_bfloat162 *>(out + orow) = __floats2bfloat162_rn(O.x * inv, O.y * inv);
    } else {
      const size_t pi = ((size_t)(row0 + r) * dm.H + h) * a.splits + split;
      *reinterpret_cast<float2 *>(&a.part_o[pi * kDh + col]) = O;
      if (col == 0) { a.part_ml[pi * 2] = ml[ROWS + r]; a.part_ml[pi * 2 + 1] = ml[r]; }
    }
  }
}

static int self_attn_tc_smem(int P, int mt) {
  int ring = SW * SDEPTH * 2 * P * 128;
  int merge = SW * 16 * mt * (SMROW + 2) * 4;
  return ring > merge ? ring : merge;
}

bool self_attn_tc_supported(const Dims &dm) {
  return dm.C <= 32 && (dm.P == 16 || dm.P == 32) && dm.SM * dm.PPS <= SMAXLIST &&
         (dm.pos_mode != PD_POS_T5_BIAS || dm.n_dist <= SMAXDIST);
}

template <int MT, int P>
static cudaError_t prepare_one() {
  return cudaFuncSetAttribute(self_attn_tc_kernel<MT, P>, cudaFuncAttributeMaxDynamicSharedMemorySize, self_attn_tc_smem(P, MT));
}

cudaError_t self_attn_tc_prepare() {
  cudaError_t e = prepare_one<1, 16>();
  if (e == cudaSuccess) e = prepare_one<2, 16>();
  if (e == cudaSuccess) e = prepare_one<1, 32>();
  if (e == cudaSuccess) e = prepare_one<2, 32>();
  return e;
}

cudaError_t launch_self_attn_tc(const AttnArgs &a, cudaStream_t s) {
  dim3 grid(a.splits, a.dm.H, a.batch);
  const int mt = (a.dm.C + 15) / 16;
  const int smem = self_attn_tc_smem(a.dm.P, mt);
  if (mt == 1 && a.dm.P == 16) self_attn_tc_kernel<1, 16><<<grid, STHREADS, smem, s>>>(a);
  else if (mt == 2 && a.dm.P == 16) self_attn_tc_kernel<2, 16><<<grid, STHREADS, smem, s>>>(a);
  else if (mt == 1 && a.dm.P == 32) self_attn_tc_kernel<1, 32><<<grid, STHREADS, smem, s>>>(a);
  else if (mt == 2 && a.dm.P == 32) self_attn_tc_kernel<2, 32><<<grid, STHREADS, smem, s>>>(a);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace pd
