// Pipelined self-attention for bf16 storage (sm_100a): decode attention of all active
// subsequences of a sequence over the paged per-subsequence KV cache, with the dependency rule
// of Section 3.2 (a query of subsequence i sees subsequences i' <= i as generated so far)
// evaluated per key from (subsequence, position) metadata - no mask is ever stored -
// and the step's KV-append with its positional write (Eq. 2: the entry's position is tau + i)
// done by the same launch.
//
// All S active rows of a sequence share its cache, so one key/value block serves up to S
// queries: with S around 8-16 the scores are far too many flops for the plain ALUs to keep
// up with HBM, so scores and P.V run on tensor cores (mma.sync m16n8k16, bf16 in, fp32
// accumulate) with the visibility rule and the T5 bias applied to the accumulator fragment.
//
// What a launch costs is set by the number of iterations of its busiest warp, and an iteration costs
// the same whether its 16 key slots are full or not.  Pages are per subsequence, so most of a sequence's
// pages are partly filled (a 21-entry subsequence holds two pages): walking pages made a warp do up to
// three times the iterations its keys needed.  The kernel therefore walks KEYS: from the page list the
// scheduler leaves once per step (page, entries, subsequence, first position) the CTA builds, in shared
// memory, the flat list of the entries that exist - where each lies (page, slot), its subsequence and
// its distance base - and its warps take tiles of 16 consecutive keys of that list, whatever pages
// they come from.  A tile is gathered into the warp's private two-slot ring with 16-byte cp.async
// (the cache rows are stored pre-swizzled by their slot; the copy re-swizzles them by their place in
// the tile, so that ldmatrix reads without bank conflicts); one CTA = one (split, head, sequence).
//
// Fused append: the entries the rows feed at this step are written to the cache by the same launch,
// in its prologue: warp w takes rows w, w + 4, ...; their keys and values of this head come straight from
// the projection's output (bf16 when nothing is rotated; fp32, rotated by the position tau + i and
// rounded, in rotary mode), requested in the first round of loads and stored once the rows' slots are
// known.  After the CTA's barrier they are cache entries like any other.  Queries come from the same
// projection output (rotated likewise).  Split CTAs of one (sequence, head) write the same bits.
//
// Splits: the number of splits in use follows the key list's length (a CTA whose split is not needed
// leaves at once).  Warps merge through shared memory; split CTAs leave a partial record, take a
// ticket, and the last one to arrive merges the records in split order (deterministic) and writes
// the output - no merge launch, and no CTA ever waits for another.
#include "pd_internal.h"

namespace pd {

constexpr int SW = 4;                      // worker warps per CTA
constexpr int STHREADS = SW * 32;
constexpr int SDEPTH = 2;                  // ring slots per warp: the tile in use and the next one
constexpr int STK = 16;                    // keys per tile
constexpr uint32_t SSLOT = STK * 256u;     // keys + values of one tile of one head (4 KB)
constexpr int SMAXLIST = 256;              // page-list entries of one sequence held in shared memory
constexpr int SMAXDIST = 512;
constexpr int SMROW = kDh + 8;             // row stride of the merge scratch in floats (spreads the eight fragment rows over the banks)
// Tiles a warp walks before another split is used: a tile costs a warp ~0.75 us, a split ~4 us of fixed cost
// (partial records, fence, ticket, the last CTA's read-back), so a split pays once it saves about six tiles per warp.
constexpr int STILES_PER_WARP = 10;
constexpr int SBIAS_PER_THREAD = (SMAXDIST + STHREADS - 1) / STHREADS;

__device__ __forceinline__ uint32_t s_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// 16-byte asynchronous copy global -> shared
__device__ __forceinline__ void s_cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void s_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void s_cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void s_st_shared_u32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
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
// Byte offset of 16-byte chunk `chunk` of key row `row` inside a batch slot (256 bytes per entry:
// swizzled key row, then swizzled value row at + 128).  Pages are 16 or 32 entries, so the
// swizzle phase (row & 7) of an entry is the same in the slot as in its page.
__device__ __forceinline__ uint32_t s_swz(int row, int chunk) { return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4)); }

// Bytes of the rings (or of the merge scratch that reuses them, whichever is larger).
__host__ __device__ constexpr int self_attn_tc_ring_bytes(int mt) {
  return SW * SDEPTH * (int)SSLOT > SW * 16 * mt * (SMROW + 2) * 4 ? SW * SDEPTH * (int)SSLOT : SW * 16 * mt * (SMROW + 2) * 4;
}

// MT = 16-row query tiles (rows per sequence <= 16 * MT); P = page_tokens; MODE 0 = the launch follows the append
// kernel (queries in a.q); 1 = it appends the step's keys/values itself from the projection's bf16 output a.qkv;
// 2 = the same from an fp32 output that it rotates by the rows' positions first (rotary mode)
// OCC = CTAs per SM the register budget is set for: four leave the compiler 128 registers (nothing spills),
// five 96 (more CTAs resident, which wins when there are more (sequence, head) pairs than four per SM)
template <int MT, int P, int MODE, int OCC>
__global__ void __launch_bounds__(STHREADS, MT == 1 ? OCC : 2) self_attn_tc_kernel(AttnArgs a) {
  // dynamic shared memory: the warps' rings (reused as merge scratch), the sequence's page list, the exclusive
  // prefix of its entry counts, the flat key list (where the key lies; its subsequence and distance base), and
  // this head's bias row
  extern __shared__ __align__(128) uint8_t s_ring_raw[];
  __shared__ int rsub_s[16 * MT];          // subsequence of row r
  __shared__ int last_s, n_keys_s;

  const Dims &dm = a.dm;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row0 = b * dm.C;
  __nv_bfloat16 *out = (__nv_bfloat16 *)a.out;
  const int g = lane >> 2, tig = lane & 3;
  const int list_cap = dm.SM * dm.PPS;
  int4 *plist_s = reinterpret_cast<int4 *>(s_ring_raw + self_attn_tc_ring_bytes(MT));
  int *off_s = reinterpret_cast<int *>(plist_s + list_cap);                  // [list_cap + 1]
  int2 *key_s = reinterpret_cast<int2 *>(off_s + ((list_cap + 1 + 1) & ~1));   // [list_cap * P]: (page * 32 + slot, subsequence | (distance base + 1024) << 8)
  float *bias_s = reinterpret_cast<float *>(key_s + (size_t)list_cap * P);

  // ---- ONE round of independent global loads, none waiting for another: active-row count, page list, row ->
  // subsequence, where every row's new entry goes, bias row of this head, query fragments, and (fused modes) the
  // new keys/values of the rows this warp appends.  What turns out to be unused is masked afterwards.
  const int S = a.st.n_active[b];
  const int n_list = a.st.plist_n[b];
  const int4 *pl = a.st.plist + (size_t)b * list_cap;
  int4 my_entry[(SMAXLIST + STHREADS - 1) / STHREADS];
#pragma unroll
  for (int k = 0; k < (SMAXLIST + STHREADS - 1) / STHREADS; ++k)
    my_entry[k] = k * STHREADS + tid < list_cap ? pl[k * STHREADS + tid] : make_int4(0, 0, 0, 0);
  int my_rsub = 0;
  if (tid < dm.C) my_rsub = a.st.row_sub[row0 + tid];
  // (page, slot, position tau + i, subsequence) of the entry row `lane` of this sequence appends at this step
  const int4 meta = (MODE != 0 && lane < dm.C) ? a.st.row_meta[row0 + lane] : make_int4(-1, 0, 0, 0);
  const bool use_bias = a.bias_tab != nullptr;
  float my_bias[SBIAS_PER_THREAD];
#pragma unroll
  for (int k = 0; k < SBIAS_PER_THREAD; ++k) {
    const int dd = k * STHREADS + tid;
    my_bias[k] = (use_bias && dd < dm.n_dist) ? a.bias_tab[h * dm.n_dist + dd] : 0.f;
  }
  uint32_t qf[MT][4][4];
  if (MODE != 2) {
    const __nv_bfloat16 *qsrc = MODE == 1 ? (const __nv_bfloat16 *)a.qkv : (const __nv_bfloat16 *)a.q;
    const size_t qstride = MODE == 1 ? 3 * (size_t)dm.d : (size_t)dm.d;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
      const __nv_bfloat16 *q_lo = qsrc + (size_t)(row0 + r_lo) * qstride + h * kDh + 2 * tig;
      const __nv_bfloat16 *q_hi = qsrc + (size_t)(row0 + r_hi) * qstride + h * kDh + 2 * tig;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        qf[mt][kk][0] = r_lo < dm.C ? *reinterpret_cast<const uint32_t *>(q_lo + kk * 16) : 0u;
        qf[mt][kk][1] = r_hi < dm.C ? *reinterpret_cast<const uint32_t *>(q_hi + kk * 16) : 0u;
        qf[mt][kk][2] = r_lo < dm.C ? *reinterpret_cast<const uint32_t *>(q_lo + kk * 16 + 8) : 0u;
        qf[mt][kk][3] = r_hi < dm.C ? *reinterpret_cast<const uint32_t *>(q_hi + kk * 16 + 8) : 0u;
      }
    }
  }
  // the new entries this warp appends (rows warp, warp + SW, ...): lane l holds columns 2 l, 2 l + 1 of key and value
  constexpr int APW = (16 * MT + SW - 1) / SW;
  uint32_t new_k[APW], new_v[APW];
  float2 new_kf[MODE == 2 ? APW : 1], new_vf[MODE == 2 ? APW : 1];
  if (MODE == 1) {
#pragma unroll
    for (int j = 0; j < APW; ++j) {
      const int c = warp + j * SW;
      new_k[j] = new_v[j] = 0u;
      if (c < dm.C) {
        const __nv_bfloat16 *src = (const __nv_bfloat16 *)a.qkv + (size_t)(row0 + c) * 3 * dm.d + dm.d + (size_t)h * kDh + 2 * lane;
        new_k[j] = *reinterpret_cast<const uint32_t *>(src);
        new_v[j] = *reinterpret_cast<const uint32_t *>(src + dm.d);
      }
    }
  } else if (MODE == 2) {
#pragma unroll
    for (int j = 0; j < APW; ++j) {
      const int c = warp + j * SW;
      new_kf[j] = new_vf[j] = make_float2(0.f, 0.f);
      if (c < dm.C) {
        const float *src = (const float *)a.qkv + (size_t)(row0 + c) * 3 * dm.d + dm.d + (size_t)h * kDh + 2 * lane;
        new_kf[j] = *reinterpret_cast<const float2 *>(src);
        new_vf[j] = *reinterpret_cast<const float2 *>(src + dm.d);
      }
    }
  }

  if (S == 0) {   // nothing active: keep the output rows of this head defined
    if (split == 0)
      for (int idx = tid; idx < dm.C * kDh; idx += STHREADS)
        out[(size_t)(row0 + idx / kDh) * dm.d + h * kDh + idx % kDh] = __float2bfloat16_rn(0.f);
    return;
  }
  const __nv_bfloat16 *pool_lh = (const __nv_bfloat16 *)a.kv + kv_block_offset(a.layer, dm.pool, 0, dm.H, h, P);
  const size_t page_stride = (size_t)dm.H * 2 * P * kDh;      // elements from one page's block of this head to the next page's

  // ---- append (every CTA of the (sequence, head) pair writes the same bits) and, in rotary mode, the queries
  if (MODE == 2) {
    const float *qkv32 = reinterpret_cast<const float *>(a.qkv);
#pragma unroll
    for (int j = 0; j < APW; ++j) {
      const int c = warp + j * SW;
      if (c < S) {
        const int pos = __shfl_sync(0xffffffffu, meta.z, c);
        const float2 cs = a.rope_tab[(size_t)pos * (kDh / 2) + lane];
        new_k[j] = s_pack_bf16(new_kf[j].x * cs.x - new_kf[j].y * cs.y, new_kf[j].x * cs.y + new_kf[j].y * cs.x);
        new_v[j] = s_pack_bf16(new_vf[j].x, new_vf[j].y);
      }
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int r = mt * 16 + g + 8 * hh;
        const int pos = __shfl_sync(0xffffffffu, meta.z, r & 31);
        float2 v[8], c2[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {         // columns kk * 16 + 2 tig (+ 8): j = 2 kk + half
          const int col = (j >> 1) * 16 + 2 * tig + (j & 1) * 8;
          v[j] = make_float2(0.f, 0.f); c2[j] = make_float2(1.f, 0.f);
          if (r < S) {
            v[j] = *reinterpret_cast<const float2 *>(qkv32 + (size_t)(row0 + r) * 3 * dm.d + (size_t)h * kDh + col);
            c2[j] = a.rope_tab[(size_t)pos * (kDh / 2) + col / 2];
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
          qf[mt][j >> 1][hh + 2 * (j & 1)] = s_pack_bf16(v[j].x * c2[j].x - v[j].y * c2[j].y, v[j].x * c2[j].y + v[j].y * c2[j].x);
      }
    }
  }
  if (MODE != 0) {
#pragma unroll
    for (int j = 0; j < APW; ++j) {
      const int c = warp + j * SW;
      if (c < S) {
        const int page = __shfl_sync(0xffffffffu, meta.x, c), slot = __shfl_sync(0xffffffffu, meta.y, c);
        __nv_bfloat16 *cache = const_cast<__nv_bfloat16 *>(pool_lh) + page * page_stride + kv_entry_offset<__nv_bfloat16>(slot, 2 * lane, 0);
        *reinterpret_cast<uint32_t *>(cache) = new_k[j];
        *reinterpret_cast<uint32_t *>(cache + kDh) = new_v[j];      // the value row follows the key row of the same entry
      }
    }
  }

  // ---- the page list in shared memory, the exclusive prefix of its entry counts, the flat key list
#pragma unroll
  for (int k = 0; k < (SMAXLIST + STHREADS - 1) / STHREADS; ++k)
    if (k * STHREADS + tid < list_cap) plist_s[k * STHREADS + tid] = my_entry[k];
  if (tid < 16 * MT) rsub_s[tid] = my_rsub;
#pragma unroll
  for (int k = 0; k < SBIAS_PER_THREAD; ++k)
    if (use_bias && k * STHREADS + tid < dm.n_dist) bias_s[k * STHREADS + tid] = my_bias[k];
  __syncthreads();          // (also: this CTA's appended entries are in the cache for all its warps)
  if (warp == 0) {
    int carry = 0;
    for (int j0 = 0; j0 < n_list; j0 += 32) {
      const int nv = j0 + lane < n_list ? plist_s[j0 + lane].y : 0;
      int incl = nv;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += u; }
      if (j0 + lane < n_list) off_s[j0 + lane] = carry + incl - nv;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) n_keys_s = carry;
  }
  __syncthreads();
  for (int j = tid; j < n_list; j += STHREADS) {
    const int4 e = plist_s[j];
    const int o0 = off_s[j];
    for (int k = 0; k < e.y; ++k)      // entry k of the page: its distance base is the page's minus its offset
      key_s[o0 + k] = make_int2(e.x * 32 + k, e.z | ((e.w - k + 1024) << 8));
  }
  __syncthreads();
  const int n_keys = n_keys_s;

  // splits in use: enough that a warp gets about STILES_PER_WARP tiles, at most the launched ones
  const int n_tiles = (n_keys + STK - 1) / STK;
  const int n_eff = min(a.splits, max(1, (n_tiles + SW * STILES_PER_WARP - 1) / (SW * STILES_PER_WARP)));
  if (split >= n_eff) return;
  const int W = n_eff * SW, g0 = split * SW + warp;
  const int n_mine = n_tiles > g0 ? (n_tiles - g0 + W - 1) / W : 0;
  const uint32_t my_ring = s_smem_u32(s_ring_raw) + warp * SDEPTH * SSLOT;

  // Tile n of this warp = keys 16 (g0 + n W) ... of the flat list.  Lane l copies, in eight rounds, one 16-byte chunk
  // each: round k covers keys 2 k and 2 k + 1, chunks 0-7 = the key row, 8-15 = the value row.  A cache row's chunk c
  // lies at place c ^ (slot & 7) of its row; in the tile it goes to place c ^ (row in tile & 7).
  auto fetch = [&](int n) {
    const int first = STK * (g0 + n * W);
    const uint32_t dst = my_ring + (n % SDEPTH) * SSLOT;
#pragma unroll
    for (int k = 0; k < STK / 2; ++k) {
      const int r = 2 * k + (lane >> 4), p = lane & 15;
      if (first + r < n_keys) {
        const int src = key_s[first + r].x;
        const int page = src >> 5, slot = src & 31;
        const uint8_t *from = reinterpret_cast<const uint8_t *>(pool_lh + page * page_stride) + slot * 256 + p * 16;
        const int place = (p & 7) ^ (slot & 7) ^ (r & 7);
        s_cp_async16(dst + r * 256 + (p & 8) * 16 + place * 16, from);
      }
    }
  };
  // Nothing is ever cleared: what a slot holds beyond the list's last key (anything) gets score -inf, and the value
  // fragments of those keys are zeroed in registers after ldmatrix.
#pragma unroll
  for (int n = 0; n < SDEPTH; ++n) {
    if (n < n_mine) fetch(n);
    s_cp_async_commit();
  }

  int rs[MT][2];                     // subsequence of rows g and g + 8 of every query tile
  int tile_last[MT];                 // subsequence of the tile's last active row (rows are sorted)
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    rs[mt][0] = rsub_s[min(mt * 16 + g, S - 1)];           // unused rows repeat the last active one
    rs[mt][1] = rsub_s[min(mt * 16 + g + 8, S - 1)];
    tile_last[mt] = 16 * mt < S ? rsub_s[min(16 * mt + 15, S - 1)] : 0;
  }
  const int sub_first = rsub_s[0];   // the smallest active subsequence: a key it sees, every row sees
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
    s_cp_async_wait<SDEPTH - 1>();     // everything but the newest group has landed: tile n is in its slot
    __syncwarp();
    const int first = STK * (g0 + n * W);
    const int nv = min(STK, n_keys - first);           // keys of this tile that exist
    // this thread's four keys of the tile (two per 8-key score tile): subsequence and distance base
    int ksub[2][2], kd[2][2];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const int e = nt * 8 + 2 * tig + x;
        const int m = e < nv ? key_s[first + e].y : 0x7f;     // absent: a subsequence no row reaches
        ksub[nt][x] = m & 0xff; kd[nt][x] = (m >> 8) - 1024;
      }
    const int k_first = key_s[first].y & 0xff, k_last = key_s[first + nv - 1].y & 0xff;   // keys are sorted by subsequence
    const uint32_t kbase = my_ring + (n % SDEPTH) * SSLOT, vbase = kbase + 128u;
    // Dependency rule: a row of subsequence i sees a key iff i' <= i (every stored entry was generated
    // before the current step).  A query tile none of whose rows sees the tile's first key is skipped;
    // a full tile that every row sees needs no masking at all.
    bool act[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) act[mt] = tile_last[mt] >= k_first;
    const bool plain = nv == STK && sub_first >= k_last;

    // ---- scores: Q (16 x 64) . K^T (64 x 16 keys); two accumulators per tile halve the mma chain
    float sc[MT][2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
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
    // ---- scale, positional bias on the Manhattan distance (the key's distance base + the row's subsequence),
    // visibility, online softmax (log2 domain)
    uint32_t pf[MT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      if (!act[mt]) continue;
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int kx = x & 1, hh = x >> 1;
          const bool vis = plain || (ksub[nt][kx] <= rs[mt][hh]);       // (an absent key's subsequence is beyond every row)
          float v = -INFINITY;
          if (vis) {
            const float bias = use_bias ? bias_s[kd[nt][kx] + rs[mt][hh]] : 0.f;
            v = fmaf(sc[mt][nt][x], sl2, bias);
          }
          sc[mt][nt][x] = v;
        }
        mx0 = fmaxf(mx0, fmaxf(sc[mt][nt][0], sc[mt][nt][1]));
        mx1 = fmaxf(mx1, fmaxf(sc[mt][nt][2], sc[mt][nt][3]));
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
      for (int nt = 0; nt < 2; ++nt) {
        float p0 = s_ex2(sc[mt][nt][0] - ref0), p1 = s_ex2(sc[mt][nt][1] - ref0);
        float p2 = s_ex2(sc[mt][nt][2] - ref1), p3 = s_ex2(sc[mt][nt][3] - ref1);
        s0 += p0 + p1; s1 += p2 + p3;
        pf[mt][nt * 2 + 0] = s_pack_bf16(p0, p1);
        pf[mt][nt * 2 + 1] = s_pack_bf16(p2, p3);
      }
      l_run[mt][0] = l_run[mt][0] * cr0 + s0;
      l_run[mt][1] = l_run[mt][1] * cr1 + s1;
      if (__any_sync(0xffffffffu, cr0 != 1.f || cr1 != 1.f)) {   // some row's running maximum moved
#pragma unroll
        for (int dn = 0; dn < 8; ++dn) { o[mt][dn][0] *= cr0; o[mt][dn][1] *= cr0; o[mt][dn][2] *= cr1; o[mt][dn][3] *= cr1; }
      }
    }
    // ---- O += P (16 x 16 keys) . V (16 keys x 64)
    {
      const int vkey = ((lane >> 3) & 1) * 8 + (lane & 7);
      // this lane's fragment halves hold keys k0, k0 + 1 (b0, b2) and k0 + 8, k0 + 9 (b1, b3) of the tile;
      // keys that do not exist have weight exactly 0 and must not contribute whatever the slot holds
      const bool ragged = nv < STK;
      uint32_t keep_a = 0xffffffffu, keep_b = 0xffffffffu;
      if (ragged) {
        const int k0 = 2 * tig;
        keep_a = (k0 < nv ? 0x0000ffffu : 0u) | (k0 + 1 < nv ? 0xffff0000u : 0u);
        keep_b = (k0 + 8 < nv ? 0x0000ffffu : 0u) | (k0 + 9 < nv ? 0xffff0000u : 0u);
      }
#pragma unroll
      for (int dp = 0; dp < 4; ++dp) {
        uint32_t b0, b1, b2, b3;
        s_ldsm_x4_t(vbase + s_swz(vkey, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
        if (ragged) { b0 &= keep_a; b1 &= keep_b; b2 &= keep_a; b3 &= keep_b; }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          if (!act[mt]) continue;
          s_mma_bf16(o[mt][2 * dp], pf[mt][0], pf[mt][1], pf[mt][2], pf[mt][3], b0, b1);
          s_mma_bf16(o[mt][2 * dp + 1], pf[mt][0], pf[mt][1], pf[mt][2], pf[mt][3], b2, b3);
        }
      }
    }
    __syncwarp();   // every lane is done reading the slot
    if (n + SDEPTH < n_mine) fetch(n + SDEPTH);
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
  __syncthreads();   // every warp is past its last batch: the ring can be reused
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
    if (n_eff == 1) {
      const float inv = 1.f / ml[r];
      *reinterpret_cast<__nv_bfloat162 *>(out + orow) = __floats2bfloat162_rn(O.x * inv, O.y * inv);
    } else {
      const size_t pi = ((size_t)(row0 + r) * dm.H + h) * a.splits + split;
      *reinterpret_cast<float2 *>(&a.part_o[pi * kDh + col]) = O;
      if (col == 0) { a.part_ml[pi * 2] = ml[ROWS + r]; a.part_ml[pi * 2 + 1] = ml[r]; }
    }
  }
  if (n_eff == 1) return;

  // ---- several splits: the CTA that arrives last for this (sequence, head) merges the records in split order
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(&a.tickets[b * dm.H + h], 1);
    last_s = ticket == n_eff - 1;
    if (last_s) a.tickets[b * dm.H + h] = 0;     // zero again for the next launch (every other CTA of the pair has arrived)
  }
  __syncthreads();
  if (!last_s) return;
  __threadfence();
  for (int idx = tid; idx < S * (kDh / 2); idx += STHREADS) {
    const int r = idx / (kDh / 2), col = 2 * (idx % (kDh / 2));
    const size_t p0 = ((size_t)(row0 + r) * dm.H + h) * a.splits;
    float M = -INFINITY;
    for (int s = 0; s < n_eff; ++s) M = fmaxf(M, __ldcg(&a.part_ml[(p0 + s) * 2]));
    float L = 0.f;
    float2 O = make_float2(0.f, 0.f);
    for (int s = 0; s < n_eff; ++s) {
      const float m = __ldcg(&a.part_ml[(p0 + s) * 2]);
      if (m == -INFINITY) continue;
      const float w = s_ex2(m - M);
      L += __ldcg(&a.part_ml[(p0 + s) * 2 + 1]) * w;
      const float2 v = __ldcg(reinterpret_cast<const float2 *>(&a.part_o[(p0 + s) * kDh + col]));
      O.x += v.x * w; O.y += v.y * w;
    }
    const float inv = 1.f / L;
    *reinterpret_cast<__nv_bfloat162 *>(out + (size_t)(row0 + r) * dm.d + h * kDh + col) = __floats2bfloat162_rn(O.x * inv, O.y * inv);
  }
}

static int self_attn_tc_smem(const Dims &dm) {
  const int mt = (dm.C + 15) / 16, list_cap = dm.SM * dm.PPS;
  return self_attn_tc_ring_bytes(mt) + list_cap * (int)sizeof(int4) + ((list_cap + 2) & ~1) * 4 + list_cap * dm.P * (int)sizeof(int2) +
         (dm.pos_mode == PD_POS_T5_BIAS ? dm.n_dist * 4 : 0);
}

bool self_attn_tc_supported(const Dims &dm) {
  return dm.C <= 32 && (dm.P == 16 || dm.P == 32) && dm.SM * dm.PPS <= SMAXLIST && dm.SM <= 127 &&
         (dm.pos_mode != PD_POS_T5_BIAS || dm.n_dist <= SMAXDIST) && self_attn_tc_smem(dm) <= 200 * 1024;
}

// Splits to launch for `pairs` (sequence, head) pairs on a device with `sms` SMs: enough for the
// longest key list a sequence can have (CTAs whose split the current lists do not need leave at
// once), but never more CTAs than are resident at the same time - a second wave costs a whole
// CTA lifetime, a longer walk per warp a fraction of one.
int self_attn_tc_splits(const Dims &dm, int pairs, int sms) {
  const int tiles = (dm.SM * (dm.MSL + 2) + STK - 1) / STK;
  int s = (tiles + SW * STILES_PER_WARP - 1) / (SW * STILES_PER_WARP);
  // CTAs an SM holds: five by registers (two with 32 rows), and what 227 KB of shared memory allow
  const int by_smem = (227 * 1024) / (self_attn_tc_smem(dm) + 1024 + 256);
  const int per_sm = dm.C <= 16 ? (by_smem < 5 ? by_smem : 5) : (by_smem < 2 ? by_smem : 2);
  const int resident = (per_sm < 1 ? 1 : per_sm) * sms;
  if (s > resident / (pairs > 0 ? pairs : 1)) s = resident / (pairs > 0 ? pairs : 1);
  return s < 1 ? 1 : (s > 8 ? 8 : s);
}

template <int MT, int P>
static cudaError_t prepare_one() {
  const int smem = 200 * 1024;
  cudaError_t e = cudaFuncSetAttribute(self_attn_tc_kernel<MT, P, 0, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(self_attn_tc_kernel<MT, P, 1, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(self_attn_tc_kernel<MT, P, 2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(self_attn_tc_kernel<MT, P, 0, 5>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(self_attn_tc_kernel<MT, P, 1, 5>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(self_attn_tc_kernel<MT, P, 2, 5>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  return e;
}

cudaError_t self_attn_tc_prepare() {
  cudaError_t e = prepare_one<1, 16>();
  if (e == cudaSuccess) e = prepare_one<2, 16>();
  if (e == cudaSuccess) e = prepare_one<1, 32>();
  if (e == cudaSuccess) e = prepare_one<2, 32>();
  return e;
}

// a.fused_append 1: a.qkv = the projection's output [rows][3 d] in bf16; 2: in fp32, rotated here with a.rope_tab;
// 0: a.q = the queries the append kernel left.  a.tickets one zeroed int32 per (sequence, head) (the kernel leaves them zeroed), a.part_o /
// a.part_ml sized for a.splits records per (row, head).
cudaError_t launch_self_attn_tc(const AttnArgs &a, cudaStream_t s) {
  dim3 grid(a.splits, a.dm.H, a.batch);
  const int mt = (a.dm.C + 15) / 16;
  const int smem = self_attn_tc_smem(a.dm);
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const bool roomy = (long long)a.splits * a.dm.H * a.batch <= 4LL * sms;      // all CTAs resident at four per SM
#define PD_SELF_LAUNCH(MT_, P_)                                                                            \
  do {                                                                                                   \
    if (a.fused_append == 1 && roomy) self_attn_tc_kernel<MT_, P_, 1, 4><<<grid, STHREADS, smem, s>>>(a);        \
    else if (a.fused_append == 1) self_attn_tc_kernel<MT_, P_, 1, 5><<<grid, STHREADS, smem, s>>>(a);            \
    else if (a.fused_append == 2 && roomy) self_attn_tc_kernel<MT_, P_, 2, 4><<<grid, STHREADS, smem, s>>>(a);   \
    else if (a.fused_append == 2) self_attn_tc_kernel<MT_, P_, 2, 5><<<grid, STHREADS, smem, s>>>(a);            \
    else if (roomy) self_attn_tc_kernel<MT_, P_, 0, 4><<<grid, STHREADS, smem, s>>>(a);                          \
    else self_attn_tc_kernel<MT_, P_, 0, 5><<<grid, STHREADS, smem, s>>>(a);                                     \
  } while (0)
  if (mt == 1 && a.dm.P == 16) PD_SELF_LAUNCH(1, 16);
  else if (mt == 2 && a.dm.P == 16) PD_SELF_LAUNCH(2, 16);
  else if (mt == 1 && a.dm.P == 32) PD_SELF_LAUNCH(1, 32);
  else if (mt == 2 && a.dm.P == 32) PD_SELF_LAUNCH(2, 32);
  else return cudaErrorInvalidValue;
#undef PD_SELF_LAUNCH
  return cudaGetLastError();
}

}  // namespace pd
