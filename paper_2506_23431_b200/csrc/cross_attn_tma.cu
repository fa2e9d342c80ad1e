// Batched cross-attention for the bf16 path (sm_100a): every active subsequence of a sequence
// is a query row against the shared encoder keys/values (all context positions < ctx_len
// visible, no positional term).  This is the one part of the step that is a dense S x L_ctx
// contraction, so it runs on tensor cores; it stays HBM-bound (about S flop per byte).
//
// Persistent kernel, two CTAs per SM.  The 128-key tiles of all (sequence with an active row,
// head) pairs form one flat list.  With enough (sequence, head) segments every CTA takes the same
// number of whole segments (nothing is cut: no partial records, no merge); with few segments left
// the list is cut into equal contiguous ranges, one per CTA, so that the GPU stays full.  Either
// way there are no partial waves.  In every CTA a producer warp streams the K and V tiles of its range
// (16 KB each, contiguous) through a ring of shared-memory stages with TMA (cp.async.bulk.tensor.2d,
// 128-byte swizzle, completion on an mbarrier) without stopping at (sequence, head) boundaries;
// four consumer warps each take 32 keys of every tile: S = Q K^T with mma.sync m16n8k16 (bf16 in,
// fp32 accumulate), online softmax in the log2 domain with quad shuffles, O += P V.  At the end
// of a (sequence, head) segment the warps' (m, l, O) are tree-merged through shared memory into
// warp 0.  A segment that covers the whole context is written out; otherwise warp 0 stores the
// partial record, takes a ticket, and the CTA that arrives last for that (sequence, head) merges
// all records in CTA order (deterministic) and writes the output - no CTA ever waits for another.
// Every mbarrier wait is bounded: on expiry the kernel records PD_ERR_TIMEOUT and drains.
//
// 8-bit variant (FP8 = true): the context keys/values are E4M3 codes with one scale per (layer,
// sequence, head, keys | values) - half the bytes of the dominant term of a decode step.  Keys are
// stored [position][64] (a 128-key tile is 64 lines of 128 bytes), values transposed [dim][position],
// so that both reach the tensor cores through plain ldmatrix: a thread's 32-bit fragment word holds
// four consecutive codes (four dims of a key, or four keys of a dim), widened to two f16 pairs in
// registers (cvt.rn.f16x2.e4m3x2, exact).  The order of the sixteen dims (keys) inside a k16 step is
// therefore 4 tig + {0, 1} | 4 tig + {2, 3} instead of 2 tig + {0, 1} | 2 tig + 8 + {0, 1}; queries
// (score columns) are loaded with the same permutation, which a contraction does not see.  Queries and
// softmax weights go through f16 (exact for bf16 queries in f16's range; 11 bits for the weights), the
// key scale is folded into the score scale and the value scale into the final 1 / l.  Stages are 16 KB,
// the ring six deep.
#include <cuda_fp16.h>

#include "pd_internal.h"

namespace pd {

constexpr int XK = 128;                   // keys per tile
// ring: three 32 KB stages (bf16) or six 16 KB stages (8-bit); with the merge scratch two CTAs fit an SM
__host__ __device__ constexpr int xring_bytes(bool fp8) { return fp8 ? 96 * 1024 : 96 * 1024; }
// consumer warps: four, each taking 32 keys of a tile.  (Eight warps of 16 keys each were measured in both
// variants and lost: 50.3 against 49.2 us per full bf16 launch, 31.9 against 28.7 us per 8-bit launch.)
__host__ __device__ constexpr int xcw(bool fp8) { return fp8 ? 4 : 4; }
__host__ __device__ constexpr int xthreads(bool fp8) { return (xcw(fp8) + 1) * 32; }
constexpr int XMIN_TILES = 4;              // fewest tiles worth a CTA of its own
constexpr int XMIN_WHOLE = 64;             // fewest CTAs for which whole (sequence, head) segments per CTA still beat cutting the tile list
constexpr int XLONG_SEG = 24;              // tiles from which a segment is worth two CTAs when there are fewer segments than SMs
constexpr int XMAXB = 256;                // sequences per launch the tile prefix table holds
constexpr int XREC_WORDS = 36;            // per lane and 16-row tile: 32 output values, 2 maxima, 2 sums
constexpr int XREC_FLOATS = XREC_WORDS * 32;
__host__ __device__ constexpr int xscratch_bytes(bool fp8) { return (xcw(fp8) / 2) * XREC_FLOATS * 4; }   // half the consumer warps' records for the tree merge
__host__ __device__ constexpr int xsmem(bool fp8) { return xring_bytes(fp8) + xscratch_bytes(fp8) + 128 /*barriers*/ + 1024 /*alignment slack*/; }
constexpr uint32_t XSPIN_LIMIT = 1u << 24;

int cross_attn_tma_smem_bytes() { return xsmem(false); }
size_t cross_attn_tma_partial_bytes(int n_ctas, int rows_per_seq) {
  return (size_t)n_ctas * 2 * ((rows_per_seq + 15) / 16) * XREC_FLOATS * sizeof(float);
}
bool cross_attn_tma_supported(const Dims &dm, int batch) { return dm.C <= 32 && batch <= XMAXB; }

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
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tmap, uint32_t bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tmap), "r"(bar), "r"(x), "r"(y), "r"(z)
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
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
// two E4M3 codes (the low or the high half of a fragment word) -> f16 pair; every E4M3 value is an f16 value.
// (Widening with integer instructions instead - byte permute, shift, mask: the codes' values times 2^-8 -
// gave the same results and a slower kernel: 39 against 30 us per launch.)
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t word, int high) {
  uint32_t r;
  const unsigned short v = (unsigned short)(high ? (word >> 16) : (word & 0xffffu));
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
  return r;
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&w);
  const __half2 hh = __float22half2_rn(__bfloat1622float2(b));
  return *reinterpret_cast<const uint32_t *>(&hh);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
template <int THREADS> __device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory"); }

// Byte offset of (row, 16-byte chunk) inside a 128-byte-swizzled tile whose rows are 128 bytes.
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ float ex2f(float x) {   // 2^x; ex2(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// One warp's (or one CTA's) state for a 16-row query tile in mma fragment layout: this lane holds
// columns dn*8 + 2*tig, +1 of rows g (o[dn][0..1], m0, l0) and g + 8 (o[dn][2..3], m1, l1).
struct TileAcc {
  float o[8][4];
  float m0, m1, l0, l1;
  __device__ __forceinline__ void clear() {
    m0 = m1 = -INFINITY; l0 = l1 = 0.f;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) o[dn][0] = o[dn][1] = o[dn][2] = o[dn][3] = 0.f;
  }
  // record layout [word][lane]: consecutive lanes touch consecutive words (coalesced, no bank conflicts)
  __device__ __forceinline__ void store(float *rec, int lane) const {
#pragma unroll
    for (int dn = 0; dn < 8; ++dn)
#pragma unroll
      for (int x = 0; x < 4; ++x) rec[(dn * 4 + x) * 32 + lane] = o[dn][x];
    rec[32 * 32 + lane] = m0; rec[33 * 32 + lane] = m1; rec[34 * 32 + lane] = l0; rec[35 * 32 + lane] = l1;
  }
  // acc <- acc (+) record, the log-sum-exp merge of two partial softmax states
  template <bool GLOBAL>
  __device__ __forceinline__ void merge(const float *rec, int lane) {
    auto ld = [&](int w) { return GLOBAL ? __ldcg(rec + w * 32 + lane) : rec[w * 32 + lane]; };
    const float om0 = ld(32), om1 = ld(33), ol0 = ld(34), ol1 = ld(35);
    const float M0 = fmaxf(m0, om0), M1 = fmaxf(m1, om1);
    const float r0 = M0 == -INFINITY ? 0.f : M0, r1 = M1 == -INFINITY ? 0.f : M1;
    const float a0 = ex2f(m0 - r0), b0 = ex2f(om0 - r0), a1 = ex2f(m1 - r1), b1 = ex2f(om1 - r1);
    m0 = M0; m1 = M1;
    l0 = l0 * a0 + ol0 * b0; l1 = l1 * a1 + ol1 * b1;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) {
      o[dn][0] = o[dn][0] * a0 + ld(dn * 4 + 0) * b0;
      o[dn][1] = o[dn][1] * a0 + ld(dn * 4 + 1) * b0;
      o[dn][2] = o[dn][2] * a1 + ld(dn * 4 + 2) * b1;
      o[dn][3] = o[dn][3] * a1 + ld(dn * 4 + 3) * b1;
    }
  }
};

// The flat tile list: sequence-major, then head, then tile.  pfx[b] = tiles per head of the
// active sequences before b; a sequence without an active row contributes none.
struct TileCursor {
  int b, h, tile, nt;   // current sequence, head, tile within the head's context, tiles per head of b
  __device__ __forceinline__ void locate(const int *pfx, int batch, int H, int f) {
    b = 0;
    while (b + 1 < batch && (long long)H * pfx[b + 1] <= f) ++b;
    nt = pfx[b + 1] - pfx[b];
    const int rem = f - H * pfx[b];
    h = rem / nt; tile = rem % nt;
  }
  __device__ __forceinline__ void next_segment(const int *pfx, int batch, int H) {
    tile = 0;
    if (++h == H) {
      h = 0;
      do { ++b; } while (b + 1 < batch && pfx[b + 1] == pfx[b]);
      nt = b < batch ? pfx[b + 1] - pfx[b] : 1;
    }
  }
};

// MT = 16-row query tiles (rows per sequence <= 16 * MT); FP8 = keys/values are E4M3 codes (tmap: the keys'
// 128-byte lines, tmap_v: the transposed values), else bf16 (tmap alone: rows of 64 values)
template <int MT, bool FP8>
__global__ void __launch_bounds__(xthreads(FP8), 2) cross_attn_tma_kernel(const __grid_constant__ CUtensorMap tmap,
                                                                          const __grid_constant__ CUtensorMap tmap_v, AttnArgs a) {
  constexpr int XCW = xcw(FP8), XTHREADS = xthreads(FP8);
  constexpr int KPW = XK / XCW;                            // keys of a tile per consumer warp: 32 or 16
  constexpr int NTW = KPW / 8, KSW = KPW / 16;             // 8-key score tiles and 16-key P.V steps per warp and tile
  constexpr int XTILE_BYTES = XK * kDh * (FP8 ? 1 : 2);    // keys (or values) of one tile: 8 or 16 KB
  constexpr int XSTAGE_BYTES = 2 * XTILE_BYTES;
  constexpr int XSTAGES = xring_bytes(FP8) / XSTAGE_BYTES;
  constexpr int XSCRATCH_BYTES = xscratch_bytes(FP8);
  extern __shared__ uint8_t smem_raw[];
  __shared__ int pfx_s[XMAXB + 1];
  __shared__ int aseq_s[XMAXB];             // the a-th sequence that has an active row
  __shared__ int n_aseq_s;
  __shared__ unsigned char nact_s[XMAXB];   // active rows of every sequence (at most 32 here)
  const Dims &dm = a.dm;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, G = gridDim.x, H = dm.H, batch = a.batch;
  __nv_bfloat16 *out = (__nv_bfloat16 *)a.out;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *smem_al = smem_raw + (base - smem_u32(smem_raw));
  float *scratch = reinterpret_cast<float *>(smem_al + XSTAGES * XSTAGE_BYTES);     // [2][XREC_FLOATS]
  const uint32_t bar_full = base + XSTAGES * XSTAGE_BYTES + XSCRATCH_BYTES;
  const uint32_t bar_empty = bar_full + 8 * XSTAGES;

  // ---- tiles per head of every sequence, prefix sums, this CTA's range of the flat list
  for (int b = tid; b < batch; b += XTHREADS) {
    // counts the caller wrote (stand-alone op) are clamped to the tensors' extents
    const int S = min(max(a.st.n_active[b], 0), min(dm.C, 16 * MT));
    nact_s[b] = (unsigned char)S;
    pfx_s[b + 1] = S > 0 ? (min(max(a.st.ctx_len[b], 1), dm.ctx) + XK - 1) / XK : 0;
  }
  if (tid == 0) {
    pfx_s[0] = 0;
    for (int s = 0; s < XSTAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, XCW); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 0) {   // inclusive scan in chunks of 32
    int carry = 0;
    for (int c0 = 0; c0 < batch; c0 += 32) {
      int v = c0 + lane < batch ? pfx_s[c0 + lane + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { int u = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += u; }
      if (c0 + lane < batch) pfx_s[c0 + lane + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  } else if (warp == 1) {   // the sequences that have an active row, in order
    int n = 0;
    for (int c0 = 0; c0 < batch; c0 += 32) {
      const bool on = c0 + lane < batch && nact_s[c0 + lane] > 0;
      const unsigned m = __ballot_sync(0xffffffffu, on);
      if (on) aseq_s[n + __popc(m & ((1u << lane) - 1u))] = c0 + lane;
      n += __popc(m);
    }
    if (lane == 0) n_aseq_s = n;
  }
  // rows of a sequence beyond its active ones come back as zeros (all heads)
  for (int b = cta; b < batch && a.row_base == nullptr; b += G) {
    const int S = nact_s[b];
    uint4 *z = reinterpret_cast<uint4 *>(out + (size_t)(b * dm.C + S) * dm.d);      // rows are d * 2 bytes, d a multiple of 64
    for (int idx = tid; idx < (dm.C - S) * dm.d / 8; idx += XTHREADS) z[idx] = make_uint4(0u, 0u, 0u, 0u);
  }
  __syncthreads();
  const long long T = (long long)H * pfx_s[batch];
  // CTAs that get work: every one of them at least XMIN_TILES tiles (when there are that many), so
  // that few tiles do not turn into many one-tile CTAs whose records one CTA then merges serially
  const long long want = (T + XMIN_TILES - 1) / XMIN_TILES;
  int Ge = (int)(want < G ? want : G);
  int lo, hi;
  // With enough (sequence, head) segments to keep at least one CTA per SM streaming, every CTA takes
  // whole segments (the same number each): nothing is cut, so there are no partial records, no
  // tickets and no merge after the last tile.  Otherwise the tile list itself is cut into equal
  // ranges.  Fewer segments than SMs, but long ones (a lone CTA streams 32 tiles too slowly): two
  // CTAs per segment.
  const int n_seg = n_aseq_s * H;
  const int seg_per_cta = (n_seg + G - 1) / G;
  const bool two_per_segment = n_seg > 0 && 2 * n_seg <= G && T >= (long long)XLONG_SEG * n_seg;
  const bool whole_segments = n_seg > 0 && (n_seg + seg_per_cta - 1) / seg_per_cta >= XMIN_WHOLE && !two_per_segment;
  if (two_per_segment && 2 * n_seg < Ge) Ge = 2 * n_seg;
  if (whole_segments) {
    Ge = (n_seg + seg_per_cta - 1) / seg_per_cta;
    if (cta >= Ge) return;
    auto seg_tile = [&](int sidx) {    // first tile of segment sidx in the flat list
      if (sidx >= n_seg) return (int)T;
      const int bb = aseq_s[sidx / H], hh = sidx % H;
      return H * pfx_s[bb] + hh * (pfx_s[bb + 1] - pfx_s[bb]);
    };
    lo = seg_tile(cta * seg_per_cta);
    hi = seg_tile((cta + 1) * seg_per_cta);
  } else {
    if (cta >= Ge) return;
    lo = (int)(cta * T / Ge); hi = (int)((cta + 1) * T / Ge);
  }

  if (warp == XCW) {
    // ------------------------------------------------------------------ producer (one lane)
    if (lane == 0) {
      TileCursor cur;
      cur.locate(pfx_s, batch, H, lo);
      for (int it = 0; it < hi - lo; ++it) {
        const int s = it % XSTAGES;
        const uint32_t u = (uint32_t)(it / XSTAGES);
        if (!mbar_wait(bar_empty + 8 * s, (u & 1u) ^ 1u)) { atomicExch(&a.st.hdr[HDR_STATUS], (int)PD_ERR_TIMEOUT); break; }
        mbar_expect_tx(bar_full + 8 * s, XSTAGE_BYTES);
        const uint32_t dst = base + s * XSTAGE_BYTES;
        const int kv_b = a.kv_seq != nullptr ? a.kv_seq[cur.b] : cur.b;     // the sequence whose context this group reads
        if (FP8) {
          // block (layer, sequence, head) = max_ctx * 64 bytes of keys, then as many of transposed values
          const int blk = (((a.layer * dm.B + kv_b) * H + cur.h) << 1);
          tma_load_2d(dst, &tmap, bar_full + 8 * s, 0, blk * (dm.ctx >> 1) + cur.tile * (XK / 2));    // 64 lines = 128 keys
          tma_load_3d(dst + XTILE_BYTES, &tmap_v, bar_full + 8 * s, cur.tile * XK, 0, blk + 1);       // 64 dims x 128 keys
        } else {
          const int y = (int)(ctx_kv_offset(a.layer, dm.B, kv_b, H, cur.h, 0, dm.ctx) / kDh) + cur.tile * XK;
          tma_load_2d(dst, &tmap, bar_full + 8 * s, 0, y);                         // K tile
          tma_load_2d(dst + XTILE_BYTES, &tmap, bar_full + 8 * s, 0, y + dm.ctx);  // V tile
        }
        if (++cur.tile == cur.nt) cur.next_segment(pfx_s, batch, H);
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int g = lane >> 2, tig = lane & 3;
  const __nv_bfloat16 *qbuf = (const __nv_bfloat16 *)a.q;
  const int kb = warp * KPW;         // this warp's keys inside every tile
  const float sl2 = dm.scale_log2e;
  bool ok = true;
  int it = 0;
  TileCursor cur;
  cur.locate(pfx_s, batch, H, lo);
  for (int f = lo; f < hi;) {
    const int b = cur.b, h = cur.h;
    const int seg_start = H * pfx_s[b] + h * cur.nt, seg_end = seg_start + cur.nt;
    const int my_end = min(hi, seg_end);
    const int S = nact_s[b], ctx_len = min(max(a.st.ctx_len[b], 1), dm.ctx);
    const int row0 = a.row_base != nullptr ? a.row_base[b] : b * dm.C;
    float seg_sl2 = sl2, seg_vscale = 1.f;          // 8-bit: the key scale joins the score scale, the value scale the final 1 / l
    if (FP8) {
      const int kv_b = a.kv_seq != nullptr ? a.kv_seq[b] : b;
      const float2 sc2 = *reinterpret_cast<const float2 *>(a.kv_scale + ((((size_t)a.layer * dm.B + kv_b) * H + h) << 1));
      seg_sl2 = sl2 * sc2.x; seg_vscale = sc2.y;
    }
    uint32_t qf[MT][4][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      int r_lo = mt * 16 + g, r_hi = r_lo + 8;
      if (FP8) {
        // f16 queries, dims 4 tig + {0, 1} | 4 tig + {2, 3} of every 16: the order the key codes come in
        const __nv_bfloat16 *q_lo = qbuf + (size_t)(row0 + r_lo) * dm.d + h * kDh + 4 * tig;
        const __nv_bfloat16 *q_hi = qbuf + (size_t)(row0 + r_hi) * dm.d + h * kDh + 4 * tig;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const uint2 lo = r_lo < S ? *reinterpret_cast<const uint2 *>(q_lo + kk * 16) : make_uint2(0u, 0u);
          const uint2 hi = r_hi < S ? *reinterpret_cast<const uint2 *>(q_hi + kk * 16) : make_uint2(0u, 0u);
          qf[mt][kk][0] = bf16x2_to_f16x2(lo.x); qf[mt][kk][2] = bf16x2_to_f16x2(lo.y);
          qf[mt][kk][1] = bf16x2_to_f16x2(hi.x); qf[mt][kk][3] = bf16x2_to_f16x2(hi.y);
        }
      } else {
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
    }
    TileAcc acc[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) acc[mt].clear();

    for (int tile = f - seg_start; tile < my_end - seg_start; ++tile, ++it) {
      const int s = it % XSTAGES;
      const uint32_t u = (uint32_t)(it / XSTAGES);
      if (ok && !mbar_wait(bar_full + 8 * s, u & 1u)) ok = false;
      if (!ok) continue;             // drained mode: keep the control flow (barriers below) intact
      const uint32_t kbase = base + s * XSTAGE_BYTES, vbase = kbase + XTILE_BYTES;
      const int key0 = tile * XK + kb;               // context position of this warp's first key
      const bool ragged = key0 + KPW > ctx_len;
      // Rows at or beyond ctx_len hold whatever follows in memory.  Their weights are exactly 0 below;
      // the value fragments of those keys are cleared in registers after ldmatrix, so that 0 never
      // multiplies a non-finite.  (Nothing but TMA ever writes a stage: zeroing the rows in shared
      // memory raced with the next bulk copy into the stage, proxy fence or not.)
      // ---- scores: S[mt][nt] = Q (16 x 64) . K^T (64 x 8 keys)
      float sc[MT][NTW][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) sc[mt][nt][0] = sc[mt][nt][1] = sc[mt][nt][2] = sc[mt][nt][3] = 0.f;
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        if (FP8) {
          // column c of score tile nt = 2 ks + u is key 16 ks + 4 (c >> 1) + 2 u + (c & 1) of this warp's 32: the
          // order in which the value codes of a 16-key step come out of ldmatrix (see the P.V loop).  The keys
          // of every group of 16 are STORED in that order (tile u's eight keys in lines 4 u .. 4 u + 3), so that
          // the eight rows of an ldmatrix fall into eight different 16-byte bank groups.
          const int key = kb + nt * 8 + (lane & 7);                                 // position in stored order
          const int line = key >> 1, chunk = ((key & 1) << 2) + (lane >> 3);       // two keys per 128-byte line
          uint32_t r[4];
          ldsm_x4(kbase + (uint32_t)(line * 128 + ((chunk ^ (line & 7)) << 4)), r[0], r[1], r[2], r[3]);   // all 64 dims of 8 keys
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t b0 = e4m3x2_to_f16x2(r[j], 0), b1 = e4m3x2_to_f16x2(r[j], 1);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) mma_f16(sc[mt][nt], qf[mt][j][0], qf[mt][j][1], qf[mt][j][2], qf[mt][j][3], b0, b1);
          }
        } else {
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
      }
      // ---- scale, mask the ragged end of the context, online softmax
      uint32_t pf[MT][KSW][4];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float v = sc[mt][nt][e] * seg_sl2;
            const int kidx = FP8 ? key0 + 16 * (nt >> 1) + 4 * tig + 2 * (nt & 1) + (e & 1) : key0 + nt * 8 + 2 * tig + (e & 1);
            if (ragged && kidx >= ctx_len) v = -INFINITY;
            sc[mt][nt][e] = v;
          }
          mx0 = fmaxf(mx0, fmaxf(sc[mt][nt][0], sc[mt][nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sc[mt][nt][2], sc[mt][nt][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        TileAcc &A = acc[mt];
        const float mn0 = fmaxf(A.m0, mx0), mn1 = fmaxf(A.m1, mx1);
        const float ref0 = mn0 == -INFINITY ? 0.f : mn0, ref1 = mn1 == -INFINITY ? 0.f : mn1;
        const float c0 = ex2f(A.m0 - ref0), c1 = ex2f(A.m1 - ref1);
        A.m0 = mn0; A.m1 = mn1;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) {
          float p0 = ex2f(sc[mt][nt][0] - ref0), p1 = ex2f(sc[mt][nt][1] - ref0);
          float p2 = ex2f(sc[mt][nt][2] - ref1), p3 = ex2f(sc[mt][nt][3] - ref1);
          s0 += p0 + p1; s1 += p2 + p3;
          pf[mt][nt >> 1][(nt & 1) * 2 + 0] = FP8 ? pack_f16(p0, p1) : pack_bf16(p0, p1);
          pf[mt][nt >> 1][(nt & 1) * 2 + 1] = FP8 ? pack_f16(p2, p3) : pack_bf16(p2, p3);
        }
        A.l0 = A.l0 * c0 + s0;
        A.l1 = A.l1 * c1 + s1;
        if (__any_sync(0xffffffffu, c0 != 1.f || c1 != 1.f)) {   // some row's running maximum moved
#pragma unroll
          for (int dn = 0; dn < 8; ++dn) { A.o[dn][0] *= c0; A.o[dn][1] *= c0; A.o[dn][2] *= c1; A.o[dn][3] *= c1; }
        }
      }
      // ---- O += P (16 x 32 keys) . V (32 keys x 64)
      if (FP8) {
        // transposed values: a line is one dim, a 16-byte chunk sixteen keys; positions at or beyond ctx_len
        // hold zero codes (written so, or filled by the copy beyond max_ctx), so nothing needs masking
#pragma unroll
        for (int ks = 0; ks < KSW; ++ks) {
          const int chunk = (kb + ks * 16) >> 4;
#pragma unroll
          for (int dq = 0; dq < 2; ++dq) {      // four 8-wide slices of the head per ldmatrix.x4
            const int dim = (dq * 4 + (lane >> 3)) * 8 + (lane & 7);
            uint32_t r[4];
            ldsm_x4(vbase + (uint32_t)(dim * 128 + ((chunk ^ (dim & 7)) << 4)), r[0], r[1], r[2], r[3]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t b0 = e4m3x2_to_f16x2(r[j], 0), b1 = e4m3x2_to_f16x2(r[j], 1);
#pragma unroll
              for (int mt = 0; mt < MT; ++mt)
                mma_f16(acc[mt].o[dq * 4 + j], pf[mt][ks][0], pf[mt][ks][1], pf[mt][ks][2], pf[mt][ks][3], b0, b1);
            }
          }
        }
      } else {
#pragma unroll
      for (int ks = 0; ks < KSW; ++ks) {
        const int key = kb + ks * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
        // this lane's fragment halves hold keys k0, k0 + 1 (b0, b2) and k0 + 8, k0 + 9 (b1, b3)
        uint32_t keep_a = 0xffffffffu, keep_b = 0xffffffffu;
        if (ragged) {
          const int k0 = key0 + ks * 16 + 2 * tig;
          keep_a = (k0 < ctx_len ? 0x0000ffffu : 0u) | (k0 + 1 < ctx_len ? 0xffff0000u : 0u);
          keep_b = (k0 + 8 < ctx_len ? 0x0000ffffu : 0u) | (k0 + 9 < ctx_len ? 0xffff0000u : 0u);
        }
#pragma unroll
        for (int dp = 0; dp < 4; ++dp) {      // two 8-wide slices of the head per ldmatrix.x4
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(vbase + swz(key, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
          if (ragged) { b0 &= keep_a; b1 &= keep_b; b2 &= keep_a; b3 &= keep_b; }
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            mma_bf16(acc[mt].o[2 * dp], pf[mt][ks][0], pf[mt][ks][1], pf[mt][ks][2], pf[mt][ks][3], b0, b1);
            mma_bf16(acc[mt].o[2 * dp + 1], pf[mt][ks][0], pf[mt][ks][1], pf[mt][ks][2], pf[mt][ks][3], b2, b3);
          }
        }
      }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * s);
    }

    // ---- end of this CTA's part of the (sequence, head) segment: row sums across the quad, then
    // tree-merge the consumer warps into warp 0, one 16-row tile at a time
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      TileAcc &A = acc[mt];
      A.l0 += __shfl_xor_sync(0xffffffffu, A.l0, 1); A.l0 += __shfl_xor_sync(0xffffffffu, A.l0, 2);
      A.l1 += __shfl_xor_sync(0xffffffffu, A.l1, 1); A.l1 += __shfl_xor_sync(0xffffffffu, A.l1, 2);
#pragma unroll
      for (int stride = XCW / 2; stride >= 1; stride >>= 1) {                 // the upper half hands its state to the lower half
        if (warp >= stride && warp < 2 * stride) A.store(scratch + (warp - stride) * XREC_FLOATS, lane);
        consumer_bar_sync<XCW * 32>();
        if (warp < stride) A.template merge<false>(scratch + warp * XREC_FLOATS, lane);
        consumer_bar_sync<XCW * 32>();
      }
    }
    if (warp == 0) {
      const bool whole = f == seg_start && my_end == seg_end;
      bool write_out = whole;
      if (!whole) {
        // Partial segment: store the record, take a ticket; the last CTA to arrive merges them all.
        const int which = lo >= seg_start ? 0 : 1;     // this CTA's first segment, or its last one
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) acc[mt].store(a.part_o + (size_t)((cta * 2 + which) * MT + mt) * XREC_FLOATS, lane);
        __threadfence();
        __syncwarp();
        const int c_first = (int)((((long long)seg_start + 1) * Ge - 1) / T), c_last = (int)(((long long)seg_end * Ge - 1) / T);
        int last = 0;
        if (lane == 0) last = atomicAdd(&a.tickets[b * H + h], 1) == c_last - c_first;
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          __threadfence();
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) acc[mt].clear();
          for (int c2 = c_first; c2 <= c_last; ++c2) {          // fixed order: the result does not depend on arrival order
            const int w2 = (int)(c2 * T / Ge) >= seg_start ? 0 : 1;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
              acc[mt].template merge<true>(a.part_o + (size_t)((c2 * 2 + w2) * MT + mt) * XREC_FLOATS, lane);
          }
          if (lane == 0) a.tickets[b * H + h] = 0;
          write_out = true;
        }
      }
      if (write_out) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const TileAcc &A = acc[mt];
          const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
          const float i0 = seg_vscale / A.l0, i1 = seg_vscale / A.l1;
          __nv_bfloat16 *o_lo = out + (size_t)(row0 + r_lo) * dm.d + h * kDh + 2 * tig;
          __nv_bfloat16 *o_hi = out + (size_t)(row0 + r_hi) * dm.d + h * kDh + 2 * tig;
#pragma unroll
          for (int dn = 0; dn < 8; ++dn) {
            if (r_lo < S) *reinterpret_cast<__nv_bfloat162 *>(o_lo + dn * 8) = __floats2bfloat162_rn(A.o[dn][0] * i0, A.o[dn][1] * i0);
            if (r_hi < S) *reinterpret_cast<__nv_bfloat162 *>(o_hi + dn * 8) = __floats2bfloat162_rn(A.o[dn][2] * i1, A.o[dn][3] * i1);
          }
        }
      }
    }
    f = my_end;
    if (f < hi) cur.next_segment(pfx_s, batch, H);
  }
  if (!ok && lane == 0) atomicExch(&a.st.hdr[HDR_STATUS], (int)PD_ERR_TIMEOUT);
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

int cross_attn_ctas() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    sms = 148;
  return 2 * sms < kMaxCrossCtas ? 2 * sms : kMaxCrossCtas;
}

// Tensor maps of the 8-bit context keys/values, n_blocks = layers * sequences * heads blocks of
// max_ctx * 64 bytes of keys followed by max_ctx * 64 bytes of transposed values.  Keys: the whole buffer
// as lines of 128 bytes (two keys each), boxes of 64 lines; values: [block][64 dims][max_ctx], boxes of
// 128 keys x 64 dims.  Both with the 128-byte swizzle; reads beyond max_ctx are filled with zeros.
cudaError_t encode_ctx_kv8_tensor_maps(CUtensorMap *map_k, CUtensorMap *map_v, const void *base, uint64_t n_blocks, uint64_t ctx,
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
  {
    cuuint64_t gdim[2] = {128, (cuuint64_t)(n_blocks * 2 * ctx * kDh / 128)};
    cuuint64_t gstride[1] = {128};
    cuuint32_t box[2] = {128, (cuuint32_t)(XK / 2)};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = ((EncodeFn)fn)(map_k, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), gdim, gstride, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { if (driver_code) *driver_code = (int)r; return cudaErrorInvalidValue; }
  }
  {
    cuuint64_t gdim[3] = {(cuuint64_t)ctx, (cuuint64_t)kDh, (cuuint64_t)(n_blocks * 2)};
    cuuint64_t gstride[2] = {(cuuint64_t)ctx, (cuuint64_t)ctx * kDh};
    cuuint32_t box[3] = {(cuuint32_t)XK, (cuuint32_t)kDh, 1u};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult r = ((EncodeFn)fn)(map_v, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), gdim, gstride, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { if (driver_code) *driver_code = (int)r; return cudaErrorInvalidValue; }
  }
  return cudaSuccess;
}

cudaError_t cross_attn_tma_prepare() {
  cudaError_t e = cudaFuncSetAttribute(cross_attn_tma_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, xsmem(false));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(cross_attn_tma_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, xsmem(false));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(cross_attn_tma_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, xsmem(true));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(cross_attn_tma_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, xsmem(true));
  return e;
}

// n_ctas persistent CTAs (two per SM); a.part_o holds cross_attn_tma_partial_bytes(n_ctas, C),
// a.tickets one zeroed int32 per (sequence, head) (the kernel leaves them zeroed).
// 8-bit keys/values (a.kv_scale set): tmap = the keys' lines, tmap_v = the transposed values; else tmap alone.
cudaError_t launch_cross_attn_tma(const AttnArgs &a, const CUtensorMap &tmap, const CUtensorMap &tmap_v, int n_ctas, cudaStream_t s) {
  int mt = (a.dm.C + 15) / 16;
  const bool fp8 = a.kv_scale != nullptr;
  if (mt == 1 && !fp8) cross_attn_tma_kernel<1, false><<<n_ctas, xthreads(false), xsmem(false), s>>>(tmap, tmap_v, a);
  else if (mt == 2 && !fp8) cross_attn_tma_kernel<2, false><<<n_ctas, xthreads(false), xsmem(false), s>>>(tmap, tmap_v, a);
  else if (mt == 1) cross_attn_tma_kernel<1, true><<<n_ctas, xthreads(true), xsmem(true), s>>>(tmap, tmap_v, a);
  else if (mt == 2) cross_attn_tma_kernel<2, true><<<n_ctas, xthreads(true), xsmem(true), s>>>(tmap, tmap_v, a);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace pd
