// Warp-level building blocks of the mma.sync attention kernels: ldmatrix / mma wrappers, the 128-byte
// swizzle, and the (m, l, O) state of a 16-row query tile in mma fragment layout with its log-sum-exp merge.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace pd {
namespace mt {

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float ex2f(float x) {   // 2^x; ex2(-inf) = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Byte offset of (row, 16-byte chunk) inside a tile whose rows are 128 bytes (64 bf16), chunks swizzled by the row.
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// One warp's state for a 16-row query tile: this lane holds columns dn*8 + 2*tig, +1 of rows g (o[dn][0..1], m0, l0)
// and g + 8 (o[dn][2..3], m1, l1).
struct TileAcc {
  float o[8][4];
  float m0, m1, l0, l1;
  __device__ __forceinline__ void clear() {
    m0 = m1 = -INFINITY; l0 = l1 = 0.f;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) o[dn][0] = o[dn][1] = o[dn][2] = o[dn][3] = 0.f;
  }
  // record layout [word][lane]: 36 words per lane
  __device__ __forceinline__ void store(float *rec, int lane) const {
#pragma unroll
    for (int dn = 0; dn < 8; ++dn)
#pragma unroll
      for (int x = 0; x < 4; ++x) rec[(dn * 4 + x) * 32 + lane] = o[dn][x];
    rec[32 * 32 + lane] = m0; rec[33 * 32 + lane] = m1; rec[34 * 32 + lane] = l0; rec[35 * 32 + lane] = l1;
  }
  // acc <- acc (+) record: the log-sum-exp merge of two partial softmax states (log2 domain)
  __device__ __forceinline__ void merge(const float *rec, int lane) {
    const float om0 = rec[32 * 32 + lane], om1 = rec[33 * 32 + lane], ol0 = rec[34 * 32 + lane], ol1 = rec[35 * 32 + lane];
    const float M0 = fmaxf(m0, om0), M1 = fmaxf(m1, om1);
    const float r0 = M0 == -INFINITY ? 0.f : M0, r1 = M1 == -INFINITY ? 0.f : M1;
    const float a0 = ex2f(m0 - r0), b0 = ex2f(om0 - r0), a1 = ex2f(m1 - r1), b1 = ex2f(om1 - r1);
    m0 = M0; m1 = M1;
    l0 = l0 * a0 + ol0 * b0; l1 = l1 * a1 + ol1 * b1;
#pragma unroll
    for (int dn = 0; dn < 8; ++dn) {
      o[dn][0] = o[dn][0] * a0 + rec[(dn * 4 + 0) * 32 + lane] * b0;
      o[dn][1] = o[dn][1] * a0 + rec[(dn * 4 + 1) * 32 + lane] * b0;
      o[dn][2] = o[dn][2] * a1 + rec[(dn * 4 + 2) * 32 + lane] * b1;
      o[dn][3] = o[dn][3] * a1 + rec[(dn * 4 + 3) * 32 + lane] * b1;
    }
  }
};
constexpr int kRecFloats = 36 * 32;

}  // namespace mt
}  // namespace pd
