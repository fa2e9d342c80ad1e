// Kernels of the teacher-forced forward of Section 3.3 (Eq. 6): the whole target of every sequence in one
// pass, every token attending to the tokens the dependency rule of Section 3.2 lets it see - evaluated per
// (query, key) pair from (subsequence, timestamp) and never stored as a mask.  Off the decode hot path
// (scoring, perplexity).  One CTA per group of up to 32 query rows and head, on tensor cores (mma.sync, 64-key tiles).
#include "mma_tile.cuh"
#include "pd_internal.h"

namespace pd {

namespace {

// Four warps; a tile = 64 keys of the sequence, staged by all threads as swizzled bf16 rows (keys rotated on the way
// in rotary mode), each warp taking 16 of them: scores with mma.sync against the group's two 16-row query tiles, the
// dependency rule and the T5 bias applied to the accumulator fragment per (query, key) pair, online softmax, P.V.
// The warps' states are tree-merged through shared memory at the end.
constexpr int TQ = 32, TK = 64, TT = 128, TW = 4, TMAXD = 640;

__global__ void __launch_bounds__(TT) dense_self_attn_tc_kernel(DenseAttnArgs a) {
  using namespace mt;
  const int grp = blockIdx.x, h = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const int q0 = a.grp_row0[grp], nq = a.grp_n[grp];
  const int k0 = a.grp_seq_row0[grp], nk = a.grp_seq_rows[grp];
  __shared__ __align__(1024) uint8_t ks[TK * 128];
  __shared__ __align__(1024) uint8_t vs[TK * 128];
  __shared__ int ki_s[TK], kt_s[TK], qi_s[TQ], qt_s[TQ];
  __shared__ float bias_s[TMAXD];
  __shared__ float scratch[2 * kRecFloats];
  const size_t ld = 3 * (size_t)a.d;
  const bool rope = a.rope_tab != nullptr, use_bias = a.bias_tab != nullptr;
  if (tid < TQ) {
    qi_s[tid] = tid < nq ? a.row_sub[q0 + tid] : 0;
    qt_s[tid] = tid < nq ? a.row_tau[q0 + tid] : 0;
  }
  if (use_bias)
    for (int dd = tid; dd < a.n_dist; dd += TT) bias_s[dd] = a.bias_tab[(size_t)h * a.n_dist + dd];
  __syncthreads();
  // query fragments (rows beyond the group's are zero and masked anyway)
  uint32_t qf[2][4][4];
  int qi[2][2], qp[2][2];               // subsequence and position tau + i of rows g / g + 8 of both query tiles
#pragma unroll
  for (int mt_ = 0; mt_ < 2; ++mt_) {
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int r = mt_ * 16 + g + hh * 8;
      qi[mt_][hh] = r < nq ? qi_s[r] : -1;                       // -1: sees nothing
      qp[mt_][hh] = r < nq ? qt_s[r] + qi_s[r] : 0;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t w = 0u;
          if (r < nq) {
            const int col = kk * 16 + 2 * tig + half * 8;
            const size_t o = (size_t)(q0 + r) * ld + (size_t)h * kDh + col;
            if (!a.qkv_f32) {
              w = *reinterpret_cast<const uint32_t *>(reinterpret_cast<const __nv_bfloat16 *>(a.qkv) + o);
            } else {
              float2 v = *reinterpret_cast<const float2 *>(reinterpret_cast<const float *>(a.qkv) + o);
              if (rope) {
                const float2 cs = a.rope_tab[(size_t)qp[mt_][hh] * (kDh / 2) + col / 2];
                const float t = v.x * cs.x - v.y * cs.y;
                v.y = v.x * cs.y + v.y * cs.x; v.x = t;
              }
              w = pack_bf16(v.x, v.y);
            }
          }
          qf[mt_][kk][hh + 2 * half] = w;
        }
    }
  }
  const int qt_row[2][2] = {{qp[0][0] - qi[0][0], qp[0][1] - qi[0][1]}, {qp[1][0] - qi[1][0], qp[1][1] - qi[1][1]}};
  TileAcc acc[2];
  acc[0].clear(); acc[1].clear();
  const int q_i_max = qi_s[nq - 1];
  const uint32_t kbase = smem_u32(ks), vbase = smem_u32(vs);
  const int kb = warp * 16;              // this warp's keys inside every tile

  for (int kt0 = 0; kt0 < nk; kt0 += TK) {
    if (a.row_sub[k0 + kt0] > q_i_max) break;     // rows are sorted by subsequence: nothing further on is visible
    const int nv = min(TK, nk - kt0);
    __syncthreads();                    // the previous tile is consumed
    if (tid < TK) {
      ki_s[tid] = tid < nv ? a.row_sub[k0 + kt0 + tid] : 0x3fffffff;
      kt_s[tid] = tid < nv ? a.row_tau[k0 + kt0 + tid] : 0x3fffffff;
    }
    {
      // thread = (key, half of the head): 32 columns of its key row and of its value row
      const int e = tid >> 1, c0 = (tid & 1) * 32;
      uint4 kq[4], vq[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) kq[j] = vq[j] = make_uint4(0u, 0u, 0u, 0u);
      if (e < nv) {
        const size_t ob = (size_t)(k0 + kt0 + e) * ld + (size_t)h * kDh + c0;
        if (!a.qkv_f32) {
          const __nv_bfloat16 *src = reinterpret_cast<const __nv_bfloat16 *>(a.qkv) + ob;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            kq[j] = *reinterpret_cast<const uint4 *>(src + a.d + 8 * j);
            vq[j] = *reinterpret_cast<const uint4 *>(src + 2 * (size_t)a.d + 8 * j);
          }
        } else {
          const float *src = reinterpret_cast<const float *>(a.qkv) + ob;
          const int pos = a.row_tau[k0 + kt0 + e] + a.row_sub[k0 + kt0 + e];
          uint32_t kw[16], vw[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            float2 kf = *reinterpret_cast<const float2 *>(src + a.d + 2 * j);
            const float2 vf = *reinterpret_cast<const float2 *>(src + 2 * (size_t)a.d + 2 * j);
            if (rope) {
              const float2 cs = a.rope_tab[(size_t)pos * (kDh / 2) + c0 / 2 + j];
              const float t = kf.x * cs.x - kf.y * cs.y;
              kf.y = kf.x * cs.y + kf.y * cs.x; kf.x = t;
            }
            kw[j] = pack_bf16(kf.x, kf.y); vw[j] = pack_bf16(vf.x, vf.y);
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            kq[j] = make_uint4(kw[4 * j], kw[4 * j + 1], kw[4 * j + 2], kw[4 * j + 3]);
            vq[j] = make_uint4(vw[4 * j], vw[4 * j + 1], vw[4 * j + 2], vw[4 * j + 3]);
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        *reinterpret_cast<uint4 *>(ks + swz(e, (tid & 1) * 4 + j)) = kq[j];
        *reinterpret_cast<uint4 *>(vs + swz(e, (tid & 1) * 4 + j)) = vq[j];      // absent keys: zero rows
      }
    }
    __syncthreads();
    if (kb >= nv) continue;              // (the barriers above are reached by every warp on every tile)
    // ---- scores of this warp's 16 keys
    float sc[2][2][4];
#pragma unroll
    for (int mt_ = 0; mt_ < 2; ++mt_)
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) sc[mt_][nt][0] = sc[mt_][nt][1] = sc[mt_][nt][2] = sc[mt_][nt][3] = 0.f;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int key = kb + nt * 8 + (lane & 7);
#pragma unroll
      for (int kp = 0; kp < 2; ++kp) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(kbase + swz(key, kp * 4 + (lane >> 3)), b0, b1, b2, b3);
#pragma unroll
        for (int mt_ = 0; mt_ < 2; ++mt_) {
          mma_bf16(sc[mt_][nt], qf[mt_][2 * kp][0], qf[mt_][2 * kp][1], qf[mt_][2 * kp][2], qf[mt_][2 * kp][3], b0, b1);
          mma_bf16(sc[mt_][nt], qf[mt_][2 * kp + 1][0], qf[mt_][2 * kp + 1][1], qf[mt_][2 * kp + 1][2], qf[mt_][2 * kp + 1][3], b2, b3);
        }
      }
    }
    // ---- the dependency rule per pair (i' <= i and tau' <= tau), bias on the Manhattan distance, online softmax
    uint32_t pf[2][4];
#pragma unroll
    for (int mt_ = 0; mt_ < 2; ++mt_) {
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int e = kb + nt * 8 + 2 * tig + (x & 1), hh = x >> 1;
          const int ki = ki_s[e], ktau = kt_s[e];
          float v = -INFINITY;
          if (ki <= qi[mt_][hh] && ktau <= qt_row[mt_][hh]) {
            v = sc[mt_][nt][x] * a.scale_log2e;
            if (use_bias) v += bias_s[qp[mt_][hh] - (ktau + ki)];
          }
          sc[mt_][nt][x] = v;
          if (hh == 0) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
        }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      TileAcc &A = acc[mt_];
      const float mn0 = fmaxf(A.m0, mx0), mn1 = fmaxf(A.m1, mx1);
      const float ref0 = mn0 == -INFINITY ? 0.f : mn0, ref1 = mn1 == -INFINITY ? 0.f : mn1;
      const float c0 = ex2f(A.m0 - ref0), c1 = ex2f(A.m1 - ref1);
      A.m0 = mn0; A.m1 = mn1;
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const float p0 = ex2f(sc[mt_][nt][0] - ref0), p1 = ex2f(sc[mt_][nt][1] - ref0);
        const float p2 = ex2f(sc[mt_][nt][2] - ref1), p3 = ex2f(sc[mt_][nt][3] - ref1);
        s0 += p0 + p1; s1 += p2 + p3;
        pf[mt_][nt * 2 + 0] = pack_bf16(p0, p1);
        pf[mt_][nt * 2 + 1] = pack_bf16(p2, p3);
      }
      A.l0 = A.l0 * c0 + s0; A.l1 = A.l1 * c1 + s1;
#pragma unroll
      for (int dn = 0; dn < 8; ++dn) { A.o[dn][0] *= c0; A.o[dn][1] *= c0; A.o[dn][2] *= c1; A.o[dn][3] *= c1; }
    }
    // ---- O += P (16 x 16 keys) . V (16 keys x 64)
    {
      const int key = kb + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
      for (int dp = 0; dp < 4; ++dp) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vbase + swz(key, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
#pragma unroll
        for (int mt_ = 0; mt_ < 2; ++mt_) {
          mma_bf16(acc[mt_].o[2 * dp], pf[mt_][0], pf[mt_][1], pf[mt_][2], pf[mt_][3], b0, b1);
          mma_bf16(acc[mt_].o[2 * dp + 1], pf[mt_][0], pf[mt_][1], pf[mt_][2], pf[mt_][3], b2, b3);
        }
      }
    }
  }
  // ---- row sums across the quad, tree merge of the four warps, output
#pragma unroll
  for (int mt_ = 0; mt_ < 2; ++mt_) {
    TileAcc &A = acc[mt_];
    A.l0 += __shfl_xor_sync(0xffffffffu, A.l0, 1); A.l0 += __shfl_xor_sync(0xffffffffu, A.l0, 2);
    A.l1 += __shfl_xor_sync(0xffffffffu, A.l1, 1); A.l1 += __shfl_xor_sync(0xffffffffu, A.l1, 2);
#pragma unroll
    for (int stride = TW / 2; stride >= 1; stride >>= 1) {
      __syncthreads();
      if (warp >= stride && warp < 2 * stride) A.store(scratch + (warp - stride) * kRecFloats, lane);
      __syncthreads();
      if (warp < stride) A.merge(scratch + warp * kRecFloats, lane);
    }
    if (warp == 0) {
      const int r_lo = mt_ * 16 + g, r_hi = r_lo + 8;
      const float i0 = 1.f / A.l0, i1 = 1.f / A.l1;
      __nv_bfloat16 *o_lo = a.out + (size_t)(q0 + r_lo) * a.d + (size_t)h * kDh + 2 * tig;
      __nv_bfloat16 *o_hi = a.out + (size_t)(q0 + r_hi) * a.d + (size_t)h * kDh + 2 * tig;
#pragma unroll
      for (int dn = 0; dn < 8; ++dn) {
        if (r_lo < nq) *reinterpret_cast<__nv_bfloat162 *>(o_lo + dn * 8) = __floats2bfloat162_rn(A.o[dn][0] * i0, A.o[dn][1] * i0);
        if (r_hi < nq) *reinterpret_cast<__nv_bfloat162 *>(o_hi + dn * 8) = __floats2bfloat162_rn(A.o[dn][2] * i1, A.o[dn][3] * i1);
      }
    }
  }
}

// x[r] = embedding of the row's input token (fp32 residual stream)
__global__ void gather_rows_kernel(int d, const int32_t *__restrict__ row_tok, const __nv_bfloat16 *__restrict__ embed,
                                   float *__restrict__ x) {
  const int r = blockIdx.x;
  const __nv_bfloat16 *e = embed + (size_t)row_tok[r] * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) x[(size_t)r * d + c] = __bfloat162float(e[c]);
}

// logprob[r] = logits[r][target] - log sum_v exp(logits[r][v])   (the row's term of Eq. 6)
__global__ void __launch_bounds__(256) target_logprob_kernel(int V, const float *__restrict__ logits, const int32_t *__restrict__ targets,
                                                             float *__restrict__ logprob) {
  __shared__ float red[8];
  __shared__ float mx_s;
  const float *row = logits + (size_t)blockIdx.x * V;
  float mx = -INFINITY;
  for (int v = threadIdx.x; v < V; v += 256) mx = fmaxf(mx, row[v]);
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) { float m = red[0]; for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]); mx_s = m; }
  __syncthreads();
  mx = mx_s;
  float sum = 0.f;
  for (int v = threadIdx.x; v < V; v += 256) sum += expf(row[v] - mx);
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
    for (int w = 0; w < 8; ++w) s += red[w];
    logprob[blockIdx.x] = row[targets[blockIdx.x]] - (mx + logf(s));
  }
}

}  // namespace

cudaError_t launch_dense_self_attn(const DenseAttnArgs &a, cudaStream_t s) {
  if (a.n_groups < 1) return cudaSuccess;
  if (a.bias_tab != nullptr && a.n_dist > TMAXD) return cudaErrorInvalidValue;      // the head's bias row is held in shared memory
  dense_self_attn_tc_kernel<<<dim3(a.n_groups, a.H), TT, 0, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(int rows, int d, const int32_t *row_tok, const void *embed, float *x, cudaStream_t s) {
  gather_rows_kernel<<<rows, 128, 0, s>>>(d, row_tok, (const __nv_bfloat16 *)embed, x);
  return cudaGetLastError();
}

cudaError_t launch_target_logprob(int rows, int V, const float *logits, const int32_t *targets, float *logprob, cudaStream_t s) {
  target_logprob_kernel<<<rows, 256, 0, s>>>(V, logits, targets, logprob);
  return cudaGetLastError();
}

}  // namespace pd
