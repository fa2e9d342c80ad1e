// Kernels of the teacher-forced forward of Section 3.3 (Eq. 6): the whole target of every sequence in one
// pass, every token attending to the tokens the dependency rule of Section 3.2 lets it see - evaluated per
// (query, key) pair from (subsequence, timestamp) and never stored as a mask.  Off the decode hot path
// (scoring, perplexity): plain-ALU fp32 arithmetic, one CTA per group of up to 32 query rows and head.
#include "pd_internal.h"

namespace pd {

namespace {

constexpr int DQ = 32;            // query rows per CTA
constexpr int DK = 32;            // keys per tile
constexpr int DT = 256;           // threads
constexpr int DSG = DT / kDh;     // 4 row groups in the P.V phase
constexpr int DRPT = DQ / DSG;    // 8 rows per thread there
constexpr int DMAXD = 640;        // longest distance table held in shared memory

__device__ __forceinline__ float ld_qkv(const void *base, int f32, size_t idx) {
  return f32 ? reinterpret_cast<const float *>(base)[idx] : __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(base)[idx]);
}

__global__ void __launch_bounds__(DT) dense_self_attn_kernel(DenseAttnArgs a) {
  const int grp = blockIdx.x, h = blockIdx.y, tid = threadIdx.x;
  const int q0 = a.grp_row0[grp], nq = a.grp_n[grp];
  const int k0 = a.grp_seq_row0[grp], nk = a.grp_seq_rows[grp];
  __shared__ float Qs[DQ][kDh];
  __shared__ float Ks[DK][kDh + 1];
  __shared__ float Vs[DK][kDh];
  __shared__ float Ps[DQ][DK];
  __shared__ float m_s[DQ], l_s[DQ], corr_s[DQ];
  __shared__ int qi_s[DQ], qt_s[DQ], ki_s[DK], kt_s[DK];
  __shared__ float bias_d[DMAXD];
  const size_t ld = 3 * (size_t)a.d;
  const bool rope = a.rope_tab != nullptr, use_bias = a.bias_tab != nullptr;

  if (tid < DQ) {
    m_s[tid] = -INFINITY; l_s[tid] = 0.f; corr_s[tid] = 1.f;
    qi_s[tid] = tid < nq ? a.row_sub[q0 + tid] : 0;
    qt_s[tid] = tid < nq ? a.row_tau[q0 + tid] : 0;
  }
  if (use_bias)
    for (int dd = tid; dd < a.n_dist && dd < DMAXD; dd += DT) bias_d[dd] = a.bias_tab[(size_t)h * a.n_dist + dd];
  __syncthreads();
  // queries (rotated by the row's position tau + i in rotary mode): pairs of columns
  for (int idx = tid; idx < DQ * (kDh / 2); idx += DT) {
    const int r = idx / (kDh / 2), j = idx % (kDh / 2);
    float x0 = 0.f, x1 = 0.f;
    if (r < nq) {
      const size_t o = (size_t)(q0 + r) * ld + (size_t)h * kDh + 2 * j;
      x0 = ld_qkv(a.qkv, a.qkv_f32, o); x1 = ld_qkv(a.qkv, a.qkv_f32, o + 1);
      if (rope) {
        const float2 cs = a.rope_tab[(size_t)(qt_s[r] + qi_s[r]) * (kDh / 2) + j];
        const float t = x0 * cs.x - x1 * cs.y;
        x1 = x0 * cs.y + x1 * cs.x; x0 = t;
      }
    }
    Qs[r][2 * j] = x0; Qs[r][2 * j + 1] = x1;
  }
  float o[DRPT];
#pragma unroll
  for (int u = 0; u < DRPT; ++u) o[u] = 0.f;
  const int dim = tid & (kDh - 1), sg = tid >> 6;

  for (int kt0 = 0; kt0 < nk; kt0 += DK) {
    const int nv = min(DK, nk - kt0);
    __syncthreads();                     // the previous tile is consumed (and the queries are in place)
    if (tid < DK) {
      ki_s[tid] = tid < nv ? a.row_sub[k0 + kt0 + tid] : 0x7fffffff;
      kt_s[tid] = tid < nv ? a.row_tau[k0 + kt0 + tid] : 0x7fffffff;
    }
    for (int idx = tid; idx < DK * (kDh / 2); idx += DT) {
      const int e = idx / (kDh / 2), j = idx % (kDh / 2);
      float x0 = 0.f, x1 = 0.f, v0 = 0.f, v1 = 0.f;
      if (e < nv) {
        const size_t ob = (size_t)(k0 + kt0 + e) * ld + (size_t)h * kDh + 2 * j;
        x0 = ld_qkv(a.qkv, a.qkv_f32, ob + a.d); x1 = ld_qkv(a.qkv, a.qkv_f32, ob + a.d + 1);
        v0 = ld_qkv(a.qkv, a.qkv_f32, ob + 2 * (size_t)a.d); v1 = ld_qkv(a.qkv, a.qkv_f32, ob + 2 * (size_t)a.d + 1);
        if (rope) {
          const int pos = a.row_tau[k0 + kt0 + e] + a.row_sub[k0 + kt0 + e];
          const float2 cs = a.rope_tab[(size_t)pos * (kDh / 2) + j];
          const float t = x0 * cs.x - x1 * cs.y;
          x1 = x0 * cs.y + x1 * cs.x; x0 = t;
        }
        if (!a.qkv_f32) { /* bf16 inputs are used as they are */ }
      }
      Ks[e][2 * j] = x0; Ks[e][2 * j + 1] = x1;
      Vs[e][2 * j] = v0; Vs[e][2 * j + 1] = v1;
    }
    __syncthreads();
    // scores in the log2 domain; the dependency rule per pair: i' <= i and tau' <= tau
    for (int idx = tid; idx < DQ * DK; idx += DT) {
      const int r = idx / DK, e = idx % DK;
      float sc = -INFINITY;
      if (r < nq && ki_s[e] <= qi_s[r] && kt_s[e] <= qt_s[r]) {
        float acc = 0.f;
#pragma unroll 16
        for (int c = 0; c < kDh; ++c) acc = fmaf(Qs[r][c], Ks[e][c], acc);
        sc = acc * a.scale_log2e;
        if (use_bias) sc += bias_d[(qt_s[r] + qi_s[r]) - (kt_s[e] + ki_s[e])];   // = |dtau| + |di| on a visible pair
      }
      Ps[r][e] = sc;
    }
    __syncthreads();
    if (tid < nq) {
      const int r = tid;
      float mt = m_s[r];
      for (int e = 0; e < DK; ++e) mt = fmaxf(mt, Ps[r][e]);
      float corr = 1.f, sum = 0.f;
      if (mt == -INFINITY) {
        for (int e = 0; e < DK; ++e) Ps[r][e] = 0.f;
      } else {
        corr = exp2f(m_s[r] - mt);
        for (int e = 0; e < DK; ++e) { const float p = exp2f(Ps[r][e] - mt); Ps[r][e] = p; sum += p; }
      }
      l_s[r] = l_s[r] * corr + sum;
      m_s[r] = mt;
      corr_s[r] = corr;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < DRPT; ++u) {
      const int r = sg + u * DSG;
      if (r < nq) {
        float acc = o[u] * corr_s[r];
        for (int e = 0; e < nv; ++e) acc = fmaf(Ps[r][e], Vs[e][dim], acc);
        o[u] = acc;
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int u = 0; u < DRPT; ++u) {
    const int r = sg + u * DSG;
    if (r < nq) a.out[(size_t)(q0 + r) * a.d + (size_t)h * kDh + dim] = __float2bfloat16_rn(o[u] / l_s[r]);
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
  if (a.bias_tab != nullptr && a.n_dist > DMAXD) return cudaErrorInvalidValue;
  dense_self_attn_kernel<<<dim3(a.n_groups, a.H), DT, 0, s>>>(a);
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
