// CUDA-core attention kernels (fp32 arithmetic) for both storage types:
//   * pipelined self-attention over the paged per-subsequence KV cache, with the visibility
//     rule of Section 3.2 evaluated from (subsequence, start step, entry) metadata per page;
//   * cross-attention over the shared context keys/values (all context rows < ctx_len visible);
//   * the split-K merge.
// These are the fp32 path of every configuration and the bf16 path when a sequence has more
// than 32 rows; otherwise bf16 runs the tensor-core kernels in self_attn_tc.cu and
// cross_attn_tma.cu.
#include "pd_internal.h"

namespace pd {

template <typename T> __device__ __forceinline__ float ld_f(const T *p);
template <> __device__ __forceinline__ float ld_f<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ld_f<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st_f(T *p, float v);
template <> __device__ __forceinline__ void st_f<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void st_f<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

constexpr int TK = 32;            // keys per tile
constexpr int NT = 256;           // threads per CTA
constexpr int SG = NT / kDh;      // 4 row groups
constexpr int RPT = kMaxRows / SG;  // rows per thread in the PV phase (16)
constexpr int MAXD = 512;         // longest distance table held in shared memory

// One CTA = one (split, head, sequence).  All active subsequences of the sequence are processed
// together so that each key/value tile is read once for all of them.
template <typename T, bool SELF>
__global__ void __launch_bounds__(NT) attn_core_kernel(AttnArgs a) {
  const Dims &dm = a.dm;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x;
  // (the stand-alone op reads caller-written counts: clamped, so that no access leaves the tensors)
  const int S = min(max(a.st.n_active[b], 0), min(dm.C, kMaxRows));
  const int row0 = b * dm.C;
  const int t = SELF ? a.st.hdr[HDR_STEP_T] - a.st.t0[b] : 0;        // the sequence's own step
  const T *qbuf = (const T *)a.q;
  T *out = (T *)a.out;

  __shared__ float Qs[kMaxRows][kDh];
  __shared__ float Ks[TK][kDh + 1];
  __shared__ float Vs[TK][kDh];
  __shared__ float Ps[kMaxRows][TK];
  __shared__ float m_s[kMaxRows], l_s[kMaxRows], corr_s[kMaxRows];
  __shared__ int sub_s[kMaxRows];
  __shared__ float bias_d[SELF ? MAXD : 1];

  if (S == 0) {   // nothing active: keep the output rows of this head defined
    if (split == 0)
      for (int idx = tid; idx < dm.C * kDh; idx += NT)
        st_f<T>(out + (size_t)(row0 + idx / kDh) * dm.d + h * kDh + idx % kDh, 0.f);
    return;
  }

  for (int idx = tid; idx < S * kDh; idx += NT) {
    int s = idx / kDh, c = idx % kDh;
    Qs[s][c] = ld_f<T>(qbuf + (size_t)(row0 + s) * dm.d + h * kDh + c);
  }
  if (tid < kMaxRows) {
    m_s[tid] = -INFINITY; l_s[tid] = 0.f; corr_s[tid] = 1.f;
    sub_s[tid] = (SELF && tid < S) ? a.st.row_sub[row0 + tid] : 0;
  }
  const bool use_bias = SELF && dm.pos_mode == PD_POS_T5_BIAS;
  if (use_bias)
    for (int dd = tid; dd < dm.n_dist && dd < MAXD; dd += NT)
      bias_d[dd] = a.rel_bias[h * a.rel_buckets + a.dist_bucket[dd]] * 1.4426950408889634f;  // log2 domain
  __syncthreads();

  float o[RPT];
#pragma unroll
  for (int u = 0; u < RPT; ++u) o[u] = 0.f;
  const int dim = tid & (kDh - 1), sg = tid >> 6;

  // tile enumeration
  int n_tiles, i_max = 0, ctx_len = 0;
  if (SELF) {
    i_max = sub_s[S - 1];                  // rows are in increasing subsequence order
    n_tiles = a.st.k[b] * dm.PPS;          // one tile per page (page_tokens <= TK)
  } else {
    ctx_len = min(max(a.st.ctx_len[b], 1), dm.ctx);
    n_tiles = (ctx_len + TK - 1) / TK;
  }
  for (int tile = split; tile < n_tiles; tile += a.splits) {
    int n_valid;           // keys of this tile that exist
    int k_sub = 0, k_tau0 = 0;
    const T *kp, *vp;
    size_t kstride;
    if (SELF) {
      int ksub = tile / dm.PPS + 1, j = tile % dm.PPS;
      if (ksub > i_max) break;             // later subsequences are invisible to every row
      int sidx = b * dm.SM + ksub - 1;
      int n_entries = a.st.len[sidx] + 1;  // bos + content tokens, including this step's input
      int e0 = j * dm.P;
      n_valid = min(dm.P, n_entries - e0);
      if (n_valid <= 0) continue;
      int page = a.st.page_table[(size_t)sidx * dm.PPS + j];
      kp = (const T *)a.kv + kv_block_offset(a.layer, dm.pool, page, dm.H, h, dm.P);
      vp = kp;             // values interleaved with the keys, entry by entry
      kstride = kDh;
      k_sub = ksub;
      k_tau0 = a.st.start[sidx] - 1 + e0;  // timestamp of the tile's first entry
    } else {
      int pos0 = tile * TK;
      n_valid = min(TK, ctx_len - pos0);
      kp = (const T *)a.kv + ctx_kv_offset(a.layer, dm.B, b, dm.H, h, 0, dm.ctx) + (size_t)pos0 * kDh;
      vp = kp + (size_t)dm.ctx * kDh;
      kstride = kDh;
    }
    __syncthreads();   // previous tile fully consumed
    for (int idx = tid; idx < n_valid * kDh; idx += NT) {
      int e = idx / kDh, c = idx % kDh;
      Ks[e][c] = ld_f<T>(kp + (SELF ? kv_entry_offset<T>(e, c, 0) : e * kstride + c));
      Vs[e][c] = ld_f<T>(vp + (SELF ? kv_entry_offset<T>(e, c, 1) : e * kstride + c));
    }
    __syncthreads();
    // scores in the log2 domain
    for (int idx = tid; idx < S * TK; idx += NT) {
      int s = idx / TK, e = idx % TK;
      float sc = -INFINITY;
      bool vis = e < n_valid;
      if (SELF && vis) {
        // dependency rule: subsequence index not larger than the query's, timestamp not later
        vis = (k_sub <= sub_s[s]) && (k_tau0 + e <= t - 1);
      }
      if (vis) {
        float acc = 0.f;
#pragma unroll 16
        for (int c = 0; c < kDh; ++c) acc = fmaf(Qs[s][c], Ks[e][c], acc);
        sc = acc * dm.scale_log2e;
        if (use_bias) {
          int dist = (t - 1 + sub_s[s]) - (k_tau0 + e + k_sub);   // = |dtau| + |di| on a visible pair
          sc += bias_d[dist];
        }
      }
      Ps[s][e] = sc;
    }
    __syncthreads();
    if (tid < S) {
      int s = tid;
      float mt = m_s[s];
      for (int e = 0; e < TK; ++e) mt = fmaxf(mt, Ps[s][e]);
      float corr = 1.f, sum = 0.f;
      if (mt == -INFINITY) {
        for (int e = 0; e < TK; ++e) Ps[s][e] = 0.f;
      } else {
        corr = exp2f(m_s[s] - mt);
        for (int e = 0; e < TK; ++e) { float p = exp2f(Ps[s][e] - mt); Ps[s][e] = p; sum += p; }
      }
      l_s[s] = l_s[s] * corr + sum;
      m_s[s] = mt;
      corr_s[s] = corr;
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < RPT; ++u) {
      int s = sg + u * SG;
      if (s < S) {
        float acc = o[u] * corr_s[s];
        for (int e = 0; e < n_valid; ++e) acc = fmaf(Ps[s][e], Vs[e][dim], acc);
        o[u] = acc;
      }
    }
  }
  __syncthreads();

#pragma unroll
  for (int u = 0; u < RPT; ++u) {
    int s = sg + u * SG;
    if (s >= S) continue;
    int r = row0 + s;
    if (a.splits == 1) {
      st_f<T>(out + (size_t)r * dm.d + h * kDh + dim, o[u] / l_s[s]);
    } else {
      size_t pi = ((size_t)r * dm.H + h) * a.splits + split;
      a.part_o[pi * kDh + dim] = o[u];
      if (dim == 0) { a.part_ml[pi * 2] = m_s[s]; a.part_ml[pi * 2 + 1] = l_s[s]; }
    }
  }
  if (a.splits == 1 || split == 0)   // rows beyond the active ones stay zero
    for (int idx = tid; idx < (dm.C - S) * kDh; idx += NT)
      st_f<T>(out + (size_t)(row0 + S + idx / kDh) * dm.d + h * kDh + idx % kDh, 0.f);
}

cudaError_t launch_attn_core(const AttnArgs &a, int dtype, bool self, cudaStream_t s) {
  dim3 grid(a.splits, a.dm.H, a.batch);
  if (dtype == PD_DTYPE_BF16) {
    if (self) attn_core_kernel<__nv_bfloat16, true><<<grid, NT, 0, s>>>(a);
    else attn_core_kernel<__nv_bfloat16, false><<<grid, NT, 0, s>>>(a);
  } else {
    if (self) attn_core_kernel<float, true><<<grid, NT, 0, s>>>(a);
    else attn_core_kernel<float, false><<<grid, NT, 0, s>>>(a);
  }
  return cudaGetLastError();
}

// Merge of the split-K partials (m, l, o) of one row and head: the usual log-sum-exp rescale.
template <typename T>
__global__ void attn_merge_kernel(AttnArgs a) {
  const Dims &dm = a.dm;
  int r = blockIdx.x;
  int b = r / dm.C, c = r % dm.C;
  if (c >= min(a.st.n_active[b], dm.C)) return;       // the attention kernel already zeroed unused rows
  T *out = (T *)a.out;
  for (int idx = threadIdx.x; idx < dm.d; idx += blockDim.x) {
    int h = idx / kDh, dim = idx % kDh;
    size_t p0 = ((size_t)r * dm.H + h) * a.splits;
    float M = -INFINITY;
    for (int s = 0; s < a.splits; ++s) M = fmaxf(M, a.part_ml[(p0 + s) * 2]);
    float L = 0.f, O = 0.f;
    for (int s = 0; s < a.splits; ++s) {
      float m = a.part_ml[(p0 + s) * 2];
      if (m == -INFINITY) continue;
      float w = exp2f(m - M);
      L += a.part_ml[(p0 + s) * 2 + 1] * w;
      O += a.part_o[(p0 + s) * kDh + dim] * w;
    }
    st_f<T>(out + (size_t)r * dm.d + idx, O / L);
  }
}

cudaError_t launch_attn_merge(const AttnArgs &a, int dtype, cudaStream_t s) {
  int rows = a.batch * a.dm.C;
  if (dtype == PD_DTYPE_BF16) attn_merge_kernel<__nv_bfloat16><<<rows, 256, 0, s>>>(a);
  else attn_merge_kernel<float><<<rows, 256, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace pd
