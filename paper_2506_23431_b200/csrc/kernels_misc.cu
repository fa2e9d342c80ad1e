// Small kernels of the decode step: state reset, embedding gather, RMSNorm, ReLU,
// KV-append with the positional write.
#include <cuda_fp8.h>

#include "pd_internal.h"

namespace pd {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------------
// Reset (the initialisation of Algorithm 1 plus the admission of subsequence 1 at step 1): clears the
// whole state block, then gives every sequence its first subsequence, first KV page and row.
__global__ void reset_state_kernel(Dims dm, DecState st, int batch, const int32_t *ctx_len,
                                   const int32_t *forced_len, size_t state_words, int32_t *state_base, int phase) {
  size_t gid = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  size_t stride = (size_t)gridDim.x * blockDim.x;
  if (phase == 0) {
    for (size_t i = gid; i < state_words; i += stride) state_base[i] = 0;
    return;
  }
  // phase 1 (after phase 0 has completed on the stream)
  for (size_t i = gid; i < (size_t)batch * dm.SM; i += stride) {
    st.forced_len[i] = forced_len ? forced_len[i] : -1;
    st.last_tok[i] = dm.bos;
    st.plan[i] = (int)(i % dm.SM) * dm.dt + 1;          // Eq. 2: s_i = (i-1) delta_t + 1
  }
  for (size_t i = gid; i < (size_t)dm.B * dm.SM * (dm.MSL + 1); i += stride) st.chosen[i] = -1;
  for (size_t i = gid; i < (size_t)dm.B * dm.SM * dm.MSL; i += stride) st.tokens[i] = -1;
  for (size_t b = gid; b < (size_t)batch; b += stride) {
    st.ctx_len[b] = ctx_len[b];
    st.k[b] = 1;
    st.n_active[b] = 1;
    st.start[b * dm.SM] = 1;
    st.state[b * dm.SM] = SUB_ACTIVE;
    st.row_sub[b * dm.C] = 1;
    const int pg = dm.pool_static ? (int)b * dm.SM * dm.PPS : (int)b;    // bump allocation: pages 0..batch-1 go to the first subsequences
    st.page_table[(size_t)b * dm.SM * dm.PPS] = pg;
    st.plist[(size_t)b * dm.SM * dm.PPS] = make_int4(pg, 1, 1, -1);      // step 1: bos of subsequence 1 at position 1, d0 = 0 - 1
    st.plist_n[b] = 1;
    st.row_meta[b * dm.C] = make_int4(pg, 0, 1, 1);                      // bos goes to slot 0 of that page, position 0 + 1
    for (int c = 1; c < dm.C; ++c) st.row_meta[b * dm.C + c] = make_int4(0, 0, 0, 0);
  }
  if (gid == 0) {
    st.hdr[HDR_STEP_T] = 1;
    st.hdr[HDR_BATCH] = batch;
    st.hdr[HDR_PAGE_BUMP] = batch;
    if (batch > dm.pool) st.hdr[HDR_STATUS] = PD_ERR_POOL_EXHAUSTED;
  }
}

// A new sequence in row b between two steps (the initialisation of Algorithm 1 for this row alone): the row's
// state as reset_state leaves it, with the row's step origin at the step before the coming one, so that the
// coming step is its step 1.  Only with the static page mapping (the row's pages are its own).
__global__ void admit_row_kernel(Dims dm, DecState st, int b, int ctx_len, const int32_t *forced_len) {
  const int tid = threadIdx.x, n = blockDim.x;
  const int SM = dm.SM, C = dm.C, NPT = dm.SM * dm.PPS;
  for (int i = tid; i < SM; i += n) {
    const int sidx = b * SM + i;
    st.forced_len[sidx] = forced_len ? forced_len[i] : -1;
    st.last_tok[sidx] = dm.bos;
    st.plan[sidx] = i * dm.dt + 1;
    st.start[sidx] = i == 0 ? 1 : 0; st.len[sidx] = 0; st.state[sidx] = i == 0 ? SUB_ACTIVE : SUB_NONE; st.flag[sidx] = 0;
  }
  for (int i = tid; i < SM * (dm.MSL + 1); i += n) st.chosen[(size_t)b * SM * (dm.MSL + 1) + i] = -1;
  for (int i = tid; i < SM * dm.MSL; i += n) st.tokens[(size_t)b * SM * dm.MSL + i] = -1;
  for (int i = tid; i < NPT; i += n) st.page_table[(size_t)b * NPT + i] = 0;
  for (int c = tid; c < C; c += n) {
    st.row_sub[b * C + c] = c == 0 ? 1 : 0; st.prev_row_sub[b * C + c] = 0; st.row_tok[b * C + c] = 0;
    st.row_meta[b * C + c] = make_int4(0, 0, 0, 0);
  }
  for (int t = tid; t < dm.T; t += n) st.trace[(size_t)t * dm.B + b] = 0ull;
  __syncthreads();
  if (tid == 0) {
    const int pg = b * NPT;
    st.ctx_len[b] = ctx_len;
    st.k[b] = 1; st.n_active[b] = 1; st.steps[b] = 0; st.seq_ticket[b] = 0;
    st.page_table[(size_t)b * NPT] = pg;
    st.plist[(size_t)b * NPT] = make_int4(pg, 1, 1, -1);
    st.plist_n[b] = 1;
    st.row_meta[b * C] = make_int4(pg, 0, 1, 1);
    st.t0[b] = st.hdr[HDR_STEP_T] - 1;
    if (st.done[b]) { st.done[b] = 0; atomicSub(&st.hdr[HDR_N_DONE], 1); }
    st.hdr[HDR_ALL_DONE] = 0;
  }
}

cudaError_t launch_admit_row(const Dims &dm, const DecState &st, int row, int ctx_len, const int32_t *forced_len_dev, cudaStream_t s) {
  admit_row_kernel<<<1, 256, 0, s>>>(dm, st, row, ctx_len, forced_len_dev);
  return cudaGetLastError();
}

cudaError_t launch_reset_state(const Dims &dm, const DecState &st, int batch, const int32_t *ctx_len_dev,
                               const int32_t *forced_len_dev, size_t state_words, int32_t *state_base,
                               cudaStream_t s) {
  reset_state_kernel<<<148, 256, 0, s>>>(dm, st, batch, ctx_len_dev, forced_len_dev, state_words, state_base, 0);
  reset_state_kernel<<<148, 256, 0, s>>>(dm, st, batch, ctx_len_dev, forced_len_dev, state_words, state_base, 1);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// bias_tab[h][dist] = rel_bias[h][bucket(dist)] * log2(e): the positional term of a score in the
// log2 domain, indexed by the Manhattan distance itself.  Built once per handle.
__global__ void build_bias_table_kernel(int H, int n_dist, int rel_buckets, const float *__restrict__ rel_bias,
                                        const int32_t *__restrict__ dist_bucket, float *__restrict__ bias_tab) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= H * n_dist) return;
  int h = i / n_dist, dd = i % n_dist;
  bias_tab[i] = rel_bias[h * rel_buckets + dist_bucket[dd]] * 1.4426950408889634f;
}

cudaError_t launch_build_bias_table(const Dims &dm, const float *rel_bias, int rel_buckets, const int32_t *dist_bucket,
                                    float *bias_tab, cudaStream_t s) {
  int n = dm.H * dm.n_dist;
  build_bias_table_kernel<<<(n + 255) / 256, 256, 0, s>>>(dm.H, dm.n_dist, rel_buckets, rel_bias, dist_bucket, bias_tab);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Embedding gather: row (b, c) takes the embedding of the last token of its subsequence (the
// decoder input of Eq. 3); unused rows are zero so that they stay zero through the layer stack.
// The first layer's RMSNorm of the row rides along (the CTA holds the whole row): h = norm(x) * gain.
template <typename T>
__global__ void __launch_bounds__(128) embed_kernel(Dims dm, DecState st, const T *__restrict__ embed, float *__restrict__ x,
                                                    const T *__restrict__ gain, T *__restrict__ h) {
  __shared__ float red[4];
  int r = blockIdx.x;
  int b = r / dm.C;
  int i = st.row_sub[r];
  float *xr = x + (size_t)r * dm.d;
  T *hr = h + (size_t)r * dm.d;
  if (i <= 0) {
    for (int c = threadIdx.x; c < dm.d; c += blockDim.x) { xr[c] = 0.f; hr[c] = from_f<T>(0.f); }
    return;
  }
  int tok = st.last_tok[b * dm.SM + i - 1];
  const T *e = embed + (size_t)tok * dm.d;
  float ss = 0.f;
  for (int c = threadIdx.x; c < dm.d; c += blockDim.x) { const float v = to_f<T>(e[c]); xr[c] = v; ss += v * v; }
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  const float inv = rsqrtf((red[0] + red[1] + red[2] + red[3]) / (float)dm.d + dm.eps);
  for (int c = threadIdx.x; c < dm.d; c += blockDim.x) hr[c] = from_f<T>(to_f<T>(e[c]) * inv * to_f<T>(gain[c]));
}

// gain, h: the first layer's norm gain and the buffer its normalised rows go to (the input of that layer's Q/K/V projection)
cudaError_t launch_embed(const Dims &dm, const DecState &st, int batch, int dtype, const void *embed, float *x, const void *gain,
                         void *h, cudaStream_t s) {
  int rows = batch * dm.C;
  if (dtype == PD_DTYPE_BF16)
    embed_kernel<__nv_bfloat16><<<rows, 128, 0, s>>>(dm, st, (const __nv_bfloat16 *)embed, x, (const __nv_bfloat16 *)gain, (__nv_bfloat16 *)h);
  else
    embed_kernel<float><<<rows, 128, 0, s>>>(dm, st, (const float *)embed, x, (const float *)gain, (float *)h);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// RMSNorm of the fp32 residual stream, output in the GEMM input type.  One CTA per row; a thread
// keeps its part of the row in registers (one pass over memory) when the row fits RN_REGS values
// per thread, else the row is read twice.
constexpr int RN_THREADS = 256, RN_REGS = 8;

template <typename T>
__global__ void __launch_bounds__(RN_THREADS) rmsnorm_kernel(int d, float eps, const float *__restrict__ x,
                                                             const T *__restrict__ gain, T *__restrict__ out) {
  __shared__ float red[RN_THREADS / 32];
  const float *xr = x + (size_t)blockIdx.x * d;
  T *orow = out + (size_t)blockIdx.x * d;
  const bool in_regs = d <= RN_THREADS * RN_REGS;
  float v[RN_REGS];
  float ss = 0.f;
  if (in_regs) {
#pragma unroll
    for (int k = 0; k < RN_REGS; ++k) {
      const int c = k * RN_THREADS + threadIdx.x;
      v[k] = c < d ? xr[c] : 0.f;
      ss += v[k] * v[k];
    }
  } else {
    for (int c = threadIdx.x; c < d; c += RN_THREADS) { float t = xr[c]; ss += t * t; }
  }
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < RN_THREADS / 32; ++w) tot += red[w];     // every thread sums the warps' parts in the same order
  const float inv = rsqrtf(tot / (float)d + eps);
  if (in_regs) {
#pragma unroll
    for (int k = 0; k < RN_REGS; ++k) {
      const int c = k * RN_THREADS + threadIdx.x;
      if (c < d) orow[c] = from_f<T>(v[k] * inv * to_f<T>(gain[c]));
    }
  } else {
    for (int c = threadIdx.x; c < d; c += RN_THREADS) orow[c] = from_f<T>(xr[c] * inv * to_f<T>(gain[c]));
  }
}

cudaError_t launch_rmsnorm(const Dims &dm, int rows, int dtype, const float *x, const void *gain, void *out,
                           cudaStream_t s) {
  if (dtype == PD_DTYPE_BF16)
    rmsnorm_kernel<__nv_bfloat16><<<rows, RN_THREADS, 0, s>>>(dm.d, dm.eps, x, (const __nv_bfloat16 *)gain, (__nv_bfloat16 *)out);
  else
    rmsnorm_kernel<float><<<rows, RN_THREADS, 0, s>>>(dm.d, dm.eps, x, (const float *)gain, (float *)out);
  return cudaGetLastError();
}

// The same norm for the rows that feed the vocabulary projection: only active rows are written,
// packed back to back in (sequence, row) order, so that the projection's work follows the rows
// that exist.  Row (b, c) goes to crow[b] + c with crow[b] = active rows of the sequences before b;
// the CTA of row (b, 0) publishes crow[b] for the kernels that follow.
template <typename T>
__global__ void __launch_bounds__(RN_THREADS) rmsnorm_packed_kernel(int d, float eps, int C, DecState st,
                                                                    const float *__restrict__ x, const T *__restrict__ gain,
                                                                    T *__restrict__ out) {
  __shared__ float red[RN_THREADS / 32];
  __shared__ int redi[RN_THREADS / 32];
  // the vocabulary projection that follows may start its set-up and its first lm_head copies now (it waits for
  // this kernel's rows where it needs them)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int b = blockIdx.x / C, c = blockIdx.x % C;
  int before = 0;
  for (int bb = threadIdx.x; bb < b; bb += RN_THREADS) before += st.n_active[bb];
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
  if ((threadIdx.x & 31) == 0) redi[threadIdx.x >> 5] = before;
  __syncthreads();
  before = 0;
#pragma unroll
  for (int w = 0; w < RN_THREADS / 32; ++w) before += redi[w];
  if (c == 0 && threadIdx.x == 0) st.crow[b] = before;
  if (c >= st.n_active[b]) return;
  const float *xr = x + (size_t)blockIdx.x * d;
  T *orow = out + (size_t)(before + c) * d;
  float ss = 0.f;
  for (int col = threadIdx.x; col < d; col += RN_THREADS) { const float t = xr[col]; ss += t * t; }
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < RN_THREADS / 32; ++w) tot += red[w];
  const float inv = rsqrtf(tot / (float)d + eps);
  for (int col = threadIdx.x; col < d; col += RN_THREADS) orow[col] = from_f<T>(xr[col] * inv * to_f<T>(gain[col]));
}

cudaError_t launch_rmsnorm_packed(const Dims &dm, const DecState &st, int batch, int dtype, const float *x, const void *gain,
                                  void *out, cudaStream_t s) {
  if (dtype == PD_DTYPE_BF16)
    rmsnorm_packed_kernel<__nv_bfloat16><<<batch * dm.C, RN_THREADS, 0, s>>>(dm.d, dm.eps, dm.C, st, x, (const __nv_bfloat16 *)gain,
                                                                             (__nv_bfloat16 *)out);
  else
    rmsnorm_packed_kernel<float><<<batch * dm.C, RN_THREADS, 0, s>>>(dm.d, dm.eps, dm.C, st, x, (const float *)gain, (float *)out);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void relu_kernel(T *buf, size_t n) {
  size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) { float v = to_f<T>(buf[i]); buf[i] = from_f<T>(v > 0.f ? v : 0.f); }
}

cudaError_t launch_relu(int dtype, void *buf, size_t n, cudaStream_t s) {
  int blocks = (int)((n + 1023) / 1024);
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  if (dtype == PD_DTYPE_BF16) relu_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>((__nv_bfloat16 *)buf, n);
  else relu_kernel<float><<<blocks, 256, 0, s>>>((float *)buf, n);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// KV-append + positional write.  Row (b, c) belongs to subsequence i; its input token is cache
// entry p = len (p = 0 is bos) with timestamp tau = s_i - 1 + p (Eq. 2) and position tau + i, so
// that the difference of two positions is the Manhattan distance of Section 4.3 on every visible
// pair.  Writes k and v to slot p of the subsequence's page list and q to the query buffer; in
// RoPE mode q and k are rotated by the position first.  All rows of a step are appended before
// any attends: tokens fed by earlier subsequences at the same step are visible (tau' <= t - 1).
// The same step when q, k, v arrive already in the storage type (no rotation to apply, so the
// projection's own epilogue did the one rounding): eight columns (16 bytes) per thread, pure copies.
__global__ void append_copy_bf16_kernel(Dims dm, DecState st, int layer, const __nv_bfloat16 *__restrict__ qkv,
                                        __nv_bfloat16 *__restrict__ q_out, __nv_bfloat16 *__restrict__ kv_pool) {
  const int r = blockIdx.x;
  const __nv_bfloat16 *row = qkv + (size_t)r * 3 * dm.d;
  const int4 meta = st.row_meta[r];                 // (page, slot, position tau + i, subsequence i or 0)
  const int col = 8 * threadIdx.x;                  // blockDim.x = d / 8; one 16-byte chunk of one head
  const uint4 q = *reinterpret_cast<const uint4 *>(row + col);
  const uint4 k = *reinterpret_cast<const uint4 *>(row + dm.d + col);
  const uint4 v = *reinterpret_cast<const uint4 *>(row + 2 * dm.d + col);
  if (meta.w <= 0) return;
  const int h = col / kDh, dd = col % kDh;
  __nv_bfloat16 *ko = kv_pool + kv_block_offset(layer, dm.pool, meta.x, dm.H, h, dm.P) + kv_entry_offset<__nv_bfloat16>(meta.y, dd, 0);
  *reinterpret_cast<uint4 *>(q_out + (size_t)r * dm.d + col) = q;
  *reinterpret_cast<uint4 *>(ko) = k;
  *reinterpret_cast<uint4 *>(ko + kDh) = v;         // the value row follows the key row of the same entry
}

template <typename T>
__global__ void append_kernel(Dims dm, DecState st, int layer, const float *__restrict__ qkv, T *__restrict__ q_out,
                              T *__restrict__ kv_pool, const float2 *__restrict__ rope_tab) {
  const int r = blockIdx.x;
  const float *row = qkv + (size_t)r * 3 * dm.d;
  // one round of independent loads: where the row goes, and this thread's four columns of q, k, v
  const int4 meta = st.row_meta[r];                 // (page, slot, position tau + i, subsequence i or 0)
  const int col = 4 * threadIdx.x;                  // blockDim.x = d / 4; four columns never straddle a 16-byte chunk or a head
  float4 q = *reinterpret_cast<const float4 *>(row + col);
  float4 k = *reinterpret_cast<const float4 *>(row + dm.d + col);
  const float4 v = *reinterpret_cast<const float4 *>(row + 2 * dm.d + col);
  if (meta.w <= 0) return;
  const int h = col / kDh, dd = col % kDh;
  if (dm.pos_mode == PD_POS_ROPE) {
    const float2 c0 = rope_tab[(size_t)meta.z * (kDh / 2) + dd / 2], c1 = rope_tab[(size_t)meta.z * (kDh / 2) + dd / 2 + 1];
    float a;
    a = q.x * c0.x - q.y * c0.y; q.y = q.x * c0.y + q.y * c0.x; q.x = a;
    a = q.z * c1.x - q.w * c1.y; q.w = q.z * c1.y + q.w * c1.x; q.z = a;
    a = k.x * c0.x - k.y * c0.y; k.y = k.x * c0.y + k.y * c0.x; k.x = a;
    a = k.z * c1.x - k.w * c1.y; k.w = k.z * c1.y + k.w * c1.x; k.z = a;
  }
  T *qo = q_out + (size_t)r * dm.d + col;
  T *ko = kv_pool + kv_block_offset(layer, dm.pool, meta.x, dm.H, h, dm.P) + kv_entry_offset<T>(meta.y, dd, 0);
  T *vo = ko + kDh;                                 // the value row follows the key row of the same entry
  qo[0] = from_f<T>(q.x); qo[1] = from_f<T>(q.y); qo[2] = from_f<T>(q.z); qo[3] = from_f<T>(q.w);
  ko[0] = from_f<T>(k.x); ko[1] = from_f<T>(k.y); ko[2] = from_f<T>(k.z); ko[3] = from_f<T>(k.w);
  vo[0] = from_f<T>(v.x); vo[1] = from_f<T>(v.y); vo[2] = from_f<T>(v.z); vo[3] = from_f<T>(v.w);
}

cudaError_t launch_append_copy_bf16(const Dims &dm, const DecState &st, int batch, int layer, const void *qkv, void *q_out,
                                    void *kv_pool, cudaStream_t s) {
  append_copy_bf16_kernel<<<batch * dm.C, dm.d / 8, 0, s>>>(dm, st, layer, (const __nv_bfloat16 *)qkv, (__nv_bfloat16 *)q_out,
                                                           (__nv_bfloat16 *)kv_pool);
  return cudaGetLastError();
}

cudaError_t launch_append(const Dims &dm, const DecState &st, int batch, int layer, int dtype, const float *qkv,
                          void *q_out, void *kv_pool, const float2 *rope_tab, cudaStream_t s) {
  int rows = batch * dm.C;
  int threads = dm.d / 4;                           // d is a multiple of 64 and at most 4096 (checked at init)
  if (dtype == PD_DTYPE_BF16)
    append_kernel<__nv_bfloat16><<<rows, threads, 0, s>>>(dm, st, layer, qkv, (__nv_bfloat16 *)q_out,
                                                         (__nv_bfloat16 *)kv_pool, rope_tab);
  else
    append_kernel<float><<<rows, threads, 0, s>>>(dm, st, layer, qkv, (float *)q_out, (float *)kv_pool, rope_tab);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// The context projection writes [position][k of all heads | v of all heads]; the attention
// kernels read head-major blocks.  One 16-byte chunk per thread and iteration.
__global__ void ctx_kv_relayout_kernel(Dims dm, int b0, int batch, int layer, int esize, const uint4 *__restrict__ proj,
                                       uint4 *__restrict__ kv_c) {
  const int cpr = kDh * esize / 16;                        // 16-byte chunks of one head's row
  const size_t per_pos = (size_t)2 * dm.H * cpr;           // chunks of one projected position
  const size_t total = (size_t)batch * dm.ctx * per_pos;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(i % cpr);
    const int h = (int)((i / cpr) % dm.H);
    const int is_v = (int)((i / ((size_t)cpr * dm.H)) % 2);
    const size_t bp = i / per_pos;
    const int pos = (int)(bp % dm.ctx), b = (int)(bp / dm.ctx);
    const size_t dst = (ctx_kv_offset(layer, dm.B, b0 + b, dm.H, h, is_v, dm.ctx) + (size_t)pos * kDh) * esize / 16 + c;
    kv_c[dst] = proj[i];
  }
}

// proj holds the projections of sequences b0 .. b0 + batch - 1.
cudaError_t launch_ctx_kv_relayout(const Dims &dm, int b0, int batch, int layer, int dtype, const void *proj, void *kv_c,
                                   cudaStream_t s) {
  const int esize = dtype == PD_DTYPE_BF16 ? 2 : 4;
  ctx_kv_relayout_kernel<<<148 * 8, 256, 0, s>>>(dm, b0, batch, layer, esize, (const uint4 *)proj, (uint4 *)kv_c);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// 8-bit storage of the context keys/values (E4M3, one scale per (layer, sequence, head, keys | values)).
// proj holds [position][k of all heads | v of all heads] in bf16 for sequences b0 .. b0 + nb - 1.
// Pass 1: scale = max|.| / 448 over the positions below ctx_len (1 when all are zero).
__global__ void __launch_bounds__(256) ctx_kv_amax_kernel(Dims dm, int b0, int layer, const __nv_bfloat16 *__restrict__ proj,
                                                          const int32_t *__restrict__ ctx_len, float *__restrict__ scale,
                                                          float *__restrict__ amax) {
  __shared__ float red[8];
  const int h = blockIdx.x >> 1, kv = blockIdx.x & 1, b = blockIdx.y;
  const int n = min(max(ctx_len[b0 + b], 0), dm.ctx);
  const __nv_bfloat16 *base = proj + (size_t)b * dm.ctx * 2 * dm.d + (size_t)kv * dm.d + (size_t)h * kDh;
  float m = 0.f;
  for (int idx = threadIdx.x; idx < n * 8; idx += 256) {               // one 16-byte chunk (8 values) per thread and iteration
    const int pos = idx >> 3, c = idx & 7;
    const uint4 v = *reinterpret_cast<const uint4 *>(base + (size_t)pos * 2 * dm.d + c * 8);
    const __nv_bfloat162 *p2 = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int j = 0; j < 4; ++j) m = fmaxf(m, fmaxf(fabsf(__low2float(p2[j])), fabsf(__high2float(p2[j]))));
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]);
    const size_t i = ((((size_t)layer * dm.B + b0 + b) * dm.H + h) << 1) + kv;
    scale[i] = m > 0.f ? __fdiv_rn(m, 448.f) : 1.f;
    amax[i] = m;
  }
}

// Pass 2: codes.  Keys as [position][64] (two keys per 128-byte line; inside every group of 16 positions
// key g sits at place 8 * ((g >> 1) & 1) + 2 * (g >> 2) + (g & 1): the order the attention kernel's score
// tiles take them in, which keeps its ldmatrix rows in different banks), values transposed as [dim][max_ctx],
// both inside the block of (layer, sequence, head): keys at + 0, values at + max_ctx * 64 bytes.  A value's
// code is the nearest E4M3 number (ties to even, saturating) of value * (448 / max|.|), the product
// rounded to fp32; positions at or beyond ctx_len become zeros.
__global__ void __launch_bounds__(256) ctx_kv_quant_kernel(Dims dm, int b0, int layer, const __nv_bfloat16 *__restrict__ proj,
                                                           const int32_t *__restrict__ ctx_len, const float *__restrict__ amax,
                                                           uint8_t *__restrict__ kv8) {
  __shared__ uint8_t vt[64][80];                      // this tile's value codes, [position][dim], rows padded to 80 bytes
  const int tile = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int n = min(max(ctx_len[b0 + b], 0), dm.ctx);
  const size_t blk = (((size_t)layer * dm.B + b0 + b) * dm.H + h) * 2;
  const float mk = amax[blk], mv = amax[blk + 1];
  const float ik = mk > 0.f ? __fdiv_rn(448.f, mk) : 1.f, iv = mv > 0.f ? __fdiv_rn(448.f, mv) : 1.f;
  uint8_t *kblock = kv8 + blk * (size_t)dm.ctx * kDh, *vblock = kblock + (size_t)dm.ctx * kDh;
  const int t = threadIdx.x, pl = t >> 2, c = t & 3;          // position within the tile, 16-value chunk
  const int pos = tile * 64 + pl;
  const __nv_bfloat16 *row = proj + ((size_t)b * dm.ctx + pos) * 2 * dm.d + (size_t)h * kDh + c * 16;
  uint32_t kc[4] = {0u, 0u, 0u, 0u}, vc[4] = {0u, 0u, 0u, 0u};
  if (pos < n) {
    uint4 kin[2], vin[2];
    kin[0] = *reinterpret_cast<const uint4 *>(row); kin[1] = *reinterpret_cast<const uint4 *>(row + 8);
    vin[0] = *reinterpret_cast<const uint4 *>(row + dm.d); vin[1] = *reinterpret_cast<const uint4 *>(row + dm.d + 8);
    const __nv_bfloat162 *k2 = reinterpret_cast<const __nv_bfloat162 *>(kin), *v2 = reinterpret_cast<const __nv_bfloat162 *>(vin);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float2 kf = make_float2(__fmul_rn(__low2float(k2[j]), ik), __fmul_rn(__high2float(k2[j]), ik));
      const float2 vf = make_float2(__fmul_rn(__low2float(v2[j]), iv), __fmul_rn(__high2float(v2[j]), iv));
      kc[j >> 1] |= (uint32_t)__nv_cvt_float2_to_fp8x2(kf, __NV_SATFINITE, __NV_E4M3) << (16 * (j & 1));
      vc[j >> 1] |= (uint32_t)__nv_cvt_float2_to_fp8x2(vf, __NV_SATFINITE, __NV_E4M3) << (16 * (j & 1));
    }
  }
  const int g16 = pos & 15, place = (pos & ~15) | ((((g16 >> 1) & 1) << 3) + ((g16 >> 2) << 1) + (g16 & 1));
  if (pos < dm.ctx) *reinterpret_cast<uint4 *>(kblock + (size_t)place * kDh + c * 16) = make_uint4(kc[0], kc[1], kc[2], kc[3]);
  *reinterpret_cast<uint4 *>(&vt[pl][c * 16]) = make_uint4(vc[0], vc[1], vc[2], vc[3]);
  __syncthreads();
  // transposed write: thread = (dim, 16 positions)
  const int dim = t >> 2, p0 = (t & 3) * 16;
  uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j >> 2] |= (uint32_t)vt[p0 + j][dim] << (8 * (j & 3));
  if (tile * 64 + p0 < dm.ctx)                       // max_ctx is a multiple of 16: a chunk is inside or outside as a whole
    *reinterpret_cast<uint4 *>(vblock + (size_t)dim * dm.ctx + tile * 64 + p0) = make_uint4(o[0], o[1], o[2], o[3]);
}

// scale, amax: [layer][sequence][head][keys | values] fp32 each.
cudaError_t launch_ctx_kv_quantize(const Dims &dm, int b0, int batch, int layer, const void *proj, const int32_t *ctx_len_dev,
                                   float *scale, float *amax, void *kv8, cudaStream_t s) {
  ctx_kv_amax_kernel<<<dim3(dm.H * 2, batch), 256, 0, s>>>(dm, b0, layer, (const __nv_bfloat16 *)proj, ctx_len_dev, scale, amax);
  ctx_kv_quant_kernel<<<dim3((dm.ctx + 63) / 64, dm.H, batch), 256, 0, s>>>(dm, b0, layer, (const __nv_bfloat16 *)proj, ctx_len_dev,
                                                                            amax, (uint8_t *)kv8);
  return cudaGetLastError();
}

}  // namespace pd
