// Fused logits-argmax + scheduler.  One CTA per row scans the row's fp32 logits for the
// greedy choice of Eq. 4 (ties to the lowest id); the CTA that finishes a sequence's last row
// then runs that sequence's part of Algorithm 1 for the step: append the tokens, retire
// subsequences on eos/sep, the stop test, the admission that the loop performs at the top of
// the next step, and the compaction of the active rows for it.  No CTA
// ever waits for another: the hand-over is an atomic ticket after a memory fence.
#include <limits.h>

#include "pd_internal.h"

namespace pd {

constexpr int AT = 512;

__device__ __forceinline__ void better(float &bv, int &bi, float v, int i) {
  if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

// One sequence's integer state for the step, staged in shared memory by the CTA that runs its
// scheduler: the scheduler itself is one thread walking dependent loads, which on global memory
// costs a round trip each; the CTA copies the arrays in (and the changed ones back out) with all
// its threads instead.  Indices are local to the sequence: subsequence i at [i - 1], row c at [c].
struct SeqStage {
  int32_t *row_sub, *row_tok;                                        // [C]
  int32_t *len, *forced_len, *state, *flag, *start, *last_tok, *teacher;   // [SM]
  int32_t *page_table;                                               // [SM * PPS]
  int4 *row_meta;                                                    // [C]
  int4 *plist;                                                       // [SM * PPS]
};
__host__ __device__ inline size_t seq_stage_bytes(const Dims &dm) {
  return ((size_t)(2 * dm.C + 7 * dm.SM + dm.SM * dm.PPS + 3) / 4 * 4) * sizeof(int32_t) + ((size_t)dm.C + (size_t)dm.SM * dm.PPS) * sizeof(int4);
}

// Algorithm 1 for one sequence and one step, after the step's tokens have been chosen: the append,
// the retirement on eos/sep, the stop test, the admission the loop performs at the top of the next
// step, and the compaction of the active rows for it.  Runs in one thread on the staged state.
__device__ void schedule_sequence(const Dims &dm, const DecState &st, const SeqStage &v, int b, bool have_teacher) {
  const int t = st.hdr[HDR_STEP_T];
  const int C = dm.C, SM = dm.SM;
  int nact = st.n_active[b];
  int k = st.k[b];
  if (st.done[b] || st.hdr[HDR_STATUS] != 0) {
    if (!st.done[b]) { st.done[b] = 1; st.steps[b] = t; atomicAdd(&st.hdr[HDR_N_DONE], 1); }
    for (int c = 0; c < C; ++c) { v.row_sub[c] = 0; v.row_meta[c] = make_int4(0, 0, 0, 0); }
    st.n_active[b] = 0;
    st.plist_n[b] = 0;
    return;
  }
  // traffic counters of the step just executed (before any length changes)
  int i_max = 0;
  for (int c = 0; c < nact; ++c) i_max = max(i_max, v.row_sub[c]);
  unsigned long long nvis = 0;
  for (int i = 1; i <= i_max; ++i) nvis += (unsigned long long)(v.len[i - 1] + 1);
  atomicAdd(&st.stats[PD_STAT_SELF_ENTRIES], nvis);
  if (nact > 0) atomicAdd(&st.stats[PD_STAT_CROSS_KEYS], (unsigned long long)st.ctx_len[b]);
  atomicAdd(&st.stats[PD_STAT_TOKENS], (unsigned long long)nact);

  unsigned long long mask = 0ull;
  for (int c = 0; c < nact; ++c) {
    const int i = v.row_sub[c];
    const int sidx = b * SM + i - 1;
    const int len = v.len[i - 1];
    const int fl = v.forced_len[i - 1];
    int own = v.row_tok[c];
    if (fl >= 0) { if (len >= fl) own = dm.sep; }
    else if (len >= dm.MSL) own = dm.sep;
    st.chosen[(size_t)sidx * (dm.MSL + 1) + len] = own;
    int tok = own;
    if (have_teacher) { int tt = v.teacher[i - 1]; if (tt >= 0) tok = tt; }
    if (len >= dm.MSL) { tok = dm.sep; if (fl < 0) v.flag[i - 1] |= PD_FLAG_CAPPED; }
    if (tok == dm.eos || tok == dm.sep) {
      v.state[i - 1] = SUB_ENDED;
      v.flag[i - 1] |= PD_FLAG_COMPLETE;
    } else {
      st.tokens[(size_t)sidx * dm.MSL + len] = tok;
      v.len[i - 1] = len + 1;
      v.last_tok[i - 1] = tok;
    }
    mask |= 1ull << (i - 1);
  }
  st.trace[(size_t)(t - 1) * dm.B + b] = mask;

  int ended = 0;
  for (int i = 1; i <= k; ++i) ended += v.state[i - 1] == SUB_ENDED;
  bool done = false;
  if (ended == k) {
    done = true;                                   // every subsequence has produced its terminator
  } else if (t >= dm.T) {
    done = true;                                   // time_max reached with subsequences still open
    for (int i = 1; i <= k; ++i)
      if (v.state[i - 1] == SUB_ACTIVE) v.flag[i - 1] |= PD_FLAG_TRUNCATED;
  } else if (t % dm.dt == 0 && k < SM) {           // step t+1 satisfies (t+1-1) mod delta_t == 0
    k += 1;
    st.k[b] = k;
    v.start[k - 1] = t + 1;
    v.len[k - 1] = 0;
    v.state[k - 1] = SUB_ACTIVE;
    v.flag[k - 1] = 0;
    v.last_tok[k - 1] = dm.bos;
  }
  int n = 0;
  if (done) {
    st.done[b] = 1;
    st.steps[b] = t;
    atomicAdd(&st.hdr[HDR_N_DONE], 1);
  } else {
    for (int i = 1; i <= k; ++i) {
      if (v.state[i - 1] != SUB_ACTIVE) continue;
      if (n >= C) { atomicExch(&st.hdr[HDR_STATUS], (int)PD_ERR_STATE); break; }
      const int p = v.len[i - 1];                  // entry the next step will write
      if (p % dm.P == 0) {
        int pg = atomicAdd(&st.hdr[HDR_PAGE_BUMP], 1);
        if (pg >= dm.pool) { atomicExch(&st.hdr[HDR_STATUS], (int)PD_ERR_POOL_EXHAUSTED); pg = 0; }
        v.page_table[(i - 1) * dm.PPS + p / dm.P] = pg;
        atomicAdd(&st.stats[PD_STAT_PAGES], 1ull);
      }
      // where the append kernels of the coming step put this row's key/value, and its position tau + i
      v.row_meta[n] = make_int4(v.page_table[(i - 1) * dm.PPS + p / dm.P], p % dm.P, v.start[i - 1] - 1 + p + i, i);
      v.row_sub[n++] = i;
    }
  }
  for (int c = n; c < C; ++c) { v.row_sub[c] = 0; v.row_meta[c] = make_int4(0, 0, 0, 0); }
  st.n_active[b] = n;
  // Page list of the coming step for the self-attention kernels: every page of subsequences
  // 1..i_max (i_max = last active one; later ones are invisible to every row), with the number
  // of entries it will hold once the step's inputs are appended (bos + content = len + 1 per
  // subsequence), its subsequence i', and the Manhattan distance from a query of "subsequence 0"
  // at that step to its first entry, d0 = t - (tau' + i') (the coming step is t + 1, whose queries sit
  // at position t + i; a kernel adds the query's i and subtracts the key's offset in the page).
  int np = 0;
  if (n > 0) {
    const int i_last = v.row_sub[n - 1];
    for (int i = 1; i <= i_last; ++i) {
      const int entries = v.len[i - 1] + 1;
      const int pos0 = v.start[i - 1] - 1 + i;
      for (int j = 0; j * dm.P < entries; ++j)
        v.plist[np++] = make_int4(v.page_table[(i - 1) * dm.PPS + j], min(dm.P, entries - j * dm.P), i, t - (pos0 + j * dm.P));
    }
  }
  st.plist_n[b] = np;
}

// Called by every thread of a row's CTA once the row's choice is in row_tok: the CTA that arrives
// last for its sequence stages the sequence's state, runs its scheduler and writes the state back;
// the last sequence advances the step.  No CTA ever waits for another.
__device__ void row_done(const Dims &dm, const DecState &st, int batch, int b, const int32_t *teacher, int *is_last) {
  extern __shared__ __align__(16) uint8_t sched_smem[];
  const int tid = threadIdx.x, nthr = blockDim.x;
  if (tid == 0) {
    __threadfence();
    int ticket = atomicAdd(&st.seq_ticket[b], 1);
    *is_last = ticket == dm.C - 1;
  }
  __syncthreads();
  if (!*is_last) return;
  __threadfence();
  const int C = dm.C, SM = dm.SM, NPT = dm.SM * dm.PPS;
  SeqStage v;
  int32_t *w = reinterpret_cast<int32_t *>(sched_smem);
  v.row_sub = w; w += C;
  v.row_tok = w; w += C;
  v.len = w; w += SM; v.forced_len = w; w += SM; v.state = w; w += SM; v.flag = w; w += SM;
  v.start = w; w += SM; v.last_tok = w; w += SM; v.teacher = w; w += SM;
  v.page_table = w; w += NPT;
  w = reinterpret_cast<int32_t *>(sched_smem) + (size_t)(2 * C + 7 * SM + NPT + 3) / 4 * 4;     // 16-byte aligned
  v.row_meta = reinterpret_cast<int4 *>(w);
  v.plist = v.row_meta + C;
  for (int c = tid; c < C; c += nthr) {
    v.row_sub[c] = st.row_sub[b * C + c];
    v.row_tok[c] = __ldcg(&st.row_tok[b * C + c]);            // written by other CTAs of this launch
    st.prev_row_sub[b * C + c] = v.row_sub[c];
  }
  for (int i = tid; i < SM; i += nthr) {
    const int sidx = b * SM + i;
    v.len[i] = st.len[sidx]; v.forced_len[i] = st.forced_len[sidx]; v.state[i] = st.state[sidx]; v.flag[i] = st.flag[sidx];
    v.start[i] = st.start[sidx]; v.last_tok[i] = st.last_tok[sidx];
    v.teacher[i] = teacher != nullptr ? teacher[sidx] : -1;
  }
  for (int i = tid; i < NPT; i += nthr) v.page_table[i] = st.page_table[(size_t)b * NPT + i];
  __syncthreads();
  if (tid == 0) {
    st.seq_ticket[b] = 0;
    schedule_sequence(dm, st, v, b, teacher != nullptr);
  }
  __syncthreads();
  for (int c = tid; c < C; c += nthr) { st.row_sub[b * C + c] = v.row_sub[c]; st.row_meta[b * C + c] = v.row_meta[c]; }
  for (int i = tid; i < SM; i += nthr) {
    const int sidx = b * SM + i;
    st.len[sidx] = v.len[i]; st.state[sidx] = v.state[i]; st.flag[sidx] = v.flag[i]; st.start[sidx] = v.start[i];
    st.last_tok[sidx] = v.last_tok[i];
  }
  for (int i = tid; i < NPT; i += nthr) st.page_table[(size_t)b * NPT + i] = v.page_table[i];
  const int np = st.plist_n[b];                        // written by thread 0 before the barrier above
  for (int i = tid; i < np; i += nthr) st.plist[(size_t)b * NPT + i] = v.plist[i];
  __threadfence();
  __syncthreads();
  if (tid != 0) return;
  if (atomicAdd(&st.hdr[HDR_TICKET], 1) == batch - 1) {   // last sequence of the step
    __threadfence();
    st.hdr[HDR_TICKET] = 0;
    const int n_done = atomicAdd(&st.hdr[HDR_N_DONE], 0);
    if (st.hdr[HDR_ALL_DONE] == 0) {
      atomicAdd(&st.stats[PD_STAT_STEPS], 1ull);
      if (n_done >= batch) st.hdr[HDR_ALL_DONE] = 1;
      else st.hdr[HDR_STEP_T] = st.hdr[HDR_STEP_T] + 1;
    }
  }
}

__global__ void __launch_bounds__(AT) argmax_sched_kernel(Dims dm, DecState st, int batch, const float *__restrict__ logits,
                                                          const int32_t *__restrict__ teacher) {
  __shared__ float sv[AT / 32];
  __shared__ int si[AT / 32];
  __shared__ int is_last;
  const int r = blockIdx.x, tid = threadIdx.x;
  const int b = r / dm.C;
  const int i = st.row_sub[r];
  if (i > 0) {
    const int sidx = b * dm.SM + i - 1;
    const int fl = st.forced_len[sidx];
    const bool bar = fl >= 0 && st.len[sidx] < fl;     // terminators cannot win before the forced length
    const float *row = logits + (size_t)r * dm.V;
    float bv = -INFINITY;
    int bi = INT_MAX;
    // 16-byte streaming loads over the aligned body of the row, scalar loads for its ragged ends
    const int head = min(dm.V, (int)((4u - (unsigned)(((size_t)r * dm.V) & 3u)) & 3u));
    const int nvec = (dm.V - head) / 4;
    auto take = [&](float x, int v) {
      if (bar && (v == dm.eos || v == dm.sep)) return;
      better(bv, bi, x, v);
    };
    if (tid < head) take(__ldcs(row + tid), tid);
    const float4 *body = reinterpret_cast<const float4 *>(row + head);
    constexpr int UN = 4;   // loads in flight per thread
    int q = tid;
    for (; q + (UN - 1) * AT < nvec; q += UN * AT) {
      float4 x[UN];
#pragma unroll
      for (int u = 0; u < UN; ++u) x[u] = __ldcs(body + q + u * AT);
#pragma unroll
      for (int u = 0; u < UN; ++u) {
        const int v = head + 4 * (q + u * AT);
        take(x[u].x, v); take(x[u].y, v + 1); take(x[u].z, v + 2); take(x[u].w, v + 3);
      }
    }
    for (; q < nvec; q += AT) {
      const float4 x = __ldcs(body + q);
      const int v = head + 4 * q;
      take(x.x, v); take(x.y, v + 1); take(x.z, v + 2); take(x.w, v + 3);
    }
    for (int v = head + 4 * nvec + tid; v < dm.V; v += AT) take(__ldcs(row + v), v);
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      better(bv, bi, ov, oi);
    }
    if ((tid & 31) == 0) { sv[tid >> 5] = bv; si[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < AT / 32; ++w) better(bv, bi, sv[w], si[w]);
      st.row_tok[r] = bi == INT_MAX ? 0 : bi;
    }
  }
  row_done(dm, st, batch, b, teacher, &is_last);
}

cudaError_t launch_argmax_sched(const Dims &dm, const DecState &st, int batch, const float *logits,
                                const int32_t *teacher, cudaStream_t s) {
  argmax_sched_kernel<<<batch * dm.C, AT, seq_stage_bytes(dm), s>>>(dm, st, batch, logits, teacher);
  return cudaGetLastError();
}

// The same step when the vocabulary projection has already reduced every row to one candidate per
// vocabulary slice (vocab_tc.cu): one warp-sized CTA per row finishes the greedy choice over the
// slices' maxima - ties to the lowest id; eos and sep, kept apart by the projection, join unless the
// forced length bars them - and hands over to the scheduler exactly as above.
constexpr int PT = 64;

__global__ void __launch_bounds__(PT) pick_sched_kernel(Dims dm, DecState st, int batch, int tiles, int rows_cap,
                                                        const float *__restrict__ part_val, const int32_t *__restrict__ part_idx,
                                                        const float *__restrict__ term_val, const int32_t *__restrict__ teacher) {
  __shared__ float sv[PT / 32];
  __shared__ int si[PT / 32];
  __shared__ int is_last;
  const int r = blockIdx.x, tid = threadIdx.x;
  const int b = r / dm.C;
  const int i = st.row_sub[r];
  if (i > 0) {
    const int sidx = b * dm.SM + i - 1;
    const int fl = st.forced_len[sidx];
    const bool bar = fl >= 0 && st.len[sidx] < fl;     // terminators cannot win before the forced length
    const int m = st.crow[b] + r % dm.C;               // the row's place among the packed rows
    float bv = -INFINITY;
    int bi = INT_MAX;
    for (int t = tid; t < tiles; t += PT) better(bv, bi, __ldcg(part_val + (size_t)t * rows_cap + m), __ldcg(part_idx + (size_t)t * rows_cap + m));
    if (tid == 0 && !bar) {
      better(bv, bi, __ldcg(term_val + 2 * m), dm.eos);
      if (dm.sep != dm.eos) better(bv, bi, __ldcg(term_val + 2 * m + 1), dm.sep);
    }
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      better(bv, bi, ov, oi);
    }
    if ((tid & 31) == 0) { sv[tid >> 5] = bv; si[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < PT / 32; ++w) better(bv, bi, sv[w], si[w]);
      st.row_tok[r] = bi == INT_MAX ? 0 : bi;
    }
  }
  row_done(dm, st, batch, b, teacher, &is_last);
}

cudaError_t launch_pick_sched(const Dims &dm, const DecState &st, int batch, int tiles, const float *part_val,
                              const int32_t *part_idx, const float *term_val, const int32_t *teacher, cudaStream_t s) {
  pick_sched_kernel<<<batch * dm.C, PT, seq_stage_bytes(dm), s>>>(dm, st, batch, tiles, batch * dm.C, part_val, part_idx, term_val, teacher);
  return cudaGetLastError();
}

}  // namespace pd
