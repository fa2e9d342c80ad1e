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
  int32_t *len, *forced_len, *state, *flag, *start, *last_tok, *teacher, *plan;   // [SM]
  int32_t *page_table;                                               // [SM * PPS]
  int4 *row_meta;                                                    // [C]
  int4 *plist;                                                       // [SM * PPS]
};
__host__ __device__ inline size_t seq_stage_bytes(const Dims &dm) {
  return ((size_t)(2 * dm.C + 8 * dm.SM + dm.SM * dm.PPS + 3) / 4 * 4) * sizeof(int32_t) + ((size_t)dm.C + (size_t)dm.SM * dm.PPS) * sizeof(int4);
}

// Scalars of the sequence that only its own scheduler changes, read at the top of the kernel.
struct SeqScalars { int t, nact, k, done, status; };

__device__ __forceinline__ SeqStage seq_stage_views(const Dims &dm, uint8_t *smem) {
  const int C = dm.C, SM = dm.SM, NPT = dm.SM * dm.PPS;
  SeqStage v;
  int32_t *w = reinterpret_cast<int32_t *>(smem);
  v.row_sub = w; w += C;
  v.row_tok = w; w += C;
  v.len = w; w += SM; v.forced_len = w; w += SM; v.state = w; w += SM; v.flag = w; w += SM;
  v.start = w; w += SM; v.last_tok = w; w += SM; v.teacher = w; w += SM; v.plan = w; w += SM;
  v.page_table = w; w += NPT;
  w = reinterpret_cast<int32_t *>(smem) + (size_t)(2 * C + 8 * SM + NPT + 3) / 4 * 4;     // 16-byte aligned
  v.row_meta = reinterpret_cast<int4 *>(w);
  v.plist = v.row_meta + C;
  return v;
}

// Every CTA of a sequence copies the sequence's state in at its very top, while its own row's loads
// are in flight (nothing of it changes during the launch except row_tok, which the CTA that ends up
// running the scheduler fetches afterwards): the copy is then off the critical path.
__device__ __forceinline__ SeqScalars stage_in(const Dims &dm, const DecState &st, int b, const int32_t *teacher, const SeqStage &v) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int C = dm.C, SM = dm.SM, NPT = dm.SM * dm.PPS;
  SeqScalars sc;
  sc.t = st.hdr[HDR_STEP_T] - st.t0[b];        // the sequence's own step (Algorithm 1 runs per sequence)
  sc.nact = st.n_active[b]; sc.k = st.k[b]; sc.done = st.done[b]; sc.status = st.hdr[HDR_STATUS];
  for (int c = tid; c < C; c += nthr) v.row_sub[c] = st.row_sub[b * C + c];
  for (int i = tid; i < SM; i += nthr) {
    const int sidx = b * SM + i;
    v.len[i] = st.len[sidx]; v.forced_len[i] = st.forced_len[sidx]; v.state[i] = st.state[sidx]; v.flag[i] = st.flag[sidx];
    v.start[i] = st.start[sidx]; v.last_tok[i] = st.last_tok[sidx];
    v.teacher[i] = teacher != nullptr ? teacher[sidx] : -1;
    v.plan[i] = st.plan[sidx];
  }
  for (int i = tid; i < NPT; i += nthr) v.page_table[i] = st.page_table[(size_t)b * NPT + i];
  return sc;
}

__device__ __forceinline__ int warp_sum(int x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// Algorithm 1 for one sequence and one step, after the step's tokens have been chosen: the append,
// the retirement on eos/sep, the stop test, the admission the loop performs at the top of the next
// step, and the compaction of the active rows for it.  Runs in one warp on the staged state: lanes
// take rows, then subsequences; order-dependent results (row order, page ids, page-list offsets) come
// from ballots and prefix sums, so they equal what a loop over increasing i would give.
__device__ void schedule_sequence(const Dims &dm, const DecState &st, const SeqStage &v, int b, bool have_teacher, const SeqScalars &sc) {
  const unsigned FULL = 0xffffffffu;
  const int lane = threadIdx.x & 31;
  const unsigned lt_mask = (1u << lane) - 1u;
  const int t = sc.t;
  const int C = dm.C, SM = dm.SM, P = dm.P;
  const int nact = sc.nact;
  int k = sc.k;
  if (sc.done || sc.status != 0) {
    if (lane == 0 && !sc.done) { st.done[b] = 1; st.steps[b] = t; atomicAdd(&st.hdr[HDR_N_DONE], 1); }
    for (int c = lane; c < C; c += 32) { v.row_sub[c] = 0; v.row_meta[c] = make_int4(0, 0, 0, 0); }
    if (lane == 0) { st.n_active[b] = 0; st.plist_n[b] = 0; }
    return;
  }
  // traffic counters of the step just executed (before any length changes)
  int i_max = 0;
  for (int c = lane; c < nact; c += 32) i_max = max(i_max, v.row_sub[c]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) i_max = max(i_max, __shfl_xor_sync(FULL, i_max, o));
  int nvis = 0;
  for (int i = lane + 1; i <= i_max; i += 32) nvis += v.len[i - 1] + 1;
  nvis = warp_sum(nvis);
  if (lane == 0) {
    atomicAdd(&st.stats[PD_STAT_SELF_ENTRIES], (unsigned long long)nvis);
    if (nact > 0) atomicAdd(&st.stats[PD_STAT_CROSS_KEYS], (unsigned long long)st.ctx_len[b]);
    atomicAdd(&st.stats[PD_STAT_TOKENS], (unsigned long long)nact);
  }
  __syncwarp();

  // ---- the step's tokens: one row per lane (every row belongs to a different subsequence)
  unsigned mask_lo = 0u, mask_hi = 0u;
  for (int c = lane; c < nact; c += 32) {
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
    if (i <= 32) mask_lo |= 1u << (i - 1); else mask_hi |= 1u << (i - 33);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { mask_lo |= __shfl_xor_sync(FULL, mask_lo, o); mask_hi |= __shfl_xor_sync(FULL, mask_hi, o); }
  if (lane == 0) st.trace[(size_t)(t - 1) * dm.B + b] = ((unsigned long long)mask_hi << 32) | mask_lo;
  __syncwarp();

  // ---- stop test, time limit, admission
  int ended = 0;
  for (int i = lane + 1; i <= k; i += 32) ended += v.state[i - 1] == SUB_ENDED;
  ended = warp_sum(ended);
  bool done = false;
  if (ended == k) {
    done = true;                                   // every subsequence has produced its terminator
  } else if (t >= dm.T) {
    done = true;                                   // time_max reached with subsequences still open
    for (int i = lane + 1; i <= k; i += 32)
      if (v.state[i - 1] == SUB_ACTIVE) v.flag[i - 1] |= PD_FLAG_TRUNCATED;
  } else if (k < SM && v.plan[k] == t + 1) {       // the next subsequence starts at step t + 1 (Eq. 2: (t+1-1) mod delta_t == 0 unless a plan was set)
    if (lane == 0) {
      st.k[b] = k + 1;
      v.start[k] = t + 1;
      v.len[k] = 0;
      v.state[k] = SUB_ACTIVE;
      v.flag[k] = 0;
      v.last_tok[k] = dm.bos;
    }
    k += 1;
  }
  __syncwarp();

  // ---- rows of the coming step: the active subsequences in increasing i
  int n = 0;
  if (done) {
    if (lane == 0) { st.done[b] = 1; st.steps[b] = t; atomicAdd(&st.hdr[HDR_N_DONE], 1); }
  } else {
    int pages = 0;
    for (int i0 = 0; i0 < k; i0 += 32) {
      const int i = i0 + lane + 1;
      const bool on = i <= k && v.state[i - 1] == SUB_ACTIVE;
      const unsigned bal = __ballot_sync(FULL, on);
      const int my_n = n + __popc(bal & lt_mask);
      const int p = on ? v.len[i - 1] : 0;                       // entry the next step will write
      const bool need = on && my_n < C && p % P == 0;            // it opens a new page
      const unsigned nb = __ballot_sync(FULL, need);
      int pg0 = 0;
      if (nb != 0u) {
        if (!dm.pool_static) {
          if (lane == 0) pg0 = atomicAdd(&st.hdr[HDR_PAGE_BUMP], __popc(nb));
          pg0 = __shfl_sync(FULL, pg0, 0);
        }
        pages += __popc(nb);
      }
      if (on) {
        if (my_n >= C) {
          atomicExch(&st.hdr[HDR_STATUS], (int)PD_ERR_STATE);
        } else {
          if (need) {
            int pg = dm.pool_static ? (b * SM + i - 1) * dm.PPS + p / P : pg0 + __popc(nb & lt_mask);
            if (pg >= dm.pool) { atomicExch(&st.hdr[HDR_STATUS], (int)PD_ERR_POOL_EXHAUSTED); pg = 0; }
            v.page_table[(i - 1) * dm.PPS + p / P] = pg;
          }
          // where the append kernels of the coming step put this row's key/value, and its position tau + i
          v.row_meta[my_n] = make_int4(v.page_table[(i - 1) * dm.PPS + p / P], p % P, v.start[i - 1] - 1 + p + i, i);
          v.row_sub[my_n] = i;
        }
      }
      n += __popc(bal);
    }
    if (n > C) n = C;
    if (lane == 0 && pages > 0) atomicAdd(&st.stats[PD_STAT_PAGES], (unsigned long long)pages);
  }
  for (int c = n + lane; c < C; c += 32) { v.row_sub[c] = 0; v.row_meta[c] = make_int4(0, 0, 0, 0); }
  if (lane == 0) st.n_active[b] = n;
  __syncwarp();
  // Page list of the coming step for the self-attention kernels: every page of subsequences
  // 1..i_max (i_max = last active one; later ones are invisible to every row), with the number
  // of entries it will hold once the step's inputs are appended (bos + content = len + 1 per
  // subsequence), its subsequence i', and the Manhattan distance from a query of "subsequence 0"
  // at that step to its first entry, d0 = t - (tau' + i') (the coming step is t + 1, whose queries sit
  // at position t + i; a kernel adds the query's i and subtracts the key's offset in the page).
  int np = 0;
  if (n > 0) {
    const int i_last = v.row_sub[n - 1];
    for (int i0 = 0; i0 < i_last; i0 += 32) {
      const int i = i0 + lane + 1;
      const bool on = i <= i_last;
      const int entries = on ? v.len[i - 1] + 1 : 0;
      const int cnt = (entries + P - 1) / P;
      int incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(FULL, incl, o); if (lane >= o) incl += u; }
      if (on) {
        const int off = np + incl - cnt;
        const int pos0 = v.start[i - 1] - 1 + i;
        for (int j = 0; j < cnt; ++j)
          v.plist[off + j] = make_int4(v.page_table[(i - 1) * dm.PPS + j], min(P, entries - j * P), i, t - (pos0 + j * P));
      }
      np += __shfl_sync(FULL, incl, 31);
    }
  }
  if (lane == 0) st.plist_n[b] = np;
}

// Called by every thread of a row's CTA once the row's choice is in row_tok: the CTA that arrives
// last for its sequence fetches the rows' choices, runs the sequence's scheduler in its first warp
// and writes the state back; the last sequence advances the step.  No CTA ever waits for another.
__device__ void row_done(const Dims &dm, const DecState &st, int batch, int b, const int32_t *teacher, int *is_last,
                         const SeqStage &v, const SeqScalars &sc) {
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
  for (int c = tid; c < C; c += nthr) {
    v.row_tok[c] = __ldcg(&st.row_tok[b * C + c]);            // written by other CTAs of this launch
    st.prev_row_sub[b * C + c] = v.row_sub[c];
  }
  __syncthreads();
  if (tid < 32) {
    if (tid == 0) st.seq_ticket[b] = 0;
    schedule_sequence(dm, st, v, b, teacher != nullptr, sc);
  }
  __syncthreads();
  for (int c = tid; c < C; c += nthr) { st.row_sub[b * C + c] = v.row_sub[c]; st.row_meta[b * C + c] = v.row_meta[c]; }
  for (int i = tid; i < SM; i += nthr) {
    const int sidx = b * SM + i;
    st.len[sidx] = v.len[i]; st.state[sidx] = v.state[i]; st.flag[sidx] = v.flag[i]; st.start[sidx] = v.start[i];
    st.last_tok[sidx] = v.last_tok[i];
  }
  for (int i = tid; i < NPT; i += nthr) st.page_table[(size_t)b * NPT + i] = v.page_table[i];
  const int np = st.plist_n[b];                        // written by lane 0 before the barrier above
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
  extern __shared__ __align__(16) uint8_t sched_smem[];
  __shared__ float sv[AT / 32];
  __shared__ int si[AT / 32];
  __shared__ int is_last;
  const int r = blockIdx.x, tid = threadIdx.x;
  const int b = r / dm.C;
  const SeqStage stage = seq_stage_views(dm, sched_smem);
  const SeqScalars sc = stage_in(dm, st, b, teacher, stage);
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
  row_done(dm, st, batch, b, teacher, &is_last, stage, sc);
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
  extern __shared__ __align__(16) uint8_t sched_smem[];
  __shared__ float sv[PT / 32];
  __shared__ int si[PT / 32];
  __shared__ int is_last;
  const int r = blockIdx.x, tid = threadIdx.x;
  const int b = r / dm.C;
  // first round of loads: the row's subsequence, the sequence's place among the packed rows, and the
  // sequence's state for the scheduler
  const int i = st.row_sub[r];
  const int m = st.crow[b] + r % dm.C;                 // the row's place among the packed rows (meaningful when i > 0)
  const SeqStage stage = seq_stage_views(dm, sched_smem);
  const SeqScalars sc = stage_in(dm, st, b, teacher, stage);
  if (i > 0) {
    const int sidx = b * dm.SM + i - 1;
    // second round: the forced-length rule's inputs and the row's candidates
    const int fl = st.forced_len[sidx], len = st.len[sidx];
    float bv = -INFINITY;
    int bi = INT_MAX;
    for (int t = tid; t < tiles; t += PT) better(bv, bi, __ldcg(part_val + (size_t)t * rows_cap + m), __ldcg(part_idx + (size_t)t * rows_cap + m));
    const bool bar = fl >= 0 && len < fl;              // terminators cannot win before the forced length
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
  row_done(dm, st, batch, b, teacher, &is_last, stage, sc);
}

cudaError_t launch_pick_sched(const Dims &dm, const DecState &st, int batch, int tiles, const float *part_val,
                              const int32_t *part_idx, const float *term_val, const int32_t *teacher, cudaStream_t s) {
  pick_sched_kernel<<<batch * dm.C, PT, seq_stage_bytes(dm), s>>>(dm, st, batch, tiles, batch * dm.C, part_val, part_idx, term_val, teacher);
  return cudaGetLastError();
}

}  // namespace pd
