/* pd.h - C ABI of the pipelined-decoder decode path for NVIDIA B200 (sm_100a).
 *
 * The library runs the per-time-step decode of the pipelined decoder: up to sub_max
 * subsequences of one target, each started delta_t steps after the previous one, each
 * emitting one token per step while attending to the encoder memory H^E and to the earlier
 * subsequences as generated so far (Section 3.2, Eq. 2-4; Algorithm 1 in Section 3.4).
 * Encoder memory goes in, per-subsequence token streams come out.
 *
 * Conventions
 *  - Every function returns a pd_status (0 = PD_OK, negative = error) unless stated.  Nothing
 *    throws, aborts or exits.  pd_last_error() gives a text for the last failure on a handle.
 *  - "device" pointers are CUDA device memory on cfg.device; "host" pointers are ordinary
 *    host memory.  The caller owns every buffer it passes, including the workspace and the
 *    weights, and must keep them alive and unmodified until pd_destroy().  The library owns
 *    only the host-side handle.  pd_init..pd_step allocate no device memory of their own
 *    (cuBLAS is given a slice of the workspace).
 *  - All work is enqueued on the CUDA stream given to pd_init.  pd_step and pd_encode_context
 *    do not synchronise; pd_done, pd_collect and the pd_get_* readers do.
 *  - Errors found on the device (page pool exhausted, a bounded wait that expired) are written
 *    to a status word in the workspace, turn the remaining steps into no-ops and are returned
 *    by the next synchronising call.
 *  - Time-steps t and subsequence indices i are 1-based as in the paper.  Subsequence i is
 *    admitted at step s_i = (i-1)*delta_t + 1.  Its cache entry p (p = 0 is <bos>, p >= 1 the
 *    p-th content token) carries the timestamp tau = s_i - 1 + p (Eq. 2: token j of
 *    subsequence i is generated at step (i-1)*delta_t + j) and the position tau + i.
 */
#ifndef PD_H_
#define PD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define PD_API __attribute__((visibility("default")))
#else
#define PD_API
#endif

typedef struct pd_handle pd_handle; /* opaque; host memory owned by the library */

typedef enum {
  PD_OK = 0,
  PD_ERR_ARG = -1,            /* null pointer, size out of range, unsupported shape        */
  PD_ERR_STATE = -2,          /* call out of order (e.g. pd_step before pd_encode_context) */
  PD_ERR_WORKSPACE = -3,      /* workspace too small or misaligned                         */
  PD_ERR_POOL_EXHAUSTED = -4, /* the KV page pool ran out (set on the device)              */
  PD_ERR_CUDA = -5,           /* a CUDA or cuBLAS call failed                              */
  PD_ERR_TIMEOUT = -6,        /* a bounded device-side wait expired (set on the device)    */
  PD_ERR_UNSUPPORTED = -7     /* valid request the build does not implement                */
} pd_status;

enum { PD_DTYPE_FP32 = 0, PD_DTYPE_BF16 = 1 };
enum { PD_POS_T5_BIAS = 0, PD_POS_ROPE = 1 };
enum { PD_KV_SAME = 0, PD_KV_E4M3 = 1 };
/* per-subsequence flags returned by pd_collect */
enum { PD_FLAG_COMPLETE = 1, PD_FLAG_TRUNCATED = 2, PD_FLAG_CAPPED = 4 };
/* intermediate buffers readable with pd_debug_read (values of the last layer of the last step) */
enum {
  PD_BUF_X = 0,        /* residual stream after the last layer, fp32 [rows, d_model]          */
  PD_BUF_QKV = 1,      /* self-attention projection [rows, 3*d_model]: fp32, except bf16 on the
                          bf16 path without rotary positions (the projection rounds itself)   */
  PD_BUF_SELF_OUT = 2, /* self-attention output, dtype [rows, d_model]                        */
  PD_BUF_CROSS_Q = 3,  /* cross-attention queries, dtype [rows, d_model]                      */
  PD_BUF_CROSS_OUT = 4,/* cross-attention output, dtype [rows, d_model]                       */
  PD_BUF_STATE = 5     /* the integer decode state block, int32                               */
};

typedef struct {
  int32_t n_layers, d_model, n_heads, d_head, d_ff, vocab; /* d_head must be 64, n_heads*d_head == d_model */
  int32_t dtype;          /* PD_DTYPE_FP32 or PD_DTYPE_BF16: storage type of weights, H^E, K/V, GEMM inputs */
  int32_t max_batch, max_ctx;
  int32_t sub_max, delta_t, time_max; /* the three parameters of Algorithm 1; sub_max <= 64     */
  int32_t max_sub_len;    /* cap on content tokens per subsequence; a subsequence that reaches
                             it ends with sep_id at its next emission (flag PD_FLAG_CAPPED)      */
  int32_t bos_id, eos_id, sep_id; /* eos_id and sep_id both end a subsequence                   */
  int32_t pos_mode;       /* PD_POS_T5_BIAS: bucketed bias on the Manhattan distance of
                             Section 4.3; PD_POS_ROPE: rotary embedding at position tau + i      */
  int32_t rel_buckets, rel_max_dist; /* T5 causal bucketing (32, 128 in T5)                     */
  float rope_theta, attn_scale, norm_eps;
  int32_t page_tokens;    /* KV page size in tokens: 16 or 32                                   */
  int32_t pool_pages;     /* KV pool size in pages; 0 = worst case (never exhausts)             */
  int32_t self_splits, cross_splits; /* split-K factors of the attention kernels; 0 = auto.  The
                             bf16 tensor-core cross-attention kernel ignores cross_splits: it
                             divides the context tiles over the GPU by itself                      */
  int32_t use_graph;      /* 1: pd_step replays a CUDA graph captured at the first step         */
  int32_t store_logits;   /* 1: every step leaves its fp32 logits behind for pd_get_logits.  0: on the
                             bf16 path the vocabulary projection keeps the logits on chip (only the
                             greedy choice of Eq. 4 leaves the kernel) and pd_get_logits returns
                             PD_ERR_STATE; the fp32 path stores them either way                    */
  int32_t kv_c_dtype;     /* storage of the cross-attention keys/values (the projected encoder memory, the
                             dominant byte term of a step).  PD_KV_SAME: cfg.dtype.  PD_KV_E4M3 (bf16 path,
                             at most 32 rows per sequence, max_ctx a multiple of 16): 8-bit floats (1-4-3,
                             largest value 448) with one fp32 scale per (layer, sequence, head, keys | values)
                             = max|.| / 448 over the sequence's context; attention runs over the de-quantised
                             values - half the bytes per step, logits within the same tolerance of an oracle
                             that quantises likewise                                                  */
  int32_t device;         /* CUDA device ordinal                                                */
} pd_config;

/* Device pointers to the parameters, all of cfg.dtype except rel_bias (fp32).  Linear weights
 * are row-major [in, out] (y = x W).  Per layer, in this order: norm1 [d], wqkv [d, 3d]
 * (columns q | k | v, head-major), wo [d, d], norm2 [d], wq_c [d, d], wkv_c [d, 2d] (columns
 * k | v), wo_c [d, d], norm3 [d], w1 [d, d_ff], w2 [d_ff, d].  The decoder layer is pre-RMSNorm,
 * bias-free, ReLU feed-forward, untied output head. */
typedef struct {
  const void *embed;        /* [vocab, d]                                   */
  const void *const *layer; /* host array of n_layers*10 device pointers    */
  const void *final_norm;   /* [d]                                          */
  const void *lm_head;      /* [vocab, d]                                   */
  const float *rel_bias;    /* [n_heads, rel_buckets], shared by all layers; may be NULL in RoPE mode */
} pd_weights;

/* PD_OK if pd_init would accept cfg; PD_ERR_ARG for a field out of range; PD_ERR_UNSUPPORTED for a valid request
 * beyond a limit of this build: T5-bias mode needs time_max + sub_max + 2 <= 512 (one bias value per distance is
 * kept in shared memory); 8-bit context keys/values need the bf16 path, max_ctx a multiple of 16 and at most 32
 * rows per sequence.  *reason (may be NULL) receives a static text.  Not a limit but a slower path: with more than
 * 32 rows per sequence (pd_rows_per_seq) the bf16 attention steps run on the plain-ALU kernels instead of the
 * tensor-core ones.  Pure function; no CUDA call. */
PD_API pd_status pd_config_check(const pd_config *cfg, const char **reason);

/* Bytes of device workspace pd_init needs for this configuration (0 if pd_config_check(cfg) fails).
 * Pure function; no CUDA call. */
PD_API size_t pd_workspace_bytes(const pd_config *cfg);

/* Creates a handle: validates cfg, carves the workspace (device, 256-byte aligned, at least
 * pd_workspace_bytes(cfg)), creates the cuBLAS handles and the TMA descriptor of the context
 * keys/values, builds the position tables.  Returns what pd_config_check returns for a configuration it
 * does not take.  `cuda_stream` is a cudaStream_t (NULL = legacy default stream).  Algorithm 1's inputs delta_t, time_max,
 * sub_max are fixed here. */
PD_API pd_status pd_init(const pd_config *cfg, const pd_weights *weights, void *workspace, size_t workspace_bytes,
                  void *cuda_stream, pd_handle **out);

/* The initialisation of Algorithm 1 with H^E supplied: resets all decode state, projects the encoder
 * memory to per-layer cross-attention keys/values, admits subsequence 1 of every sequence.
 * enc_mem: device [batch, max_ctx, d_model] of cfg.dtype (rows at or beyond ctx_len[b] are
 * ignored).  ctx_len: host [batch], 1..max_ctx.  forced_len: host [batch, sub_max] or NULL;
 * forced_len[b][i-1] = m >= 0 makes subsequence i hold exactly m content tokens (terminators
 * are barred from the argmax before that and sep_id is emitted at emission m+1); NULL or a
 * negative entry = free-running greedy decoding. */
PD_API pd_status pd_encode_context(pd_handle *h, const void *enc_mem, const int32_t *ctx_len, int32_t batch,
                            const int32_t *forced_len);

/* One iteration of Algorithm 1's loop for every sequence of the batch: one
 * decoder pass (Eq. 3) for all active subsequences, greedy choice (Eq. 4), append, retire on
 * eos/sep, stop test, and the admission the loop would do at the top of the next step.
 * teacher_tokens: device [batch, sub_max] int32 or NULL; an entry >= 0 replaces the chosen
 * token of that subsequence as the one appended (the library's own choice is still recorded);
 * -1 keeps the own choice.  Enqueues only; a no-op for sequences that are done. */
PD_API pd_status pd_step(pd_handle *h, const int32_t *teacher_tokens);

/* Runs pd_step(NULL) until every sequence is done or time_max is reached.  The host follows the
 * device min(poll_every, 2) steps behind (poll_every >= 1) through header snapshots copied on a
 * stream of the handle's own, so the decode stream is never drained to look; at most that many
 * steps are enqueued past the end (they are no-ops).  Returns the number of steps enqueued in
 * *steps_run.  Synchronises at the end. */
PD_API pd_status pd_run(pd_handle *h, int32_t poll_every, int32_t *steps_run);

/* Synchronises the stream; *all_done = 1 when every sequence has ended or hit time_max. */
PD_API pd_status pd_done(pd_handle *h, int32_t *all_done);

/* The result of Algorithm 1: the subsequences without bos and terminator.  Host outputs (any may be
 * NULL): tokens [batch, sub_max, max_sub_len] (unused tail = -1), lens [batch, sub_max],
 * n_sub [batch] (k at the end), flags [batch, sub_max] (PD_FLAG_*), steps [batch] (the step
 * at which the sequence stopped).  Synchronises; returns a pending device error if any. */
PD_API pd_status pd_collect(pd_handle *h, int32_t *tokens, int32_t *lens, int32_t *n_sub, int32_t *flags,
                     int32_t *steps);

/* Start steps that are not at fixed intervals (Section 6 names "new subsequences adaptively rather than at fixed time
 * intervals" as future work; the policy is the caller's, the library takes its outcome): plan[b][i-1] = the step of
 * sequence b's own clock at which subsequence i is admitted, instead of Eq. 2's (i-1)*delta_t + 1.  Host
 * [batch, sub_max]; every plan starts at 1 and its start steps are at least cfg.delta_t apart (which keeps the bound on
 * concurrently open subsequences the workspace is sized for), else PD_ERR_ARG.  Entry p of a subsequence started at s
 * carries the timestamp s - 1 + p; the dependency rule, the Manhattan distance and the stop test are unchanged (a
 * sequence whose held subsequences have all ended stops, later planned starts or not).  Call it after
 * pd_encode_context and before the first pd_step (PD_ERR_STATE otherwise); pd_encode_context and pd_admit put the
 * fixed-interval plan back.  pd_teacher_forward uses the plan in force.  Synchronises. */
PD_API pd_status pd_set_start_plan(pd_handle *h, const int32_t *plan);

/* Continuous batching: a new sequence in a row whose sequence has ended, between two steps (Algorithm 1
 * runs per sequence; rows only share the step clock).  The row starts over as pd_encode_context would leave
 * it - state cleared, subsequence 1 admitted, its own step counter at 1 for the coming pd_step, its pages its
 * own again - and the context's keys/values are projected into the row's slice.  The other rows carry on
 * untouched; the result of the row's sequence is what the sequence gives decoded alone.  Take the previous
 * sequence's result first (pd_collect_row).
 *   row        0 .. batch-1 of the last pd_encode_context; its sequence should have ended (pd_rows_done)
 *   enc_mem    device [max_ctx, d_model] of cfg.dtype;  ctx_len 1..max_ctx;  forced_len host [sub_max] or NULL
 * Needs the default page pool (cfg.pool_pages = 0), else PD_ERR_UNSUPPORTED.  Enqueues on the handle's stream;
 * call it between pd_step calls (not while pd_run is running).  pd_run / pd_done report "all done" again only
 * when every row's current sequence has ended. */
PD_API pd_status pd_admit(pd_handle *h, int32_t row, const void *enc_mem, int32_t ctx_len, const int32_t *forced_len);

/* done[b] = 1 when row b's current sequence has ended (host [batch]); steps[b] (host [batch] or NULL) = the step
 * of the sequence's own clock at which it stopped.  Synchronises; returns a pending device error if any. */
PD_API pd_status pd_rows_done(pd_handle *h, int32_t *done, int32_t *steps);

/* pd_collect for one row: tokens host [sub_max, max_sub_len], lens [sub_max], n_sub [1], flags [sub_max],
 * steps [1] (any may be NULL).  Synchronises. */
PD_API pd_status pd_collect_row(pd_handle *h, int32_t row, int32_t *tokens, int32_t *lens, int32_t *n_sub, int32_t *flags,
                                int32_t *steps);

/* The teacher-forced forward of Section 3.3 (Eq. 6): the whole target of every sequence in one pass instead of
 * one time-step at a time.  Subsequence i of sequence b is given as its lens[b][i-1] content tokens; row (b, i, p),
 * p = 0 .. lens, has the input <bos> (p = 0) or content token p, the timestamp (i-1)*delta_t + p, and attends to the
 * rows the dependency rule lets it see (subsequence i' <= i, timestamp tau' <= tau - evaluated per pair, no mask is
 * stored) and to the sequence's context; its target is content token p+1 or, at p = lens, the subsequence's
 * terminator.  Row r's logits are the ones pd_step computes at step s_i + p when it is fed the same tokens.
 * Uses the context keys/values of the last pd_encode_context (any kv_c_dtype); leaves the decode state untouched.
 *   n_sub        host [batch]: subsequences of every sequence (0..sub_max; an empty one, lens = 0, is one row)
 *   lens, tokens host [batch, sub_max], [batch, sub_max, max_sub_len]
 *   terminators  host [batch, sub_max] or NULL (= sep_id everywhere)
 *   scratch      device, 256-byte aligned, at least pd_teacher_forward_scratch_bytes(h, rows, own_logits) for the
 *                sum over all subsequences of lens + 1 rows (own_logits = 1 when `logits` is NULL: the library then
 *                works through the vocabulary projection in chunks of rows inside the scratch)
 *   logprob      host [rows] or NULL: log P(target) per row, rows in (sequence, subsequence, position) order
 *   logits       device fp32 [rows, vocab] or NULL: every row's logits (tests)
 *   rows_out, loss_out  host or NULL: the row count, and Eq. 6's L = - sum of logprob
 * bf16 path with at most 32 rows per sequence in pd_step (the tensor-core cross-attention kernel) only, else
 * PD_ERR_UNSUPPORTED.  Synchronises. */
PD_API size_t pd_teacher_forward_scratch_bytes(const pd_handle *h, int32_t max_rows, int32_t own_logits);
PD_API pd_status pd_teacher_forward(pd_handle *h, const int32_t *n_sub, const int32_t *lens, const int32_t *tokens,
                                    const int32_t *terminators, void *scratch, size_t scratch_bytes, float *logprob,
                                    float *logits, int32_t *rows_out, double *loss_out);

/* Whole Algorithm 1 from host buffers: copies enc_mem (host [batch, max_ctx, d_model], dtype;
 * pinned memory lets the copy overlap) to the device in chunks of sequences on a copy stream of
 * the handle's own while the context projection of the chunks already there runs on the handle's
 * stream, decodes until done, copies the streams back.  Output arguments as in pd_collect.
 * Synchronises. */
PD_API pd_status pd_generate_host(pd_handle *h, const void *enc_mem_host, const int32_t *ctx_len, int32_t batch,
                           const int32_t *forced_len, int32_t *tokens, int32_t *lens, int32_t *n_sub,
                           int32_t *flags, int32_t *steps);

/* Schedule trace: active_mask[(t-1)*batch + b] has bit i-1 set iff subsequence i of sequence b
 * emitted a token at step t of the sequence's own clock (a row's column starts over with pd_admit).
 * Host [time_max, batch].  Synchronises. */
PD_API pd_status pd_get_trace(pd_handle *h, uint64_t *active_mask);

/* Parity/debug: fp32 logits of the last executed step, host [rows, vocab] with
 * rows = batch * pd_rows_per_seq(); row_sub host [rows] = subsequence index (1-based) the row
 * belonged to in that step, 0 = unused row.  Either may be NULL.  Synchronises. */
PD_API pd_status pd_get_logits(pd_handle *h, float *logits, int32_t *row_sub);

/* The library's own greedy choices: chosen[b][i-1][n] = token chosen at emission n (0-based)
 * of subsequence i, -1 where none.  Host [batch, sub_max, max_sub_len + 1].  Synchronises. */
PD_API pd_status pd_get_chosen(pd_handle *h, int32_t *chosen);

/* Rows per sequence in the step's row block: min(sub_max, floor(max_sub_len/delta_t) + 1), the
 * largest number of subsequences that can be active at once. */
PD_API int32_t pd_rows_per_seq(const pd_handle *h);

/* Copies an intermediate buffer (PD_BUF_*) to host; *bytes_out = bytes written (<= max_bytes).
 * Synchronises.  For tests. */
PD_API pd_status pd_debug_read(pd_handle *h, int32_t which, void *dst_host, size_t max_bytes, size_t *bytes_out);

/* Counters since pd_init (or the last pd_reset_counters): kernels of this library launched
 * (graph replays count their kernel nodes) and cuBLAS GEMM calls issued. */
PD_API pd_status pd_get_counters(const pd_handle *h, int64_t *own_kernel_launches, int64_t *gemm_calls);
PD_API pd_status pd_reset_counters(pd_handle *h);

/* Per-kernel timing.  pd_profile_enable(h, 1) makes every following pd_step bracket each hot
 * kernel with CUDA events on the stream (steps then run without the CUDA graph);
 * pd_profile_read sums them up (synchronises): for kind k in PD_PROF_*, ms[k] = total device
 * time, launches[k] = launches.  Arrays of PD_PROF_COUNT entries. */
enum { PD_PROF_APPEND = 0, PD_PROF_SELF_ATTN = 1, PD_PROF_CROSS_ATTN = 2, PD_PROF_ARGMAX_SCHED = 3,
       PD_PROF_GEMM = 4, PD_PROF_OTHER = 5, PD_PROF_VOCAB = 6 /* tensor-core vocabulary projection */, PD_PROF_COUNT = 7 };
PD_API pd_status pd_profile_enable(pd_handle *h, int32_t on);
PD_API pd_status pd_profile_read(pd_handle *h, double *ms, int64_t *launches);

/* Times one attention step in isolation on the decoder's current state: enqueues the
 * self-attention (which = PD_PROF_SELF_ATTN) or cross-attention (PD_PROF_CROSS_ATTN) launches of
 * all layers, one layer after the other, `reps` times back to back after one warm-up pass,
 * between two CUDA events, and returns the average device time per layer launch (merge kernel
 * included when the step is split) in microseconds.  Successive layers read different memory, so
 * with per-layer keys/values beyond the L2 size the launches stay HBM-bound.  The decode state is
 * not changed (the attention outputs of the last layer are rewritten with the same values).
 * Synchronises. */
PD_API pd_status pd_time_attention(pd_handle *h, int32_t which, int32_t reps, float *avg_us);

/* Counters accumulated on the device since the last pd_encode_context, host int64 [PD_STAT_COUNT]:
 * tokens emitted (terminators included), steps executed, and the two sums the attention
 * kernels' algorithmic traffic follows from: over all (step, sequence), the number of cache
 * entries of subsequences 1..max active i (each is read once per layer and head as K and V),
 * and ctx_len of every sequence that had an active subsequence (each context key/value is read
 * once per layer).  Synchronises. */
enum { PD_STAT_TOKENS = 0, PD_STAT_STEPS = 1, PD_STAT_SELF_ENTRIES = 2, PD_STAT_CROSS_KEYS = 3,
       PD_STAT_PAGES = 4, PD_STAT_COUNT = 8 };
PD_API pd_status pd_get_stats(pd_handle *h, int64_t *stats);

/* The batched cross-attention step alone (Section 3.2: every generated token attends to all
 * context tokens; Eq. 3's Decoder(G, H^E) reads H^E only through this step), on caller-supplied
 * tensors and without a handle: the kernels are the ones pd_step launches.  For sequence b,
 * rows b*rows_per_seq .. b*rows_per_seq + n_rows[b] - 1 of q are the queries of its active
 * subsequences; each attends, per head, to context positions 0 .. ctx_len[b]-1 with weights
 * softmax(attn_scale * q.k) and no positional term:  out = softmax(attn_scale * q K^T) V.
 *   dtype        PD_DTYPE_FP32 or PD_DTYPE_BF16: element type of q, kv and out
 *   q, out       device [batch*rows_per_seq, n_heads*64], 16-byte aligned; rows at or beyond n_rows[b] of a
 *                sequence are not read and come back as zeros
 *   kv           device [batch, n_heads, 2, max_ctx, 64], 16-byte aligned: per sequence and head
 *                the keys of all context positions, then the values (the layout the decoder keeps
 *                its projected context in); positions at or beyond ctx_len[b] are ignored (they
 *                may hold anything)
 *   n_rows       device int32 [batch], 0..rows_per_seq;  ctx_len  device int32 [batch], 1..max_ctx
 *                (the kernels clamp what they read to these ranges, so a bad value gives a wrong
 *                result for that sequence, never an access outside the tensors)
 *   splits       1..32: split-K factor over the context of the plain-ALU kernel (fp32, or more
 *                than 32 rows per sequence; partials are merged by a second kernel).  The bf16
 *                tensor-core kernel divides the context tiles of all sequences evenly over the
 *                GPU by itself and merges its partials in the same launch.
 *   scratch      device, 256-byte aligned, at least pd_cross_attention_scratch_bytes(...): a
 *                256-byte header (int32 word 2 receives PD_ERR_TIMEOUT if a bounded wait inside
 *                the kernel expired) and per-(sequence, head) arrival counters, both cleared by
 *                the call, then the partial results
 * rows_per_seq <= 64.  Enqueues on cuda_stream (a cudaStream_t) and returns; allocates nothing on
 * the device.  The caller owns every buffer and keeps it alive until the stream has passed the
 * call.  PD_ERR_ARG for null pointers or sizes out of range, PD_ERR_WORKSPACE for a scratch
 * that is too small, PD_ERR_CUDA if a launch fails. */
PD_API size_t pd_cross_attention_scratch_bytes(int32_t batch, int32_t rows_per_seq, int32_t n_heads, int32_t splits);
PD_API pd_status pd_cross_attention(int32_t dtype, int32_t batch, int32_t rows_per_seq, int32_t n_heads, int32_t max_ctx,
                             float attn_scale, int32_t splits, const void *q, const void *kv, const int32_t *n_rows,
                             const int32_t *ctx_len, void *out, void *scratch, size_t scratch_bytes, void *cuda_stream);

/* The vocabulary projection and greedy choice alone (Eq. 4: the token with the highest
 * probability, i.e. the largest logit, ties to the lowest id), on caller-supplied rows and
 * without a handle: logits[r][v] = sum_k hidden[r][k] * lm_head[v][k] in bf16 with fp32
 * accumulation on the tcgen05 tensor cores, the per-row maximum taken inside the same kernel -
 * the [rows, vocab] logits are only written when `logits` is given.
 *   hidden     device bf16 [rows, d_model], 16-byte aligned; d_model a multiple of 64
 *   lm_head    device bf16 [vocab, d_model], 16-byte aligned
 *   best_id    device int32 [rows] out;  best_val  device fp32 [rows] out, or NULL
 *   logits     device fp32 [rows, vocab] out, or NULL
 *   scratch    device, 256-byte aligned, at least pd_vocab_argmax_scratch_bytes(rows, vocab): a
 *              256-byte header (int32 word 2 receives PD_ERR_TIMEOUT if a bounded wait inside the
 *              kernel expired; cleared by the call), then per-slice partial maxima
 * Enqueues on cuda_stream and returns; allocates nothing on the device; the caller owns every
 * buffer.  PD_ERR_ARG for null pointers, misaligned buffers or sizes out of range,
 * PD_ERR_WORKSPACE for a scratch that is too small, PD_ERR_CUDA if a launch fails. */
PD_API size_t pd_vocab_argmax_scratch_bytes(int32_t rows, int32_t vocab);
PD_API pd_status pd_vocab_argmax(int32_t rows, int32_t d_model, int32_t vocab, const void *hidden, const void *lm_head,
                                 int32_t *best_id, float *best_val, float *logits, void *scratch, size_t scratch_bytes,
                                 void *cuda_stream);

/* One linear layer of the decoder stack alone (Section 3.2, Eq. 3: the Decoder is a stacked transformer
 * decoder; every projection in it - Q/K/V, attention output, feed-forward - is  y = x W  on the step's few
 * hundred active rows), on caller-supplied tensors and without a handle: the tcgen05 kernel pd_step uses
 * for the bf16 projections, with the work around the product fused into it.
 *   rows, d_in, d_out   rows >= 1; d_in a multiple of 64; d_out a multiple of 16
 *   a          device bf16 [rows, d_in], 16-byte aligned: the layer's input.  When it is the
 *              un-normalised RMSNorm input times the norm's gain, pass row_sumsq
 *   w          device bf16 [d_in, d_out] row-major (y = x W), 16-byte aligned
 *   row_sumsq  device fp32 [rows] or NULL: sum over d_in of the squared norm inputs of every row; the
 *              product's row m is then scaled by rsqrt(row_sumsq[m] / d_in + eps) (the norm applied after
 *              the product instead of before it)
 *   mode 0     out (device bf16 [rows, d_out]) = a W (scaled);  mode 1: the same through max(., 0)
 *   mode 2     residual form: x (device fp32 [rows, d_out], in and out) += a W;  xg (device bf16
 *              [rows, d_out]) = x * gain_next (device bf16 [d_out]), the next layer's GEMM input;
 *              sumsq_out (device fp32 [*sumsq_parts, rows], or NULL): partial sums over column slices of
 *              the new x squared - their sum over the parts is the next norm's row_sumsq
 *   sumsq_parts host int32 out or NULL: number of parts the kernel writes for this shape on the current
 *              device (pd_linear_sumsq_parts(d_in, d_out) gives it beforehand, to size sumsq_out)
 *   scratch    device, 256-byte aligned, at least pd_linear_scratch_bytes(d_in, d_out): a 256-byte header
 *              (int32 word 2 receives PD_ERR_TIMEOUT if a bounded wait inside the kernel expired; cleared
 *              by the call), then the weight re-laid as [d_out, d_in] (the decoder does this once per
 *              handle, the stand-alone call every time)
 * Enqueues on cuda_stream and returns; allocates nothing on the device; the caller owns every buffer.
 * PD_ERR_ARG for null pointers, misaligned buffers or unsupported sizes, PD_ERR_WORKSPACE for a scratch
 * that is too small, PD_ERR_CUDA if a launch fails. */
PD_API size_t pd_linear_scratch_bytes(int32_t d_in, int32_t d_out);
PD_API int32_t pd_linear_sumsq_parts(int32_t d_in, int32_t d_out);
PD_API pd_status pd_linear(int32_t rows, int32_t d_in, int32_t d_out, int32_t mode, const void *a, const void *w,
                           const float *row_sumsq, float eps, void *out, float *x, const void *gain_next, void *xg,
                           float *sumsq_out, int32_t *sumsq_parts, void *scratch, size_t scratch_bytes, void *cuda_stream);

/* pd_cross_attention without a scratch argument (an addition of this library; the paper has no
 * counterpart).  Some callers have no way to obtain device memory at the moment they need the
 * op: a plug-in that runs inside a host framework which owns the whole device heap and hands
 * out no raw allocations; a serving loop that must not call cudaMalloc/cudaFree because those
 * synchronise the device and stall every stream; a process started with all memory already
 * reserved by another pool.  For them the split-K partials live in a fixed 8 MiB array inside
 * the library image (pd_cross_attention_static_max_bytes()), which every GPU that loads the
 * library carries until the process exits.  The caller still passes q, kv, n_rows, ctx_len and
 * out exactly as for pd_cross_attention; results are the same.
 *  - Sizes whose partials would not fit are refused with PD_ERR_WORKSPACE and a message in
 *    pd_static_last_error(); use fewer splits, fewer sequences or rows per call, or
 *    pd_cross_attention with a buffer of your own.  What is needed depends on the kernel that
 *    runs: the bf16 tensor-core kernel (at most 32 rows per sequence) keeps per-CTA records
 *    (2.9 MiB up to 16 rows, 5.9 MiB up to 32, whatever the batch), the plain-ALU kernel (fp32,
 *    or 33..64 rows) batch*rows*heads*splits*264 bytes; pd_cross_attention_scratch_bytes() is
 *    the larger of the two.
 *  - Calls no cudaMalloc, cudaFree or any other allocating routine.  The first call on a device
 *    looks up the array's device address (cudaGetSymbolAddress, with the current device, which
 *    must be the device of the stream and of the buffers); make that first call before any
 *    stream capture begins.
 *  - All calls on a device share the one array.  The call clears the header it needs at zero
 *    and overwrites the partials it reads, so stale contents of earlier calls never matter, but
 *    two calls that may overlap on the GPU (different streams, no dependency) race on it:
 *    order them on one stream or with events.
 *  - The kernel's status word (PD_ERR_TIMEOUT when a bounded wait inside it expired) lives in
 *    that array too, where the caller cannot read it: pd_cross_attention_static_status() copies
 *    it to *status_out (host) after synchronising cuda_stream; it allocates nothing either.  A
 *    non-zero status means that `out` of the last call on this device is not valid.
 * pd_static_last_error() returns the calling thread's message of the last failed
 * pd_cross_attention_static or pd_cross_attention_static_status (empty after a success). */
PD_API size_t pd_cross_attention_static_max_bytes(void);
PD_API pd_status pd_cross_attention_static(int32_t dtype, int32_t batch, int32_t rows_per_seq, int32_t n_heads,
                                    int32_t max_ctx, float attn_scale, int32_t splits, const void *q, const void *kv,
                                    const int32_t *n_rows, const int32_t *ctx_len, void *out, void *cuda_stream);
PD_API pd_status pd_cross_attention_static_status(void *cuda_stream, int32_t *status_out);
PD_API const char *pd_static_last_error(void);

PD_API const char *pd_last_error(const pd_handle *h);
PD_API const char *pd_version(void);

/* Frees the host-side handle (cuBLAS handle, graph, events).  The workspace stays the caller's. */
PD_API void pd_destroy(pd_handle *h);

#ifdef __cplusplus
}
#endif
#endif /* PD_H_ */
