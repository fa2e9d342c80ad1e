"""CPU fp64 oracle of the pipelined decoder.  TEST INFRASTRUCTURE, NOT A PRODUCT PATH.

Only the test-suite, the smoke check and the benchmark's cpu-baseline leg may import
this file.  It shares no code with the CUDA library and imports nothing from it.  It is
written to be checked against the paper by eye: plain numpy in float64, Python loops
wherever a loop is what the paper states, a library matmul as the only primitive, no
blocking, no paging, no fusion.

What follows the paper and what is a reading of it:

* `decode`             - the decoding procedure of Section 3.4 driven by Eq. 2's closed form: at
                         step t the sequence holds k(t) = min(sub_max, ceil(t / delta_t))
                         subsequences (subsequence i starts at s_i = (i-1) delta_t + 1), every
                         subsequence that has not ended gets one token from one decoder call,
                         a terminator ends it, and the procedure stops after the first step at
                         which every subsequence it holds has ended (or at time_max).
* `visible`            - the dependency rule of Section 3.2 (the set G^{<=t}_{<=i} under
                         Eq. 3): a query of subsequence i whose input token was generated
                         at step tau_q sees token (i', tau') iff i' <= i and tau' <= tau_q.
* `timestamp`          - Eq. 2's prose: token j of subsequence i is generated at step
                         (i-1)*delta_t + j; bos counts as j = 0 (a reading).
* `manhattan`          - Section 4.3: distance |t1-t2| + |i1-i2| between two tokens.
* `relative_bucket`    - the published T5 causal bucketing of a distance (a reading: the
                         paper only says "the attention layer of T5").
* `PipelinedDecoderOracle.step_dense`       - formulation A: every step recomputes every
                         token of G from scratch under the dense mask (the teacher-forced
                         form of Eq. 6).
* `PipelinedDecoderOracle.step_incremental` - formulation B: keeps a plain growing list of
                         keys and values per layer and applies the same predicate.
* Layer internals (pre-RMSNorm, bias-free projections, ReLU FFN, untied output head) are a
  property of the backbone, not stated in the paper: PARITY UNPINNED BY THE PAPER for those;
  they are pinned only against a separately written textbook causal decoder (sub_max = 1).
* The terminator of an ended subsequence is output only; it is never fed back and never
  becomes a key (a reading).  eos and sep both end a subsequence.
* `PipelinedDecoderOracle.teacher_forward`  - Section 3.3, Eq. 6: one pass over the whole target
                         (every subsequence as [bos, Y_i], inputs given) under the dense dependency
                         mask; returns the logits of every position and the loss
                         L = - sum_(i,t) log P(target_i^(t+1) | targets seen under the rule; H^E).
* start plans          - an option of this build for Section 6's "new subsequences adaptively rather
                         than at fixed time intervals": `decode`, `run` and `teacher_forward` take the
                         start step of every subsequence (increasing, the first one 1) instead of
                         deriving it from delta_t; entry p of a subsequence started at s carries the
                         timestamp s - 1 + p, which is Eq. 2's (i-1) delta_t + p for the fixed plan
                         s_i = (i-1) delta_t + 1.  Everything else (rule, distance, stop test) is unchanged.
* `e4m3_round`, `quantize_context_kv` - an option of this build, not of the paper (hp["kv_c_dtype"] =
  "e4m3"): the cross-attention keys/values of Eq. 1's encoder memory are stored as 8-bit floats
  (OCP FP8 E4M3: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest
  finite value 448) with one scale per (layer, head, keys | values) of a sequence, and attention
  runs over the de-quantised values.  The rounding decisions are taken in the precision the CUDA
  path takes them in (bf16 projections, float32 scale arithmetic); everything after that is
  float64 as elsewhere.
"""
from __future__ import annotations

import math
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np

POS_T5_BIAS = 0
POS_ROPE = 1

FLAG_OPEN = 0         # admitted, still generating
FLAG_COMPLETE = 1     # ended with a terminator
FLAG_TRUNCATED = 2    # still open when time_max was reached
FLAG_CAPPED = 4      # terminator imposed because max_sub_len content tokens were reached


# --------------------------------------------------------------------------- schedule
def timestamp(i: int, p: int, delta_t: int) -> int:
    """Step at which entry p of subsequence i was generated (p = 0 is bos).  Eq. 2 prose."""
    return (i - 1) * delta_t + p


def fixed_plan(delta_t: int, sub_max: int) -> List[int]:
    """Eq. 2's start steps: s_i = (i-1) delta_t + 1."""
    return [(i - 1) * delta_t + 1 for i in range(1, sub_max + 1)]


def visible(i_q: int, tau_q: int, i_k: int, tau_k: int) -> bool:
    """Dependency rule of Section 3.2: first i subsequences, as generated until tau_q."""
    return i_k <= i_q and tau_k <= tau_q


def manhattan(tau_q: int, i_q: int, tau_k: int, i_k: int) -> int:
    """Relative distance of Section 4.3."""
    return abs(tau_q - tau_k) + abs(i_q - i_k)


def relative_bucket(dist: int, num_buckets: int = 32, max_dist: int = 128) -> int:
    """T5's causal bucketing: exact below num_buckets/2, logarithmic up to max_dist."""
    if dist < 0:
        raise ValueError("causal bucketing takes a non-negative distance")
    exact = num_buckets // 2
    if dist < exact:
        return dist
    b = exact + int(math.floor(math.log(dist / exact) / math.log(max_dist / exact) * (num_buckets - exact)))
    return min(b, num_buckets - 1)


class Sub:
    """One subsequence G_i: its tokens (bos first), start step and end state."""

    def __init__(self, index: int, start: int, bos: int):
        self.index = index          # i, 1-based
        self.start = start          # s_i, the step of admission
        self.tokens = [bos]         # bos + content tokens; the terminator is kept aside
        self.ended = False
        self.terminator: Optional[int] = None
        self.flag = FLAG_OPEN

    @property
    def n_content(self) -> int:
        return len(self.tokens) - 1


def decode(step_fn: Callable[[List[Sub], int, List[int]], Dict[int, int]], delta_t: int, time_max: int,
           sub_max: int, bos: int, terminators: Sequence[int], start_plan: Optional[Sequence[int]] = None):
    """The decoding procedure of Section 3.4.  `step_fn(G, t, active)` plays Decoder(G, H^E): it returns
    the new token of every active (not yet ended) subsequence.  Returns (G, steps_used, trace) where
    trace[t-1] = (active list, {i: token}) and G keeps bos (callers strip with `strip`).

    The schedule comes from Eq. 2: while the procedure runs, the number of subsequences at step t is
    k(t) = min(sub_max, ceil(t / delta_t)), so subsequence i appears exactly at s_i = (i-1) delta_t + 1;
    k(t) grows by at most one per step, which is the paper's "a new subsequence every delta_t steps while
    fewer than sub_max exist".  With `start_plan` (increasing start steps, the first one 1, at most sub_max of them)
    subsequence i appears at start_plan[i-1] instead: k(t) = number of planned starts <= t."""
    if start_plan is not None:
        plan = [int(x) for x in start_plan][:sub_max]
        if not plan or plan[0] != 1 or any(b <= a for a, b in zip(plan, plan[1:])):
            raise ValueError("a start plan begins at step 1 and increases")
    G: List[Sub] = []
    trace = []
    t = 0
    while t < time_max:
        t += 1
        if start_plan is None:
            k_t = min(sub_max, -(-t // delta_t))             # Eq. 2, capped
        else:
            k_t = sum(1 for s_i in plan if s_i <= t)
        if len(G) < k_t:
            i = len(G) + 1
            assert k_t == i and (plan[i - 1] if start_plan is not None else (i - 1) * delta_t + 1) == t   # one at a time, at its start step
            G.append(Sub(i, t, bos))
        active = [s.index for s in G if not s.ended]
        new = step_fn(G, t, active)
        for s in (G[i - 1] for i in active):
            tok = int(new[s.index])
            if tok in terminators:
                s.ended, s.terminator = True, tok
                s.flag |= FLAG_COMPLETE
            else:
                s.tokens.append(tok)
        trace.append((active, {i: int(new[i]) for i in active}))
        if all(s.ended for s in G):                          # every subsequence the sequence holds has ended
            break
    for s in G:
        if not s.ended:
            s.flag |= FLAG_TRUNCATED
    return G, t, trace


def strip(G: List[Sub]) -> List[List[int]]:
    """Last line of Algorithm 1: the subsequences without bos and without terminator."""
    return [list(s.tokens[1:]) for s in G]


def select_token(logits: np.ndarray, n_content: int, forced_len: Optional[int], max_sub_len: int,
                 eos: int, sep: int):
    """Greedy choice (Eq. 4 prose) under the workload's length rules.  Returns (token, capped).

    forced_len = m: while fewer than m content tokens exist the terminators cannot win; the
    (m+1)-th emission is sep whatever the logits say.  Free-running: plain argmax, except
    that a subsequence holding max_sub_len content tokens must end (sep, capped).  Ties go
    to the lowest id (np.argmax returns the first maximum)."""
    if forced_len is not None:
        if n_content >= forced_len:
            return sep, False
        masked = np.array(logits, dtype=np.float64, copy=True)
        masked[eos] = -np.inf
        masked[sep] = -np.inf
        return int(np.argmax(masked)), False
    if n_content >= max_sub_len:
        return sep, True
    return int(np.argmax(logits)), False


# --------------------------------------------------------------------------- arithmetic
def rms_norm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * gain


def rope_rotate(x: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotate consecutive pairs (x[2j], x[2j+1]) of the last axis by pos * theta^(-2j/dh)."""
    dh = x.shape[-1]
    j = np.arange(dh // 2, dtype=np.float64)
    ang = float(pos) * theta ** (-2.0 * j / dh)
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty_like(x)
    out[..., 0::2] = x[..., 0::2] * c - x[..., 1::2] * s
    out[..., 1::2] = x[..., 0::2] * s + x[..., 1::2] * c
    return out


def bf16_round(a: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bfloat16 (ties to even), as float32: bfloat16 keeps the
    upper 16 bits of a float32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32)


E4M3_MAX = 448.0


def e4m3_round(a: np.ndarray) -> np.ndarray:
    """Round to the nearest value of the E4M3 grid, ties to the even mantissa, saturating at +-448.
    The grid: +-2^(e-7) * (1 + m/8) for e = 1..15 (m = 0..7, without e = 15, m = 7, which is NaN), and
    the subnormals +-2^-6 * m/8.  Below 2^-6 the spacing is 2^-9; in [2^k, 2^(k+1)) it is 2^(k-3)."""
    x = np.asarray(a, dtype=np.float64)
    mag = np.minimum(np.abs(x), E4M3_MAX)
    k = np.floor(np.log2(np.maximum(mag, 2.0 ** -6)))          # exponent of the binade (subnormals share 2^-6's spacing)
    step = 2.0 ** (k - 3)
    q = np.rint(mag / step) * step                               # np.rint rounds halves to even, and mag / step is exact
    return np.copysign(np.minimum(q, E4M3_MAX), x)


def quantize_context_kv(kv: np.ndarray, ctx_rows: int):
    """kv [N, dh] (one head's keys or values of one sequence, float64).  Returns (the de-quantised
    array, scale).  Decisions in the CUDA path's precision: the projection is rounded to bfloat16, the
    scale is max|.| / 448 in float32 (1 when everything is zero), a value's code is
    e4m3_round(float32(value) * float32(448 / max|.|))."""
    v = bf16_round(np.asarray(kv, dtype=np.float64).astype(np.float32))[:ctx_rows]
    amax = np.float32(np.abs(v).max()) if v.size else np.float32(0)
    if amax == 0:
        return np.zeros(v.shape, dtype=np.float64), 1.0
    inv = np.float32(E4M3_MAX) / amax
    scale = amax / np.float32(E4M3_MAX)
    codes = e4m3_round((v * inv).astype(np.float32))
    return codes.astype(np.float64) * np.float64(scale), float(scale)


def masked_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, mask: np.ndarray, scale: float,
                     bias: Optional[np.ndarray] = None) -> np.ndarray:
    """softmax(scale * q.k + bias) over exactly the visible keys, times V.
    q [S,H,dh]; K,V [H,N,dh]; mask [S,N] bool; bias [S,H,N] or None.  Returns [S,H,dh].
    An invisible key gets score -inf, i.e. weight exactly 0; a row with no visible key is
    an error."""
    if not mask.any(axis=1).all():
        raise ValueError("query with an empty visible set")
    sc = scale * np.matmul(q.transpose(1, 0, 2), K.transpose(0, 2, 1))      # [H,S,N]
    if bias is not None:
        sc = sc + bias.transpose(1, 0, 2)
    sc = np.where(mask[None, :, :], sc, -np.inf)
    sc = sc - sc.max(axis=-1, keepdims=True)
    p = np.exp(sc)
    p = p / p.sum(axis=-1, keepdims=True)
    return np.matmul(p, V).transpose(1, 0, 2)


class PipelinedDecoderOracle:
    """The decoder of Eq. 3-4 around Algorithm 1, one sequence at a time, float64.

    `weights`: dict of arrays (embed, l{n}.norm1, l{n}.wqkv, l{n}.wo, l{n}.norm2, l{n}.wq_c,
    l{n}.wkv_c, l{n}.wo_c, l{n}.norm3, l{n}.w1, l{n}.w2, final_norm, lm_head, rel_bias; linear
    weights [in, out], wqkv columns [q | k | v], wkv_c columns [k | v], heads major), any float
    dtype; widened to float64 here.  `hp`: dict with n_layers, d_model, n_heads, d_head,
    delta_t, time_max, sub_max, max_sub_len, bos_id, eos_id, sep_id, pos_mode, rel_buckets,
    rel_max_dist, rope_theta, attn_scale, norm_eps."""

    def __init__(self, weights: Dict[str, np.ndarray], hp: Dict):
        self.hp = dict(hp)
        self.w = {k: np.asarray(v, dtype=np.float64) for k, v in weights.items()}
        self.L, self.d = hp["n_layers"], hp["d_model"]
        self.H, self.dh = hp["n_heads"], hp["d_head"]
        self.scale = float(hp["attn_scale"])
        self.eps = float(hp["norm_eps"])
        self.pos_mode = hp["pos_mode"]

    def _heads(self, a: np.ndarray) -> np.ndarray:
        """[N, H*dh] -> [H, N, dh]."""
        return np.ascontiguousarray(a.reshape(a.shape[0], self.H, self.dh).transpose(1, 0, 2))

    # ---- context: H^E is handed over (Algorithm 1, initialisation); its per-layer keys/values are fixed
    def encode_context(self, enc_mem: np.ndarray, ctx_len: int):
        mem = np.asarray(enc_mem, dtype=np.float64)[:ctx_len]
        hd = self.H * self.dh
        ctx = []
        for l in range(self.L):
            kv = mem @ self.w[f"l{l}.wkv_c"]
            K, V = self._heads(kv[:, :hd]), self._heads(kv[:, hd:])
            if self.hp.get("kv_c_dtype", "same") == "e4m3":
                K = np.stack([quantize_context_kv(K[h], ctx_len)[0] for h in range(self.H)])
                V = np.stack([quantize_context_kv(V[h], ctx_len)[0] for h in range(self.H)])
            ctx.append((K, V))
        return ctx

    # ---- the dependency rule and the positional term, by brute force over all token pairs
    @staticmethod
    def visibility_matrix(q_meta, k_meta) -> np.ndarray:
        """mask[s, n] = visible(query s, token n); metas are (subsequence, timestamp) pairs."""
        m = np.zeros((len(q_meta), len(k_meta)), dtype=bool)
        for s, (iq, tq) in enumerate(q_meta):
            for n, (ik, tk) in enumerate(k_meta):
                m[s, n] = visible(iq, tq, ik, tk)
        return m

    def position_bias(self, q_meta, k_meta) -> np.ndarray:
        """bias[s, h, n] = rel_bias[h, bucket(Manhattan distance)] on visible pairs, else 0."""
        hp = self.hp
        bias = np.zeros((len(q_meta), self.H, len(k_meta)), dtype=np.float64)
        for s, (iq, tq) in enumerate(q_meta):
            for n, (ik, tk) in enumerate(k_meta):
                if visible(iq, tq, ik, tk):
                    b = relative_bucket(manhattan(tq, iq, tk, ik), hp["rel_buckets"], hp["rel_max_dist"])
                    bias[s, :, n] = self.w["rel_bias"][:, b]
        return bias

    # ---- one decoder layer (Eq. 3: a stacked transformer decoder)
    def _layer(self, l, x, q_meta, K_prev, V_prev, mask, bias, ctx):
        """Rows x[S,d] carry (subsequence, timestamp) = q_meta.  Their own keys/values are
        appended to K_prev/V_prev ([H,N,dh] or None) BEFORE attending: a query sees its own
        input token and the tokens that earlier subsequences feed at the same step.
        mask/bias are over (rows, previous tokens + rows).  Returns (x_out, K_all, V_all)."""
        w, H, dh = self.w, self.H, self.dh
        hd = H * dh
        S = x.shape[0]
        h = rms_norm(x, w[f"l{l}.norm1"], self.eps)
        qkv = h @ w[f"l{l}.wqkv"]
        q = qkv[:, :hd].reshape(S, H, dh).copy()
        k = qkv[:, hd:2 * hd].reshape(S, H, dh).copy()
        v = qkv[:, 2 * hd:].reshape(S, H, dh)
        if self.pos_mode == POS_ROPE:
            for s, (iq, tq) in enumerate(q_meta):
                q[s] = rope_rotate(q[s], tq + iq, self.hp["rope_theta"])
                k[s] = rope_rotate(k[s], tq + iq, self.hp["rope_theta"])
        k, v = k.transpose(1, 0, 2), v.transpose(1, 0, 2)
        K_all = k if K_prev is None else np.concatenate([K_prev, k], axis=1)
        V_all = v if V_prev is None else np.concatenate([V_prev, v], axis=1)
        a = masked_attention(q, K_all, V_all, mask, self.scale, bias)
        x = x + a.reshape(S, hd) @ w[f"l{l}.wo"]
        h = rms_norm(x, w[f"l{l}.norm2"], self.eps)
        qc = (h @ w[f"l{l}.wq_c"]).reshape(S, H, dh)
        Kc, Vc = ctx[l]
        c = masked_attention(qc, Kc, Vc, np.ones((S, Kc.shape[1]), dtype=bool), self.scale, None)
        x = x + c.reshape(S, hd) @ w[f"l{l}.wo_c"]
        h = rms_norm(x, w[f"l{l}.norm3"], self.eps)
        x = x + np.maximum(h @ w[f"l{l}.w1"], 0.0) @ w[f"l{l}.w2"]
        return x, K_all, V_all

    def _logits(self, x):
        return rms_norm(x, self.w["final_norm"], self.eps) @ self.w["lm_head"].T

    # ---- formulation B: incremental, plain growing key/value arrays
    def new_cache(self):
        return {"K": [None] * self.L, "V": [None] * self.L, "meta": []}

    def step_incremental(self, cache, rows, ctx):
        """rows: (i, tau, token) of every active subsequence (tau = t - 1).  Appends their
        keys/values to `cache` and returns logits [S, vocab]."""
        q_meta = [(i, tau) for (i, tau, _) in rows]
        meta_all = list(cache["meta"]) + q_meta
        mask = self.visibility_matrix(q_meta, meta_all)
        bias = self.position_bias(q_meta, meta_all) if self.pos_mode == POS_T5_BIAS else None
        x = self.w["embed"][[tok for (_, _, tok) in rows]]
        for l in range(self.L):
            x, cache["K"][l], cache["V"][l] = self._layer(l, x, q_meta, cache["K"][l], cache["V"][l],
                                                          mask, bias, ctx)
        cache["meta"] = meta_all
        return self._logits(x)

    # ---- formulation A: recompute every token of G under the dense mask (Eq. 6 form)
    def step_dense(self, G: List[Sub], active: List[int], ctx):
        dt = self.hp["delta_t"]
        toks, meta = [], []
        for s in G:
            for p, tok in enumerate(s.tokens):
                toks.append(tok)
                meta.append((s.index, s.start - 1 + p))
        mask = self.visibility_matrix(meta, meta)
        bias = self.position_bias(meta, meta) if self.pos_mode == POS_T5_BIAS else None
        x = self.w["embed"][toks]
        for l in range(self.L):
            x, _, _ = self._layer(l, x, meta, None, None, mask, bias, ctx)
        last = [meta.index((i, G[i - 1].start - 1 + G[i - 1].n_content)) for i in active]
        return self._logits(x[last])

    # ---- Eq. 6: the whole target in one teacher-forced pass under the dense mask
    def teacher_forward(self, enc_mem: np.ndarray, ctx_len: int, subsequences: Sequence[Sequence[int]],
                        terminators: Optional[Sequence[int]] = None, start_plan: Optional[Sequence[int]] = None):
        """subsequences[i-1] = the content tokens of subsequence i.  Row (i, p), p = 0..m_i, has input bos
        (p = 0) or content token p, timestamp (i-1) delta_t + p, and target content token p + 1 or, at
        p = m_i, the subsequence's terminator (sep unless given).  Returns a dict: rows [(i, p)], targets,
        logits [R, vocab], logprob [R] (log-softmax of the logits at the target) and loss = -sum(logprob)."""
        hp = self.hp
        starts = fixed_plan(hp["delta_t"], len(subsequences)) if start_plan is None else [int(x) for x in start_plan]
        ctx = self.encode_context(enc_mem, ctx_len)
        rows, toks, meta, targets = [], [], [], []
        for i, sub in enumerate(subsequences, start=1):
            term = hp["sep_id"] if terminators is None else int(terminators[i - 1])
            seq = [hp["bos_id"]] + [int(t) for t in sub]
            for p, tok in enumerate(seq):
                rows.append((i, p))
                toks.append(tok)
                meta.append((i, starts[i - 1] - 1 + p))
                targets.append(seq[p + 1] if p + 1 < len(seq) else term)
        mask = self.visibility_matrix(meta, meta)
        bias = self.position_bias(meta, meta) if self.pos_mode == POS_T5_BIAS else None
        x = self.w["embed"][toks]
        for l in range(self.L):
            x, _, _ = self._layer(l, x, meta, None, None, mask, bias, ctx)
        logits = self._logits(x)
        mx = logits.max(axis=-1, keepdims=True)
        lse = mx[:, 0] + np.log(np.exp(logits - mx).sum(axis=-1))
        logprob = logits[np.arange(len(rows)), targets] - lse
        return {"rows": rows, "targets": targets, "logits": logits, "logprob": logprob, "loss": float(-logprob.sum())}

    # ---- Algorithm 1 around either formulation
    def run(self, enc_mem: np.ndarray, ctx_len: int, forced_len: Optional[Sequence[int]] = None,
            teacher: Optional[Callable[[int, int], Optional[int]]] = None, formulation: str = "B",
            keep_logits: bool = True, start_plan: Optional[Sequence[int]] = None):
        """Decode one sequence.  `teacher(i, t)`, when given and not None for that (i, t),
        replaces the chosen token as the one appended (the oracle's own choice is still
        recorded).  A subsequence that already holds max_sub_len content tokens ends with sep
        whatever was chosen or taught.  Returns a dict: subsequences (stripped), flags, n_sub,
        steps, starts and, per step, the active list, input tokens, chosen tokens, appended
        tokens and logits [S, vocab]."""
        hp = self.hp
        dt = hp["delta_t"]
        ctx = self.encode_context(enc_mem, ctx_len)
        cache = self.new_cache()
        steps_log = []
        capped = set()

        def step_fn(G, t, active):
            if formulation == "B":
                rows = [(i, t - 1, G[i - 1].tokens[-1]) for i in active]
                for (i, tau, _) in rows:
                    assert tau == G[i - 1].start - 1 + G[i - 1].n_content
                    assert start_plan is not None or tau == timestamp(i, G[i - 1].n_content, dt)
                logits = self.step_incremental(cache, rows, ctx)
            elif formulation == "A":
                logits = self.step_dense(G, active, ctx)
            else:
                raise ValueError(formulation)
            chosen, appended = {}, {}
            for r, i in enumerate(active):
                s = G[i - 1]
                fl = None if forced_len is None else int(forced_len[i - 1])
                tok, _ = select_token(logits[r], s.n_content, fl, hp["max_sub_len"], hp["eos_id"], hp["sep_id"])
                chosen[i] = tok
                t_tok = teacher(i, t) if teacher is not None else None
                appended[i] = tok if t_tok is None else int(t_tok)
                if s.n_content >= hp["max_sub_len"]:
                    appended[i] = hp["sep_id"]
                    if forced_len is None:
                        capped.add(i)
            steps_log.append({"t": t, "active": list(active),
                              "inputs": {i: G[i - 1].tokens[-1] for i in active},
                              "chosen": chosen, "appended": dict(appended),
                              "logits": logits if keep_logits else None})
            return appended

        G, steps, _ = decode(step_fn, dt, hp["time_max"], hp["sub_max"], hp["bos_id"],
                             (hp["eos_id"], hp["sep_id"]), start_plan)
        for i in capped:
            G[i - 1].flag |= FLAG_CAPPED
        return {"subsequences": strip(G), "flags": [s.flag for s in G], "n_sub": len(G), "steps": steps,
                "starts": [s.start for s in G], "trace": steps_log}
