"""Seeded synthetic inputs for the pipelined-decoder hot path.

This module is DATA ONLY: shapes, seeds, random draws and the bf16 rounding of
the drawn values.  It holds none of the method's arithmetic (no attention, no
schedule, no position rule) and is the one module that both the CUDA path's
callers and the CPU oracle's callers may import, so that both sides see the
same numbers.

The five workloads stand in for the paper's datasets (Table 1: phrase-level
targets = many short subsequences, sentence-level targets = few long ones, all
over a long input context), which are not available offline.  Random numbers
come from numpy's Philox counter-based generator, one independent stream per
kind of tensor, so a workload is a pure function of (name, seed).
"""
from __future__ import annotations

from dataclasses import dataclass, replace, asdict
from typing import Dict, Optional, Tuple

import numpy as np

POS_T5_BIAS = 0   # bucketed relative bias on the Manhattan distance (Section 4.3)
POS_ROPE = 1      # rotary embedding at position tau + i

STREAM_WEIGHTS, STREAM_MEMORY, STREAM_LENGTHS, STREAM_CTXLEN, STREAM_TOKENS = range(5)


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    d_ff: int
    vocab: int
    dtype: str            # "fp32" | "bf16"
    batch: int
    ctx: int
    sub_max: int
    delta_t: int
    time_max: int
    max_sub_len: int
    length_dist: Tuple    # ("uniform", lo, hi) | ("geometric", mean, cap) | ("lognormal", mu, sigma, cap)
    pos_mode: int
    seed: int
    d_head: int = 64
    page_tokens: int = 16
    bos_id: int = 0
    eos_id: int = 1
    sep_id: int = 2
    rel_buckets: int = 32
    rel_max_dist: int = 128
    rope_theta: float = 10000.0
    norm_eps: float = 1e-6
    weight_std: float = 0.02
    rel_bias_std: float = 0.5
    norm_gain_std: float = 0.0   # 0 => all norm gains are exactly 1
    kv_c_dtype: str = "same"     # "e4m3": cross-attention keys/values stored as 8-bit floats (an option of the build)

    @property
    def attn_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.d_head))

    def hyper(self) -> Dict:
        """Plain-dict view (what the oracle and the binding take)."""
        h = asdict(self)
        h["attn_scale"] = self.attn_scale
        return h

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations named by the benchmark definition.  Seeds: 0, 2, 3, 4, 5.
CONFIGS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 2, 256, 4, 1024, 8192, "fp32", 1, 256, 4, 2, 64, 16,
                     ("uniform", 8, 16), POS_T5_BIAS, 0),
    "bart_base": Workload("bart_base", 6, 768, 12, 3072, 50265, "bf16", 16, 1024, 8, 3, 128, 48,
                          ("geometric", 20.0, 48), POS_ROPE, 2),
    "long_context": Workload("long_context", 12, 1024, 16, 4096, 32128, "bf16", 8, 4096, 8, 4, 160, 40,
                             ("uniform", 16, 40), POS_T5_BIAS, 3),
    "summarisation": Workload("summarisation", 12, 1024, 16, 4096, 32128, "bf16", 32, 2048, 16, 2, 256, 64,
                              ("lognormal", 3.0, 0.4, 64), POS_T5_BIAS, 4),
    "keyphrase": Workload("keyphrase", 6, 768, 12, 3072, 50265, "bf16", 64, 1024, 32, 1, 48, 8,
                          ("uniform", 3, 8), POS_ROPE, 5),
}
CONFIG_ORDER = ["tiny", "bart_base", "long_context", "summarisation", "keyphrase"]


def _rng(seed: int, stream: int) -> np.random.Generator:
    key = np.array([np.uint64(seed), np.uint64(stream)], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bfloat16, returned as float32."""
    return (bf16_bits(a).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(a: np.ndarray, dtype: str) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return bf16_round(a) if dtype == "bf16" else a


def make_weights(w: Workload) -> Dict[str, np.ndarray]:
    """All decoder parameters as float32 arrays (bf16-representable when dtype == "bf16").

    Linear weights are stored [in, out] (y = x @ W); lm_head and embed are [vocab, d].
    wqkv columns are [q | k | v], each n_heads*d_head wide, head-major; wkv_c is [k | v].
    rel_bias is always float32 [n_heads, rel_buckets] and shared by all layers.
    """
    g = _rng(w.seed, STREAM_WEIGHTS)
    d, ff, v, hd = w.d_model, w.d_ff, w.vocab, w.n_heads * w.d_head

    def normal(*shape):
        return _store(g.standard_normal(shape, dtype=np.float32) * np.float32(w.weight_std), w.dtype)

    def gain():
        a = np.ones(d, dtype=np.float32)
        if w.norm_gain_std > 0:
            a = a + g.standard_normal(d, dtype=np.float32) * np.float32(w.norm_gain_std)
        return _store(a, w.dtype)

    out: Dict[str, np.ndarray] = {"embed": normal(v, d)}
    for l in range(w.n_layers):
        out[f"l{l}.norm1"] = gain()
        out[f"l{l}.wqkv"] = normal(d, 3 * hd)
        out[f"l{l}.wo"] = normal(hd, d)
        out[f"l{l}.norm2"] = gain()
        out[f"l{l}.wq_c"] = normal(d, hd)
        out[f"l{l}.wkv_c"] = normal(d, 2 * hd)
        out[f"l{l}.wo_c"] = normal(hd, d)
        out[f"l{l}.norm3"] = gain()
        out[f"l{l}.w1"] = normal(d, ff)
        out[f"l{l}.w2"] = normal(ff, d)
    out["final_norm"] = gain()
    out["lm_head"] = normal(v, d)
    out["rel_bias"] = (g.standard_normal((w.n_heads, w.rel_buckets), dtype=np.float32)
                       * np.float32(w.rel_bias_std)).astype(np.float32)
    return out


LAYER_TENSORS = ["norm1", "wqkv", "wo", "norm2", "wq_c", "wkv_c", "wo_c", "norm3", "w1", "w2"]


def make_encoder_memory(w: Workload, rows: Optional[range] = None) -> np.ndarray:
    """Encoder hidden states H^E, iid N(0,1), [batch, ctx, d] float32 (bf16-representable
    for bf16 workloads).  Every batch row has its own stream, so a subset of rows can be
    drawn without drawing the rest."""
    rows = range(w.batch) if rows is None else rows
    out = np.empty((len(rows), w.ctx, w.d_model), dtype=np.float32)
    for j, b in enumerate(rows):
        g = _rng(w.seed, STREAM_MEMORY + 16 * (b + 1))
        out[j] = _store(g.standard_normal((w.ctx, w.d_model), dtype=np.float32), w.dtype)
    return out


def make_ctx_len(w: Workload, ragged: bool = False) -> np.ndarray:
    if not ragged:
        return np.full(w.batch, w.ctx, dtype=np.int32)
    g = _rng(w.seed, STREAM_CTXLEN)
    return g.integers(max(1, w.ctx // 2), w.ctx + 1, size=w.batch).astype(np.int32)


def make_forced_len(w: Workload) -> np.ndarray:
    """Content-token count of every subsequence, [batch, sub_max] int32, 0 <= m <= max_sub_len."""
    g = _rng(w.seed, STREAM_LENGTHS)
    shape = (w.batch, w.sub_max)
    kind = w.length_dist[0]
    if kind == "uniform":
        _, lo, hi = w.length_dist
        m = g.integers(lo, hi + 1, size=shape)
    elif kind == "geometric":
        _, mean, cap = w.length_dist
        m = np.minimum(g.geometric(1.0 / mean, size=shape), cap)
    elif kind == "lognormal":
        _, mu, sigma, cap = w.length_dist
        z = g.standard_normal(shape)
        m = np.clip(np.rint(np.exp(mu + sigma * z)), 1, cap)
    else:
        raise ValueError(kind)
    return np.minimum(m, w.max_sub_len).astype(np.int32)


def make_random_tokens(w: Workload, shape) -> np.ndarray:
    """Content token ids (never bos/eos/sep) for scripted or teacher-forced runs."""
    g = _rng(w.seed, STREAM_TOKENS)
    return g.integers(3, w.vocab, size=shape).astype(np.int32)
