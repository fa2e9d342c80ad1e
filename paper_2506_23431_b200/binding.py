"""ctypes binding of the C ABI in include/pd.h.  Argument marshalling only: every step of the
decode path runs inside libpd.so.  torch is used for device memory and the CUDA stream.

There is no fallback: if libpd.so is missing or does not load, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpd.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it first (python -m paper_2506_23431_b200.build); "
                      "there is no CPU or PyTorch fallback for the decode path")
_lib = C.CDLL(LIB_PATH)

PD_OK = 0
PD_DTYPE_FP32, PD_DTYPE_BF16 = 0, 1
PD_POS_T5_BIAS, PD_POS_ROPE = 0, 1
PD_FLAG_COMPLETE, PD_FLAG_TRUNCATED, PD_FLAG_CAPPED = 1, 2, 4
PD_BUF_X, PD_BUF_QKV, PD_BUF_SELF_OUT, PD_BUF_CROSS_Q, PD_BUF_CROSS_OUT, PD_BUF_STATE = range(6)
PD_PROF_NAMES = ["append", "self_attn", "cross_attn", "argmax_sched", "gemm", "other", "vocab"]
PD_STAT_TOKENS, PD_STAT_STEPS, PD_STAT_SELF_ENTRIES, PD_STAT_CROSS_KEYS, PD_STAT_PAGES = range(5)
PD_STAT_COUNT = 8
LAYER_TENSORS = ["norm1", "wqkv", "wo", "norm2", "wq_c", "wkv_c", "wo_c", "norm3", "w1", "w2"]


class PdConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "d_head", "d_ff", "vocab", "dtype",
                                         "max_batch", "max_ctx", "sub_max", "delta_t", "time_max", "max_sub_len",
                                         "bos_id", "eos_id", "sep_id", "pos_mode", "rel_buckets", "rel_max_dist")] + \
               [(n, C.c_float) for n in ("rope_theta", "attn_scale", "norm_eps")] + \
               [(n, C.c_int32) for n in ("page_tokens", "pool_pages", "self_splits", "cross_splits", "use_graph",
                                         "store_logits", "kv_c_dtype", "device")]


class PdWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("layer", C.POINTER(C.c_void_p)), ("final_norm", C.c_void_p),
                ("lm_head", C.c_void_p), ("rel_bias", C.c_void_p)]


_H = C.c_void_p
_i32p = C.POINTER(C.c_int32)
_SIGS = {
    "pd_config_check": (C.c_int, [C.POINTER(PdConfig), C.POINTER(C.c_char_p)]),
    "pd_workspace_bytes": (C.c_size_t, [C.POINTER(PdConfig)]),
    "pd_init": (C.c_int, [C.POINTER(PdConfig), C.POINTER(PdWeights), C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(_H)]),
    "pd_encode_context": (C.c_int, [_H, C.c_void_p, _i32p, C.c_int32, _i32p]),
    "pd_step": (C.c_int, [_H, C.c_void_p]),
    "pd_run": (C.c_int, [_H, C.c_int32, _i32p]),
    "pd_done": (C.c_int, [_H, _i32p]),
    "pd_collect": (C.c_int, [_H, _i32p, _i32p, _i32p, _i32p, _i32p]),
    "pd_set_start_plan": (C.c_int, [_H, _i32p]),
    "pd_admit": (C.c_int, [_H, C.c_int32, C.c_void_p, C.c_int32, _i32p]),
    "pd_rows_done": (C.c_int, [_H, _i32p, _i32p]),
    "pd_collect_row": (C.c_int, [_H, C.c_int32, _i32p, _i32p, _i32p, _i32p, _i32p]),
    "pd_teacher_forward_scratch_bytes": (C.c_size_t, [_H, C.c_int32, C.c_int32]),
    "pd_teacher_forward": (C.c_int, [_H, _i32p, _i32p, _i32p, _i32p, C.c_void_p, C.c_size_t, C.POINTER(C.c_float), C.c_void_p,
                                     _i32p, C.POINTER(C.c_double)]),
    "pd_generate_host": (C.c_int, [_H, C.c_void_p, _i32p, C.c_int32, _i32p, _i32p, _i32p, _i32p, _i32p, _i32p]),
    "pd_get_trace": (C.c_int, [_H, C.POINTER(C.c_uint64)]),
    "pd_get_logits": (C.c_int, [_H, C.POINTER(C.c_float), _i32p]),
    "pd_get_chosen": (C.c_int, [_H, _i32p]),
    "pd_rows_per_seq": (C.c_int32, [_H]),
    "pd_debug_read": (C.c_int, [_H, C.c_int32, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]),
    "pd_get_counters": (C.c_int, [_H, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "pd_reset_counters": (C.c_int, [_H]),
    "pd_profile_enable": (C.c_int, [_H, C.c_int32]),
    "pd_profile_read": (C.c_int, [_H, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "pd_time_attention": (C.c_int, [_H, C.c_int32, C.c_int32, C.POINTER(C.c_float)]),
    "pd_get_stats": (C.c_int, [_H, C.POINTER(C.c_int64)]),
    "pd_cross_attention_scratch_bytes": (C.c_size_t, [C.c_int32] * 4),
    "pd_cross_attention": (C.c_int, [C.c_int32] * 5 + [C.c_float, C.c_int32] + [C.c_void_p] * 5 + [C.c_void_p, C.c_size_t,
                                                                                                  C.c_void_p]),
    "pd_vocab_argmax_scratch_bytes": (C.c_size_t, [C.c_int32, C.c_int32]),
    "pd_vocab_argmax": (C.c_int, [C.c_int32] * 3 + [C.c_void_p] * 6 + [C.c_size_t, C.c_void_p]),
    "pd_linear_scratch_bytes": (C.c_size_t, [C.c_int32, C.c_int32]),
    "pd_linear_sumsq_parts": (C.c_int32, [C.c_int32, C.c_int32]),
    "pd_linear": (C.c_int, [C.c_int32] * 4 + [C.c_void_p] * 3 + [C.c_float] + [C.c_void_p] * 5 + [_i32p, C.c_void_p, C.c_size_t,
                                                                                                C.c_void_p]),
    "pd_cross_attention_static_max_bytes": (C.c_size_t, []),
    "pd_cross_attention_static": (C.c_int, [C.c_int32] * 5 + [C.c_float, C.c_int32] + [C.c_void_p] * 5 + [C.c_void_p]),
    "pd_cross_attention_static_status": (C.c_int, [C.c_void_p, _i32p]),
    "pd_static_last_error": (C.c_char_p, []),
    "pd_last_error": (C.c_char_p, [_H]),
    "pd_version": (C.c_char_p, []),
    "pd_destroy": (None, [_H]),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(_lib, _name)          # AttributeError here = the library does not export the symbol
    _fn.restype, _fn.argtypes = _res, _args
EXPORTS = sorted(_SIGS)


class PdError(RuntimeError):
    def __init__(self, status: int, where: str, msg: str = ""):
        super().__init__(f"{where} failed with pd_status {status}" + (f": {msg}" if msg else ""))
        self.status = status


def _np_i32(a, shape=None) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int32)
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def _p(a: Optional[np.ndarray], typ=_i32p):
    return None if a is None else a.ctypes.data_as(typ)


def make_config(hp: Dict, max_batch: int, device: int = 0, use_graph: bool = True, self_splits: int = 0,
                cross_splits: int = 0, pool_pages: int = 0, store_logits: bool = True, kv_c_dtype: Optional[str] = None) -> PdConfig:
    """pd_config from a plain hyper-parameter dict (keys as in Workload.hyper())."""
    c = PdConfig()
    for k in ("n_layers", "d_model", "n_heads", "d_head", "d_ff", "vocab", "sub_max", "delta_t", "time_max",
              "max_sub_len", "bos_id", "eos_id", "sep_id", "pos_mode", "rel_buckets", "rel_max_dist", "page_tokens"):
        setattr(c, k, int(hp[k]))
    c.dtype = PD_DTYPE_BF16 if hp["dtype"] == "bf16" else PD_DTYPE_FP32
    c.max_batch, c.max_ctx = int(max_batch), int(hp["ctx"])
    c.rope_theta, c.attn_scale, c.norm_eps = float(hp["rope_theta"]), float(hp["attn_scale"]), float(hp["norm_eps"])
    c.pool_pages, c.self_splits, c.cross_splits = pool_pages, self_splits, cross_splits
    c.use_graph, c.store_logits, c.device = int(use_graph), int(store_logits), device
    kv = hp.get("kv_c_dtype", "same") if kv_c_dtype is None else kv_c_dtype
    c.kv_c_dtype = 1 if kv == "e4m3" else 0
    return c


class PipelinedDecoder:
    """One pd_handle plus the torch tensors (weights, workspace) it points into."""

    def __init__(self, hp: Dict, weights: Dict[str, np.ndarray], max_batch: int, device: int = 0, stream=None,
                 **cfg_kw):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("the pipelined-decoder library needs a CUDA device; there is no CPU path")
        self.torch = torch
        self.hp = dict(hp)
        self.device = torch.device("cuda", device)
        self.cfg = make_config(hp, max_batch, device, **cfg_kw)
        self.tdtype = torch.bfloat16 if hp["dtype"] == "bf16" else torch.float32
        self.np_out_dtype = np.float32
        nbytes = _lib.pd_workspace_bytes(C.byref(self.cfg))
        if nbytes == 0:
            raise PdError(-1, "pd_workspace_bytes", "invalid configuration")
        self.workspace_bytes = int(nbytes)
        with torch.cuda.device(self.device):
            self._w = {}
            for k, v in weights.items():
                t = torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32))
                self._w[k] = t.to(self.device, torch.float32 if k == "rel_bias" else self.tdtype).contiguous()
            self._ws = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
            self.stream = stream if stream is not None else torch.cuda.Stream(device=self.device)
        ws_ptr = (self._ws.data_ptr() + 255) // 256 * 256
        L = int(hp["n_layers"])
        self._layer_ptrs = (C.c_void_p * (L * len(LAYER_TENSORS)))()
        for l in range(L):
            for j, name in enumerate(LAYER_TENSORS):
                self._layer_ptrs[l * len(LAYER_TENSORS) + j] = self._w[f"l{l}.{name}"].data_ptr()
        w = PdWeights()
        w.embed = self._w["embed"].data_ptr()
        w.layer = C.cast(self._layer_ptrs, C.POINTER(C.c_void_p))
        w.final_norm = self._w["final_norm"].data_ptr()
        w.lm_head = self._w["lm_head"].data_ptr()
        w.rel_bias = self._w["rel_bias"].data_ptr() if "rel_bias" in self._w else None
        self._h = _H()
        torch.cuda.synchronize(self.device)
        st = _lib.pd_init(C.byref(self.cfg), C.byref(w), C.c_void_p(ws_ptr), C.c_size_t(self.workspace_bytes),
                          C.c_void_p(self.stream.cuda_stream), C.byref(self._h))
        if st != PD_OK:
            raise PdError(st, "pd_init")
        self.batch = 0
        self.rows_per_seq = int(_lib.pd_rows_per_seq(self._h))
        self._keep = []

    # -- helpers
    def _check(self, st: int, where: str):
        if st != PD_OK:
            raise PdError(st, where, (_lib.pd_last_error(self._h) or b"").decode())

    def close(self):
        if getattr(self, "_h", None):
            self.torch.cuda.synchronize(self.device)
            _lib.pd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def device_memory(self, enc_mem: np.ndarray):
        """Host float32 [batch, ctx, d] -> device tensor of the configured dtype."""
        t = self.torch.from_numpy(np.ascontiguousarray(enc_mem, dtype=np.float32))
        return t.to(self.device, self.tdtype).contiguous()

    # -- the C ABI, one method per entry point
    def encode_context(self, enc_mem, ctx_len: Sequence[int], forced_len=None):
        """enc_mem: torch CUDA tensor [batch, ctx, d] of the configured dtype."""
        batch = int(enc_mem.shape[0])
        if tuple(enc_mem.shape[1:]) != (self.cfg.max_ctx, self.cfg.d_model) or enc_mem.dtype != self.tdtype \
                or not enc_mem.is_contiguous() or not enc_mem.is_cuda:
            raise ValueError("enc_mem must be a contiguous CUDA tensor [batch, max_ctx, d_model] of the model dtype")
        cl = _np_i32(ctx_len, (batch,))
        fl = None if forced_len is None else _np_i32(forced_len, (batch, self.cfg.sub_max))
        self.stream.wait_stream(self.torch.cuda.current_stream(self.device))
        self._keep = [enc_mem]
        self._check(_lib.pd_encode_context(self._h, C.c_void_p(enc_mem.data_ptr()), _p(cl), batch, _p(fl)),
                    "pd_encode_context")
        self.batch = batch

    def step(self, teacher_tokens=None):
        """teacher_tokens: torch CUDA int32 tensor [batch, sub_max] or None."""
        ptr = None
        if teacher_tokens is not None:
            if teacher_tokens.dtype != self.torch.int32 or tuple(teacher_tokens.shape) != (self.batch, self.cfg.sub_max) \
                    or not teacher_tokens.is_contiguous() or not teacher_tokens.is_cuda:
                raise ValueError("teacher_tokens must be a contiguous CUDA int32 tensor [batch, sub_max]")
            self.stream.wait_stream(self.torch.cuda.current_stream(self.device))
            self._keep.append(teacher_tokens)
            ptr = C.c_void_p(teacher_tokens.data_ptr())
        self._check(_lib.pd_step(self._h, ptr), "pd_step")

    def run(self, poll_every: int = 8) -> int:
        n = C.c_int32(0)
        self._check(_lib.pd_run(self._h, poll_every, C.byref(n)), "pd_run")
        return n.value

    def done(self) -> bool:
        d = C.c_int32(0)
        self._check(_lib.pd_done(self._h, C.byref(d)), "pd_done")
        return bool(d.value)

    def collect(self):
        b, sm, msl = self.batch, self.cfg.sub_max, self.cfg.max_sub_len
        tokens = np.empty((b, sm, msl), np.int32)
        lens = np.empty((b, sm), np.int32)
        n_sub = np.empty((b,), np.int32)
        flags = np.empty((b, sm), np.int32)
        steps = np.empty((b,), np.int32)
        self._check(_lib.pd_collect(self._h, _p(tokens), _p(lens), _p(n_sub), _p(flags), _p(steps)), "pd_collect")
        return {"tokens": tokens, "lens": lens, "n_sub": n_sub, "flags": flags, "steps": steps}

    def set_start_plan(self, plan):
        """plan [batch, sub_max]: start step of every subsequence (after encode_context, before the first step)."""
        pl = _np_i32(plan, (self.batch, self.cfg.sub_max))
        self._check(_lib.pd_set_start_plan(self._h, _p(pl)), "pd_set_start_plan")

    def admit(self, row: int, enc_mem, ctx_len: int, forced_len=None):
        """A new sequence in `row` (whose sequence has ended): enc_mem torch CUDA tensor [ctx, d] of the model dtype."""
        if tuple(enc_mem.shape) != (self.cfg.max_ctx, self.cfg.d_model) or enc_mem.dtype != self.tdtype \
                or not enc_mem.is_contiguous() or not enc_mem.is_cuda:
            raise ValueError("enc_mem must be a contiguous CUDA tensor [max_ctx, d_model] of the model dtype")
        fl = None if forced_len is None else _np_i32(forced_len, (self.cfg.sub_max,))
        self.stream.wait_stream(self.torch.cuda.current_stream(self.device))
        self._keep.append(enc_mem)
        self._check(_lib.pd_admit(self._h, int(row), C.c_void_p(enc_mem.data_ptr()), int(ctx_len), _p(fl)), "pd_admit")

    def rows_done(self):
        done = np.empty((self.batch,), np.int32)
        steps = np.empty((self.batch,), np.int32)
        self._check(_lib.pd_rows_done(self._h, _p(done), _p(steps)), "pd_rows_done")
        return done, steps

    def collect_row(self, row: int):
        sm, msl = self.cfg.sub_max, self.cfg.max_sub_len
        tokens = np.empty((sm, msl), np.int32)
        lens = np.empty((sm,), np.int32)
        flags = np.empty((sm,), np.int32)
        n_sub, steps = np.empty((1,), np.int32), np.empty((1,), np.int32)
        self._check(_lib.pd_collect_row(self._h, int(row), _p(tokens), _p(lens), _p(n_sub), _p(flags), _p(steps)), "pd_collect_row")
        return {"tokens": tokens, "lens": lens, "n_sub": int(n_sub[0]), "flags": flags, "steps": int(steps[0])}

    def teacher_forward(self, subsequences, terminators=None, want_logits: bool = False):
        """Eq. 6 in one pass.  subsequences[b] = list of content-token lists of sequence b (after encode_context).
        Returns (logprob float32 [rows], loss, logits torch CUDA float32 [rows, vocab] or None), rows in
        (sequence, subsequence, position) order."""
        torch = self.torch
        sm, msl, B = self.cfg.sub_max, self.cfg.max_sub_len, self.batch
        n_sub = np.zeros((B,), np.int32)
        lens = np.zeros((B, sm), np.int32)
        toks = np.zeros((B, sm, msl), np.int32)
        term = None if terminators is None else np.zeros((B, sm), np.int32)
        for b, subs in enumerate(subsequences):
            n_sub[b] = len(subs)
            for i, sub in enumerate(subs):
                lens[b, i] = len(sub)
                toks[b, i, :len(sub)] = sub
                if term is not None:
                    term[b, i] = terminators[b][i]
        rows = int((lens + 1)[np.arange(sm)[None, :] < n_sub[:, None]].sum())
        nbytes = int(_lib.pd_teacher_forward_scratch_bytes(self._h, max(rows, 1), 0 if want_logits else 1))
        scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        sptr = (scratch.data_ptr() + 255) // 256 * 256
        logits = torch.empty((max(rows, 1), self.cfg.vocab), dtype=torch.float32, device=self.device) if want_logits else None
        lp = np.empty((max(rows, 1),), np.float32)
        n_rows, loss = C.c_int32(0), C.c_double(0.0)
        self.stream.wait_stream(torch.cuda.current_stream(self.device))
        self._check(_lib.pd_teacher_forward(self._h, _p(n_sub), _p(lens), _p(toks), _p(term), C.c_void_p(sptr), C.c_size_t(nbytes),
                                            lp.ctypes.data_as(C.POINTER(C.c_float)),
                                            C.c_void_p(logits.data_ptr()) if want_logits else None, C.byref(n_rows), C.byref(loss)),
                    "pd_teacher_forward")
        assert n_rows.value == rows
        return lp[:rows], loss.value, (logits[:rows] if want_logits else None)

    def generate_host(self, enc_mem_host, ctx_len, forced_len=None):
        """enc_mem_host: host buffer (torch CPU tensor, ideally pinned, or numpy array) of the model
        dtype's bit pattern, [batch, ctx, d].  Returns the same dict as collect()."""
        batch = int(enc_mem_host.shape[0])
        ptr = enc_mem_host.data_ptr() if hasattr(enc_mem_host, "data_ptr") else enc_mem_host.ctypes.data
        cl = _np_i32(ctx_len, (batch,))
        fl = None if forced_len is None else _np_i32(forced_len, (batch, self.cfg.sub_max))
        sm, msl = self.cfg.sub_max, self.cfg.max_sub_len
        tokens = np.empty((batch, sm, msl), np.int32)
        lens = np.empty((batch, sm), np.int32)
        n_sub = np.empty((batch,), np.int32)
        flags = np.empty((batch, sm), np.int32)
        steps = np.empty((batch,), np.int32)
        self._check(_lib.pd_generate_host(self._h, C.c_void_p(ptr), _p(cl), batch, _p(fl), _p(tokens), _p(lens),
                                          _p(n_sub), _p(flags), _p(steps)), "pd_generate_host")
        self.batch = batch
        return {"tokens": tokens, "lens": lens, "n_sub": n_sub, "flags": flags, "steps": steps}

    def get_trace(self) -> np.ndarray:
        m = np.zeros((self.cfg.time_max, self.batch), np.uint64)
        self._check(_lib.pd_get_trace(self._h, m.ctypes.data_as(C.POINTER(C.c_uint64))), "pd_get_trace")
        return m

    def get_logits(self, want_logits: bool = True):
        rows = self.batch * self.rows_per_seq
        lg = np.empty((rows, self.cfg.vocab), np.float32) if want_logits else None
        rs = np.empty((rows,), np.int32)
        self._check(_lib.pd_get_logits(self._h, _p(lg, C.POINTER(C.c_float)), _p(rs)), "pd_get_logits")
        return lg, rs.reshape(self.batch, self.rows_per_seq)

    def get_chosen(self) -> np.ndarray:
        a = np.empty((self.batch, self.cfg.sub_max, self.cfg.max_sub_len + 1), np.int32)
        self._check(_lib.pd_get_chosen(self._h, _p(a)), "pd_get_chosen")
        return a

    def debug_read(self, which: int, dtype, count: int) -> np.ndarray:
        a = np.empty(count, dtype)
        n = C.c_size_t(0)
        self._check(_lib.pd_debug_read(self._h, which, a.ctypes.data_as(C.c_void_p), a.nbytes, C.byref(n)),
                    "pd_debug_read")
        return a[: n.value // a.itemsize]

    def counters(self):
        a, b = C.c_int64(0), C.c_int64(0)
        self._check(_lib.pd_get_counters(self._h, C.byref(a), C.byref(b)), "pd_get_counters")
        return a.value, b.value

    def reset_counters(self):
        self._check(_lib.pd_reset_counters(self._h), "pd_reset_counters")

    def profile_enable(self, on: bool):
        self._check(_lib.pd_profile_enable(self._h, int(on)), "pd_profile_enable")

    def profile_read(self):
        ms = (C.c_double * len(PD_PROF_NAMES))()
        n = (C.c_int64 * len(PD_PROF_NAMES))()
        self._check(_lib.pd_profile_read(self._h, ms, n), "pd_profile_read")
        return {k: (ms[i], n[i]) for i, k in enumerate(PD_PROF_NAMES)}

    def time_attention(self, which: str, reps: int = 5) -> float:
        """Average device microseconds per layer launch of 'self_attn' or 'cross_attn' on the current state."""
        us = C.c_float(0)
        self._check(_lib.pd_time_attention(self._h, PD_PROF_NAMES.index(which), reps, C.byref(us)), "pd_time_attention")
        return us.value

    def stats(self) -> Dict[str, int]:
        a = (C.c_int64 * PD_STAT_COUNT)()
        self._check(_lib.pd_get_stats(self._h, a), "pd_get_stats")
        return {"tokens": a[PD_STAT_TOKENS], "steps": a[PD_STAT_STEPS], "self_entries": a[PD_STAT_SELF_ENTRIES],
                "cross_keys": a[PD_STAT_CROSS_KEYS], "pages": a[PD_STAT_PAGES]}


def _attention_call(fn_name: str, q, kv, n_rows, ctx_len, attn_scale: float, splits: int, scratch):
    """Shared marshalling of the stand-alone cross-attention entry points.  q [batch, rows, heads*64],
    kv [batch, heads, 2, ctx, 64] (keys, then values, per head) CUDA tensors of one dtype (float32 or
    bfloat16); n_rows, ctx_len CUDA int32 [batch].  Runs on torch's current stream; returns out
    (same shape as q)."""
    import torch
    if q.dtype not in (torch.float32, torch.bfloat16) or kv.dtype != q.dtype:
        raise ValueError("q and kv must both be float32 or both bfloat16")
    for t in (q, kv, n_rows, ctx_len):
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")
    batch, rows, hd = q.shape
    heads = hd // 64
    if hd % 64 or tuple(kv.shape[:3]) != (batch, heads, 2) or kv.dim() != 5 or kv.shape[4] != 64 \
            or n_rows.dtype != torch.int32 \
            or ctx_len.dtype != torch.int32 or n_rows.numel() != batch or ctx_len.numel() != batch:
        raise ValueError("shape mismatch")
    out = torch.empty_like(q)
    dt = PD_DTYPE_BF16 if q.dtype == torch.bfloat16 else PD_DTYPE_FP32
    stream = torch.cuda.current_stream(q.device).cuda_stream
    args = [dt, batch, rows, heads, int(kv.shape[3]), float(attn_scale), int(splits), C.c_void_p(q.data_ptr()),
            C.c_void_p(kv.data_ptr()), C.c_void_p(n_rows.data_ptr()), C.c_void_p(ctx_len.data_ptr()),
            C.c_void_p(out.data_ptr())]
    if scratch is not None:
        args += [C.c_void_p(scratch.data_ptr()), C.c_size_t(scratch.numel() * scratch.element_size())]
    args.append(C.c_void_p(stream))
    st = getattr(_lib, fn_name)(*args)
    if st != PD_OK:
        msg = (_lib.pd_static_last_error() or b"").decode() if fn_name == "pd_cross_attention_static" else ""
        raise PdError(st, fn_name, msg)
    return out


def cross_attention_scratch_bytes(batch: int, rows_per_seq: int, n_heads: int, splits: int) -> int:
    return int(_lib.pd_cross_attention_scratch_bytes(batch, rows_per_seq, n_heads, splits))


def cross_attention(q, kv, n_rows, ctx_len, attn_scale: float, splits: int = 1, scratch=None):
    """pd_cross_attention on torch CUDA tensors; `scratch` (uint8 CUDA tensor, 256-byte aligned) is
    allocated here when not given."""
    import torch
    if scratch is None:
        n = cross_attention_scratch_bytes(q.shape[0], q.shape[1], q.shape[2] // 64, splits)
        scratch = torch.empty(max(n, 256), dtype=torch.uint8, device=q.device)
    return _attention_call("pd_cross_attention", q, kv, n_rows, ctx_len, attn_scale, splits, scratch)


def cross_attention_static(q, kv, n_rows, ctx_len, attn_scale: float, splits: int = 1):
    """pd_cross_attention_static: the same op with the split-K partials in the library's built-in
    scratch array, for callers that cannot allocate device memory.  Calls sharing a device must not
    overlap on the GPU."""
    return _attention_call("pd_cross_attention_static", q, kv, n_rows, ctx_len, attn_scale, splits, None)


def cross_attention_static_status(device=None) -> int:
    """Status word the last pd_cross_attention_static call on the current device left behind (0 = fine);
    synchronises torch's current stream."""
    import torch
    word = C.c_int32(-99)
    st = _lib.pd_cross_attention_static_status(C.c_void_p(torch.cuda.current_stream(device).cuda_stream), C.byref(word))
    if st != PD_OK:
        raise PdError(st, "pd_cross_attention_static_status", (_lib.pd_static_last_error() or b"").decode())
    return word.value


def cross_attention_static_max_bytes() -> int:
    return int(_lib.pd_cross_attention_static_max_bytes())


def vocab_argmax(hidden, lm_head, want_logits: bool = False, scratch=None):
    """pd_vocab_argmax on torch CUDA tensors: hidden [rows, d] and lm_head [vocab, d], both bfloat16.
    Runs on torch's current stream; returns (best_id int32 [rows], best_val float32 [rows], logits
    float32 [rows, vocab] or None)."""
    import torch
    if hidden.dtype != torch.bfloat16 or lm_head.dtype != torch.bfloat16:
        raise ValueError("hidden and lm_head must be bfloat16")
    hidden, lm_head = hidden.contiguous(), lm_head.contiguous()
    rows, d = hidden.shape
    vocab = lm_head.shape[0]
    if scratch is None:
        n = int(_lib.pd_vocab_argmax_scratch_bytes(rows, vocab))
        scratch = torch.empty(max(n, 256), dtype=torch.uint8, device=hidden.device)
    best_id = torch.empty(rows, dtype=torch.int32, device=hidden.device)
    best_val = torch.empty(rows, dtype=torch.float32, device=hidden.device)
    logits = torch.empty(rows, vocab, dtype=torch.float32, device=hidden.device) if want_logits else None
    st = _lib.pd_vocab_argmax(rows, d, vocab, hidden.data_ptr(), lm_head.data_ptr(), best_id.data_ptr(), best_val.data_ptr(),
                              logits.data_ptr() if want_logits else None, scratch.data_ptr(), scratch.numel(),
                              torch.cuda.current_stream(hidden.device).cuda_stream)
    if st != 0:
        raise PdError(st, "pd_vocab_argmax")
    return best_id, best_val, logits


def linear(a, w, mode: int = 0, row_sumsq=None, eps: float = 1e-6, x=None, gain_next=None):
    """pd_linear on torch CUDA tensors: a bf16 [rows, d_in], w bf16 [d_in, d_out].  mode 0 / 1: returns out
    bf16 [rows, d_out] (1 = through ReLU).  mode 2 (residual): x fp32 [rows, d_out] is updated in place;
    returns (xg bf16 [rows, d_out], sumsq fp32 [parts, rows]).  Runs on torch's current stream."""
    import torch
    if a.dtype != torch.bfloat16 or w.dtype != torch.bfloat16:
        raise ValueError("a and w must be bfloat16")
    a, w = a.contiguous(), w.contiguous()
    rows, d_in = a.shape
    d_out = w.shape[1]
    dev = a.device
    n = int(_lib.pd_linear_scratch_bytes(d_in, d_out))
    scratch = torch.empty(max(n, 256), dtype=torch.uint8, device=dev)
    out = xg = ssq = None
    parts = C.c_int32(0)
    if mode == 2:
        xg = torch.empty(rows, d_out, dtype=torch.bfloat16, device=dev)
        ssq = torch.full((max(1, int(_lib.pd_linear_sumsq_parts(d_in, d_out))), rows), float("nan"), dtype=torch.float32, device=dev)
    else:
        out = torch.empty(rows, d_out, dtype=torch.bfloat16, device=dev)
    ptr = lambda t: None if t is None else C.c_void_p(t.data_ptr())
    st = _lib.pd_linear(rows, d_in, d_out, mode, ptr(a), ptr(w), ptr(row_sumsq), C.c_float(eps), ptr(out), ptr(x), ptr(gain_next),
                        ptr(xg), ptr(ssq), C.byref(parts), ptr(scratch), scratch.numel(),
                        C.c_void_p(torch.cuda.current_stream(dev).cuda_stream))
    if st != 0:
        raise PdError(st, "pd_linear")
    torch.cuda.current_stream(dev).synchronize()
    status = int(scratch[:16].view(torch.int32)[2].item())
    if status != 0:
        raise PdError(status, "pd_linear (device status)")
    if mode == 2:
        return xg, ssq[: parts.value]
    return out


def version() -> str:
    return _lib.pd_version().decode()
