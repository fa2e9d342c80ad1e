"""Element-by-element comparison of the CUDA library with the CPU oracle on the same seeded
inputs.  Used by the GPU tests and by the smoke check.  Everything the CUDA side is compared
with comes from `oracle/`; nothing here feeds CUDA results back into an expectation."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np

from oracle import pipelined_decoder as O
from paper_2506_23431_b200 import workload as W

MARGIN = 5e-2            # greedy ids are compared only where the oracle's top-2 margin exceeds this
TOL = {"fp32": 1e-4, "bf16": 2e-2}   # max-abs logit error allowed per storage type


def oracle_runs(wl: W.Workload, weights, mem_rows: Dict[int, np.ndarray], ctx_len, forced_len,
                keep_logits: bool = True, start_plan=None) -> Dict[int, dict]:
    """Decode the given batch rows with the oracle (formulation B).  mem_rows: {b: [ctx, d]}; start_plan
    [batch, sub_max] or None (Eq. 2's fixed intervals)."""
    orc = O.PipelinedDecoderOracle(weights, wl.hyper())
    out = {}
    for b, mem in mem_rows.items():
        fl = None if forced_len is None else forced_len[b]
        plan = None if start_plan is None else [int(x) for x in start_plan[b]]
        out[b] = orc.run(mem, int(ctx_len[b]), fl, keep_logits=keep_logits, start_plan=plan)
    return out


def _margin(logits: np.ndarray, barred: Sequence[int]) -> float:
    x = np.array(logits, dtype=np.float64, copy=True)
    if barred:
        x[list(barred)] = -np.inf
    top2 = np.partition(x, -2)[-2:]
    return float(top2[1] - top2[0])


def replay_compare(dec, wl: W.Workload, mem_dev, ctx_len, forced_len, runs: Dict[int, dict],
                   tol: Optional[float] = None, max_steps: Optional[int] = None, use_logits: bool = True, start_plan=None) -> dict:
    """Teacher-forced replay: the library consumes the oracle's appended tokens on the rows the
    oracle decoded (other rows run free), so every step's logits stay comparable.  Asserts:
    active sets bit-exact, logits within tol, own greedy choice equal where the oracle's margin
    exceeds MARGIN, and at the end streams / lengths / flags / steps / trace identical.
    With use_logits = False (a decoder that keeps its logits on chip, as the benchmark runs it)
    the logits are not read; everything else - active sets per step, the library's own choices
    under the margin rule, streams, lengths, flags, steps, trace - is compared all the same.
    Returns statistics (max error, compared logits, compared / skipped choices)."""
    import torch
    tol = TOL[wl.dtype] if tol is None else tol
    hp = wl.hyper()
    dec.encode_context(mem_dev, ctx_len, forced_len)
    if start_plan is not None:
        dec.set_start_plan(start_plan)
    batch, sm = dec.batch, wl.sub_max
    t_end = max(r["steps"] for r in runs.values())
    stats = {"max_err": 0.0, "logits": 0, "choices": 0, "low_margin": 0, "steps": 0}
    t = 0
    while True:
        t += 1
        teacher = np.full((batch, sm), -1, np.int32)
        for b, r in runs.items():
            if t <= r["steps"]:
                for i, tok in r["trace"][t - 1]["appended"].items():
                    teacher[b, i - 1] = tok
        dec.step(torch.from_numpy(teacher).to(dec.device))
        need_logits = use_logits and any(t <= r["steps"] for r in runs.values())
        logits, row_sub = dec.get_logits(want_logits=need_logits)
        if need_logits:
            logits = logits.reshape(batch, dec.rows_per_seq, wl.vocab)
        for b, r in runs.items():
            if t > r["steps"]:
                assert not (row_sub[b] > 0).any(), f"row {b}: active after the oracle stopped (step {t})"
                continue
            step = r["trace"][t - 1]
            act = [int(i) for i in row_sub[b] if i > 0]
            assert act == step["active"], f"row {b} step {t}: active {act} vs oracle {step['active']}"
            for c, i in enumerate(act if use_logits else []):
                ref = step["logits"][c]
                err = float(np.abs(logits[b, c].astype(np.float64) - ref).max())
                stats["max_err"] = max(stats["max_err"], err)
                stats["logits"] += ref.size
                assert err <= tol, f"row {b} step {t} subsequence {i}: logit error {err:.3e} > {tol:g}"
        stats["steps"] = t
        if dec.done() or (max_steps is not None and t >= max_steps):
            break
        assert t <= wl.time_max
    if max_steps is None:
        assert t >= t_end
    res = dec.collect()
    chosen = dec.get_chosen()
    trace = dec.get_trace()
    for b, r in runs.items():
        if max_steps is not None and r["steps"] > max_steps:
            continue
        assert int(res["n_sub"][b]) == r["n_sub"]
        assert int(res["steps"][b]) == r["steps"]
        for i, sub in enumerate(r["subsequences"]):
            n = int(res["lens"][b, i])
            assert n == len(sub) and res["tokens"][b, i, :n].tolist() == sub, f"row {b} subsequence {i + 1}"
            assert int(res["flags"][b, i]) == r["flags"][i]
        for s in r["trace"]:
            mask = sum(1 << (i - 1) for i in s["active"])
            assert int(trace[s["t"] - 1, b]) == mask
        assert not trace[r["steps"]:, b].any()
        # own greedy choices under the margin rule
        emitted = {i: 0 for i in range(1, r["n_sub"] + 1)}
        for s in r["trace"]:
            for c, i in enumerate(s["active"]):
                n = emitted[i]
                emitted[i] += 1
                fl = None if forced_len is None else int(forced_len[b][i - 1])
                n_content = n
                forced_sep = (fl is not None and n_content >= fl) or (fl is None and n_content >= hp["max_sub_len"])
                barred = [hp["eos_id"], hp["sep_id"]] if (fl is not None and not forced_sep) else []
                if forced_sep or _margin(s["logits"][c], barred) > MARGIN:
                    assert int(chosen[b, i - 1, n]) == s["chosen"][i], f"row {b} step {s['t']} sub {i}"
                    stats["choices"] += 1
                else:
                    stats["low_margin"] += 1
    return stats


def free_run_compare(dec, wl: W.Workload, mem_dev, ctx_len, forced_len, runs: Dict[int, dict]) -> dict:
    """Free-running decode on the library; per oracle row the streams must agree up to (not
    including) the first step at which some oracle margin fell below MARGIN.  Schedule facts that
    do not depend on tokens (forced lengths) must agree entirely."""
    hp = wl.hyper()
    dec.encode_context(mem_dev, ctx_len, forced_len)
    dec.run(poll_every=4)
    res = dec.collect()
    trace = dec.get_trace()
    out = {"rows_fully_equal": 0, "rows": 0}
    for b, r in runs.items():
        out["rows"] += 1
        safe_t = r["steps"] + 1
        for s in r["trace"]:
            for c, i in enumerate(s["active"]):
                fl = None if forced_len is None else int(forced_len[b][i - 1])
                n_content = s["t"] - r["starts"][i - 1]
                forced_sep = (fl is not None and n_content >= fl) or (fl is None and n_content >= hp["max_sub_len"])
                barred = [hp["eos_id"], hp["sep_id"]] if (fl is not None and not forced_sep) else []
                if not forced_sep and _margin(s["logits"][c], barred) <= MARGIN:
                    safe_t = min(safe_t, s["t"])
        # tokens emitted before safe_t must be identical
        for i, sub in enumerate(r["subsequences"], start=1):
            n_safe = max(0, min(len(sub), safe_t - r["starts"][i - 1]))
            got = res["tokens"][b, i - 1, :n_safe].tolist()
            assert got == sub[:n_safe], f"row {b} subsequence {i}: diverged before any low-margin step"
        for s in r["trace"]:
            if s["t"] < safe_t or forced_len is not None:
                assert int(trace[s["t"] - 1, b]) == sum(1 << (i - 1) for i in s["active"])
        if forced_len is not None:
            assert int(res["steps"][b]) == r["steps"] and int(res["n_sub"][b]) == r["n_sub"]
            assert res["lens"][b, : r["n_sub"]].tolist() == [len(x) for x in r["subsequences"]]
        if safe_t > r["steps"]:
            out["rows_fully_equal"] += 1
    return out
