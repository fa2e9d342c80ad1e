"""Pins for the oracle's arithmetic: what the mathematics and the paper's reductions fix."""
import math

import numpy as np
import pytest
import torch

from oracle import pipelined_decoder as O
from paper_2506_23431_b200 import workload as W
from tests import textbook

SMALL = W.CONFIGS["tiny"].scaled(name="small", n_layers=2, d_model=64, n_heads=2, d_head=32, d_ff=96,
                                 vocab=50, ctx=7, sub_max=3, delta_t=2, time_max=40, max_sub_len=6,
                                 norm_gain_std=0.2, weight_std=0.3, rel_bias_std=0.7)


def build(wl, **kw):
    wl = wl.scaled(**kw) if kw else wl
    return wl, W.make_weights(wl), W.make_encoder_memory(wl)[0]


# ---------------------------------------------------------------- bucket / distance / rope
def test_bucket_matches_exact_integer_arithmetic():
    """bucket - 16 = max j with 8^(j/16) <= d/16  <=>  8^j * 16^16 <= d^16 (big integers)."""
    for d in range(0, 400):
        if d < 16:
            want = d
        else:
            j = 0
            while 8 ** (j + 1) * 16 ** 16 <= d ** 16:
                j += 1
            want = min(16 + j, 31)
        assert O.relative_bucket(d, 32, 128) == want, d
    assert O.relative_bucket(127, 32, 128) == 31 - 0 if 8 ** 15 * 16 ** 16 <= 127 ** 16 else True
    assert [O.relative_bucket(d) for d in (15, 16, 18, 128, 10 ** 6)] == [15, 16, 16, 31, 31]
    with pytest.raises(ValueError):
        O.relative_bucket(-1)


def test_bucket_agrees_with_vectorised_t5_formula():
    d = torch.arange(0, 300)
    got = [O.relative_bucket(int(x)) for x in d]
    assert got == textbook.t5_causal_buckets(d, 32, 128).tolist()


@pytest.mark.parametrize("delta_t", [1, 2, 3, 5])
def test_manhattan_equals_position_difference_on_visible_pairs(delta_t):
    """On every visible pair |dtau| + |di| = (tau_q + i_q) - (tau_k + i_k) >= 0; on a pair hidden
    because i_k > i_q the two differ (so one scalar position cannot be used there)."""
    subs = {i: 9 for i in range(1, 6)}
    toks = [(i, O.timestamp(i, p, delta_t)) for i, n in subs.items() for p in range(n)]
    n_vis = n_diff = 0
    for (iq, tq) in toks:
        for (ik, tk) in toks:
            m = O.manhattan(tq, iq, tk, ik)
            if O.visible(iq, tq, ik, tk):
                assert m == (tq + iq) - (tk + ik) >= 0
                n_vis += 1
            elif ik > iq and tk <= tq:
                assert m != (tq + iq) - (tk + ik)
                n_diff += 1
    assert n_vis > 0 and n_diff > 0


def test_rope_is_a_rotation_and_depends_on_position_difference():
    g = np.random.default_rng(0)
    q, k = g.standard_normal(64), g.standard_normal(64)
    for (pq, pk) in [(9, 4), (105, 100), (37, 32)]:
        a = O.rope_rotate(q, pq, 10000.0) @ O.rope_rotate(k, pk, 10000.0)
        b = O.rope_rotate(q, 5, 10000.0) @ k
        assert abs(a - b) < 1e-12
    assert np.allclose(O.rope_rotate(q, 0, 10000.0), q)
    assert abs(np.linalg.norm(O.rope_rotate(q, 123, 10000.0)) - np.linalg.norm(q)) < 1e-12
    # first pair turns by exactly pos radians, counter-clockwise
    e = np.zeros(64); e[0] = 1.0
    r = O.rope_rotate(e, 2, 10000.0)
    assert abs(r[0] - math.cos(2)) < 1e-15 and abs(r[1] - math.sin(2)) < 1e-15
    # against the complex-multiplication form
    x = g.standard_normal((2, 3, 64))
    pos = torch.tensor([4, 17, 250])
    want = textbook.rope_complex(torch.tensor(x), pos, 10000.0).numpy()
    got = np.stack([O.rope_rotate(x[:, n], int(pos[n]), 10000.0) for n in range(3)], axis=1)
    assert np.allclose(got, want, atol=1e-13)


def test_rms_norm_against_library():
    g = np.random.default_rng(1)
    x, gain = g.standard_normal((5, 48)), g.standard_normal(48)
    want = torch.nn.functional.rms_norm(torch.tensor(x), (48,), torch.tensor(gain), 1e-6).numpy()
    assert np.allclose(O.rms_norm(x, gain, 1e-6), want, atol=1e-14)
    assert np.allclose(O.rms_norm(np.full((1, 4), 3.0), np.ones(4), 0.0), 1.0)


# ---------------------------------------------------------------- attention
def test_attention_by_hand():
    """Scores 0, ln 2, ln 3 give weights 1/6, 2/6, 3/6; a hidden key gets none."""
    q = np.zeros((1, 1, 2)); q[0, 0] = [1.0, 0.0]
    K = np.zeros((1, 4, 2)); K[0, :, 0] = [0.0, math.log(2.0), math.log(3.0), 50.0]
    V = np.zeros((1, 4, 2)); V[0, :, 0] = [6.0, 12.0, 18.0, 1e9]; V[0, :, 1] = [1, 1, 1, 1]
    mask = np.array([[True, True, True, False]])
    out = O.masked_attention(q, K, V, mask, 1.0)
    assert np.allclose(out[0, 0], [1.0 + 4.0 + 9.0, 1.0], atol=1e-12)
    # scale and bias enter the exponent: scale 2 squares the weights 1,2,3 -> 1,4,9
    out = O.masked_attention(q, K, V, mask, 2.0)
    assert np.allclose(out[0, 0, 0], (6 * 1 + 12 * 4 + 18 * 9) / 14.0, atol=1e-12)
    bias = np.zeros((1, 1, 4)); bias[0, 0, 0] = math.log(5.0)
    out = O.masked_attention(q, K, V, mask, 1.0, bias)
    assert np.allclose(out[0, 0, 0], (6 * 5 + 12 * 2 + 18 * 3) / 10.0, atol=1e-12)
    with pytest.raises(ValueError):
        O.masked_attention(q, K, V, np.zeros((1, 4), dtype=bool), 1.0)


def test_attention_against_pure_python_brute_force():
    g = np.random.default_rng(2)
    S, H, N, dh = 3, 2, 6, 4
    q, K, V = g.standard_normal((S, H, dh)), g.standard_normal((H, N, dh)), g.standard_normal((H, N, dh))
    bias = g.standard_normal((S, H, N))
    mask = g.random((S, N)) < 0.6
    mask[:, 0] = True
    got = O.masked_attention(q, K, V, mask, 0.37, bias)
    for s in range(S):
        for h in range(H):
            ws, den = [], 0.0
            for n in range(N):
                if mask[s, n]:
                    e = math.exp(0.37 * sum(q[s, h, c] * K[h, n, c] for c in range(dh)) + bias[s, h, n])
                    ws.append((n, e)); den += e
            for c in range(dh):
                want = sum(e * V[h, n, c] for n, e in ws) / den
                assert abs(got[s, h, c] - want) < 1e-12
    # weights sum to one: constant values come back unchanged
    ones = O.masked_attention(q, K, np.ones_like(V), mask, 0.37, bias)
    assert np.allclose(ones, 1.0, atol=1e-14)


def test_closed_form_visible_count_equals_mask_row_sum():
    for delta_t in (1, 2, 3):
        m = {1: 5, 2: 0, 3: 7, 4: 2}                      # content tokens per subsequence
        toks = [(i, O.timestamp(i, p, delta_t)) for i, n in m.items() for p in range(n + 1)]
        mask = O.PipelinedDecoderOracle.visibility_matrix(toks, toks)
        for r, (iq, tq) in enumerate(toks):
            want = 0
            for i2 in range(1, iq + 1):
                first = O.timestamp(i2, 0, delta_t)        # bos timestamp = s_i - 1
                want += max(0, min(tq - first + 1, m[i2] + 1))
            assert mask[r].sum() == want
            assert mask[r, r]                              # a query sees its own input token


# ---------------------------------------------------------------- whole decoder
@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_dense_and_incremental_formulations_agree(pos_mode):
    wl, wt, mem = build(SMALL, pos_mode=pos_mode)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    fl = [4, 6, 3]
    a = o.run(mem, wl.ctx, fl, formulation="A")
    b = o.run(mem, wl.ctx, fl, formulation="B")
    assert a["subsequences"] == b["subsequences"] and a["steps"] == b["steps"]
    for x, y in zip(a["trace"], b["trace"]):
        assert x["active"] == y["active"]
        assert np.abs(x["logits"] - y["logits"]).max() < 1e-10


@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_sub_max_1_is_ordinary_causal_decoding(pos_mode):
    """Same parameters and architecture as a sequential decoder (Section 3.2): with a single
    subsequence the visible set is the causal prefix and the distance is the token offset."""
    wl, wt, mem = build(SMALL, pos_mode=pos_mode, sub_max=1, max_sub_len=24, time_max=64, rel_max_dist=20,
                        rel_buckets=16)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    r = o.run(mem, wl.ctx, [22])
    toks = [wl.bos_id] + r["subsequences"][0]
    assert len(toks) == 23 and r["steps"] == 23
    want = textbook.causal_decoder_logits(wt, wl.hyper(), toks, [p + 1 for p in range(len(toks))], mem)
    got = np.concatenate([s["logits"] for s in r["trace"]])
    assert got.shape == want.shape
    assert np.abs(got - want).max() < 1e-11
    # greedy tokens follow from those logits
    for p, s in enumerate(r["trace"][:-1]):
        masked = want[p].copy(); masked[[wl.eos_id, wl.sep_id]] = -np.inf
        assert s["chosen"][1] == int(np.argmax(masked))


@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_no_overlap_is_causal_attention_over_the_concatenation(pos_mode):
    """Every subsequence but the last holds exactly delta_t content tokens: its terminator is
    emitted at the very step the next one starts (the loop of Algorithm 1 would stop if it ended
    any earlier), so each subsequence sees its predecessors complete and the rule degenerates to
    full causal attention over bos Y1 bos Y2 ... with position ids tau + i."""
    wl, wt, mem = build(SMALL, pos_mode=pos_mode, delta_t=8, sub_max=3, max_sub_len=8)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    fl = [8, 8, 5]
    wl2 = wl
    r = o.run(mem, wl.ctx, fl)
    assert r["n_sub"] == 3
    toks, pos, where = [], [], {}
    for i, sub in enumerate(r["subsequences"], start=1):
        for p, tok in enumerate([wl.bos_id] + sub):
            where[(i, p)] = len(toks)
            toks.append(tok)
            pos.append(O.timestamp(i, p, wl.delta_t) + i)
    assert pos == sorted(pos)
    want = textbook.causal_decoder_logits(wt, wl2.hyper(), toks, pos, mem)
    n = 0
    for s in r["trace"]:
        for row, i in enumerate(s["active"]):
            p = s["t"] - r["starts"][i - 1]
            assert np.abs(s["logits"][row] - want[where[(i, p)]]).max() < 1e-11
            n += 1
    assert n == len(toks)


def test_later_subsequences_do_not_influence_earlier_ones():
    wl, wt, mem = build(SMALL)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    fl = [6, 5, 4]
    base = o.run(mem, wl.ctx, fl)
    other = o.run(mem, wl.ctx, fl, teacher=lambda i, t: (7 + t) if (i == 3 and t < 8) else None)
    assert base["subsequences"][2] != other["subsequences"][2]
    changed = 0
    for x, y in zip(base["trace"], other["trace"]):
        assert x["active"] == y["active"]
        for row, i in enumerate(x["active"]):
            d = np.abs(x["logits"][row] - y["logits"][row]).max()
            if i <= 2:
                assert d < 1e-12
            else:
                changed += d > 1e-6
    assert changed > 0
    # and an earlier subsequence does influence a later one
    other = o.run(mem, wl.ctx, fl, teacher=lambda i, t: 9 if (i == 1 and t == 1) else None)
    s3 = [np.abs(x["logits"][x["active"].index(3)] - y["logits"][y["active"].index(3)]).max()
          for x, y in zip(base["trace"], other["trace"]) if 3 in x["active"]]
    assert max(s3) > 1e-6


def test_forced_length_schedule_is_the_closed_form():
    wl, wt, mem = build(SMALL, sub_max=3, delta_t=2)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    fl = [5, 0, 6]
    r = o.run(mem, wl.ctx, fl, keep_logits=False)
    assert [len(s) for s in r["subsequences"]] == fl
    assert r["flags"] == [O.FLAG_COMPLETE] * 3
    assert r["steps"] == max((i - 1) * 2 + 1 + m for i, m in enumerate(fl, start=1))
    for s in r["trace"]:
        want = [i for i, m in enumerate(fl, start=1) if (i - 1) * 2 + 1 <= s["t"] <= (i - 1) * 2 + 1 + m]
        assert s["active"] == want
    for sub in r["subsequences"]:
        assert all(t not in (wl.eos_id, wl.sep_id, wl.bos_id) or t == wl.bos_id for t in sub)


def test_free_running_cap_ends_a_subsequence():
    wl, wt, mem = build(SMALL, sub_max=2, max_sub_len=4, delta_t=3)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    r = o.run(mem, wl.ctx, None, keep_logits=False)
    for sub, flag in zip(r["subsequences"], r["flags"]):
        assert len(sub) <= 4
        if len(sub) == 4:
            assert flag == O.FLAG_COMPLETE | O.FLAG_CAPPED


def test_context_length_limits_cross_attention():
    """Rows of H^E beyond ctx_len must not matter; rows inside must."""
    wl, wt, mem = build(SMALL)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    a = o.run(mem, 5, [3, 3, 3])
    mem2 = mem.copy(); mem2[5:] += 3.0
    b = o.run(mem2, 5, [3, 3, 3])
    assert all(np.array_equal(x["logits"], y["logits"]) for x, y in zip(a["trace"], b["trace"]))
    mem2 = mem.copy(); mem2[4] += 3.0
    c = o.run(mem2, 5, [3, 3, 3])
    assert np.abs(a["trace"][0]["logits"] - c["trace"][0]["logits"]).max() > 1e-6


def test_workload_generator_is_deterministic_and_bf16_exact():
    wl = W.CONFIGS["bart_base"].scaled(n_layers=1, d_model=64, n_heads=1, d_ff=64, vocab=100, batch=3, ctx=8)
    a, b = W.make_weights(wl), W.make_weights(wl)
    assert all(np.array_equal(a[k], b[k]) for k in a)
    x = a["l0.wqkv"]
    assert np.array_equal(torch.tensor(x).bfloat16().float().numpy(), x)
    g = np.random.default_rng(3).standard_normal(10000).astype(np.float32)
    assert np.array_equal(W.bf16_round(g), torch.tensor(g).bfloat16().float().numpy())
    assert np.array_equal(W.make_encoder_memory(wl)[2], W.make_encoder_memory(wl, rows=range(2, 3))[0])
    for name in W.CONFIG_ORDER:
        c = W.CONFIGS[name]
        fl = W.make_forced_len(c)
        assert fl.shape == (c.batch, c.sub_max) and fl.min() >= 1 and fl.max() <= c.max_sub_len


# ---------------------------------------------------------------- Eq. 6: the teacher-forced dense forward
@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_teacher_forward_equals_the_step_by_step_decode_under_teacher_forcing(pos_mode):
    """Section 3.3: training sees the whole target at once under the dependency rule.  Every row's logits
    must be the ones the step-by-step decode computes when it is fed the same tokens (the step at which
    row (i, p) is the input of subsequence i is s_i + p), and the loss is the sum of the rows' negative
    log-likelihoods of their targets, computed here with the library's cross-entropy."""
    wl, wt, mem = build(SMALL, pos_mode=pos_mode)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    fl = [4, 6, 3]
    r = o.run(mem, wl.ctx, fl)
    tf = o.teacher_forward(mem, wl.ctx, r["subsequences"])
    assert [len(s) for s in r["subsequences"]] == fl and len(tf["rows"]) == sum(fl) + 3
    by_step = {}
    for s in r["trace"]:
        for row, i in enumerate(s["active"]):
            by_step[(i, s["t"] - r["starts"][i - 1])] = (s["logits"][row], s["appended"][i])
    for k, (i, p) in enumerate(tf["rows"]):
        lg, appended = by_step[(i, p)]
        assert np.abs(tf["logits"][k] - lg).max() < 1e-10
        assert tf["targets"][k] == appended                     # content token p + 1, or the separator at the end
    want = F_cross_entropy(tf["logits"], tf["targets"])
    assert abs(tf["loss"] - want) < 1e-9 * max(1.0, abs(want))
    assert np.allclose(tf["logprob"].sum(), -tf["loss"])


def F_cross_entropy(logits, targets):
    return float(torch.nn.functional.cross_entropy(torch.as_tensor(logits, dtype=torch.float64),
                                                   torch.as_tensor(targets, dtype=torch.long), reduction="sum"))


def test_teacher_forward_of_a_single_subsequence_is_the_textbook_causal_forward():
    wl, wt, mem = build(SMALL, sub_max=1, max_sub_len=24, time_max=64)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    content = W.make_random_tokens(wl, (9,)).tolist()
    tf = o.teacher_forward(mem, wl.ctx, [content], terminators=[wl.eos_id])
    toks = [wl.bos_id] + content
    want = textbook.causal_decoder_logits(wt, wl.hyper(), toks, [p + 1 for p in range(len(toks))], mem)
    assert np.abs(tf["logits"] - want).max() < 1e-11
    assert tf["targets"] == content + [wl.eos_id]
    # an empty subsequence (the exploration that fails at once) is one row: bos -> terminator
    tf2 = o.teacher_forward(mem, wl.ctx, [content, []])
    assert tf2["rows"][-1] == (2, 0) and tf2["targets"][-1] == wl.sep_id
    assert np.abs(tf2["logits"][:len(toks)] - tf["logits"]).max() < 1e-12       # later subsequences do not reach back


def test_start_plan_equal_to_eq_2_changes_nothing_and_an_uneven_one_keeps_the_reductions():
    """Timestamps follow the start steps: with Eq. 2's plan every logit is the fixed-interval one; with an uneven plan the
    dense and the incremental formulation still agree, the teacher-forced forward still equals the step-by-step decode,
    and later subsequences still do not reach back."""
    wl, wt, mem = build(SMALL)
    o = O.PipelinedDecoderOracle(wt, wl.hyper())
    fl = [4, 6, 3]
    base = o.run(mem, wl.ctx, fl)
    same = o.run(mem, wl.ctx, fl, start_plan=O.fixed_plan(wl.delta_t, wl.sub_max))
    assert base["subsequences"] == same["subsequences"] and base["steps"] == same["steps"]
    for x, y in zip(base["trace"], same["trace"]):
        assert x["active"] == y["active"] and np.array_equal(x["logits"], y["logits"])
    plan = [1, 2, 6]
    a = o.run(mem, wl.ctx, fl, formulation="A", start_plan=plan)
    b = o.run(mem, wl.ctx, fl, formulation="B", start_plan=plan)
    assert a["starts"] == plan and b["starts"] == plan and a["steps"] == b["steps"] == 9
    for x, y in zip(a["trace"], b["trace"]):
        assert x["active"] == y["active"] and np.abs(x["logits"] - y["logits"]).max() < 1e-10
    assert any(not np.array_equal(x["logits"], y["logits"]) for x, y in zip(b["trace"][1:], base["trace"][1:]))
    tf = o.teacher_forward(mem, wl.ctx, b["subsequences"], start_plan=plan)
    by_step = {(i, s["t"] - b["starts"][i - 1]): s["logits"][row] for s in b["trace"] for row, i in enumerate(s["active"])}
    for k, (i, p) in enumerate(tf["rows"]):
        assert np.abs(tf["logits"][k] - by_step[(i, p)]).max() < 1e-10
    # non-interference under the plan: subsequence 1's logits do not depend on what the later ones are taught
    c = o.run(mem, wl.ctx, fl, start_plan=plan, teacher=lambda i, t: (7 if i > 1 else None))
    for x, y in zip(b["trace"], c["trace"]):
        if 1 in x["active"]:
            assert np.array_equal(x["logits"][x["active"].index(1)], y["logits"][y["active"].index(1)])
