"""Pins for the oracle's Algorithm 1 (Section 3.4) and the schedule arithmetic of Eq. 2."""
import json
import math
import os

import numpy as np
import pytest

from oracle import pipelined_decoder as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "fig2_walkthrough.json")))
BOS, EOS, SEP = "<bos>", "<eos>", "<sep>"


def scripted(script):
    """Token source that replays a fixed script: subsequence i emits script[i][n_content]."""
    def step_fn(G, t, active):
        return {i: script[i][G[i - 1].n_content] for i in active}
    return step_fn


def run_script(script, delta_t, time_max=50, sub_max=20):
    vocab = {}
    def enc(s):
        return vocab.setdefault(s, len(vocab) + 10)
    ids = {i: [enc(s) for s in seq] for i, seq in script.items()}
    inv = lambda: {v: k for k, v in vocab.items()}
    G, steps, trace = O.decode(scripted(ids), delta_t, time_max, sub_max, enc(BOS), (enc(EOS), enc(SEP)))
    names = inv()
    return G, steps, trace, names


def test_fig2_walkthrough_matches_the_paper():
    script = {int(k): v for k, v in GOLD["script"].items()}
    G, steps, trace, names = run_script(script, GOLD["delta_t"])
    assert steps == GOLD["steps"]
    assert len(G) == GOLD["k_final"]
    assert [[names[t] for t in s] for s in O.strip(G)] == GOLD["result"]
    assert [len(a) for a, _ in trace] == GOLD["emissions_per_step"]
    assert [a for a, _ in trace] == GOLD["active_per_step"]
    content = [sum(1 for tok in new.values() if names[tok] != EOS) for _, new in trace]
    assert content == GOLD["content_tokens_per_step"]
    assert all(s.flag == O.FLAG_COMPLETE for s in G)


def test_visible_set_of_D_matches_the_paper():
    # "D" is produced at step 2 by subsequence 2 from its bos: the query is (i=2, tau=1).
    dt = GOLD["delta_t"]
    seqs = {1: [BOS, "A", "B", "C"], 2: [BOS, "D", "E"]}
    tokens = [(i, p, s) for i, seq in seqs.items() for p, s in enumerate(seq)]
    def vis(iq, tq):
        return [[i, s] for (i, p, s) in tokens if O.visible(iq, tq, i, O.timestamp(i, p, dt))]
    assert vis(2, 1) == GOLD["visible_for_D"]
    assert len(vis(2, 1)) == 3 and GOLD["sequential_dependency_count_for_D"] == 5
    # by the same rule "E" (query i=2, tau=2) adds exactly B and D
    assert vis(2, 2) == [[1, BOS], [1, "A"], [1, "B"], [2, BOS], [2, "D"]]
    # and subsequence 1 never sees subsequence 2
    assert vis(1, 3) == [[1, BOS], [1, "A"], [1, "B"], [1, "C"]]


@pytest.mark.parametrize("delta_t,sub_max", [(1, 20), (2, 4), (3, 8), (4, 3), (7, 5)])
def test_eq2_subsequence_count_and_emission_steps(delta_t, sub_max):
    """k(t) = min(sub_max, ceil(t/delta_t)); token j of subsequence i is emitted at step
    (i-1)*delta_t + j (Eq. 2 and the sentence under it)."""
    lengths = {i: 3 + (5 * i) % 7 for i in range(1, sub_max + 1)}
    script = {i: [100 * i + j for j in range(1, m + 1)] + [1] for i, m in lengths.items()}
    seen_k = []
    def step_fn(G, t, active):
        seen_k.append(len(G))
        out = {}
        for i in active:
            j = G[i - 1].n_content + 1          # this emission is token j of subsequence i
            assert t == (i - 1) * delta_t + j
            out[i] = script[i][j - 1]
        return out
    G, steps, _ = O.decode(step_fn, delta_t, 1000, sub_max, 0, (1, 2))
    for t, k in enumerate(seen_k, start=1):
        # while earlier subsequences are still open the loop cannot have stopped, so k follows Eq. 2
        assert k == min(sub_max, math.ceil(t / delta_t))
    assert [s.start for s in G] == [(i - 1) * delta_t + 1 for i in range(1, len(G) + 1)]
    assert O.strip(G) == [script[i][:-1] for i in range(1, len(G) + 1)]
    assert steps == max((i - 1) * delta_t + lengths[i] + 1 for i in range(1, len(G) + 1))


def test_break_rule_can_stop_before_sub_max():
    # first subsequence ends at once: count(eos) == k == 1 after step 1, so the loop stops there.
    G, steps, _ = O.decode(lambda G, t, a: {i: 1 for i in a}, 3, 50, 20, 0, (1, 2))
    assert steps == 1 and len(G) == 1 and O.strip(G) == [[]]
    # with delta_t = 1 a new empty exploration is admitted each step until sub_max... but each
    # ends at once too, so the count catches up immediately.
    G, steps, _ = O.decode(lambda G, t, a: {i: 1 for i in a}, 1, 50, 20, 0, (1, 2))
    assert steps == 1 and len(G) == 1


def test_time_max_truncates_and_flags():
    G, steps, _ = O.decode(lambda G, t, a: {i: 7 for i in a}, 2, 9, 3, 0, (1, 2))
    assert steps == 9 and len(G) == 3
    assert all(s.flag == O.FLAG_TRUNCATED for s in G)
    assert [len(x) for x in O.strip(G)] == [9, 7, 5]


def test_sub_max_is_a_cap_on_the_total():
    # k only grows; once sub_max subsequences exist none is ever admitted again, even when
    # earlier ones have ended (the test is k < sub_max, not "open < sub_max").
    lengths = {1: 1, 2: 1, 3: 6}
    script = {i: [50 + i] * m + [2] for i, m in lengths.items()}
    G, steps, trace = O.decode(scripted(script), 1, 50, 3, 0, (1, 2))
    assert len(G) == 3 and steps == 3 - 1 + 6 + 1
    assert all(len(a) <= 3 for a, _ in trace)


def test_sep_and_eos_both_end_a_subsequence():
    script = {1: [5, 6, 2], 2: [7, 1]}
    G, steps, _ = O.decode(scripted(script), 2, 50, 2, 0, (1, 2))
    assert O.strip(G) == [[5, 6], [7]] and [s.terminator for s in G] == [2, 1]


def test_select_token_rules():
    logits = np.array([0.1, 9.0, 8.0, 3.0, 3.0, 2.0])
    assert O.select_token(logits, 0, None, 4, 1, 2) == (1, False)          # plain argmax may end it
    assert O.select_token(logits, 4, None, 4, 1, 2) == (2, True)           # cap forces sep
    assert O.select_token(logits, 0, 3, 4, 1, 2) == (3, False)             # terminators barred, tie -> lowest id
    assert O.select_token(logits, 3, 3, 4, 1, 2) == (2, False)             # (m+1)-th emission is sep
    assert O.select_token(np.array([1.0, 1.0, 1.0]), 0, None, 4, 7, 8)[0] == 0


# ---------------------------------------------------------------- start plans (subsequences not at fixed intervals)
def test_the_fixed_plan_is_eq_2_and_gives_the_same_decode():
    """A plan equal to Eq. 2's start steps must reproduce the fixed-interval procedure exactly; an uneven plan starts
    every subsequence at its planned step, still one per step, and stops by the same rule."""
    def scripted(lengths):
        def step_fn(G, t, active):
            return {i: (2 if G[i - 1].n_content >= lengths[i - 1] else 10 + i) for i in active}
        return step_fn
    for delta_t, sub_max in ((1, 4), (2, 5), (3, 3)):
        lengths = [5, 2, 6, 1, 4][:sub_max]
        plan = O.fixed_plan(delta_t, sub_max)
        assert plan == [(i - 1) * delta_t + 1 for i in range(1, sub_max + 1)]
        a = O.decode(scripted(lengths), delta_t, 60, sub_max, 0, (1, 2))
        b = O.decode(scripted(lengths), delta_t, 60, sub_max, 0, (1, 2), start_plan=plan)
        assert O.strip(a[0]) == O.strip(b[0]) and a[1] == b[1] and a[2] == b[2]
        assert [s.start for s in a[0]] == [s.start for s in b[0]]
    G, steps, trace = O.decode(scripted([6, 6, 2]), 2, 60, 3, 0, (1, 2), start_plan=[1, 2, 6])
    assert [s.start for s in G] == [1, 2, 6]
    assert [a for a, _ in trace][:6] == [[1], [1, 2], [1, 2], [1, 2], [1, 2], [1, 2, 3]]
    assert steps == 8 and O.strip(G) == [[11] * 6, [12] * 6, [13] * 2]
    # the plan's later starts do not keep a finished sequence alive (the stop test sees only what it holds)
    G, steps, _ = O.decode(scripted([1, 9, 9]), 2, 60, 3, 0, (1, 2), start_plan=[1, 5, 9])
    assert steps == 2 and len(G) == 1
    with pytest.raises(ValueError):
        O.decode(scripted([1]), 2, 10, 3, 0, (1, 2), start_plan=[2, 3])
    with pytest.raises(ValueError):
        O.decode(scripted([1]), 2, 10, 3, 0, (1, 2), start_plan=[1, 1])
