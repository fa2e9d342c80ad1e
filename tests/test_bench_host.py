"""Host-side logic of bench.py that needs no GPU."""
import numpy as np

import bench
from oracle import pipelined_decoder as O


def test_scheduled_tokens_equals_algorithm_1_with_a_scripted_token_source():
    g = np.random.default_rng(5)
    for _ in range(40):
        delta_t, sub_max, time_max = int(g.integers(1, 5)), int(g.integers(1, 7)), int(g.integers(3, 40))
        fl = g.integers(0, 9, size=(3, sub_max))
        want = 0
        for row in fl:
            def step_fn(G, t, active, row=row):
                return {i: (2 if G[i - 1].n_content >= row[i - 1] else 7) for i in active}   # 2 = sep, 7 = content
            _, _, trace = O.decode(step_fn, delta_t, time_max, sub_max, 0, (1, 2))
            want += sum(len(a) for a, _ in trace)
        assert bench.scheduled_tokens(fl, delta_t, sub_max, time_max) == want


def test_rank_reduction_without_a_process_group():
    t, c = bench.reduce_over_ranks([1.5, 2.5], [7])
    assert t == [1.5, 2.5] and c == [7]
