"""GPU parity tests: the CUDA library, called through the C ABI, against the CPU fp64 oracle on
the same seeded inputs.  Bars: schedule / active sets / streams bit-exact; logits within
1e-4 (fp32 storage) or 2e-2 (bf16 storage) max-abs; greedy ids identical wherever the oracle's
top-2 margin exceeds 5e-2."""
import numpy as np
import pytest

from paper_2506_23431_b200 import workload as W
from tests import parity

pytestmark = pytest.mark.gpu


def make(wl, rows=None, ragged=False, **dec_kw):
    from paper_2506_23431_b200.binding import PipelinedDecoder
    weights = W.make_weights(wl)
    mem = W.make_encoder_memory(wl)
    ctx_len = W.make_ctx_len(wl, ragged=ragged)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch, **dec_kw)
    rows = list(range(wl.batch)) if rows is None else rows
    return weights, mem, ctx_len, dec, rows


def check(wl, rows=None, ragged=False, forced=True, free_run=True, **dec_kw):
    weights, mem, ctx_len, dec, rows = make(wl, rows, ragged, **dec_kw)
    fl = W.make_forced_len(wl) if forced else None
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, fl)
    mem_dev = dec.device_memory(mem)
    stats = parity.replay_compare(dec, wl, mem_dev, ctx_len, fl, runs)
    assert stats["logits"] > 0 and stats["choices"] > 0
    if free_run:
        parity.free_run_compare(dec, wl, mem_dev, ctx_len, fl, runs)
    dec.close()
    return stats


TINY = W.CONFIGS["tiny"]
# scaled-down relatives of the bf16 configs: several tiles, ragged tails, page crossings
SMALL_BF16 = dict(n_layers=2, d_model=128, n_heads=2, d_ff=256, vocab=1000, norm_gain_std=0.1)


def test_tiny_fp32_t5_bias_full_config():
    s = check(TINY)
    assert s["max_err"] < 1e-4


def test_tiny_fp32_rope():
    check(TINY.scaled(pos_mode=W.POS_ROPE, norm_gain_std=0.1))


def test_tiny_fp32_without_graph_and_with_splits():
    check(TINY.scaled(norm_gain_std=0.1), use_graph=False, self_splits=3, cross_splits=2)


def test_fp32_batch_ragged_context_page_size_32():
    wl = TINY.scaled(batch=3, ctx=200, page_tokens=32, sub_max=5, delta_t=3, max_sub_len=40,
                     length_dist=("uniform", 1, 40), time_max=80, norm_gain_std=0.1, vocab=777)
    check(wl, ragged=True, self_splits=2, cross_splits=3)


def test_fp32_free_running_cap_and_time_max():
    # no forced lengths: random weights almost never emit a terminator, so subsequences run into
    # the max_sub_len cap; time_max then cuts the rest
    wl = TINY.scaled(batch=2, sub_max=6, delta_t=2, max_sub_len=7, time_max=15, vocab=300)
    weights, mem, ctx_len, dec, rows = make(wl)
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, None)
    assert any(f & 4 for r in runs.values() for f in r["flags"])
    assert any(f & 2 for r in runs.values() for f in r["flags"])
    parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, None, runs)
    dec.close()


def test_fp32_sub_max_1_is_sequential_decoding():
    wl = TINY.scaled(sub_max=1, max_sub_len=30, length_dist=("uniform", 30, 30), time_max=40)
    check(wl)


@pytest.mark.parametrize("page_tokens", [16, 32])
@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_small_bf16_tensor_core_attention(pos_mode, page_tokens):
    wl = W.CONFIGS["bart_base"].scaled(name="small_bf16", batch=3, ctx=300, sub_max=6, delta_t=2, max_sub_len=40,
                                       length_dist=("uniform", 1, 40), time_max=60, pos_mode=pos_mode,
                                       page_tokens=page_tokens, **SMALL_BF16)
    s = check(wl, ragged=True, cross_splits=2, self_splits=2)
    assert s["max_err"] < 2e-2


def test_small_bf16_many_short_subsequences_two_query_tiles():
    # 20 rows per sequence: exercises the two-tile (32-row) tensor-core variant
    wl = W.CONFIGS["keyphrase"].scaled(name="small_kp", batch=2, ctx=130, sub_max=24, delta_t=1, max_sub_len=19,
                                       length_dist=("uniform", 3, 19), time_max=48, **SMALL_BF16)
    check(wl, ragged=True)
    check(wl.scaled(page_tokens=32, pos_mode=W.POS_T5_BIAS), ragged=True, self_splits=3)


def test_small_bf16_wide_rows_use_cuda_core_cross_attention():
    # more than 32 rows per sequence: falls back to the CUDA-core cross-attention kernel
    wl = W.CONFIGS["keyphrase"].scaled(name="small_wide", batch=1, ctx=64, sub_max=40, delta_t=1, max_sub_len=36,
                                       length_dist=("uniform", 30, 36), time_max=80, **SMALL_BF16)
    check(wl, free_run=False)


def test_fp32_empty_subsequences_and_early_stop():
    """Lengths from 0: a subsequence can end at its first emission (returned empty), and a sequence
    whose admitted subsequences have all ended stops before the later ones are ever admitted."""
    wl = TINY.scaled(batch=4, ctx=70, sub_max=6, delta_t=3, max_sub_len=5, length_dist=("uniform", 0, 5), time_max=40,
                     vocab=300, norm_gain_std=0.1)
    weights, mem, ctx_len, dec, rows = make(wl)
    fl = W.make_forced_len(wl)
    assert (fl == 0).any()
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, fl)
    assert any(r["n_sub"] < wl.sub_max for r in runs.values()), "no early stop in this draw"
    assert any(len(sub) == 0 for r in runs.values() for sub in r["subsequences"])
    parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    parity.free_run_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    dec.close()


def test_bf16_sub_max_64_one_key_context_and_unaligned_context():
    """The largest subsequence count (a 64-bit active mask), a context of a single position, and a
    context length that is neither a multiple of the tile nor of 16."""
    wl = W.CONFIGS["keyphrase"].scaled(name="edge64", batch=3, ctx=131, sub_max=64, delta_t=1, max_sub_len=6,
                                       length_dist=("uniform", 1, 6), time_max=80, pos_mode=W.POS_T5_BIAS, **SMALL_BF16)
    weights, mem, _, dec, rows = make(wl)
    ctx_len = np.array([1, 131, 77], dtype=np.int32)
    fl = W.make_forced_len(wl)
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, fl)
    assert max(r["n_sub"] for r in runs.values()) == 64
    stats = parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    assert stats["max_err"] < 2e-2
    dec.close()


def test_bf16_long_page_lists():
    """More pages per sequence than the self-attention kernel's threads (the page list is staged in
    more than one round), long subsequences over several pages, T5 bias over long distances."""
    wl = W.CONFIGS["summarisation"].scaled(name="long_lists", batch=2, ctx=150, sub_max=48, delta_t=4, max_sub_len=50,
                                           length_dist=("uniform", 30, 50), time_max=245, **SMALL_BF16)
    weights, mem, ctx_len, dec, rows = make(wl, ragged=True)
    fl = W.make_forced_len(wl)
    runs = parity.oracle_runs(wl, weights, {0: mem[0]}, ctx_len, fl)
    stats = parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    assert dec.stats()["pages"] > 0 and stats["max_err"] < 2e-2
    import ctypes as C
    assert dec.cfg.sub_max * (-(-(wl.max_sub_len + 1) // wl.page_tokens)) > 128
    dec.close()


def test_bf16_free_running_cap_and_time_max():
    """No forced lengths on the bf16 path: subsequences run into the max_sub_len cap (ended with sep, flag capped) and
    time_max cuts the rest (flag truncated); every step replayed against the oracle."""
    wl = W.CONFIGS["summarisation"].scaled(name="bf16_cap", batch=3, ctx=80, sub_max=6, delta_t=2, max_sub_len=7, time_max=15,
                                           **SMALL_BF16)
    weights, mem, ctx_len, dec, rows = make(wl, ragged=True)
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, None)
    assert any(f & 4 for r in runs.values() for f in r["flags"]) and any(f & 2 for r in runs.values() for f in r["flags"])
    s = parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, None, runs)
    assert s["max_err"] < 2e-2
    dec.close()


@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_bf16_one_row_per_sequence_one_sequence_tiny_context(pos_mode):
    """delta_t beyond every length: at most one subsequence is open at a time (one row per sequence, the smallest row
    block), a batch of one, and a context shorter than a key tile."""
    wl = W.CONFIGS["bart_base"].scaled(name="bf16_one_row", batch=1, ctx=16, sub_max=4, delta_t=12, max_sub_len=10,
                                       length_dist=("uniform", 6, 10), time_max=60, pos_mode=pos_mode, **SMALL_BF16)
    weights, mem, _, dec, rows = make(wl)
    assert dec.rows_per_seq == 1
    ctx_len = np.array([11], dtype=np.int32)
    fl = W.make_forced_len(wl)
    runs = parity.oracle_runs(wl, weights, {0: mem[0]}, ctx_len, fl)
    s = parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    assert s["max_err"] < 2e-2 and s["choices"] > 0
    parity.free_run_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    dec.close()


def uneven_plan(wl, seed):
    """Start steps at least delta_t apart, with seeded extra gaps (what an adaptive policy might decide)."""
    g = np.random.Generator(np.random.Philox(key=np.array([seed, 808], dtype=np.uint64)))
    gaps = wl.delta_t + g.integers(0, 4, size=(wl.batch, wl.sub_max))
    gaps[:, 0] = 1
    return np.cumsum(gaps, axis=1).astype(np.int32)


@pytest.mark.parametrize("kind", ["bf16_t5", "bf16_rope", "fp32"])
def test_start_plans_not_at_fixed_intervals(kind):
    """Subsequences admitted at planned steps instead of every delta_t: the oracle decodes with the same plan; active
    sets, logits, choices, streams and the trace must agree step by step, and the teacher-forced forward must use the
    plan's timestamps too."""
    if kind == "fp32":
        wl = TINY.scaled(batch=2, ctx=64, sub_max=4, delta_t=2, max_sub_len=9, length_dist=("uniform", 2, 9), time_max=60,
                         vocab=300, norm_gain_std=0.1)
    else:
        wl = W.CONFIGS["bart_base"].scaled(name="plan", batch=3, ctx=150, sub_max=6, delta_t=2, max_sub_len=24,
                                           length_dist=("uniform", 1, 24), time_max=90,
                                           pos_mode=W.POS_T5_BIAS if kind == "bf16_t5" else W.POS_ROPE, **SMALL_BF16)
    weights, mem, ctx_len, dec, rows = make(wl, ragged=True)
    fl = W.make_forced_len(wl)
    plan = uneven_plan(wl, 3)
    assert (np.diff(plan, axis=1) >= wl.delta_t).all() and (np.diff(plan, axis=1) > wl.delta_t).any()
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, fl, start_plan=plan)
    assert all(r["starts"] == plan[b, :r["n_sub"]].tolist() for b, r in runs.items())
    mem_dev = dec.device_memory(mem)
    s = parity.replay_compare(dec, wl, mem_dev, ctx_len, fl, runs, start_plan=plan)
    assert s["choices"] > 0
    # the fixed plan comes back with the next pd_encode_context
    base = parity.oracle_runs(wl, weights, {0: mem[0]}, ctx_len, fl)
    parity.replay_compare(dec, wl, mem_dev, ctx_len, fl, base)
    if kind != "fp32":
        from oracle import pipelined_decoder as O
        dec.encode_context(mem_dev, ctx_len, fl)
        dec.set_start_plan(plan)
        subs = [runs[b]["subsequences"] for b in range(wl.batch)]
        lp, loss, logits = dec.teacher_forward(subs, want_logits=True)
        ref = O.PipelinedDecoderOracle(weights, wl.hyper()).teacher_forward(mem[0], int(ctx_len[0]), subs[0],
                                                                           start_plan=plan[0, :len(subs[0])].tolist())
        got = logits[:len(ref["rows"])].cpu().numpy().astype(np.float64)
        assert np.abs(got - ref["logits"]).max() <= 2e-2
    # plans the workspace is not sized for are refused
    from paper_2506_23431_b200.binding import PdError
    dec.encode_context(mem_dev, ctx_len, fl)
    bad = plan.copy(); bad[0, 1] = bad[0, 0] + wl.delta_t - 1
    with pytest.raises(PdError) as e:
        dec.set_start_plan(bad)
    assert e.value.status == -1
    dec.step()
    with pytest.raises(PdError) as e:
        dec.set_start_plan(plan)
    assert e.value.status == -2
    dec.close()


def test_steps_after_the_end_are_no_ops():
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = TINY.scaled(vocab=300)
    weights, mem, ctx_len, fl = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl), W.make_forced_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    dec.encode_context(dec.device_memory(mem), ctx_len, fl)
    dec.run()
    a = dec.collect()
    st = dec.stats()
    for _ in range(3):
        dec.step()
    assert dec.done()
    b = dec.collect()
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    assert dec.stats()["tokens"] == st["tokens"] and dec.stats()["steps"] == st["steps"]
    dec.close()


def test_batch_independence():
    """B sequences share a step clock and nothing else: decoding a row alone gives its streams."""
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = TINY.scaled(batch=4, ctx=96, vocab=500)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl, ragged=True)
    fl = W.make_forced_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    dec.encode_context(dec.device_memory(mem), ctx_len, fl)
    dec.run()
    full = dec.collect()
    for b in (0, 3):
        dec.encode_context(dec.device_memory(mem[b:b + 1]), ctx_len[b:b + 1], fl[b:b + 1])
        dec.run()
        one = dec.collect()
        assert np.array_equal(one["tokens"][0], full["tokens"][b])
        assert one["steps"][0] == full["steps"][b]
    dec.close()


def test_pool_exhaustion_is_reported_not_faulted():
    from paper_2506_23431_b200.binding import PipelinedDecoder, PdError
    wl = TINY.scaled(batch=2, vocab=300)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch, pool_pages=3)
    dec.encode_context(dec.device_memory(mem), ctx_len, W.make_forced_len(wl))
    with pytest.raises(PdError) as e:
        dec.run()
        dec.collect()
    assert e.value.status == -4
    dec.close()


def test_call_order_and_argument_errors():
    from paper_2506_23431_b200.binding import PipelinedDecoder, PdError
    wl = TINY.scaled(vocab=300)
    weights, mem = W.make_weights(wl), W.make_encoder_memory(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, 1)
    with pytest.raises(PdError) as e:
        dec.step()
    assert e.value.status == -2
    with pytest.raises(PdError) as e:
        dec.encode_context(dec.device_memory(mem), [wl.ctx + 1], None)
    assert e.value.status == -1
    with pytest.raises(PdError) as e:
        dec.encode_context(dec.device_memory(mem), [wl.ctx], np.full((1, wl.sub_max), wl.max_sub_len + 1))
    assert e.value.status == -1
    dec.close()


def test_generate_host_matches_stepwise_run():
    import torch
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = TINY.scaled(batch=2, vocab=400)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl)
    fl = W.make_forced_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    dec.encode_context(dec.device_memory(mem), ctx_len, fl)
    dec.run()
    a = dec.collect()
    host = torch.from_numpy(mem).pin_memory()
    b = dec.generate_host(host, ctx_len, fl)
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    own, gemms = dec.counters()
    assert own > 0 and gemms > 0
    st = dec.stats()
    assert st["tokens"] == int((fl + 1).sum()) and st["steps"] == int(a["steps"].max())
    dec.close()


def test_bf16_choices_do_not_depend_on_storing_the_logits():
    """store_logits = 0 keeps the logits inside the vocabulary kernel; the streams, the recorded
    greedy choices and the schedule must be those of a run that stores them, and pd_get_logits
    must say that there is nothing to read."""
    from paper_2506_23431_b200.binding import PipelinedDecoder, PdError
    wl = W.CONFIGS["bart_base"].scaled(name="small_nolog", batch=5, ctx=200, sub_max=7, delta_t=2, max_sub_len=30,
                                       length_dist=("uniform", 1, 30), time_max=60, **SMALL_BF16)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl, ragged=True)
    fl = W.make_forced_len(wl)
    out = []
    for store in (True, False):
        dec = PipelinedDecoder(wl.hyper(), weights, wl.batch, store_logits=store)
        dec.encode_context(dec.device_memory(mem), ctx_len, fl)
        dec.step()
        if store:
            lg, rs = dec.get_logits()
            assert np.isfinite(lg[rs.reshape(-1) > 0]).all()
        else:
            with pytest.raises(PdError) as e:
                dec.get_logits()
            assert e.value.status == -2
        dec.run()
        res = dec.collect()
        res["chosen"] = dec.get_chosen()
        res["trace"] = dec.get_trace()
        out.append(res)
        dec.close()
    for k in out[0]:
        assert np.array_equal(out[0][k], out[1][k]), k


def test_generate_host_in_uneven_chunks_matches_stepwise_run():
    """143 MB of encoder memory cross PCIe as four chunks of 4, 4, 4 and 5 sequences, each projected while
    the next is still being copied: the streams must be those of the plain encode + step path."""
    import torch
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = W.CONFIGS["bart_base"].scaled(name="chunks", batch=17, ctx=4096, sub_max=3, delta_t=2, max_sub_len=6,
                                       length_dist=("uniform", 1, 6), time_max=16, n_layers=2, d_model=1024, n_heads=16,
                                       d_ff=512, vocab=500)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl, ragged=True)
    fl = W.make_forced_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    mem_dev = dec.device_memory(mem)
    dec.encode_context(mem_dev, ctx_len, fl)
    dec.run()
    a = dec.collect()
    host = mem_dev.cpu().pin_memory()
    assert host.numel() * host.element_size() >= 2 * (64 << 20)
    for _ in range(2):                                  # the second call reuses the staging buffer
        b = dec.generate_host(host, ctx_len, fl)
        for k in a:
            assert np.array_equal(a[k], b[k]), k
    dec.close()


def test_two_identical_decodes_give_identical_logits():
    """Run-to-run reproducibility of the whole step (ragged contexts, several CTAs per (sequence, head)
    segment in cross-attention, split self-attention): the fp32 logits of every step must repeat bit
    for bit."""
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = W.CONFIGS["bart_base"].scaled(name="repeat", batch=9, ctx=4096, sub_max=3, delta_t=2, max_sub_len=6,
                                       length_dist=("uniform", 1, 6), time_max=16, n_layers=2, d_model=512, n_heads=8,
                                       d_ff=512, vocab=500)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl, ragged=True)
    fl = W.make_forced_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    mem_dev = dec.device_memory(mem)

    def trace():
        dec.encode_context(mem_dev, ctx_len, fl)
        out = []
        for _ in range(8):
            dec.step()
            out.append(dec.get_logits()[0].copy())
        return out

    first = trace()
    for _ in range(3):
        again = trace()
        for s, (x, y) in enumerate(zip(first, again)):
            assert np.array_equal(x.view(np.int32), y.view(np.int32)), f"logits of step {s + 1} differ between two identical runs"
    dec.close()


@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_small_bf16_with_e4m3_context_keys_values(pos_mode):
    """The 8-bit storage of the cross-attention keys/values against the oracle that quantises likewise:
    ragged contexts (a context of less than one tile, a tile edge, zero-filled tails), three layers."""
    wl = W.CONFIGS["bart_base"].scaled(name="small_e4m3", batch=4, ctx=304, sub_max=6, delta_t=2, max_sub_len=40,
                                       length_dist=("uniform", 1, 40), time_max=60, pos_mode=pos_mode, kv_c_dtype="e4m3",
                                       **dict(SMALL_BF16, n_layers=3))
    weights, mem, _, dec, rows = make(wl)
    ctx_len = np.array([304, 100, 257, 129], dtype=np.int32)
    fl = W.make_forced_len(wl)
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, fl)
    stats = parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    assert stats["max_err"] < 2e-2 and stats["choices"] > 0
    dec.close()


def test_small_bf16_e4m3_two_query_tiles_and_long_context():
    """Twenty rows per sequence (two 16-row query tiles) over 2000 context positions: several CTAs per
    (sequence, head) segment, partial records merged by ticket, all on 8-bit keys/values."""
    wl = W.CONFIGS["keyphrase"].scaled(name="small_kp8", batch=2, ctx=2000, sub_max=24, delta_t=1, max_sub_len=19,
                                       length_dist=("uniform", 3, 19), time_max=48, kv_c_dtype="e4m3", **SMALL_BF16)
    check(wl, ragged=True, free_run=False)


def test_split_self_attention_merges_in_the_launch_and_repeats_bit_for_bit():
    """Long page lists with four splits per (sequence, head): the split CTAs leave partial records and the
    last one to arrive merges them in split order, so twenty decodes of the same inputs must give the same
    logits bit for bit whatever the arrival order - and the logits must be the oracle's."""
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = W.CONFIGS["summarisation"].scaled(name="split_merge", batch=3, ctx=100, sub_max=40, delta_t=1, max_sub_len=40,
                                           length_dist=("uniform", 25, 40), time_max=90, **SMALL_BF16)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl, ragged=True)
    fl = W.make_forced_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch, self_splits=4)
    mem_dev = dec.device_memory(mem)
    n_steps = 45                                        # by then every sequence holds more than 64 pages

    def logits_after(steps):
        dec.encode_context(mem_dev, ctx_len, fl)
        for _ in range(steps):
            dec.step()
        return dec.get_logits()[0].copy()

    first = logits_after(n_steps)
    assert dec.stats()["pages"] > 3 * 64
    for _ in range(19):
        again = logits_after(n_steps)
        assert np.array_equal(first.view(np.int32), again.view(np.int32)), "two identical decodes gave different logits"
    runs = parity.oracle_runs(wl, weights, {1: mem[1]}, ctx_len, fl)
    stats = parity.replay_compare(dec, wl, mem_dev, ctx_len, fl, runs, max_steps=n_steps + 5)
    assert stats["max_err"] < 2e-2 and stats["logits"] > 0
    dec.close()


FULL = [("bart_base", 2e-2), ("long_context", 2e-2), ("summarisation", 2e-2), ("keyphrase", 2e-2)]
_ORACLE_CACHE = {}


def full_size_case(name, ragged):
    """Weights, encoder memory, lengths and the oracle's decode of batch rows 0 and B-1 of a full-size
    configuration; computed once per session (the oracle needs some seconds per row)."""
    key = (name, ragged)
    if key not in _ORACLE_CACHE:
        wl = W.CONFIGS[name]
        weights, mem = W.make_weights(wl), W.make_encoder_memory(wl)
        ctx_len, fl = W.make_ctx_len(wl, ragged=ragged), W.make_forced_len(wl)
        rows = sorted({0, wl.batch - 1})
        runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in rows}, ctx_len, fl)
        _ORACLE_CACHE[key] = (wl, weights, mem, ctx_len, fl, runs)
    return _ORACLE_CACHE[key]


@pytest.mark.parametrize("store_logits", [True, False])
@pytest.mark.parametrize("name,tol", FULL)
def test_full_size_configs_on_sampled_rows(name, tol, store_logits):
    """The four bf16 configurations at full size, in the launch configuration the benchmark times
    (CUDA graph, automatic splits); the oracle decodes batch rows 0 and B-1.  store_logits = False is
    the mode the benchmark runs: the logits never leave the vocabulary kernel, so the replay compares
    the active sets of every step, the library's own greedy choices under the margin rule, streams,
    lengths, flags, steps and the trace; store_logits = True adds the logits element by element."""
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl, weights, mem, ctx_len, fl, runs = full_size_case(name, False)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch, store_logits=store_logits)
    mem_dev = dec.device_memory(mem)
    s = parity.replay_compare(dec, wl, mem_dev, ctx_len, fl, runs, use_logits=store_logits)
    assert s["choices"] > 0 and s["max_err"] <= tol
    assert (s["logits"] > 0) == store_logits
    parity.free_run_compare(dec, wl, mem_dev, ctx_len, fl, runs)
    dec.close()
    print(f"{name} store_logits={store_logits}: max logit error {s['max_err']:.3e} over {s['logits']} logits, "
          f"{s['choices']} choices compared, {s['low_margin']} below margin")


@pytest.mark.parametrize("name,tol", FULL)
def test_full_size_configs_with_ragged_contexts(name, tol):
    """Full size again with context lengths drawn from [L/2, L] per sequence (ragged last tiles, unequal
    (sequence, head) segments in cross-attention), logits kept on chip as in the benchmark."""
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl, weights, mem, ctx_len, fl, runs = full_size_case(name, True)
    assert (ctx_len < wl.ctx).any()
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch, store_logits=False)
    s = parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs, use_logits=False)
    assert s["choices"] > 0
    dec.close()


def test_full_size_summarisation_with_e4m3_context_keys_values():
    """The largest configuration with the 8-bit storage of the context keys/values (half of a step's dominant
    byte term), logits element by element against the oracle that quantises likewise."""
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = W.CONFIGS["summarisation"].scaled(kv_c_dtype="e4m3")
    weights, mem = W.make_weights(wl), W.make_encoder_memory(wl)
    ctx_len, fl = W.make_ctx_len(wl, ragged=True), W.make_forced_len(wl)
    runs = parity.oracle_runs(wl, weights, {b: mem[b] for b in (0, wl.batch - 1)}, ctx_len, fl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    s = parity.replay_compare(dec, wl, dec.device_memory(mem), ctx_len, fl, runs)
    assert s["max_err"] <= 2e-2 and s["choices"] > 0
    dec.close()
    print(f"summarisation e4m3: max logit error {s['max_err']:.3e}, {s['choices']} choices, {s['low_margin']} below margin")


@pytest.mark.parametrize("store_logits", [True, False])
def test_bf16_sequential_decoder_shape_of_the_benchmark(store_logits):
    """sub_max = 1 on the concatenated targets - the workload `bench.py` times as the sequential decoder -
    on the bf16 tensor-core kernels: one long subsequence per sequence, page lists of twenty and more pages."""
    import bench
    from paper_2506_23431_b200.binding import PipelinedDecoder
    base = W.CONFIGS["bart_base"]
    swl, sfl = bench.sequential_workload(base, W.make_forced_len(base))
    assert swl.sub_max == 1 and swl.max_sub_len >= 100
    weights, mem, ctx_len = W.make_weights(swl), W.make_encoder_memory(swl), W.make_ctx_len(swl)
    rows = [0, int(np.argmax(sfl[:, 0]))]            # row 0 and the longest stream
    runs = parity.oracle_runs(swl, weights, {b: mem[b] for b in rows}, ctx_len, sfl)
    dec = PipelinedDecoder(swl.hyper(), weights, swl.batch, store_logits=store_logits)
    s = parity.replay_compare(dec, swl, dec.device_memory(mem), ctx_len, sfl, runs, use_logits=store_logits)
    assert s["choices"] > 0 and s["max_err"] <= 2e-2
    dec.close()
