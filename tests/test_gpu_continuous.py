"""Continuous batching on the GPU: a queue of sequences decoded through fewer rows, a new sequence admitted
into a row (pd_admit) as soon as the row's sequence has ended.  Algorithm 1 runs per sequence, so every
sequence - whatever step of the shared clock it was admitted at, whatever its neighbours do - must give the
oracle's result for that sequence decoded alone: active sets per step, logits, greedy choices under the margin
rule, streams, lengths, flags, steps and the trace on the sequence's own clock."""
import numpy as np
import pytest

from paper_2506_23431_b200 import workload as W
from tests import parity

pytestmark = pytest.mark.gpu

SMALL = dict(n_layers=2, d_model=128, n_heads=2, d_ff=256, vocab=600, norm_gain_std=0.1)


def queue_replay(wl_rows, n_queue, **dec_kw):
    import torch
    from paper_2506_23431_b200.binding import PipelinedDecoder
    B = wl_rows.batch
    wl_q = wl_rows.scaled(batch=n_queue)                   # the queue's data: same seed family, n_queue sequences
    weights = W.make_weights(wl_rows)
    mem, ctx_len, fl = W.make_encoder_memory(wl_q), W.make_ctx_len(wl_q, ragged=True), W.make_forced_len(wl_q)
    runs = parity.oracle_runs(wl_q, weights, {q: mem[q] for q in range(n_queue)}, ctx_len, fl)
    assert len({r["steps"] for r in runs.values()}) > 2, "the draw should end sequences at different steps"
    dec = PipelinedDecoder(wl_rows.hyper(), weights, B, **dec_kw)
    mem_dev = dec.device_memory(mem)
    tol, hp, sm = parity.TOL[wl_rows.dtype], wl_rows.hyper(), wl_rows.sub_max
    dec.encode_context(mem_dev[:B].contiguous(), ctx_len[:B], fl[:B])
    row_seq, row_t, next_q = list(range(B)), [0] * B, B
    admitted_at, finished, clock = {q: 1 for q in range(B)}, 0, 0
    max_err, n_choices = 0.0, 0
    while any(q is not None for q in row_seq):
        clock += 1
        teacher = np.full((B, sm), -1, np.int32)
        for row, q in enumerate(row_seq):
            if q is not None:
                for i, tok in runs[q]["trace"][row_t[row]]["appended"].items():
                    teacher[row, i - 1] = tok
        dec.step(torch.from_numpy(teacher).to(dec.device))
        logits, row_sub = dec.get_logits()
        logits = logits.reshape(B, dec.rows_per_seq, wl_rows.vocab)
        for row, q in enumerate(row_seq):
            if q is None:
                assert not (row_sub[row] > 0).any(), f"row {row} is empty but active at clock {clock}"
                continue
            step = runs[q]["trace"][row_t[row]]
            act = [int(i) for i in row_sub[row] if i > 0]
            assert act == step["active"], f"sequence {q} step {row_t[row] + 1} (clock {clock}): active {act} vs {step['active']}"
            for c in range(len(act)):
                err = float(np.abs(logits[row, c].astype(np.float64) - step["logits"][c]).max())
                max_err = max(max_err, err)
                assert err <= tol, f"sequence {q} step {row_t[row] + 1} (clock {clock}): logit error {err:.3e}"
            row_t[row] += 1
        for row, q in enumerate(row_seq):
            if q is None or row_t[row] < runs[q]["steps"]:
                continue
            r = runs[q]                                      # the oracle says the sequence has just ended
            done, steps = dec.rows_done()
            assert done[row] == 1 and steps[row] == r["steps"]
            res = dec.collect_row(row)
            assert res["n_sub"] == r["n_sub"] and res["steps"] == r["steps"]
            for i, sub in enumerate(r["subsequences"]):
                n = int(res["lens"][i])
                assert n == len(sub) and res["tokens"][i, :n].tolist() == sub
                assert int(res["flags"][i]) == r["flags"][i]
            trace = dec.get_trace()[:, row]
            for s in r["trace"]:
                assert int(trace[s["t"] - 1]) == sum(1 << (i - 1) for i in s["active"])   # on the sequence's own clock
            assert not trace[r["steps"]:].any()
            chosen = dec.get_chosen()[row]
            emitted = {i: 0 for i in range(1, r["n_sub"] + 1)}
            for s in r["trace"]:
                for c, i in enumerate(s["active"]):
                    n = emitted[i]; emitted[i] += 1
                    forced_sep = n >= int(fl[q][i - 1])
                    barred = [] if forced_sep else [hp["eos_id"], hp["sep_id"]]
                    if forced_sep or parity._margin(s["logits"][c], barred) > parity.MARGIN:
                        assert int(chosen[i - 1, n]) == s["chosen"][i]
                        n_choices += 1
            finished += 1
            if next_q < n_queue:
                dec.admit(row, mem_dev[next_q].contiguous(), int(ctx_len[next_q]), fl[next_q])
                admitted_at[next_q] = clock + 1
                row_seq[row], row_t[row], next_q = next_q, 0, next_q + 1
            else:
                row_seq[row] = None
        assert clock < 50 * wl_rows.time_max
    assert finished == n_queue and dec.done()
    assert len(set(admitted_at.values())) > 2, "sequences should have been admitted at several different clock steps"
    dec.step()                                               # a step after the end is a no-op
    assert dec.done()
    dec.close()
    return max_err, n_choices


@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_queue_of_sequences_through_three_rows_bf16(pos_mode):
    wl = W.CONFIGS["bart_base"].scaled(name="queue_bf16", batch=3, ctx=200, sub_max=5, delta_t=2, max_sub_len=20,
                                       length_dist=("uniform", 1, 20), time_max=60, pos_mode=pos_mode, **SMALL)
    err, n = queue_replay(wl, 9)
    assert err < 2e-2 and n > 100


def test_queue_through_two_rows_fp32_and_8_bit_context():
    wl = W.CONFIGS["tiny"].scaled(name="queue_fp32", batch=2, ctx=96, sub_max=4, delta_t=2, max_sub_len=10,
                                  length_dist=("uniform", 0, 10), time_max=40, vocab=400, norm_gain_std=0.1)
    err, _ = queue_replay(wl, 7, self_splits=2, cross_splits=2)
    assert err < 1e-4
    wl8 = W.CONFIGS["bart_base"].scaled(name="queue_e4m3", batch=2, ctx=208, sub_max=5, delta_t=3, max_sub_len=14,
                                        length_dist=("uniform", 0, 14), time_max=60, pos_mode=W.POS_T5_BIAS, kv_c_dtype="e4m3", **SMALL)
    err, _ = queue_replay(wl8, 6)
    assert err < 2e-2


def test_admit_needs_the_default_pool_and_a_valid_row():
    from paper_2506_23431_b200.binding import PipelinedDecoder, PdError
    wl = W.CONFIGS["tiny"].scaled(batch=2, vocab=300)
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch, pool_pages=64)
    mem_dev = dec.device_memory(mem)
    dec.encode_context(mem_dev, ctx_len, W.make_forced_len(wl))
    with pytest.raises(PdError) as e:
        dec.admit(0, mem_dev[0].contiguous(), wl.ctx, None)
    assert e.value.status == -7
    dec.close()
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    with pytest.raises(PdError) as e:
        dec.admit(0, mem_dev[0].contiguous(), wl.ctx, None)
    assert e.value.status == -2                      # before pd_encode_context
    dec.encode_context(mem_dev, ctx_len, W.make_forced_len(wl))
    with pytest.raises(PdError) as e:
        dec.admit(5, mem_dev[0].contiguous(), wl.ctx, None)
    assert e.value.status == -1
    dec.close()
