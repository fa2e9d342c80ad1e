"""The teacher-forced forward of Section 3.3 (Eq. 6) on the GPU against the oracle's dense-mask forward: every
row's logits (the whole target in one pass), the per-row log-probabilities of the targets and the loss."""
import numpy as np
import pytest

from oracle import pipelined_decoder as O
from paper_2506_23431_b200 import workload as W

pytestmark = pytest.mark.gpu

SMALL = dict(n_layers=2, d_model=128, n_heads=2, d_ff=256, vocab=700, norm_gain_std=0.1)


def targets_of(wl):
    """Seeded targets: content tokens of every subsequence (lengths from the workload's draw, some empty)."""
    fl = W.make_forced_len(wl)
    toks = W.make_random_tokens(wl, (wl.batch, wl.sub_max, wl.max_sub_len))
    g = np.random.Generator(np.random.Philox(key=np.array([wl.seed, 4242], dtype=np.uint64)))
    n_sub = g.integers(1, wl.sub_max + 1, size=wl.batch)
    return [[toks[b, i, :fl[b, i]].tolist() for i in range(n_sub[b])] for b in range(wl.batch)]


def run_case(wl, tol):
    import torch
    from paper_2506_23431_b200.binding import PipelinedDecoder
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl, ragged=True)
    subs = targets_of(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    dec.encode_context(dec.device_memory(mem), ctx_len, None)
    lp, loss, logits = dec.teacher_forward(subs, want_logits=True)
    lp2, loss2, none = dec.teacher_forward(subs, want_logits=False)            # logits in chunks inside the scratch
    assert none is None and np.array_equal(lp, lp2) and loss == loss2
    got = logits.cpu().numpy().astype(np.float64)
    orc = O.PipelinedDecoderOracle(weights, wl.hyper())
    r0, want_loss, worst = 0, 0.0, 0.0
    for b in range(wl.batch):
        ref = orc.teacher_forward(mem[b], int(ctx_len[b]), subs[b])
        n = len(ref["rows"])
        err = np.abs(got[r0:r0 + n] - ref["logits"]).max()
        worst = max(worst, err)
        assert err <= tol, f"sequence {b}: logit error {err:.3e}"
        assert np.abs(lp[r0:r0 + n] - ref["logprob"]).max() <= 2 * tol
        want_loss += ref["loss"]
        r0 += n
    assert r0 == len(lp)
    assert abs(loss - want_loss) <= 2 * tol * len(lp)
    # the decode state is untouched: a decode after the forward still runs
    dec.encode_context(dec.device_memory(mem), ctx_len, W.make_forced_len(wl))
    dec.run()
    dec.close()
    return worst


@pytest.mark.parametrize("pos_mode", [W.POS_T5_BIAS, W.POS_ROPE])
def test_teacher_forward_small(pos_mode):
    wl = W.CONFIGS["bart_base"].scaled(name="tf_small", batch=3, ctx=200, sub_max=6, delta_t=2, max_sub_len=40,
                                       length_dist=("uniform", 0, 40), time_max=120, pos_mode=pos_mode, **SMALL)
    assert run_case(wl, 2e-2) < 2e-2


def test_teacher_forward_8_bit_context_and_many_groups():
    """More than 256 row groups (several cross-attention launches) and the 8-bit context keys/values."""
    wl = W.CONFIGS["keyphrase"].scaled(name="tf_groups", batch=20, ctx=144, sub_max=24, delta_t=1, max_sub_len=30,
                                       length_dist=("uniform", 10, 30), time_max=60, pos_mode=W.POS_T5_BIAS, kv_c_dtype="e4m3",
                                       **dict(SMALL, n_layers=1, vocab=300))
    assert run_case(wl, 2e-2) < 2e-2


def test_teacher_forward_rejects_what_it_cannot_run():
    from paper_2506_23431_b200.binding import PipelinedDecoder, PdError
    wl = W.CONFIGS["tiny"].scaled(vocab=300)
    weights, mem = W.make_weights(wl), W.make_encoder_memory(wl)
    dec = PipelinedDecoder(wl.hyper(), weights, 1)
    with pytest.raises(PdError) as e:
        dec.batch = 1
        dec.teacher_forward([[[5, 6]]])
    assert e.value.status == -2                      # before pd_encode_context
    dec.encode_context(dec.device_memory(mem), [wl.ctx], None)
    with pytest.raises(PdError) as e:
        dec.teacher_forward([[[5, 6]]])
    assert e.value.status == -7                      # fp32 path
    dec.close()


def test_teacher_forward_full_size_summarisation_on_sampled_sequences():
    """The largest configuration: the targets the benchmark decodes (11 489 rows), the oracle's forward of batch
    rows 0 and B-1 against the corresponding rows of the one-pass result."""
    from paper_2506_23431_b200.binding import PipelinedDecoder
    wl = W.CONFIGS["summarisation"]
    weights, mem, ctx_len = W.make_weights(wl), W.make_encoder_memory(wl), W.make_ctx_len(wl)
    fl = W.make_forced_len(wl)
    toks = W.make_random_tokens(wl, (wl.batch, wl.sub_max, wl.max_sub_len))
    subs = [[toks[b, i, :fl[b, i]].tolist() for i in range(wl.sub_max)] for b in range(wl.batch)]
    dec = PipelinedDecoder(wl.hyper(), weights, wl.batch)
    dec.encode_context(dec.device_memory(mem), ctx_len, None)
    lp, loss, logits = dec.teacher_forward(subs, want_logits=True)
    assert len(lp) == int((fl + 1).sum()) and np.isfinite(lp).all() and abs(loss + float(lp.astype(np.float64).sum())) < 1e-3 * abs(loss)
    row0 = np.concatenate([[0], np.cumsum((fl + 1).sum(axis=1))])
    orc = O.PipelinedDecoderOracle(weights, wl.hyper())
    for b in (0, wl.batch - 1):
        ref = orc.teacher_forward(mem[b], int(ctx_len[b]), subs[b])
        got = logits[int(row0[b]):int(row0[b + 1])].cpu().numpy().astype(np.float64)
        err = np.abs(got - ref["logits"]).max()
        assert err <= 2e-2, f"sequence {b}: logit error {err:.3e}"
        assert np.abs(lp[int(row0[b]):int(row0[b + 1])] - ref["logprob"]).max() <= 4e-2
    dec.close()
