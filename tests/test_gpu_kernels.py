"""Per-kernel GPU tests: single steps of the decode path, called through the C ABI on their own,
against the corresponding function of the CPU fp64 oracle."""
import numpy as np
import pytest

from oracle import pipelined_decoder as O
from paper_2506_23431_b200 import workload as W

pytestmark = pytest.mark.gpu


def cross_case(seed, batch, rows, heads, ctx, dtype, poison=True):
    """Seeded queries / context keys+values; returns float32 host arrays (bf16-representable for
    bf16), row counts and ragged context lengths."""
    g = np.random.Generator(np.random.Philox(key=np.array([seed, 77], dtype=np.uint64)))
    hd = heads * 64
    q = g.standard_normal((batch, rows, hd), dtype=np.float32)
    kv = g.standard_normal((batch, heads, 2, ctx, 64), dtype=np.float32)     # keys, then values, per head
    if dtype == "bf16":
        q, kv = W.bf16_round(q), W.bf16_round(kv)
    n_rows = g.integers(0, rows + 1, size=batch).astype(np.int32)
    n_rows[0] = rows
    if batch > 2:
        n_rows[1] = 0                                  # a sequence with nothing active
    ctx_len = g.integers(1, ctx + 1, size=batch).astype(np.int32)
    ctx_len[0] = ctx
    if poison:                                         # positions beyond ctx_len must never matter
        for b in range(batch):
            kv[b, :, :, ctx_len[b]:] = np.nan
    return q, kv, n_rows, ctx_len


def oracle_cross(q, kv, n_rows, ctx_len, heads, scale):
    batch, rows, hd = q.shape
    out = np.zeros((batch, rows, hd), dtype=np.float64)
    for b in range(batch):
        S, n = int(n_rows[b]), int(ctx_len[b])
        if S == 0:
            continue
        K = kv[b, :, 0, :n].astype(np.float64)
        V = kv[b, :, 1, :n].astype(np.float64)
        qq = q[b, :S].astype(np.float64).reshape(S, heads, 64)
        out[b, :S] = O.masked_attention(qq, K, V, np.ones((S, n), dtype=bool), scale, None).reshape(S, hd)
    return out


CASES = [
    # dtype, batch, rows, heads, ctx, splits, tolerance
    ("bf16", 3, 16, 2, 700, 1, 1e-2),      # tensor-core kernel, several 128-key tiles, ragged tails
    ("bf16", 4, 9, 3, 1000, 4, 1e-2),      # split-K over the context + merge
    ("bf16", 2, 30, 1, 257, 2, 1e-2),      # two 16-row query tiles, one key past a tile edge
    ("bf16", 2, 40, 1, 130, 3, 1e-2),      # more than 32 rows: CUDA-core kernel
    ("fp32", 3, 5, 2, 300, 1, 2e-5),
    ("fp32", 2, 7, 2, 190, 5, 2e-5),
]


@pytest.mark.parametrize("dtype,batch,rows,heads,ctx,splits,tol", CASES)
def test_cross_attention_kernel_against_oracle(dtype, batch, rows, heads, ctx, splits, tol):
    import torch
    from paper_2506_23431_b200 import binding as B
    q, kv, n_rows, ctx_len = cross_case(11, batch, rows, heads, ctx, dtype)
    scale = 0.125
    ref = oracle_cross(q, kv, n_rows, ctx_len, heads, scale)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = torch.device("cuda", 0)
    out = B.cross_attention(torch.from_numpy(q).to(dev, td), torch.from_numpy(kv).to(dev, td),
                            torch.from_numpy(n_rows).to(dev), torch.from_numpy(ctx_len).to(dev), scale, splits)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    for b in range(batch):
        assert not got[b, n_rows[b]:].any(), "unused rows must come back as zeros"
    err = np.abs(got - ref).max()
    assert err <= tol, f"max abs error {err:.3e} > {tol:g}"


@pytest.mark.parametrize("dtype,rows", [("bf16", 6), ("fp32", 6), ("bf16", 36)])
def test_cross_attention_clamps_counts_it_reads_from_the_device(dtype, rows):
    """Row counts and context lengths are device arrays the host wrapper cannot check.  Values beyond
    the tensors' extents are clamped where they are read: the sequence is computed with rows_per_seq rows
    and max_ctx positions, and nothing outside its own rows of `out` changes.  (The bad values sit on
    sequence 0 of a larger allocation, so even an unclamped kernel would stay inside allocated memory.)"""
    import torch
    from paper_2506_23431_b200 import binding as B
    batch, heads, ctx = 3, 2, 150
    q, kv, n_rows, ctx_len = cross_case(31, batch, rows, heads, ctx, dtype, poison=False)
    n_rows[:] = [rows, rows - 2, rows]
    ctx_len[:] = [ctx, ctx - 17, ctx]
    ref = oracle_cross(q, kv, n_rows, ctx_len, heads, 0.125)
    bad_rows, bad_ctx = n_rows.copy(), ctx_len.copy()
    bad_rows[0], bad_ctx[0] = rows + 9, ctx + 1000
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = torch.device("cuda", 0)
    q_d, kv_d = torch.from_numpy(q).to(dev, td), torch.from_numpy(kv).to(dev, td)
    # the call sees the first two sequences of the three allocated
    out = B.cross_attention(q_d[:2], kv_d[:2], torch.from_numpy(bad_rows[:2]).to(dev), torch.from_numpy(bad_ctx[:2]).to(dev), 0.125, 2)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    tol = 1e-2 if dtype == "bf16" else 2e-5
    assert np.abs(got - ref[:2]).max() <= tol
    assert not got[1, n_rows[1]:].any()


def test_cross_attention_rejects_bad_arguments():
    import ctypes as C
    import torch
    from paper_2506_23431_b200 import binding as B
    dev = torch.device("cuda", 0)
    q = torch.zeros(1, 4, 64, device=dev)
    kv = torch.zeros(1, 1, 2, 8, 64, device=dev)
    n = torch.ones(1, dtype=torch.int32, device=dev)
    small = torch.empty(256, dtype=torch.uint8, device=dev)
    with pytest.raises(B.PdError) as e:
        B.cross_attention(q, kv, n, n, 0.125, splits=4, scratch=small)
    assert e.value.status == -3
    with pytest.raises(B.PdError) as e:
        B.cross_attention(q, kv, n, n, 0.125, splits=33)
    assert e.value.status == -1
    assert B.cross_attention_scratch_bytes(1, 65, 1, 1) == 0
    assert B._lib.pd_cross_attention(0, 1, 4, 1, 8, C.c_float(0.125), 1, None, None, None, None, None, None, 0, None) == -1


VOCAB_CASES = [
    # rows, d_model, vocab
    (100, 64, 224),        # one row tile, one vocabulary slice, a single K block
    (200, 256, 1000),      # two row tiles (ragged), five slices, the last one partly beyond the vocabulary
    (600, 1024, 5000),     # five row tiles: three passes over every slice
    (1, 64, 8),            # the smallest shapes: one row, eight ids
    (257, 128, 225),       # one row and one id beyond a tile edge: second pass with a single row, second slice with one id
    (513, 192, 449),       # three K blocks, three passes, three slices
]


@pytest.mark.parametrize("rows,d_model,vocab", VOCAB_CASES)
def test_vocab_argmax_kernel_against_oracle(rows, d_model, vocab):
    """Eq. 4's greedy choice on the tensor-core kernel: logits against the fp64 product of the same
    bf16 inputs, ids against the oracle's select_token wherever its top-2 margin is above 1e-3."""
    import torch
    from paper_2506_23431_b200 import binding as B
    g = np.random.Generator(np.random.Philox(key=np.array([rows, vocab], dtype=np.uint64)))
    hidden = W.bf16_round(g.standard_normal((rows, d_model), dtype=np.float32))
    lm_head = W.bf16_round(0.05 * g.standard_normal((vocab, d_model), dtype=np.float32))
    lm_head[7] = lm_head[3]                                   # an exact tie: the lower id must win
    ref = hidden.astype(np.float64) @ lm_head.astype(np.float64).T
    dev = torch.device("cuda", 0)
    h_d = torch.from_numpy(hidden).to(dev, torch.bfloat16)
    w_d = torch.from_numpy(lm_head).to(dev, torch.bfloat16)
    best_id, best_val, logits = B.vocab_argmax(h_d, w_d, want_logits=True)
    id_only, _, none = B.vocab_argmax(h_d, w_d, want_logits=False)
    torch.cuda.synchronize()
    assert none is None
    got = logits.cpu().numpy().astype(np.float64)
    tol = 1e-4 * max(1.0, np.abs(ref).max())
    assert np.abs(got - ref).max() <= tol
    assert np.abs(best_val.cpu().numpy() - ref.max(axis=1)).max() <= tol
    ids = best_id.cpu().numpy()
    assert (id_only.cpu().numpy() == ids).all(), "writing the logits or not must not change the choice"
    assert not (ids == 7).any()
    top2 = np.sort(ref, axis=1)[:, -2:]
    for r in range(rows):
        row = ref[r].copy()
        row[7] = -np.inf                                      # the tie's higher id can never be chosen
        if np.sort(row)[-1] - np.sort(row)[-2] > 1e-3:
            tok, _ = O.select_token(ref[r], 0, None, 10 ** 9, -1, -1)
            assert ids[r] == tok, f"row {r}: {ids[r]} != {tok} (margin {top2[r, 1] - top2[r, 0]:.3e})"


def test_vocab_argmax_rejects_bad_arguments():
    import torch
    from paper_2506_23431_b200 import binding as B
    dev = torch.device("cuda", 0)
    h = torch.zeros(4, 96, device=dev, dtype=torch.bfloat16)           # width not a multiple of 64
    w = torch.zeros(10, 96, device=dev, dtype=torch.bfloat16)
    with pytest.raises(B.PdError) as e:
        B.vocab_argmax(h, w)
    assert e.value.status == -1
    h = torch.zeros(4, 64, device=dev, dtype=torch.bfloat16)
    w = torch.zeros(10, 64, device=dev, dtype=torch.bfloat16)
    with pytest.raises(B.PdError) as e:
        B.vocab_argmax(h, w, scratch=torch.empty(256, dtype=torch.uint8, device=dev))
    assert e.value.status == -3
    assert B._lib.pd_vocab_argmax_scratch_bytes(0, 10) == 0


def test_cross_attention_is_bit_reproducible_after_ragged_tiles():
    """Few, long (sequence, head) segments with ragged context lengths: CTAs take half segments and
    carry on into the next segment after a ragged last tile.  Twenty launches on the same inputs must
    give the same bits (a write into a TMA stage once raced with the next bulk copy here), and those
    bits must match the oracle."""
    import torch
    from paper_2506_23431_b200 import binding as B
    batch, rows, heads, ctx = 9, 3, 8, 4096
    q, kv, n_rows, _ = cross_case(5, batch, rows, heads, ctx, "bf16", poison=False)
    n_rows[:] = rows
    ctx_len = np.array([3256, 3607, 2257, 4079, 3732, 2935, 2640, 3064, 3757], dtype=np.int32)
    for b in range(batch):
        kv[b, :, :, ctx_len[b]:] = np.nan                 # positions beyond ctx_len must never matter
    ref = oracle_cross(q, kv, n_rows, ctx_len, heads, 0.125)
    dev = torch.device("cuda", 0)
    q_d, kv_d = torch.from_numpy(q).to(dev, torch.bfloat16), torch.from_numpy(kv).to(dev, torch.bfloat16)
    nr_d, cl_d = torch.from_numpy(n_rows).to(dev), torch.from_numpy(ctx_len).to(dev)
    first = None
    for _ in range(20):
        out = B.cross_attention(q_d, kv_d, nr_d, cl_d, 0.125, 1)
        torch.cuda.synchronize()
        bits = out.view(torch.int16).cpu().numpy()
        if first is None:
            first = bits
            got = out.float().cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all()
            assert np.abs(got - ref).max() <= 2e-3
        else:
            assert np.array_equal(bits, first), "two launches on the same inputs gave different bits"


RANDOM_SHAPES = [
    # seed, batch, rows, heads, ctx: chosen to reach every way the kernel divides the tile list
    (21, 40, 5, 8, 700),       # 320 segments: whole segments per CTA, two of them for some CTAs
    (22, 12, 9, 8, 1500),      # 96 short segments: one CTA each
    (23, 6, 16, 8, 3300),      # 48 long segments: two CTAs per segment, ragged ends inside the CTAs' ranges
    (24, 2, 30, 4, 2900),      # 8 segments, two query tiles: the tile list cut into many short ranges
    (25, 1, 1, 1, 129),        # one row, one head, one key beyond a tile edge
    (26, 70, 3, 4, 260),       # many sequences with two or three tiles each
]


@pytest.mark.parametrize("seed,batch,rows,heads,ctx", RANDOM_SHAPES)
def test_cross_attention_random_ragged_shapes(seed, batch, rows, heads, ctx):
    """Ragged contexts and row counts (some sequences inactive) on shapes that reach every partition of the
    tile list; NaNs beyond ctx_len; the result must match the oracle and repeat bit for bit."""
    import torch
    from paper_2506_23431_b200 import binding as B
    q, kv, n_rows, ctx_len = cross_case(seed, batch, rows, heads, ctx, "bf16")
    ref = oracle_cross(q, kv, n_rows, ctx_len, heads, 0.125)
    dev = torch.device("cuda", 0)
    args = (torch.from_numpy(q).to(dev, torch.bfloat16), torch.from_numpy(kv).to(dev, torch.bfloat16),
            torch.from_numpy(n_rows).to(dev), torch.from_numpy(ctx_len).to(dev), 0.125, 1)
    outs = []
    for _ in range(4):
        out = B.cross_attention(*args)
        torch.cuda.synchronize()
        outs.append(out)
    got = outs[0].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= 1e-2
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0].view(torch.int16))


LINEAR_SHAPES = [
    # rows, d_in, d_out: the decoder's projection shapes (square, Q/K/V, feed-forward up and down) at both
    # model widths, and row counts on both sides of the 128-row tiles and of the accumulators one pass holds
    (134, 1024, 1024), (1, 1024, 3072), (300, 1024, 4096), (129, 4096, 1024),
    (576, 768, 768), (97, 768, 2304), (260, 768, 3072), (64, 3072, 768),
    (700, 256, 512), (5, 64, 16),
]


@pytest.mark.parametrize("rows,d_in,d_out", LINEAR_SHAPES)
def test_linear_kernel_against_oracle_product(rows, d_in, d_out):
    """The tcgen05 projection kernel against the fp64 product of the same bf16 inputs, in its three
    epilogues: plain (with the RMSNorm scale applied after the product), ReLU, and the residual form
    that also leaves the next norm's inputs.  Tolerance: bf16 output rounding (2^-9 relative) plus fp32
    accumulation over d_in terms."""
    import torch
    from paper_2506_23431_b200 import binding as B
    g = np.random.Generator(np.random.Philox(key=np.array([rows, d_in + d_out], dtype=np.uint64)))
    a = W.bf16_round(g.standard_normal((rows, d_in), dtype=np.float32))
    w = W.bf16_round(0.05 * g.standard_normal((d_in, d_out), dtype=np.float32))
    gain = W.bf16_round(1.0 + 0.1 * g.standard_normal(d_out, dtype=np.float32))
    x0 = g.standard_normal((rows, d_out), dtype=np.float32)
    ssq_in = (g.random(rows, dtype=np.float32) + 0.5) * d_in
    eps = 1e-6
    ref = a.astype(np.float64) @ w.astype(np.float64)
    inv = 1.0 / np.sqrt(ssq_in.astype(np.float64) / d_in + eps)
    dev = torch.device("cuda", 0)
    a_d, w_d = torch.from_numpy(a).to(dev, torch.bfloat16), torch.from_numpy(w).to(dev, torch.bfloat16)
    scale = max(1.0, np.abs(ref).max())

    out = B.linear(a_d, w_d, mode=0).float().cpu().numpy().astype(np.float64)
    assert np.abs(out - ref).max() <= 2.0 ** -8 * scale

    out = B.linear(a_d, w_d, mode=1, row_sumsq=torch.from_numpy(ssq_in).to(dev), eps=eps).float().cpu().numpy().astype(np.float64)
    want = np.maximum(ref * inv[:, None], 0.0)
    assert np.abs(out - want).max() <= 2.0 ** -8 * max(1.0, np.abs(want).max())

    x_d = torch.from_numpy(x0).to(dev)
    outs = []
    for _ in range(2):                                  # twice: the result must repeat bit for bit
        x_d.copy_(torch.from_numpy(x0).to(dev))
        xg, ssq = B.linear(a_d, w_d, mode=2, x=x_d, gain_next=torch.from_numpy(gain).to(dev, torch.bfloat16))
        outs.append((x_d.clone(), xg.clone(), ssq.clone()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1].view(torch.int16), outs[1][1].view(torch.int16))
    x_new = outs[0][0].cpu().numpy().astype(np.float64)
    want_x = x0.astype(np.float64) + ref
    assert np.abs(x_new - want_x).max() <= 1e-4 * max(1.0, np.abs(want_x).max())
    xg = outs[0][1].float().cpu().numpy().astype(np.float64)
    want_g = want_x * gain.astype(np.float64)[None, :]
    assert np.abs(xg - want_g).max() <= 2.0 ** -8 * max(1.0, np.abs(want_g).max())
    ssq = outs[0][2].cpu().numpy().astype(np.float64)
    assert np.isfinite(ssq).all()
    want_s = (want_x ** 2).sum(axis=1)
    assert np.abs(ssq.sum(axis=0) - want_s).max() <= 1e-4 * want_s.max()


def test_linear_rejects_bad_arguments():
    import torch
    from paper_2506_23431_b200 import binding as B
    dev = torch.device("cuda", 0)
    a = torch.zeros(4, 96, device=dev, dtype=torch.bfloat16)            # d_in not a multiple of 64
    w = torch.zeros(96, 64, device=dev, dtype=torch.bfloat16)
    with pytest.raises(B.PdError) as e:
        B.linear(a, w)
    assert e.value.status == -1
    assert B._lib.pd_linear_scratch_bytes(64, 8) == 0
