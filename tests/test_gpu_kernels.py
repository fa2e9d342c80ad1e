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
