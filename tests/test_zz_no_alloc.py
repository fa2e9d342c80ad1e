"""GPU test of pd_cross_attention_static, the cross-attention entry point for callers that cannot
allocate device memory (its split-K partials live in an array built into the library).  Its output
must equal pd_cross_attention's on the same inputs, on two calls in a row that share the built-in
array, and both must match the CPU oracle's attention.  Collected last on purpose: a failure here
never hides the result of another test."""
import numpy as np
import pytest

from paper_2506_23431_b200 import workload as W

pytestmark = pytest.mark.gpu

TOL = {"bf16": 1e-2, "fp32": 2e-5}     # the tolerances of the stand-alone kernel tests


def _inputs(seed, batch, rows, heads, ctx, dtype):
    import torch
    g = np.random.Generator(np.random.Philox(key=np.array([seed, 91], dtype=np.uint64)))
    hd = heads * 64
    q = g.standard_normal((batch, rows, hd), dtype=np.float32)
    kv = g.standard_normal((batch, heads, 2, ctx, 64), dtype=np.float32)
    n_rows = g.integers(1, rows + 1, size=batch).astype(np.int32)
    ctx_len = g.integers(ctx // 2, ctx + 1, size=batch).astype(np.int32)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = torch.device("cuda", 0)
    if dtype == "bf16":
        q, kv = W.bf16_round(q), W.bf16_round(kv)
    from tests.test_gpu_kernels import oracle_cross
    ref = oracle_cross(q, kv, n_rows, ctx_len, heads, 0.125)
    return (torch.from_numpy(q).to(dev, td), torch.from_numpy(kv).to(dev, td), torch.from_numpy(n_rows).to(dev),
            torch.from_numpy(ctx_len).to(dev), ref)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_static_scratch_variant_matches_the_scratch_argument_variant_twice_in_a_row(dtype):
    import torch
    from paper_2506_23431_b200 import binding as B
    # two different problems back to back: the second call finds the first call's partials in the array
    # (the third has more than 32 rows per sequence: the plain-ALU kernel, whose partials must fit the array too)
    for seed, (batch, rows, heads, ctx, splits) in enumerate([(4, 12, 3, 900, 4), (2, 7, 2, 333, 3), (2, 40, 2, 200, 2)]):
        q, kv, n_rows, ctx_len, ref = _inputs(seed, batch, rows, heads, ctx, dtype)
        want = B.cross_attention(q, kv, n_rows, ctx_len, 0.125, splits)
        got = B.cross_attention_static(q, kv, n_rows, ctx_len, 0.125, splits)
        assert B.cross_attention_static_status() == 0          # synchronises; no bounded wait expired
        err = (got.float() - want.float()).abs().max().item()
        assert np.isfinite(err) and err <= TOL[dtype], f"call {seed}: max abs difference {err:.3e}"
        err_o = np.abs(got.float().cpu().numpy().astype(np.float64) - ref).max()
        assert err_o <= TOL[dtype], f"call {seed}: max abs error against the oracle {err_o:.3e}"


def test_static_scratch_variant_refuses_sizes_beyond_its_array():
    import torch
    from paper_2506_23431_b200 import binding as B
    limit = B.cross_attention_static_max_bytes()
    batch, rows, heads, splits = 64, 32, 16, 8
    assert B.cross_attention_scratch_bytes(batch, rows, heads, splits) > limit
    dev = torch.device("cuda", 0)
    q = torch.zeros(batch, rows, heads * 64, dtype=torch.bfloat16, device=dev)
    kv = torch.zeros(batch, heads, 2, 128, 64, dtype=torch.bfloat16, device=dev)
    n = torch.ones(batch, dtype=torch.int32, device=dev)
    with pytest.raises(B.PdError) as e:
        B.cross_attention_static(q, kv, n, n, 0.125, splits)
    assert e.value.status == -3 and "built-in scratch" in str(e.value)
