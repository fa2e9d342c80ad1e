"""Pins of the oracle's 8-bit float (E4M3) rounding and of the context key/value quantisation built on
it: the format's value table written out from its definition, ties, saturation, the library's own cast,
and a worked example by hand."""
import numpy as np
import pytest

from oracle import pipelined_decoder as O


def e4m3_table():
    """All finite E4M3 magnitudes from the bit fields: exponent e (4 bits, bias 7), mantissa m (3 bits)."""
    vals = []
    for e in range(16):
        for m in range(8):
            if e == 15 and m == 7:
                continue                                   # the NaN code
            vals.append(2.0 ** -6 * m / 8 if e == 0 else 2.0 ** (e - 7) * (1 + m / 8))
    return np.array(sorted(set(vals)))


def test_grid_values_are_fixed_points_and_the_largest_is_448():
    t = e4m3_table()
    assert len(t) == 127 and t[-1] == 448.0 and t[1] == 2.0 ** -9
    assert np.array_equal(O.e4m3_round(t), t)
    assert np.array_equal(O.e4m3_round(-t), -t)


def test_nearest_with_ties_to_the_even_mantissa_by_brute_force():
    t = e4m3_table()
    g = np.random.default_rng(3)
    x = np.concatenate([g.uniform(0, 448, 20000), g.uniform(0, 0.05, 5000), (t[:-1] + t[1:]) / 2])
    got = O.e4m3_round(x)
    for xi, qi in zip(x, got):
        d = np.abs(t - xi)
        best = np.flatnonzero(d == d.min())
        if len(best) == 1:
            assert qi == t[best[0]]
        else:                                              # a tie: the neighbour whose position in the table is even has the even mantissa
            assert qi == t[[i for i in best if i % 2 == 0][0]]
    assert (np.abs(got - x) <= np.maximum(x, 2.0 ** -6) * 2.0 ** -4 + 1e-300).all()     # half a spacing: 2^-4 relative above 2^-6


def test_saturation_and_signs():
    assert O.e4m3_round(np.array([449.0, 1e9, -500.0, 463.9])).tolist() == [448.0, 448.0, -448.0, 448.0]
    assert O.e4m3_round(np.array([-0.3, 0.3])).tolist() == [-0.3125, 0.3125]


def test_against_the_library_cast():
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("no 8-bit float type in this torch")
    g = np.random.default_rng(11)
    x = np.concatenate([g.standard_normal(50000) * 30, g.standard_normal(20000) * 0.02, g.uniform(-448, 448, 20000)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(O.e4m3_round(x).astype(np.float32), want)


def test_worked_example_of_the_context_quantisation():
    """One head, four positions of one value each (padded to a row): max 448 -> scale 1, so the codes are the
    rounded values themselves: 0.3 -> 0.3125 (grid 0.28125, 0.3125), -17 -> -16 (a tie between 16 and 18:
    16 has the even mantissa), 100 -> 96 (spacing 8 in [64, 128): 96, 104; 100 is a tie, 96 = 64 * 1.5 is
    even).  With max 224 the scale is 0.5 and every value doubles before rounding."""
    col = np.array([448.0, 0.3, -17.0, 100.0])
    deq, scale = O.quantize_context_kv(col.reshape(4, 1), 4)
    assert scale == 1.0 and deq[:, 0].tolist() == [448.0, 0.3125, -16.0, 96.0]
    deq, scale = O.quantize_context_kv((col / 2).reshape(4, 1), 4)
    assert scale == 0.5 and deq[:, 0].tolist() == [224.0, 0.15625, -8.0, 48.0]
    # rows at or beyond the context length take no part in the scale
    deq, scale = O.quantize_context_kv(np.array([[1.0], [3.0], [1000.0]]), 2)
    assert scale == np.float32(3.0) / np.float32(448.0) and deq.shape == (2, 1)
    # error bound: half a grid spacing of the scaled value, i.e. at most 2^-4 of the value (above the subnormals)
    g = np.random.default_rng(5)
    kv = g.standard_normal((300, 64))
    deq, scale = O.quantize_context_kv(kv, 300)
    ref = O.bf16_round(kv.astype(np.float32)).astype(np.float64)
    assert (np.abs(deq - ref) <= np.maximum(np.abs(ref) * 2.0 ** -4, scale * 2.0 ** -10) * (1 + 1e-6)).all()
    assert O.quantize_context_kv(np.zeros((5, 64)), 5)[1] == 1.0


def test_bf16_rounding_is_the_upper_half_of_a_float32_with_ties_to_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -3.14159], dtype=np.float32)
    got = O.bf16_round(x)
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == np.float32(1.0 + 2.0 ** -7) and got[3] == np.float32(1.0 + 2.0 ** -6)
    assert got[4] == np.float32(-3.140625)
    torch = pytest.importorskip("torch")
    g = np.random.default_rng(2)
    y = g.standard_normal(100000).astype(np.float32)
    assert np.array_equal(O.bf16_round(y), torch.from_numpy(y).to(torch.bfloat16).float().numpy())


def test_decoder_with_quantised_context_stays_close_to_the_unquantised_one():
    """The option changes the cross-attention inputs by at most 2^-4 relative per element; on a small random
    decoder the logits move by a small fraction of their spread, and not at all when the option is off."""
    from paper_2506_23431_b200 import workload as W
    wl = W.CONFIGS["tiny"].scaled(n_layers=1, d_model=64, n_heads=1, d_ff=64, vocab=50, ctx=40, sub_max=2, time_max=6,
                                  max_sub_len=3, length_dist=("uniform", 2, 3))
    weights, mem, fl = W.make_weights(wl), W.make_encoder_memory(wl)[0], W.make_forced_len(wl)[0]
    hp = wl.hyper()
    a = O.PipelinedDecoderOracle(weights, hp).run(mem, wl.ctx, fl)
    b = O.PipelinedDecoderOracle(weights, dict(hp, kv_c_dtype="e4m3")).run(mem, wl.ctx, fl)
    c = O.PipelinedDecoderOracle(weights, dict(hp, kv_c_dtype="same")).run(mem, wl.ctx, fl)
    la, lb, lc = a["trace"][0]["logits"], b["trace"][0]["logits"], c["trace"][0]["logits"]
    assert np.array_equal(la, lc)
    assert 0 < np.abs(la - lb).max() < 0.1 * la.std()
