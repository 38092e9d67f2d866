"""The seeded generator: determinism, storage rounding, distributions."""
import numpy as np

import workloads as W
from workloads import generate as G


def test_bf16_round_to_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 (even mantissa) and 1 + 2^-7: goes to 1.0
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0],
                 np.float32)
    b = W.f32_to_bf16_bits(x)
    back = W.bf16_bits_to_f64(b)
    assert back[0] == 1.0 and back[1] == 1.0
    assert back[2] == 1.0 + 2.0 ** -7
    assert back[3] == 1.0 + 2.0 ** -6       # tie, odd mantissa rounds up to even
    assert back[4] == -2.5 and back[5] == 0.0
    # matches torch's conversion on random data
    import torch
    r = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    t = torch.from_numpy(r).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(W.f32_to_bf16_bits(r), t)


def test_deterministic_and_independent_streams():
    a, b = W.c2(0, 64, 32, 48), W.c2(0, 64, 32, 48)
    for k in a.params:
        assert np.array_equal(a.params[k].store, b.params[k].store)
    assert not np.array_equal(W.c2(1, 64, 32, 48).inputs["x"].store, a.inputs["x"].store)
    # changing X's shape leaves the bias draw untouched
    assert np.array_equal(W.c2(0, 8, 32, 48).params["bias"].store, a.params["bias"].store)


def test_distributions():
    w = W.c1(0)
    assert w.inputs["x"].shape == (64, 256) and w.params["W"].shape == (256, 128)
    x = w.inputs["x"].f64()
    assert abs(x.mean()) < 0.05 and abs(x.std() - 1) < 0.05
    assert abs(w.params["W"].f64().std() - (1 / 256) ** 0.5) < 0.002
    b = w.params["b"].f64()
    assert b.min() > -0.1 and b.max() < 0.1
    w3 = W.c3(0, NB=1, H=8, W=8)
    assert abs(w3.params["gamma"].f64().mean() - 1.0) < 0.01
    assert abs(w3.params["Wc"].f64().std() - (1 / 1152) ** 0.5) < 0.002
    w2 = W.c2(0, 8, 8, 4096)
    assert abs(w2.params["bias"].f64().std() - 0.02) < 0.002


def test_int_valued_exact_in_bf16():
    t = W.int_valued(3, 0, (50, 50), -4, 4, "bf16")
    v = t.f64()
    assert np.array_equal(v, np.round(v)) and v.min() >= -4 and v.max() <= 4


def test_flop_counts_match_the_workload_table():
    assert G.c1().flops == 2 * 64 * 256 * 128
    w4 = G.c4(0, B=1, H=2, S=8, D=4)          # causal work counts the exact j <= i triangle
    assert w4.flops == 4 * 1 * 2 * 4 * (8 * 9 / 2) + 2 * 8 * 8 * 8
