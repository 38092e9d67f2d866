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


def test_e4m3_codec():
    """fp8 e4m3 (the variant without infinities): every code's value from the format's definition, round to
    nearest even on conversion, saturation at 448, and torch's conversion as a second opinion."""
    t = G.E4M3_VALUES
    assert t[0x00] == 0 and t[0x80] == 0 and np.isnan(t[0x7F]) and np.isnan(t[0xFF]) and np.isnan(t).sum() == 2
    assert t[0x7E] == 448 and t[0xFE] == -448                 # largest finite: (1 + 6/8) * 2^8
    assert t[0x01] == 2.0 ** -9 and t[0x07] == 7 * 2.0 ** -9  # subnormals
    assert t[0x08] == 2.0 ** -6 and t[0x38] == 1.0 and t[0x3C] == 1.5 and t[0x40] == 2.0
    assert (np.diff(t[:0x7F]) > 0).all()                      # codes are ordered like their values
    # every finite code survives a round trip
    codes = np.array([b for b in range(256) if (b & 0x7F) != 0x7F and (b & 0x7F) != 0], np.uint8)
    assert np.array_equal(G.f32_to_e4m3_bits(t[codes].astype(np.float32)), codes)
    # ties go to the even mantissa; values past 448 saturate
    x = np.array([1.0625, 1.1875, 17.0, 19.0, 448.0, 464.0, 1000.0, -1000.0, 2.0 ** -10, 3 * 2.0 ** -10, 0.0], np.float32)
    want = np.array([1.0, 1.25, 16.0, 20.0, 448.0, 448.0, 448.0, -448.0, 0.0, 2 * 2.0 ** -9, 0.0])
    assert np.array_equal(G.e4m3_bits_to_f64(G.f32_to_e4m3_bits(x)), want)
    import torch
    r = (np.random.default_rng(1).standard_normal(20000) * 60).astype(np.float32)
    r = np.clip(r, -448, 448)
    tt = torch.from_numpy(r).to(torch.float8_e4m3fn)
    assert np.array_equal(G.f32_to_e4m3_bits(r), tt.view(torch.uint8).numpy())
    assert np.array_equal(G.e4m3_bits_to_f64(tt.view(torch.uint8).numpy()), tt.to(torch.float64).numpy())


def test_block_quantisation_recipe():
    w = W.c8(0, M=64, K=384, N=200)
    xq, sx = w.inputs["xq"], w.inputs["sx"]
    assert xq.dtype == "fp8" and xq.shape == (64, 384) and sx.dtype == "f32" and sx.shape == (64, 3)
    assert w.params["Wq"].shape == (384, 200) and w.params["sw"].shape == (2, 3)
    # every (row, block) of the activations uses the whole code range: its largest magnitude is 448
    a = np.abs(xq.f64()).reshape(64, 3, 128).max(axis=2)
    assert (a == 448).all()
    # dequantised values are close to what was quantised (relative step of e4m3: 2^-4 at worst)
    x = G._normal(0, 0, (64, 384)).astype(np.float64)
    back = xq.f64() * np.repeat(sx.f64(), 128, axis=1)
    assert np.abs(back - x).max() <= np.abs(x).max() * 2.0 ** -4
