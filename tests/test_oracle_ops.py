"""Pins for the fp64 oracle's operators: brute force in pure-Python loops on
tiny shapes, closed forms, invariants and library special cases (torch CPU
fp64 is used here only as an independent check, never as the oracle)."""
import math

import numpy as np
import pytest
import torch

from oracle import ops as O

RNG = np.random.default_rng(1234)


def rnd(*shape):
    return RNG.standard_normal(shape)


# ------------------------------------------------------------------ linear
def test_linear_brute_force():
    for (m, k, n) in [(1, 1, 1), (3, 5, 2), (8, 8, 8), (2, 7, 5)]:
        x, w = rnd(m, k), rnd(k, n)
        y = O.linear(x, w)
        for i in range(m):
            for j in range(n):
                acc = 0.0
                for t in range(k):
                    acc += float(x[i, t]) * float(w[t, j])
                assert abs(y[i, j] - acc) <= 1e-13 * max(1.0, abs(acc))


def test_linear_identity_and_orientation():
    x = rnd(4, 6)
    assert np.array_equal(O.linear(x, np.eye(6)), x)
    # a single 1 at W[k0, n0] routes column k0 of X to column n0 of Y (a
    # transposed weight would route n0 -> k0 instead)
    w = np.zeros((6, 3)); w[4, 1] = 1.0
    y = O.linear(x, w)
    assert np.array_equal(y[:, 1], x[:, 4]) and not y[:, [0, 2]].any()
    with pytest.raises(ValueError):
        O.linear(x, np.zeros((5, 3)))


def test_linear_integer_inputs_exact():
    x = RNG.integers(-4, 5, (9, 33)).astype(np.float64)
    w = RNG.integers(-4, 5, (33, 7)).astype(np.float64)
    ref = (x.astype(np.int64) @ w.astype(np.int64)).astype(np.float64)
    assert np.array_equal(O.linear(x, w), ref)


# ------------------------------------------------------------------ elementwise
def test_bias_relu_scale_clamp_residual():
    x = rnd(5, 4)
    b = rnd(4)
    y = O.bias_add(x, b)
    for i in range(5):
        for j in range(4):
            assert y[i, j] == x[i, j] + b[j]
    with pytest.raises(ValueError):
        O.bias_add(x, rnd(5))
    r = O.relu(x)
    assert (r >= 0).all() and np.array_equal(O.relu(r), r) and np.array_equal(r[x > 0], x[x > 0])
    assert np.array_equal(O.scale(x, 0.5) * 2.0, x)
    c = O.clamp(3 * x, -1.0, 1.0)
    assert c.max() <= 1.0 and c.min() >= -1.0
    inside = np.abs(3 * x) <= 1.0
    assert np.array_equal(c[inside], (3 * x)[inside])
    assert np.array_equal(O.clamp(np.array([-5.0, 0.25, 7.0]), -1.0, 1.0), np.array([-1.0, 0.25, 1.0]))
    assert np.array_equal(O.residual_add(x, -x), np.zeros_like(x))


def test_gelu_erf_pins():
    """The exact GELU is x times the standard normal's distribution function: pinned against scipy's normal CDF and
    torch's own exact GELU (neither uses the oracle's erf call), the odd-part identity, the tails, and the value at 1."""
    from scipy.stats import norm
    x = np.linspace(-6, 6, 2001)
    g = O.gelu_erf(x)
    assert O.gelu_erf(np.array([0.0]))[0] == 0.0
    assert np.allclose(g, x * norm.cdf(x), rtol=1e-13, atol=1e-15)
    assert np.allclose(g, torch.nn.functional.gelu(torch.from_numpy(x)).numpy(), rtol=1e-13, atol=1e-15)
    assert np.allclose(g - O.gelu_erf(-x), x, rtol=0, atol=1e-14)
    assert abs(O.gelu_erf(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15          # Phi(1)
    assert abs(O.gelu_erf(np.array([10.0]))[0] - 10.0) < 1e-12 and abs(O.gelu_erf(np.array([-10.0]))[0]) < 1e-12
    # not the tanh form (up to 5e-4 apart) and not the sigmoid form
    assert 1e-5 < np.abs(g - O.gelu_tanh(x)).max() < 1e-3
    assert np.abs(g - x / (1.0 + np.exp(-1.702 * x))).max() > 5e-3
    # minimum near x = -0.7518 with value -0.1700 (a sign slip in the erf argument moves it to +0.75)
    i = int(np.argmin(g))
    assert abs(x[i] + 0.7518) < 0.01 and abs(g[i] + 0.16997) < 1e-4


def test_gelu_tanh_pins():
    x = np.linspace(-6, 6, 2001)
    g = O.gelu_tanh(x)
    assert O.gelu_tanh(np.array([0.0]))[0] == 0.0
    # odd-part identity: GELU(x) - GELU(-x) = x
    assert np.allclose(g - O.gelu_tanh(-x), x, rtol=0, atol=1e-14)
    # within the known distance of the exact (erf) GELU, but not equal to it
    exact = np.array([0.5 * t * (1.0 + math.erf(t / math.sqrt(2.0))) for t in x])
    d = np.abs(g - exact).max()
    assert 1e-5 < d < 1e-3
    # the sigmoid approximation x*sigmoid(1.702x) is ~1e-2 away: a wrong activation is visible
    sig = x / (1.0 + np.exp(-1.702 * x))
    assert np.abs(g - sig).max() > 5e-3
    # tails
    assert abs(O.gelu_tanh(np.array([10.0]))[0] - 10.0) < 1e-12
    assert abs(O.gelu_tanh(np.array([-10.0]))[0]) < 1e-12
    # library special case
    t = torch.nn.functional.gelu(torch.from_numpy(x), approximate="tanh").numpy()
    assert np.allclose(g, t, rtol=1e-13, atol=1e-15)


def test_silu_swiglu():
    x = np.linspace(-8, 8, 101)
    s = O.silu(x)
    assert O.silu(np.array([0.0]))[0] == 0.0
    # silu(x) - silu(-x) = x ; silu(x) + silu(-x) = x*tanh(x/2)
    assert np.allclose(s - O.silu(-x), x, atol=1e-14, rtol=0)
    assert np.allclose(s + O.silu(-x), x * np.tanh(x / 2), atol=1e-13, rtol=0)
    for xi, si in zip(x, s):
        assert abs(si - xi / (1.0 + math.exp(-xi))) < 1e-14
    gu = rnd(3, 8)
    y = O.swiglu(gu)
    assert y.shape == (3, 4)
    for i in range(3):
        for j in range(4):
            g, u = gu[i, j], gu[i, 4 + j]
            assert abs(y[i, j] - g / (1.0 + math.exp(-g)) * u) < 1e-14
    # gate and up halves are not interchangeable
    assert not np.allclose(y, O.swiglu(np.concatenate([gu[:, 4:], gu[:, :4]], axis=1)))


# ------------------------------------------------------------------ row reductions
def test_layernorm_pins():
    x = rnd(7, 33) * 3 + 2
    g, b = rnd(33), rnd(33)
    eps = 1e-5
    y0 = O.layernorm(x, None, None, eps)
    assert np.allclose(y0.mean(axis=1), 0, atol=1e-14)
    var = x.var(axis=1)  # biased
    assert np.allclose(y0.var(axis=1), var / (var + eps), rtol=1e-12)
    # shift invariance
    assert np.allclose(O.layernorm(x + 17.0, None, None, eps), y0, atol=1e-12)
    # brute force with loops (biased variance, eps inside the root)
    y = O.layernorm(x, g, b, eps)
    for i in range(7):
        mu = sum(float(v) for v in x[i]) / 33
        vv = sum((float(v) - mu) ** 2 for v in x[i]) / 33
        for j in range(33):
            ref = (x[i, j] - mu) / math.sqrt(vv + eps) * g[j] + b[j]
            assert abs(y[i, j] - ref) < 1e-12
    t = torch.nn.functional.layer_norm(torch.from_numpy(x), (33,), torch.from_numpy(g),
                                       torch.from_numpy(b), eps).numpy()
    assert np.allclose(y, t, rtol=1e-12, atol=1e-13)
    # skipping the mean subtraction is a different function
    bad = x / np.sqrt(var + eps)[:, None]
    assert np.abs(bad - y0).max() > 0.1
    # unbiased variance (N-1) is a visibly different function at small N
    small = rnd(4, 5)
    unb = (small - small.mean(1, keepdims=True)) / np.sqrt(small.var(1, ddof=1, keepdims=True) + eps)
    assert np.abs(unb - O.layernorm(small, None, None, eps)).max() > 1e-2


def test_rmsnorm_pins():
    x = rnd(6, 40) * 2 + 0.5
    g = rnd(40)
    eps = 1e-6
    y0 = O.rmsnorm(x, None, eps)
    ms = (x * x).mean(axis=1)
    assert np.allclose((y0 * y0).mean(axis=1), ms / (ms + eps), rtol=1e-12)
    # scale invariance up to eps
    assert np.allclose(O.rmsnorm(64.0 * x, None, 0.0), O.rmsnorm(x, None, 0.0), rtol=1e-13)
    y = O.rmsnorm(x, g, eps)
    for i in range(6):
        m = sum(float(v) ** 2 for v in x[i]) / 40
        for j in range(40):
            assert abs(y[i, j] - x[i, j] / math.sqrt(m + eps) * g[j]) < 1e-13
    # not mean-centred: differs from LayerNorm on shifted data
    assert np.abs(y0 - O.layernorm(x, None, None, eps)).max() > 1e-2


def test_softmax_pins():
    x = rnd(9, 17) * 4
    p = O.softmax(x)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-15)
    assert (p > 0).all()
    assert np.allclose(O.softmax(x + 100.0), p, rtol=1e-12)
    assert np.allclose(O.softmax(np.full((2, 8), 3.3)), 1.0 / 8)
    # two-element rows: the logistic function of the difference
    z = rnd(5, 2)
    assert np.allclose(O.softmax(z)[:, 0], 1.0 / (1.0 + np.exp(-(z[:, 0] - z[:, 1]))), rtol=1e-13)
    # safe for large scores, reduction over the last dimension only
    big = np.array([[1000.0, 1001.0], [-1000.0, -1002.0]])
    pb = O.softmax(big)
    assert np.isfinite(pb).all() and np.allclose(pb.sum(axis=1), 1.0)
    assert not np.allclose(O.softmax(x).sum(axis=0), 1.0)


def test_groupnorm_pins():
    nb, h, w, c, g = 2, 3, 5, 8, 4
    x = rnd(nb, h, w, c) * 2 + 1
    gamma, beta = rnd(c), rnd(c)
    eps = 1e-5
    y0 = O.groupnorm_nhwc(x, None, None, g, eps)
    cg = c // g
    for n in range(nb):
        for gi in range(g):
            blk = y0[n, :, :, gi * cg:(gi + 1) * cg]
            src = x[n, :, :, gi * cg:(gi + 1) * cg]
            assert abs(blk.mean()) < 1e-14
            assert abs(blk.var() - src.var() / (src.var() + eps)) < 1e-12
    # brute force, one (n, g) at a time
    y = O.groupnorm_nhwc(x, gamma, beta, g, eps)
    for n in range(nb):
        for gi in range(g):
            vals = [float(x[n, i, j, ch]) for i in range(h) for j in range(w)
                    for ch in range(gi * cg, (gi + 1) * cg)]
            mu = sum(vals) / len(vals)
            var = sum((v - mu) ** 2 for v in vals) / len(vals)
            for i in range(h):
                for j in range(w):
                    for ch in range(gi * cg, (gi + 1) * cg):
                        ref = (x[n, i, j, ch] - mu) / math.sqrt(var + eps) * gamma[ch] + beta[ch]
                        assert abs(y[n, i, j, ch] - ref) < 1e-12
    # G = 1 is LayerNorm over the flattened (H, W, C) of each image
    ln = O.layernorm(x.reshape(nb, -1), None, None, eps).reshape(x.shape)
    assert np.allclose(O.groupnorm_nhwc(x, None, None, 1, eps), ln, atol=1e-13)
    # G = C is per-channel instance norm
    inst = (x - x.mean(axis=(1, 2), keepdims=True)) / np.sqrt(x.var(axis=(1, 2), keepdims=True) + eps)
    assert np.allclose(O.groupnorm_nhwc(x, None, None, c, eps), inst, atol=1e-13)
    # library special case (NCHW)
    t = torch.nn.functional.group_norm(torch.from_numpy(x).permute(0, 3, 1, 2), g,
                                       torch.from_numpy(gamma), torch.from_numpy(beta), eps)
    assert np.allclose(y, t.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-13)
    with pytest.raises(ValueError):
        O.groupnorm_nhwc(x, None, None, 3, eps)


# ------------------------------------------------------------------ convolution
def test_conv_brute_force():
    nb, h, w, c, co = 1, 4, 5, 3, 2
    x, wt = rnd(nb, h, w, c), rnd(co, 3, 3, c)
    y = O.conv2d_3x3_nhwc(x, wt)
    assert y.shape == (nb, h, w, co)
    for n in range(nb):
        for i in range(h):
            for j in range(w):
                for o in range(co):
                    acc = 0.0
                    for a in range(3):
                        for b in range(3):
                            ii, jj = i + a - 1, j + b - 1
                            if 0 <= ii < h and 0 <= jj < w:
                                for ch in range(c):
                                    acc += float(x[n, ii, jj, ch]) * float(wt[o, a, b, ch])
                    assert abs(y[n, i, j, o] - acc) < 1e-13


def test_conv_padding_delta_and_library():
    nb, h, w, c, co = 2, 5, 6, 4, 3
    y = O.conv2d_3x3_nhwc(np.ones((nb, h, w, c)), np.ones((co, 3, 3, c)))
    assert (y[:, 1:-1, 1:-1] == 9 * c).all()
    assert (y[:, 0, 1:-1] == 6 * c).all() and (y[:, 1:-1, 0] == 6 * c).all()
    assert (y[:, 0, 0] == 4 * c).all() and (y[:, -1, -1] == 4 * c).all()
    # centre-tap kernel is a pure channel mix
    x = rnd(nb, h, w, c)
    mix = rnd(co, c)
    wt = np.zeros((co, 3, 3, c)); wt[:, 1, 1, :] = mix
    assert np.allclose(O.conv2d_3x3_nhwc(x, wt), x @ mix.T, atol=1e-14)
    # off-centre tap: tap (0, 2) reads the pixel one row up, one column right (no flip)
    wt = np.zeros((1, 3, 3, c)); wt[0, 0, 2, 0] = 1.0
    y = O.conv2d_3x3_nhwc(x, wt)
    assert np.array_equal(y[:, 1:, :-1, 0], x[:, :-1, 1:, 0])
    assert not y[:, 0].any() and not y[:, :, -1].any()
    # explicit im2col x GEMM and the library routine
    wt = rnd(co, 3, 3, c)
    yref = O.conv2d_3x3_nhwc(x, wt)
    xp = np.pad(x, ((0, 0), (1, 1), (1, 1), (0, 0)))
    cols = np.stack([xp[:, a:a + h, b:b + w, :] for a in range(3) for b in range(3)], axis=3)
    assert np.allclose(cols.reshape(nb * h * w, 9 * c) @ wt.reshape(co, 9 * c).T,
                       yref.reshape(-1, co), atol=1e-13)
    t = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2),
                                   torch.from_numpy(wt).permute(0, 3, 1, 2), padding=1)
    assert np.allclose(yref, t.permute(0, 2, 3, 1).numpy(), atol=1e-13)


# ------------------------------------------------------------------ attention
def _attn_brute(q, k, v):
    b, h, s, d = q.shape
    out = np.zeros((b * s, h * d))
    for bi in range(b):
        for hi in range(h):
            for i in range(s):
                sc = [sum(float(q[bi, hi, i, t]) * float(k[bi, hi, j, t]) for t in range(d)) / math.sqrt(d)
                      for j in range(i + 1)]
                m = max(sc)
                e = [math.exp(v_ - m) for v_ in sc]
                z = sum(e)
                for t in range(d):
                    out[bi * s + i, hi * d + t] = sum(e[j] / z * float(v[bi, hi, j, t]) for j in range(i + 1))
    return out


def test_attention_brute_force_and_layout():
    b, h, s, d = 2, 3, 7, 4
    q, k, v = rnd(b, h, s, d), rnd(b, h, s, d), rnd(b, h, s, d)
    o = O.attention_causal_bhsd(q, k, v)
    assert o.shape == (b * s, h * d)
    assert np.allclose(o, _attn_brute(q, k, v), atol=1e-13)
    # packed [B*S, 3*H*D] with columns [Q | K | V], head-major
    packed = np.concatenate([t.transpose(0, 2, 1, 3).reshape(b * s, h * d) for t in (q, k, v)], axis=1)
    assert np.allclose(O.attention_causal_packed(packed, b, s, h, d), o, atol=1e-14)


def test_attention_closed_forms():
    b, h, s, d = 1, 2, 16, 8
    q, k, v = rnd(b, h, s, d), rnd(b, h, s, d), rnd(b, h, s, d)
    o = O.attention_causal_bhsd(q, k, v).reshape(b, s, h, d)
    # first query sees only the first key (diagonal kept)
    assert np.allclose(o[:, 0], v[:, :, 0], atol=1e-14)
    # identical keys -> uniform weights -> prefix mean of V
    kk = np.broadcast_to(k[:, :, :1], k.shape).copy()
    o2 = O.attention_causal_bhsd(q, kk, v).reshape(b, s, h, d)
    pm = np.cumsum(v, axis=2) / np.arange(1, s + 1)[None, None, :, None]
    assert np.allclose(o2, pm.transpose(0, 2, 1, 3), atol=1e-13)
    # scaling: q*sqrt(d) with d-scaled definition equals unscaled dot-product softmax
    t = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True)
    assert np.allclose(o, t.permute(0, 2, 1, 3).numpy(), atol=1e-12)
    # output rows are convex combinations of V rows
    assert (o.max(axis=1) <= v.transpose(0, 2, 1, 3).max(axis=1) + 1e-12).all()
    # masking the diagonal, or dropping the mask, gives a different function
    full = np.einsum("bhid,bhjd->bhij", q, k) / math.sqrt(d)
    nomask = (O.softmax(full) @ v).transpose(0, 2, 1, 3)
    assert np.abs(nomask - o).max() > 1e-2


# ------------------------------------------------------------------ unmasked (encoder) attention
def _attn_full_brute(q, k, v):
    b, h, s, d = q.shape
    out = np.zeros((b * s, h * d))
    for bi in range(b):
        for hi in range(h):
            for i in range(s):
                sc = [sum(float(q[bi, hi, i, t]) * float(k[bi, hi, j, t]) for t in range(d)) / math.sqrt(d)
                      for j in range(s)]
                m = max(sc)
                e = [math.exp(v_ - m) for v_ in sc]
                z = sum(e)
                for t in range(d):
                    out[bi * s + i, hi * d + t] = sum(e[j] / z * float(v[bi, hi, j, t]) for j in range(s))
    return out


def test_full_attention_brute_force_and_layout():
    b, h, s, d = 2, 3, 7, 4
    q, k, v = rnd(b, h, s, d), rnd(b, h, s, d), rnd(b, h, s, d)
    o = O.attention_bhsd(q, k, v)
    assert o.shape == (b * s, h * d)
    assert np.allclose(o, _attn_full_brute(q, k, v), atol=1e-13)
    packed = np.concatenate([t.transpose(0, 2, 1, 3).reshape(b * s, h * d) for t in (q, k, v)], axis=1)
    assert np.allclose(O.attention_packed(packed, b, s, h, d), o, atol=1e-14)


def test_full_attention_closed_forms_and_invariants():
    b, h, s, d = 1, 2, 16, 8
    q, k, v = rnd(b, h, s, d), rnd(b, h, s, d), rnd(b, h, s, d)
    o = O.attention_bhsd(q, k, v).reshape(b, s, h, d)
    # library special case
    t = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=False)
    assert np.allclose(o, t.permute(0, 2, 1, 3).numpy(), atol=1e-12)
    # identical keys (or zero queries) -> uniform weights -> every query gets the mean of V
    kk = np.broadcast_to(k[:, :, :1], k.shape).copy()
    mean_v = np.broadcast_to(v.mean(axis=2, keepdims=True), v.shape).transpose(0, 2, 1, 3)
    assert np.allclose(O.attention_bhsd(q, kk, v).reshape(b, s, h, d), mean_v, atol=1e-13)
    assert np.allclose(O.attention_bhsd(np.zeros_like(q), k, v).reshape(b, s, h, d), mean_v, atol=1e-13)
    # keys and values permuted together leave the output unchanged (no mask, no position);
    # the causal operator does not have this invariance
    perm = np.random.default_rng(5).permutation(s)
    assert np.allclose(O.attention_bhsd(q, k[:, :, perm], v[:, :, perm]).reshape(b, s, h, d), o, atol=1e-13)
    oc = O.attention_causal_bhsd(q, k, v).reshape(b, s, h, d)
    assert np.abs(O.attention_causal_bhsd(q, k[:, :, perm], v[:, :, perm]).reshape(b, s, h, d) - oc).max() > 1e-2
    # permuting the queries permutes the output rows
    assert np.allclose(O.attention_bhsd(q[:, :, perm], k, v).reshape(b, s, h, d), o[:, perm], atol=1e-13)
    # the last query of the causal operator sees every key: the two operators agree there and only there
    assert np.allclose(o[:, -1], oc[:, -1], atol=1e-13)
    assert np.abs(o[:, :-1] - oc[:, :-1]).max() > 1e-2
    # one key far ahead of the others takes all the weight: output = its value row
    k2 = k.copy()
    q2 = np.ones_like(q)
    k2[:, :, :, :] = 0.0
    k2[:, :, 5, :] = 100.0
    assert np.allclose(O.attention_bhsd(q2, k2, v).reshape(b, s, h, d), np.broadcast_to(v[:, :, 5][:, None], (b, s, h, d)), atol=1e-12)
    # a shift of every score of a row by a constant (k -> k + c along q's direction is not that; use q . (k + u) with u
    # orthogonal to nothing in particular) changes nothing when the shift is the same for all keys: add a vector to all keys
    u = rnd(d)
    assert np.allclose(O.attention_bhsd(q, k + u, v).reshape(b, s, h, d), o, atol=1e-12)
    # linear in V
    v2 = rnd(b, h, s, d)
    lin = O.attention_bhsd(q, k, 2.0 * v - 3.0 * v2) - (2.0 * O.attention_bhsd(q, k, v) - 3.0 * O.attention_bhsd(q, k, v2))
    assert np.abs(lin).max() < 1e-12


# ------------------------------------------------------------------ pooling
def test_pooling_brute_force_library_and_invariants():
    n, h, w, c = 2, 7, 9, 3
    x = rnd(n, h, w, c)
    for k, st in ((2, 2), (3, 2), (3, 1), (7, 7), (1, 1)):
        oh, ow = (h - k) // st + 1, (w - k) // st + 1
        avg = O.avgpool_nhwc(x, k, st)
        mx = O.maxpool_nhwc(x, k, st)
        l2 = O.lppool_nhwc(x, k, st, 2.0)
        l3 = O.lppool_nhwc(x, k, st, 3.0)
        assert avg.shape == mx.shape == l2.shape == (n, oh, ow, c)
        # brute force, one output at a time
        for ni in range(n):
            for i in range(oh):
                for j in range(ow):
                    for ci in range(c):
                        win = [float(x[ni, i * st + a, j * st + b, ci]) for a in range(k) for b in range(k)]
                        assert abs(avg[ni, i, j, ci] - sum(win) / len(win)) < 1e-13
                        assert mx[ni, i, j, ci] == max(win)
                        assert abs(l2[ni, i, j, ci] - math.sqrt(sum(v * v for v in win))) < 1e-13
                        assert abs(l3[ni, i, j, ci] - sum(abs(v) ** 3 for v in win) ** (1 / 3)) < 1e-13
        # library routines (NCHW)
        t = torch.from_numpy(x).permute(0, 3, 1, 2)
        assert np.allclose(avg, torch.nn.functional.avg_pool2d(t, k, st).permute(0, 2, 3, 1).numpy(), atol=1e-14)
        assert np.array_equal(mx, torch.nn.functional.max_pool2d(t, k, st).permute(0, 2, 3, 1).numpy())
        assert np.allclose(l2, torch.nn.functional.lp_pool2d(t, 2.0, k, st).permute(0, 2, 3, 1).numpy(), atol=1e-13)
        # invariants: max >= mean; p-norms decrease in p and are bounded below by the largest magnitude
        assert (mx >= avg - 1e-15).all()
        amax = O.maxpool_nhwc(np.abs(x), k, st)
        l1 = O.lppool_nhwc(x, k, st, 1.0)
        assert (l1 >= l2 - 1e-12).all() and (l2 >= l3 - 1e-12).all() and (l3 >= amax - 1e-12).all()
        assert np.allclose(l1, k * k * O.avgpool_nhwc(np.abs(x), k, st), atol=1e-13)
        l20 = O.lppool_nhwc(x, k, st, 20.0)                                            # p -> infinity tends to the maximum:
        assert (l20 >= amax * (1 - 1e-12)).all() and (l20 <= amax * (k * k) ** (1 / 20.0) * (1 + 1e-12)).all()
    # a constant image: mean and max return the constant, the p-norm k^(2/p) times it
    cst = np.full((1, 6, 6, 2), 1.5)
    assert np.allclose(O.avgpool_nhwc(cst, 3, 3), 1.5) and np.allclose(O.maxpool_nhwc(cst, 3, 3), 1.5)
    assert np.allclose(O.lppool_nhwc(cst, 3, 3, 2.0), 1.5 * 3.0)
    # the rows and columns that no whole window covers are dropped (floor), not padded
    assert O.avgpool_nhwc(rnd(1, 8, 8, 1), 3, 2).shape == (1, 3, 3, 1)
    with pytest.raises(ValueError):
        O.avgpool_nhwc(rnd(1, 2, 2, 1), 3, 1)


def test_linear_fp8_block_scaled():
    """Block-scaled fp8 contraction: brute force with the scale looked up per element, the special case of unit
    scales (the plain linear), a single non-zero activation (pins which scale multiplies which block, and the
    [N-block, K-block] orientation of the weight scales), homogeneity in every scale, exact integers."""
    rng = np.random.default_rng(5)
    blk = 4
    M, K, N = 5, 12, 10                       # 3 K blocks, 3 N blocks (the last one partial)
    xq = rng.integers(-8, 9, (M, K)).astype(np.float64) / 4
    wq = rng.integers(-8, 9, (K, N)).astype(np.float64) / 8
    sx = rng.uniform(0.5, 2.0, (M, K // blk))
    sw = rng.uniform(0.5, 2.0, (-(-N // blk), K // blk))
    y = O.linear_fp8_block(xq, sx, wq, sw, block=blk)
    assert y.shape == (M, N)
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += (xq[m, k] * sx[m, k // blk]) * (wq[k, n] * sw[n // blk, k // blk])
            assert abs(y[m, n] - acc) < 1e-12
    # unit scales: the plain contraction
    one_x, one_w = np.ones_like(sx), np.ones_like(sw)
    assert np.array_equal(O.linear_fp8_block(xq, one_x, wq, one_w, block=blk), O.linear(xq, wq))
    # one non-zero activation: row m0 of the result is a * sx[m0, kb0] * sw[:, kb0] (per column block) * wq[k0, :]
    m0, k0 = 3, 6
    e = np.zeros_like(xq)
    e[m0, k0] = 1.5
    y1 = O.linear_fp8_block(e, sx, wq, sw, block=blk)
    want = 1.5 * sx[m0, k0 // blk] * np.repeat(sw[:, k0 // blk], blk)[:N] * wq[k0]
    assert np.allclose(y1[m0], want, rtol=0, atol=1e-14) and not y1[np.arange(M) != m0].any()
    # a transposed scale table would change the answer (the two block counts differ only when N != K; here they are equal: use values)
    assert not np.allclose(O.linear_fp8_block(xq, sx, wq, sw.T.copy(), block=blk), y)
    # homogeneity: doubling one activation scale doubles that (row, K block)'s contribution only
    sx2 = sx.copy()
    sx2[1, 2] *= 2
    d = O.linear_fp8_block(xq, sx2, wq, sw, block=blk) - y
    contrib = (xq[1, 8:12] * sx[1, 2]) @ (wq[8:12] * np.repeat(sw[:, 2], blk)[:N])
    assert np.allclose(d[1], contrib, atol=1e-13) and not d[np.arange(M) != 1].any()
    # integers with power-of-two scales: exact
    xi = rng.integers(-4, 5, (M, K)).astype(np.float64)
    wi = rng.integers(-4, 5, (K, N)).astype(np.float64)
    s2 = 2.0 ** rng.integers(-2, 3, sx.shape)
    w2 = 2.0 ** rng.integers(-2, 3, sw.shape)
    yi = O.linear_fp8_block(xi, s2, wi, w2, block=blk)
    brute = np.zeros((M, N))
    for kb in range(K // blk):
        part = xi[:, kb * blk:(kb + 1) * blk] @ wi[kb * blk:(kb + 1) * blk]
        brute += part * s2[:, kb:kb + 1] * np.repeat(w2[:, kb], blk)[:N][None, :]
    assert np.array_equal(yi, brute)
    # the default block is the task's 128
    big = O.linear_fp8_block(np.ones((2, 256)), np.array([[1.0, 3.0], [2.0, 1.0]]), np.ones((256, 130)),
                             np.array([[1.0, 1.0], [1.0, 10.0]]))
    assert np.array_equal(big[:, 0], [128 + 384, 256 + 128]) and np.array_equal(big[:, 129], [128 + 3840, 256 + 1280])
    with pytest.raises(AssertionError):
        O.linear_fp8_block(np.ones((2, 100)), np.ones((2, 1)), np.ones((100, 4)), np.ones((1, 1)))
