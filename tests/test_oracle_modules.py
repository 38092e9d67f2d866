"""Pins for the composed-module oracle: every decomposition of a module gives
the same result; contracts expose exactly the boundary tensors; the paper's
catalogue of typical kernel bugs, injected on the CPU side, is visible to the
parity predicate."""
import numpy as np
import pytest

import workloads as W
from oracle import modules as M
from oracle import ops as O
from oracle.compare import check_close

SMALL = {
    "c1": lambda s: W.c1(s),
    "c2": lambda s: W.c2(s, M=48, K=64, N=40),
    "c3": lambda s: W.c3(s, NB=2, H=6, W=5, C=8, CO=8, G=4),
    "c4": lambda s: W.c4(s, B=2, H=2, S=12, D=8),
    "c5": lambda s: W.c5(s, B=2, S=8, E=16, H=2, F=24, L=2),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_all_decompositions_agree(name):
    w = SMALL[name](0)
    ref, inter = M.run_workload(w, None)           # per-op: every intermediate
    assert np.isfinite(ref).all()
    for pname, cuts in w.partitions.items():
        out, boundary = M.run_workload(w, cuts)
        assert np.array_equal(out, ref), pname
        for k, v in boundary.items():               # local == global intermediates
            assert np.array_equal(v, inter[k])


def test_contracts_cover_fully_and_exclusively():
    w = SMALL["c5"](0)
    cons = M.contracts(w.ops, list(w.inputs), w.partitions["fused_tails"])
    # layer 0: the out-proj + residual submodule reads the attention output and the layer input
    assert cons[3] == (["att_0", "x"], ["x1_0"])
    # gate/up GEMM + SwiGLU keeps gu inside
    assert cons[5] == (["n2_0"], ["hid_0"])
    # down-proj + residual reads the earlier residual stream through a skip edge
    assert cons[6] == (["hid_0", "x1_0"], ["x2_0"])
    for bad in ([1, 2], [0, 0], [0, 3, 2], [0, len(w.ops)], []):
        with pytest.raises(ValueError):
            M.contracts(w.ops, list(w.inputs), bad)
    # fully fused: one submodule, inputs = module inputs, output = module output
    assert M.contracts(w.ops, list(w.inputs), [0]) == [(["x"], ["y"])]


def test_c1_output_rows_are_normalised():
    y, _ = M.run_workload(W.c1(0), [0])
    assert y.shape == (64, 128)
    assert np.allclose(y.mean(axis=1), 0, atol=1e-12)
    assert np.allclose(y.var(axis=1), 1, atol=1e-3)


def test_c2_range_and_c4_c5_shapes():
    y, inter = M.run_workload(SMALL["c2"](0), None)
    assert y.min() >= -1 and y.max() <= 1
    pre = inter["y1"]                                  # x @ W + bias: unit variance by construction
    assert 0.7 < pre.std() < 1.3
    y4, _ = M.run_workload(SMALL["c4"](0), [0])
    assert y4.shape == (2 * 12, 16)
    assert np.allclose((y4 * y4).mean(axis=1), 1, atol=1e-4)   # RMSNorm, gamma = 1
    y5, _ = M.run_workload(SMALL["c5"](0), [0])
    assert y5.shape == (16, 16)
    assert np.allclose((y5 * y5).mean(axis=1), 1, atol=1e-4)


def test_c5_batch_elements_are_independent():
    """Causal attention never mixes batch elements, so an oracle run on a subset of the batch
    is exact for those rows (used to bound the CPU time at the full size)."""
    w = SMALL["c5"](0)
    full, _ = M.run_workload(w, None)
    ops = [dict(o, attrs=dict(o["attrs"])) for o in w.ops]
    for o in ops:
        if o["kind"] == "attention_causal":
            o["attrs"]["batch"] = 1
    x1 = {"x": w.inputs["x"].f64()[8:16]}               # batch element 1
    sub, _ = M.run_module(ops, x1, {k: t.f64() for k, t in w.params.items()}, None)
    assert np.array_equal(sub, full[8:16])


# ------------------------------------------------- composition written out by hand
# The dispatch and the skip edges of `apply_op` / `run_module` are pinned here against modules
# composed by hand, operator by operator, in the order the workload list gives them.  Every named
# intermediate is compared, so a slip in the middle of a chain (a residual added to itself, the
# wrong skip edge, one activation routed to another) cannot hide behind the final norm.
def _widen(w):
    return ({k: t.f64() for k, t in w.inputs.items()}, {k: t.f64() for k, t in w.params.items()})


def _hand_c1(w):
    i, p = _widen(w)
    v = {}
    v["y0"] = O.linear(i["x"], p["W"])
    v["y1"] = O.bias_add(v["y0"], p["b"])
    v["y2"] = O.relu(v["y1"])
    v["y3"] = O.layernorm(v["y2"], p["gamma"], p["beta"], 1e-5)
    return v, "y3"


def _hand_c2(w):
    i, p = _widen(w)
    v = {}
    v["y0"] = O.linear(i["x"], p["W"])
    v["y1"] = O.bias_add(v["y0"], p["bias"])
    v["y2"] = O.gelu_tanh(v["y1"])
    v["y3"] = O.scale(v["y2"], 0.5)
    v["y4"] = O.clamp(v["y3"], -1.0, 1.0)
    return v, "y4"


def _hand_c3(w):
    i, p = _widen(w)
    v = {}
    v["y0"] = O.conv2d_3x3_nhwc(i["x"], p["Wc"])
    v["y1"] = O.bias_add(v["y0"], p["bias"])
    v["y2"] = O.relu(v["y1"])
    v["y3"] = O.groupnorm_nhwc(v["y2"], p["gamma"], p["beta"], 4, 1e-5)
    return v, "y3"


def _hand_c4(w):
    i, p = _widen(w)
    v = {}
    v["a"] = O.attention_causal_bhsd(i["q"], i["k"], i["v"])
    v["p"] = O.linear(v["a"], p["Wo"])
    v["h"] = O.residual_add(v["p"], i["r"])
    v["y"] = O.rmsnorm(v["h"], p["gamma"], 1e-6)
    return v, "y"


def _hand_c5(w, B=2, S=8, H=2, D=8, L=2):
    i, p = _widen(w)
    v = {}
    x = i["x"]
    for l in range(L):
        v[f"n1_{l}"] = O.rmsnorm(x, p["ones"], 1e-6)
        v[f"qkv_{l}"] = O.linear(v[f"n1_{l}"], p[f"Wqkv{l}"])
        v[f"att_{l}"] = O.attention_causal_packed(v[f"qkv_{l}"], B, S, H, D)
        v[f"o_{l}"] = O.linear(v[f"att_{l}"], p[f"Wo{l}"])
        v[f"x1_{l}"] = O.residual_add(v[f"o_{l}"], x)                  # skip edge: the layer's input
        v[f"n2_{l}"] = O.rmsnorm(v[f"x1_{l}"], p["ones"], 1e-6)
        v[f"gu_{l}"] = O.linear(v[f"n2_{l}"], p[f"Wgu{l}"])
        v[f"hid_{l}"] = O.swiglu(v[f"gu_{l}"])
        v[f"d_{l}"] = O.linear(v[f"hid_{l}"], p[f"Wd{l}"])
        v[f"x2_{l}"] = O.residual_add(v[f"d_{l}"], v[f"x1_{l}"])       # skip edge: after attention
        x = v[f"x2_{l}"]
    v["y"] = O.rmsnorm(x, p["ones"], 1e-6)
    return v, "y"


def _hand_c6(w, B=2, S=6, H=2, D=8, L=2):
    i, p = _widen(w)
    v = {}
    x = i["x"]
    for l in range(L):
        v[f"qkv0_{l}"] = O.linear(x, p[f"Wqkv{l}"])
        v[f"qkv_{l}"] = O.bias_add(v[f"qkv0_{l}"], p[f"bqkv{l}"])
        v[f"att_{l}"] = O.attention_packed(v[f"qkv_{l}"], B, S, H, D)
        v[f"o0_{l}"] = O.linear(v[f"att_{l}"], p[f"Wo{l}"])
        v[f"o1_{l}"] = O.bias_add(v[f"o0_{l}"], p[f"bo{l}"])
        v[f"r1_{l}"] = O.residual_add(v[f"o1_{l}"], x)
        v[f"x1_{l}"] = O.layernorm(v[f"r1_{l}"], p[f"g1_{l}"], p[f"g1b_{l}"], 1e-5)
        v[f"h0_{l}"] = O.linear(v[f"x1_{l}"], p[f"W1{l}"])
        v[f"h1_{l}"] = O.bias_add(v[f"h0_{l}"], p[f"b1{l}"])
        v[f"h_{l}"] = O.relu(v[f"h1_{l}"])
        v[f"d0_{l}"] = O.linear(v[f"h_{l}"], p[f"W2{l}"])
        v[f"d1_{l}"] = O.bias_add(v[f"d0_{l}"], p[f"b2{l}"])
        v[f"r2_{l}"] = O.residual_add(v[f"d1_{l}"], v[f"x1_{l}"])
        v[f"x2_{l}"] = O.layernorm(v[f"r2_{l}"], p[f"g2_{l}"], p[f"g2b_{l}"], 1e-5)
        x = v[f"x2_{l}"]
    return v, f"x2_{L - 1}"


def _hand_c7(w, pool):
    i, p = _widen(w)
    v = {}
    v["y0"] = O.conv2d_3x3_nhwc(i["x"], p["Wc"])
    v["y1"] = O.bias_add(v["y0"], p["bias"])
    v["y2"] = O.relu(v["y1"])
    v["y3"] = {"avg": lambda t: O.avgpool_nhwc(t, 3, 2), "max": lambda t: O.maxpool_nhwc(t, 3, 2),
               "lp": lambda t: O.lppool_nhwc(t, 3, 2, 3.0)}[pool](v["y2"])
    return v, "y3"


def _hand_c8(w):
    i, p = _widen(w)
    v = {}
    v["y0"] = O.linear_fp8_block(i["xq"], i["sx"], p["Wq"], p["sw"])
    v["y1"] = O.bias_add(v["y0"], p["bias"])
    v["y2"] = O.silu(v["y1"])
    return v, "y2"


def _hand_c9(w):
    i, p = _widen(w)
    v = {}
    v["a0"] = O.linear(i["x"], p["W1"])            # a LINEAR over the channel dimension of an NHWC tensor
    v["a1"] = O.bias_add(v["a0"], p["b1"])
    v["a2"] = O.relu(v["a1"])
    v["c0"] = O.conv2d_3x3_nhwc(v["a2"], p["Wc"])
    v["c1"] = O.bias_add(v["c0"], p["b2"])
    v["c2"] = O.relu(v["c1"])
    v["d0"] = O.linear(v["c2"], p["W3"])
    v["d1"] = O.bias_add(v["d0"], p["b3"])
    v["d2"] = O.residual_add(v["d1"], i["x"])
    v["y"] = O.relu(v["d2"])
    return v, "y"


HAND = {
    "c9": (lambda s: W.c9(s, NB=2, H=5, W=6, C=16, CM=8), _hand_c9),
    "c8": (lambda s: W.c8(s, M=24, K=256, N=136, bias=True), _hand_c8),
    "c1": (lambda s: W.c1(s), _hand_c1),
    "c2": (lambda s: W.c2(s, M=48, K=64, N=40), _hand_c2),
    "c3": (lambda s: W.c3(s, NB=2, H=6, W=5, C=8, CO=8, G=4), _hand_c3),
    "c4": (lambda s: W.c4(s, B=2, H=2, S=12, D=8), _hand_c4),
    "c5": (lambda s: W.c5(s, B=2, S=8, E=16, H=2, F=24, L=2), _hand_c5),
    "c6": (lambda s: W.c6(s, B=2, S=6, E=16, H=2, F=24, L=2), _hand_c6),
    "c7 avg": (lambda s: W.c7(s, NB=2, H=7, W=6, C=8, CO=8, pool="avg", k=3, stride=2),
               lambda w: _hand_c7(w, "avg")),
    "c7 max": (lambda s: W.c7(s, NB=2, H=7, W=6, C=8, CO=8, pool="max", k=3, stride=2),
               lambda w: _hand_c7(w, "max")),
    "c7 lp": (lambda s: W.c7(s, NB=2, H=7, W=6, C=8, CO=8, pool="lp", k=3, stride=2, p=3.0),
              lambda w: _hand_c7(w, "lp")),
}


@pytest.mark.parametrize("name", list(HAND))
@pytest.mark.parametrize("seed", [0, 3])
def test_run_module_equals_the_hand_composed_module(name, seed):
    make, hand = HAND[name]
    w = make(seed)
    vals, last = hand(w)
    out, inter = M.run_workload(w, None)                 # per-operator: every intermediate is a boundary
    assert set(inter) == set(vals), (sorted(inter), sorted(vals))
    assert [o["out"] for o in w.ops] == list(vals)       # same values, same order
    for k, v in vals.items():
        assert np.array_equal(inter[k], v), k
    assert np.array_equal(out, vals[last])
    # and through every registered decomposition: boundaries are a subset of the same values
    for pname, cuts in w.partitions.items():
        o2, b2 = M.run_workload(w, cuts)
        assert np.array_equal(o2, vals[last]), pname
        for k, v in b2.items():
            assert np.array_equal(v, vals[k]), (pname, k)


def test_a_composition_slip_is_visible_to_the_hand_composed_pin():
    """The pin has teeth: each slip below changes an intermediate of the hand-composed module."""
    w = HAND["c5"][0](0)
    vals, _ = _hand_c5(w)
    i, p = _widen(w)
    # residual added to itself instead of to the skip edge
    assert not np.array_equal(O.residual_add(vals["o_0"], vals["o_0"]), vals["x1_0"])
    # second skip edge taken from the layer input instead of from after the attention
    assert not np.array_equal(O.residual_add(vals["d_0"], i["x"]), vals["x2_0"])
    # SiLU where the gated unit belongs; GELU where SiLU belongs
    assert O.silu(vals["gu_0"]).shape != vals["hid_0"].shape
    g, u = vals["gu_0"][:, :24], vals["gu_0"][:, 24:]
    assert not np.array_equal(O.gelu_tanh(g) * u, vals["hid_0"])
    assert np.array_equal(O.silu(g) * u, vals["hid_0"])


# ---------------------------------------------------------------- mutants
def _c4_with(attn_fn, w):
    inputs = {k: t.f64() for k, t in w.inputs.items()}
    params = {k: t.f64() for k, t in w.params.items()}
    a = attn_fn(inputs["q"], inputs["k"], inputs["v"])
    h = O.residual_add(O.linear(a, params["Wo"]), inputs["r"])
    return a, O.rmsnorm(h, params["gamma"], 1e-6)


def _attn_variant(q, k, v, diag=0, over_queries=False, zero_tail=0):
    b, h, s, d = q.shape
    out = np.empty((b, s, h, d))
    keep = np.tril(np.ones((s, s), bool), diag)
    for bi in range(b):
        for hi in range(h):
            kk = k[bi, hi].copy()
            if zero_tail:
                kk[:, -zero_tail:] = 0.0
            sc = np.where(keep, q[bi, hi] @ kk.T / np.sqrt(d), -np.inf)
            if over_queries:
                m = sc.max(axis=0, keepdims=True)
                e = np.exp(sc - m)
                p = e / e.sum(axis=0, keepdims=True)
            else:
                sc[0, 0] = sc[0, 0] if np.isfinite(sc[0, 0]) else 0.0
                p = O.softmax(sc)
            out[bi, :, hi] = p @ v[bi, hi]
    return out.reshape(b * s, h * d)


def test_attention_bug_catalogue_is_visible():
    w = W.c4(0, B=1, H=2, S=32, D=16)
    a_ref, y_ref = _c4_with(O.attention_causal_bhsd, w)
    assert check_close(a_ref, a_ref, "bf16")["ok"]
    mutants = {
        "diagonal masked": lambda q, k, v: _attn_variant(q, k, v, diag=-1),
        "softmax over queries": lambda q, k, v: _attn_variant(q, k, v, over_queries=True),
        "K tail of head_dim dropped": lambda q, k, v: _attn_variant(q, k, v, zero_tail=4),
    }
    for name, fn in mutants.items():
        a_bad, y_bad = _c4_with(fn, w)
        local = check_close(a_bad[1:], a_ref[1:], "bf16")     # row 0 of the masked-diagonal mutant is undefined
        assert not local["ok"], name
        # the local check at the attention boundary sees at least as much as the end-to-end one
        glob = check_close(y_bad[1:], y_ref[1:], "bf16")
        assert local["n_bad"] >= 1 and (glob["ok"] or glob["n_bad"] >= 1)


def test_ffn_bug_catalogue_is_visible():
    w = W.c2(0, M=32, K=64, N=48)
    ref, inter = M.run_workload(w, None)
    x, Wt, b = w.inputs["x"].f64(), w.params["W"].f64(), w.params["bias"].f64()
    pre = O.bias_add(O.linear(x, Wt), b)
    tail = lambda t: O.clamp(O.scale(t, 0.5), -1, 1)
    mutants = {
        "sigmoid GELU": tail(pre / (1 + np.exp(-1.702 * pre))),
        "ReLU instead of GELU": tail(O.relu(pre)),
        "K tile boundary dropped": tail(O.gelu_tanh(O.bias_add(O.linear(x[:, :48], Wt[:48]), b))),
        "missing bias": tail(O.gelu_tanh(O.linear(x, Wt))),
        "transposed weight": tail(O.gelu_tanh(O.bias_add(O.linear(x[:, :48], Wt[:48, :48].T.copy()), b))),
    }
    for name, out in mutants.items():
        # fp32-level tolerance sees all of them; the loose bf16 tolerance misses the subtle ones,
        # which is the paper's "threshold dilemma"
        assert not check_close(out, ref, "f32")["ok"], name
    assert not check_close(mutants["ReLU instead of GELU"], ref, "bf16")["ok"]
    assert not check_close(mutants["K tile boundary dropped"], ref, "bf16")["ok"]


def _bf16_round(x):
    from workloads.generate import bf16_bits_to_f32, f32_to_bf16_bits
    return bf16_bits_to_f32(f32_to_bf16_bits(np.asarray(x, np.float32))).astype(np.float64)


def _matmul_bf16_accumulator(a, b):
    """a [M, K] @ b [K, N] with the running sum rounded to bf16 after every addition (the paper's
    "bf16 accumulator" bug: the accumulator declared in the operands' type instead of fp32)."""
    acc = np.zeros((a.shape[0], b.shape[1]))
    for k in range(a.shape[1]):
        acc = _bf16_round(acc + a[:, k:k + 1] * b[k:k + 1, :])
    return acc


def test_remaining_paper_bugs_are_visible():
    """The rest of the paper's injected-bug list (appendix on correctness checking): softmax without
    the maximum subtraction, a bf16 accumulator in Q K^T and in the second FFN GEMM, a dropped
    residual.  Each is visible to the local check at the boundary where it happens."""
    w = W.c4(0, B=1, H=2, S=32, D=16)
    inputs, params = _widen(w)
    q, k, v, r = inputs["q"], inputs["k"], inputs["v"], inputs["r"]
    a_ref, y_ref = _c4_with(O.attention_causal_bhsd, w)

    def attn(q, k, v, softmax_fn, qk_fn=lambda a, b: a @ b):
        b_, h_, s_, d_ = q.shape
        out = np.empty((b_, s_, h_, d_))
        keep = np.tril(np.ones((s_, s_), bool))
        for bi in range(b_):
            for hi in range(h_):
                sc = np.where(keep, qk_fn(q[bi, hi], k[bi, hi].T.copy()) / np.sqrt(d_), -np.inf)
                out[bi, :, hi] = softmax_fn(sc) @ v[bi, hi]
        return out.reshape(b_ * s_, h_ * d_)

    def unsafe_softmax(sc):
        with np.errstate(over="ignore", invalid="ignore"):
            e = np.exp(sc)
            return e / e.sum(axis=-1, keepdims=True)

    # unsafe softmax: identical on ordinary scores, NaN once a score passes exp's range
    assert check_close(attn(q, k, v, unsafe_softmax), a_ref, "f32")["ok"]
    big = 40.0
    a_big_ref = O.attention_causal_bhsd(q * big, k * big, v)
    assert np.isfinite(a_big_ref).all()
    a_big_bad = attn(q * big, k * big, v, unsafe_softmax)
    assert not np.isfinite(a_big_bad).all()
    assert not check_close(a_big_bad, a_big_ref, "bf16")["ok"]

    # bf16 accumulator in Q K^T: far outside the fp32 tolerance, and outside the bf16 one at the boundary
    a_acc = attn(q, k, v, O.softmax, _matmul_bf16_accumulator)
    assert not check_close(a_acc, a_ref, "f32")["ok"]
    loc = check_close(a_acc, a_ref, "bf16")
    h_acc = O.residual_add(O.linear(a_acc, params["Wo"]), r)
    glob = check_close(O.rmsnorm(h_acc, params["gamma"], 1e-6), y_ref, "bf16")
    assert loc["max_abs"] > 1e-3 and loc["n_bad"] >= glob["n_bad"]      # never less visible locally

    # missing residual: the projection alone, normalised
    y_nores = O.rmsnorm(O.linear(a_ref, params["Wo"]), params["gamma"], 1e-6)
    assert not check_close(y_nores, y_ref, "bf16")["ok"]

    # bf16 accumulator in the FFN's second GEMM (K = 96 here): visible at the GEMM's own boundary
    w5 = W.c5(0, B=1, S=8, E=16, H=2, F=96, L=1)
    ref5, inter5 = M.run_workload(w5, None)
    p5 = {k_: t.f64() for k_, t in w5.params.items()}
    d_bad = _matmul_bf16_accumulator(inter5["hid_0"], p5["Wd0"])
    assert not check_close(d_bad, inter5["d_0"], "f32")["ok"]
    rel = np.abs(d_bad - inter5["d_0"]).max() / np.abs(inter5["d_0"]).max()
    assert rel > 2e-3                                  # ~ sqrt(K) roundings of 2^-9: a local calibrated check sees it
    y_bad = O.rmsnorm(O.residual_add(d_bad, inter5["x1_0"]), p5["ones"], 1e-6)
    # ... while the fixed bf16 tolerance on the module output lets it through (the threshold dilemma)
    assert check_close(y_bad, ref5, "bf16")["ok"]


def test_layernorm_without_mean_subtraction_is_visible():
    w = W.c1(0)
    ref, inter = M.run_workload(w, None)
    h = inter["y2"]
    bad = h / np.sqrt(h.var(axis=1, keepdims=True) + 1e-5)
    assert not check_close(bad, ref, "f32")["ok"]
    assert not check_close(bad, ref, "bf16")["ok"]


def test_predicate_rejects_nan_and_shape():
    a = np.ones((3, 3))
    b = a.copy(); b[1, 1] = np.nan
    assert not check_close(b, a, "bf16")["ok"]
    assert not check_close(np.ones((3, 2)), a, "bf16")["ok"]
    assert check_close(a + 1e-5, a, "f32")["ok"]
    assert not check_close(a + 2e-4, a, "f32")["ok"]
