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
