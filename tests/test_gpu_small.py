"""GPU parity at sizes the oracle finishes in well under a second: every workload, every
decomposition, five seeds (the paper's five-trial protocol), local (per-boundary) and global
checks, plus operator-level shape sweeps that cross tile boundaries and hit ragged tails."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads import generate as G
from oracle import ops as O
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


SMALL = {
    "c1": lambda s, dt: W.c1(s, dtype=dt),
    "c2": lambda s, dt: W.c2(s, M=200, K=136, N=104, dtype=dt),
    "c3": lambda s, dt: W.c3(s, NB=3, H=9, W=7, C=16, CO=24, G=4, dtype=dt),
    "c4": lambda s, dt: W.c4(s, B=2, H=3, S=40, D=32, dtype=dt),
    "c5": lambda s, dt: W.c5(s, B=2, S=24, E=64, H=2, F=96, L=2, dtype=dt),
}


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("name", list(SMALL))
def test_every_decomposition_matches_the_oracle(ctx, name, dtype):
    for seed in range(5):
        w = SMALL[name](seed, dtype)
        ref, _ = oracle(w, [0])
        for pname, cuts in w.partitions.items():
            if seed > 0 and pname not in ("fused", "split", "split3", "fused_tails"):
                continue
            dw, out = run_gpu(ctx, w, cuts)
            assert_parity(out, ref, dtype, f"{name}/{dtype}/{pname}/seed{seed}")


@pytest.mark.parametrize("name", ["c2", "c4", "c5"])
def test_local_and_global_checks_agree(ctx, name):
    """Every boundary tensor of the per-op decomposition matches the oracle's intermediate, and so
    does the final output: local and global verdicts agree (Algorithm 2 treats a disagreement as a
    broken decomposition)."""
    from paper_2607_20501_b200.runner import to_host_f64
    w = SMALL[name](0, "bf16")
    ref, inter = oracle(w, None)
    dw, out = run_gpu(ctx, w, w.partitions.get("per_op", list(range(len(w.ops)))), keep=True)
    glob = assert_parity(out, ref, "bf16", "global")
    for op in w.ops[:-1]:
        t = to_host_f64(dw.intermediate(op["out"]))
        assert_parity(t, inter[op["out"]], "bf16", f"local {op['out']}")
    assert glob["ok"]


def test_weight_layout_row_major_matches(ctx):
    from paper_2607_20501_b200 import binding as B
    w = SMALL["c2"](0, "bf16")
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0], weight_layout=B.MK_LAYOUT_ROW_MAJOR)
    assert_parity(out, ref, "bf16")


def test_integer_inputs_give_the_exact_product(ctx):
    """Integers in [-4, 4] are exact in bf16/fp32/fp64, so any mismatch is an indexing bug."""
    for dtype in ("bf16", "f32"):
        for (m, k, n) in [(1, 8, 8), (65, 40, 72), (130, 264, 136)]:
            w = G.c2(0, m, k, n, dtype=dtype)
            w.inputs["x"] = G.int_valued(1, 0, (m, k), -4, 4, dtype, "x")
            w.params["W"] = G.int_valued(1, 1, (k, n), -4, 4, dtype, "W")
            w.ops = w.ops[:1]
            ref, _ = oracle(w, [0])
            _, out = run_gpu(ctx, w, [0])
            if dtype == "f32":
                assert np.array_equal(out, ref)
            else:       # the bf16 store rounds; the fp32 accumulator itself is exact
                import workloads
                assert np.array_equal(out, workloads.bf16_bits_to_f64(workloads.f32_to_bf16_bits(ref.astype(np.float32))))


def _single(kind, x, dtype, params=None, **attrs):
    w = G.Workload("op", dtype)
    w.inputs["x"] = G.make("x", dtype, x)
    pn = {}
    for k, v in (params or {}).items():
        w.params[k] = G.make(k, dtype, v)
        pn[k] = k
    w.ops = [G._op(kind, "y", ["x"], pn, **attrs)]
    return w


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n", [8, 100, 128, 1000, 2048, 4096, 5000, 8200])
def test_row_reductions_over_row_lengths(ctx, dtype, n):
    rng = np.random.default_rng(n)
    rows = 37
    x = (rng.standard_normal((rows, n)) * 2 + 0.5).astype(np.float32)
    g = rng.standard_normal(n).astype(np.float32)
    b = rng.standard_normal(n).astype(np.float32)
    for kind, params, attrs in (("layernorm", {"gamma": g, "beta": b}, {"eps": 1e-5}),
                                ("rmsnorm", {"gamma": g}, {"eps": 1e-6}),
                                ("softmax", {}, {})):
        w = _single(kind, x, dtype, params, **attrs)
        ref, _ = oracle(w, [0])
        _, out = run_gpu(ctx, w, [0])
        assert_parity(out, ref, dtype, f"{kind} n={n}")
        if kind == "softmax":
            assert np.allclose(out.sum(axis=1), 1.0, atol=2e-2 if dtype == "bf16" else 1e-5)


def test_norm_without_affine_and_invariants(ctx):
    x = np.random.default_rng(0).standard_normal((64, 256)).astype(np.float32) * 3 + 1
    w = _single("layernorm", x, "f32", {}, eps=1e-5)
    _, out = run_gpu(ctx, w, [0])
    assert np.allclose(out.mean(axis=1), 0, atol=1e-5) and np.allclose(out.var(axis=1), 1, atol=1e-4)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,groups", [((2, 5, 7, 8), 4), ((3, 16, 16, 128), 32), ((1, 9, 9, 24), 3),
                                           ((2, 4, 4, 20), 5), ((1, 56, 56, 128), 32)])
def test_groupnorm_shapes(ctx, dtype, shape, groups):
    rng = np.random.default_rng(7)
    x = (rng.standard_normal(shape) + 0.4).astype(np.float32)
    c = shape[-1]
    w = _single("groupnorm", x, dtype, {"gamma": 1 + 0.1 * rng.standard_normal(c).astype(np.float32),
                                        "beta": 0.1 * rng.standard_normal(c).astype(np.float32)},
                groups=groups, eps=1e-5)
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0])
    assert_parity(out, ref, dtype)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,groups", [((2, 14, 14, 128), 32), ((3, 9, 7, 24), 3), ((1, 30, 30, 64), 8)])
def test_groupnorm_far_from_zero_mean(ctx, dtype, shape, groups):
    """Groups whose mean is fifty standard deviations from zero (and of either sign): sums of squares about zero
    would lose the variance to cancellation in fp32; the kernels sum about a pivot taken from the group itself."""
    rng = np.random.default_rng(11)
    c = shape[-1]
    offs = np.repeat(rng.choice([-50.0, 50.0, 37.5], groups), c // groups)
    x = (rng.standard_normal(shape) + offs).astype(np.float32)
    w = _single("groupnorm", x, dtype, {"gamma": 1 + 0.1 * rng.standard_normal(c).astype(np.float32),
                                        "beta": 0.1 * rng.standard_normal(c).astype(np.float32)},
                groups=groups, eps=1e-5)
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0])
    if dtype == "f32":
        assert_parity(out, ref, dtype)
    else:
        # bf16 input: the stored values near 50 carry steps of 0.25, which the oracle sees too; the output tolerance applies
        assert_parity(out, ref, dtype)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_elementwise_ragged_and_swiglu(ctx, dtype):
    rng = np.random.default_rng(3)
    for rows, cols in ((1, 1), (7, 13), (33, 64), (129, 1000)):
        x = rng.standard_normal((rows, 2 * cols)).astype(np.float32)
        w = G.Workload("e", dtype)
        w.inputs["x"] = G.make("x", dtype, x)
        w.inputs["r"] = G.make("r", dtype, rng.standard_normal((rows, cols)).astype(np.float32))
        w.params["b"] = G.make("b", dtype, rng.standard_normal(cols).astype(np.float32))
        w.ops = [G._op("swiglu", "h", ["x"]), G._op("bias_add", "h1", ["h"], {"b": "b"}),
                 G._op("silu", "h2", ["h1"]), G._op("residual_add", "h3", ["h2", "r"]),
                 G._op("gelu_tanh", "h4", ["h3"]), G._op("scale", "h5", ["h4"], s=-1.5),
                 G._op("clamp", "h6", ["h5"], lo=-0.75, hi=2.0), G._op("gelu_erf", "h7", ["h6"]), G._op("relu", "y", ["h7"])]
        ref, _ = oracle(w, [0])
        for cuts in ([0], [0, 1, 4], list(range(9))):
            _, out = run_gpu(ctx, w, cuts)
            assert_parity(out, ref, dtype, f"{rows}x{cols} {cuts}")


def test_attention_closed_forms_on_the_device(ctx):
    w = W.c4(0, B=1, H=2, S=33, D=64, dtype="f32")
    w.ops = w.ops[:1]
    # identical keys -> uniform weights -> prefix means of V
    k = w.inputs["k"].store
    w.inputs["k"] = G.make("k", "f32", np.broadcast_to(k[:, :, :1], k.shape).copy())
    _, out = run_gpu(ctx, w, [0])
    v = w.inputs["v"].f64()
    pm = np.cumsum(v, axis=2) / np.arange(1, 34)[None, None, :, None]
    assert_parity(out, pm.transpose(0, 2, 1, 3).reshape(33, 128), "f32")


def test_empty_batch_and_missing_param(ctx):
    from paper_2607_20501_b200 import MkError, Module, binding as B
    w = SMALL["c2"](0, "bf16")
    m = Module(ctx, w.ops, {"x": ("bf16", w.inputs["x"].shape)})
    x = torch.zeros(w.inputs["x"].shape, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((200, 104), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(MkError) as e:
        m.forward([x], y, ws, ws.numel(), 0)
    assert e.value.status == B.MK_ERR_PARAM_MISSING
    m.set_decomposition([0, 2, 3, 4])
    wt = torch.zeros((104, 136), dtype=torch.bfloat16, device="cuda")
    bias = torch.zeros((104,), dtype=torch.bfloat16, device="cuda")
    m.set_param(0, 0, wt, "bf16", (136, 104), B.MK_LAYOUT_TRANSPOSED)
    m.set_param(1, 0, bias, "bf16", (104,))
    with pytest.raises(MkError) as e:
        m.forward([x], y, ws, 16, 0)
    assert e.value.status == B.MK_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(MkError) as e:
        m.set_param(0, 0, wt, "bf16", (104, 136), B.MK_LAYOUT_TRANSPOSED)
    assert e.value.status == B.MK_ERR_SHAPE_MISMATCH
    m.forward([x], y, ws, ws.numel(), 0)
    torch.cuda.synchronize()
    assert m.launch_count() == 4


def test_profile_reports_one_time_per_submodule(ctx):
    w = SMALL["c2"](0, "bf16")
    dw, _ = run_gpu(ctx, w, w.partitions["split"])
    ms = dw.profile(iters=3)
    assert len(ms) == 4 and all(t > 0 for t in ms)
