"""Seeded random shapes against the fp64 oracle: GEMMs with every kind of tail (bias, activation, residual before
or after them; the residual ring and the register path), both attention operators at arbitrary sequence
lengths, convolution + GroupNorm at arbitrary image sizes, pooling windows.  The shapes are drawn, not
chosen, so ragged tiles, single-row problems and odd strides turn up that the hand-written cases miss."""
import numpy as np
import pytest

import workloads as W
from workloads.generate import Workload, _normal, _op, make
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def _cases(seed, n, draw):
    rng = np.random.default_rng(seed)
    return [draw(rng) for _ in range(n)]


GEMM = _cases(1, 40, lambda r: (int(r.choice([1, 7, 64, 129, 256, 300, 1000, 2048, 4096])), 8 * int(r.integers(1, 400)),
                                8 * int(r.integers(1, 300)), str(r.choice(["", "b", "ba", "r", "br", "bar", "rb"]))))
ATTN = _cases(2, 24, lambda r: (int(r.integers(1, 4)), int(r.integers(1, 6)), int(r.integers(1, 1500)),
                                str(r.choice(["attention_causal", "attention"]))))
CONV = _cases(3, 12, lambda r: (int(r.integers(1, 4)), int(r.integers(3, 40)), int(r.integers(3, 62)), int(r.choice([64, 128])),
                                int(r.choice([64, 128, 256])), int(r.choice([4, 8, 16, 32]))))
POOL = _cases(4, 16, lambda r: (int(r.integers(1, 3)), int(r.integers(4, 30)), int(r.integers(4, 30)), int(r.choice([3, 8, 24, 64])),
                                int(r.integers(1, 5)), int(r.integers(1, 4)), str(r.choice(["avg", "max", "lp"]))))


@pytest.mark.parametrize("i", range(len(GEMM)))
def test_gemm_with_random_shape_and_tail(ctx, i):
    m, n, k, tail = GEMM[i]
    w = Workload("g", "bf16")
    w.inputs["x"] = make("x", "bf16", _normal(i, 0, (m, k)))
    w.inputs["r"] = make("r", "bf16", _normal(i, 1, (m, n)))
    w.params["W"] = make("W", "bf16", _normal(i, 2, (k, n), std=0.05))
    w.params["b"] = make("b", "bf16", _normal(i, 3, (n,), std=0.1))
    w.ops = [_op("linear", "y0", ["x"], {"w": "W"}, n=n)]
    for ch in tail:
        prev = w.ops[-1]["out"]
        if ch == "b":
            w.ops.append(_op("bias_add", prev + "b", [prev], {"b": "b"}))
        elif ch == "a":
            w.ops.append(_op("gelu_tanh", prev + "a", [prev]))
        else:
            w.ops.append(_op("residual_add", prev + "r", [prev, "r"]))
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0])
    assert dw.module.bound_impl(0) in ("gemm_tc2", "gemm_tc")          # one kernel, the tail in its epilogue
    assert_parity(out, ref, "bf16", f"M{m} N{n} K{k} tail '{tail}'")


@pytest.mark.parametrize("i", range(len(ATTN)))
def test_attention_with_random_shape(ctx, i):
    b, h, s, kind = ATTN[i]
    w = W.c4(100 + i, B=b, H=h, S=s, D=128)
    w.ops = [dict(w.ops[0], kind=kind)]
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0], binds={0: "attention_tc2"})
    assert_parity(out, ref, "bf16", f"{kind} B{b} H{h} S{s}")


@pytest.mark.parametrize("i", range(len(CONV)))
def test_convolution_groupnorm_with_random_shape(ctx, i):
    nb, h, wd, c, co, g = CONV[i]
    w = W.c3(200 + i, NB=nb, H=h, W=wd, C=c, CO=co, G=g)
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, w.partitions["fused"])
    assert_parity(out, ref, "bf16", f"NB{nb} H{h} W{wd} C{c} CO{co} G{g}")


@pytest.mark.parametrize("i", range(len(POOL)))
def test_pooling_with_random_shape(ctx, i):
    nb, h, wd, c, k, st, pool = POOL[i]
    w = Workload("p", "bf16")
    w.inputs["x"] = make("x", "bf16", _normal(300 + i, 0, (nb, h, wd, c)))
    attrs = {"k": k, "stride": st}
    if pool == "lp":
        attrs["p"] = 2.0 + (i % 2)
    w.ops = [_op(pool + "pool", "y", ["x"], **attrs)]
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0])
    assert_parity(out, ref, "bf16", f"{pool} {nb}x{h}x{wd}x{c} k{k} s{st}")


FUSED = _cases(5, 36, lambda r: (int(r.integers(1, 200)), int(r.integers(1, 700)), int(r.choice([8, 9, 16, 40, 100, 128, 200, 256, 257, 300, 640, 1024])),
                                 "f32", str(r.choice(["layernorm", "rmsnorm"])), bool(r.integers(0, 2))))


@pytest.mark.parametrize("i", range(len(FUSED)))
def test_small_fused_chain_with_random_shape(ctx, i):
    """linear -> +bias -> ReLU -> row norm in one launch: the cluster form (rows up to 256 wide, any K, either weight
    layout, ragged row and column counts) and the single-CTA form beyond it; fp32, the type this kernel serves."""
    from paper_2607_20501_b200 import binding as B
    m, k, n, dtype, norm, row_major = FUSED[i]
    w = W.c1(400 + i, M=m, K=k, N=n, dtype=dtype)
    if norm == "rmsnorm":
        w.ops[-1] = dict(w.ops[-1], kind="rmsnorm", params={"gamma": "gamma"}, attrs={"eps": 1e-6})
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], weight_layout=B.MK_LAYOUT_ROW_MAJOR if row_major else None)
    assert dw.module.bound_impl(0) == "linear_rownorm_simt"
    assert_parity(out, ref, dtype, f"M{m} K{k} N{n} {dtype} {norm} row_major={row_major}")


# the small fused chain at the edges of its register form (K a multiple of 8 up to 8 * 512 / columns per CTA) and just
# beyond them, where the staged form takes over: (M, K, N, dtype, norm, row-major weight)
EDGE = [(64, 256, 128, "f32", "layernorm", False), (64, 256, 128, "f32", "layernorm", True), (61, 248, 100, "f32", "layernorm", True),
        (9, 8, 8, "f32", "rmsnorm", False), (64, 264, 128, "f32", "layernorm", False), (64, 128, 256, "f32", "rmsnorm", True),
        (64, 136, 256, "f32", "layernorm", False), (3, 512, 60, "f32", "layernorm", False), (3, 520, 60, "f32", "layernorm", True),
        (17, 256, 128, "bf16", "layernorm", False), (17, 256, 128, "bf16", "rmsnorm", True), (40, 252, 128, "f32", "layernorm", False)]


@pytest.mark.parametrize("m,k,n,dtype,norm,row_major", EDGE)
def test_small_fused_chain_at_the_edges_of_its_register_form(ctx, m, k, n, dtype, norm, row_major):
    from paper_2607_20501_b200 import binding as B
    w = W.c1(900 + m + k + n, M=m, K=k, N=n, dtype=dtype)
    if norm == "rmsnorm":
        w.ops[-1] = dict(w.ops[-1], kind="rmsnorm", params={"gamma": "gamma"}, attrs={"eps": 1e-6})
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], weight_layout=B.MK_LAYOUT_ROW_MAJOR if row_major else None)
    assert_parity(out, ref, dtype, f"M{m} K{k} N{n} {dtype} {norm} row_major={row_major}")
    _, again = run_gpu(ctx, w, [0], weight_layout=B.MK_LAYOUT_ROW_MAJOR if row_major else None)
    assert np.array_equal(out, again)     # every sum in a fixed order
