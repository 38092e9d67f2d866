"""tcgen05 GEMM (K1) against the fp64 oracle: exact on integer inputs, within tolerance on
random inputs, over shapes that span several tiles, several K blocks, ragged M/N/K tails and
more tiles than SMs; every fused tail; SwiGLU pairing; swap against the plain-ALU kernel."""
import numpy as np
import pytest

import workloads as W
from workloads import generate as G
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def _bf16_round(x):
    return W.bf16_bits_to_f64(W.f32_to_bf16_bits(np.asarray(x, np.float32)))


SHAPES = [(128, 64, 256), (128, 128, 256), (256, 512, 512), (8, 8, 8), (300, 200, 264), (129, 72, 520),
          (1000, 1032, 776), (2048, 256, 4096 + 256)]


@pytest.mark.parametrize("impl", ["gemm_tc", "gemm_tc2"])
@pytest.mark.parametrize("m,k,n", SHAPES)
def test_integer_inputs_are_exact(ctx, m, k, n, impl):
    if impl == "gemm_tc2" and m <= 128:
        pytest.skip("the two-SM form is offered only above 128 rows")
    w = G.c2(0, m, k, n)
    w.inputs["x"] = G.int_valued(1, 0, (m, k), -4, 4, "bf16", "x")
    w.params["W"] = G.int_valued(1, 1, (k, n), -4, 4, "bf16", "W")
    w.ops = w.ops[:1]
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: impl})
    assert dw.module.bound_impl(0) == impl
    bad = np.argwhere(out != _bf16_round(ref))
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}"


@pytest.mark.parametrize("m,k,n", [(256, 512, 512), (300, 200, 264), (1000, 1032, 776)])
def test_fused_tail_and_split_match_the_oracle(ctx, m, k, n):
    for seed in range(2):
        w = W.c2(seed, m, k, n)
        ref, _ = oracle(w, [0])
        for part in ("fused", "split"):
            dw, out = run_gpu(ctx, w, w.partitions[part])
            assert dw.module.bound_impl(0) == "gemm_tc2"
            assert_parity(out, ref, "bf16", f"{part} seed {seed}")


def test_swap_between_tensor_core_and_plain_alu_kernels(ctx):
    w = W.c2(0, 300, 200, 264)
    ref, _ = oracle(w, [0])
    outs = {}
    for impl in ("gemm_tc2", "gemm_tc", "gemm_simt"):
        dw, out = run_gpu(ctx, w, [0], binds={0: impl})
        assert dw.module.bound_impl(0) == impl
        assert_parity(out, ref, "bf16", impl)
        outs[impl] = out
    assert np.abs(outs["gemm_tc"] - outs["gemm_simt"]).max() <= 2e-2
    assert np.abs(outs["gemm_tc2"] - outs["gemm_tc"]).max() <= 2e-2


@pytest.mark.parametrize("impl", ["gemm_tc", "gemm_tc2"])
@pytest.mark.parametrize("t,e,f", [(136, 64, 128), (200, 136, 72), (520, 256, 392)])
def test_swiglu_and_residual_tails(ctx, t, e, f, impl):
    rng = np.random.default_rng(5)
    w = G.Workload("ffn", "bf16")
    w.inputs["x"] = G.make("x", "bf16", rng.standard_normal((t, e)).astype(np.float32))
    w.params["Wgu"] = G.make("Wgu", "bf16", (rng.standard_normal((e, 2 * f)) / np.sqrt(e)).astype(np.float32))
    w.params["Wd"] = G.make("Wd", "bf16", (rng.standard_normal((f, e)) / np.sqrt(f)).astype(np.float32))
    w.ops = [G._op("linear", "gu", ["x"], {"w": "Wgu"}, n=2 * f), G._op("swiglu", "h", ["gu"]),
             G._op("linear", "d", ["h"], {"w": "Wd"}, n=e), G._op("residual_add", "y", ["d", "x"])]
    ref, inter = oracle(w, None)
    dw, out = run_gpu(ctx, w, [0, 2], binds={0: impl, 1: impl}, keep=True)
    assert [dw.module.bound_impl(s) for s in range(2)] == [impl, impl]
    from paper_2607_20501_b200.runner import to_host_f64
    assert_parity(to_host_f64(dw.intermediate("h")), inter["h"], "bf16", "silu(gate)*up")
    assert_parity(out, ref, "bf16", "down + residual")
    # the gate and up halves are not interchangeable: integer check of the pairing
    w.inputs["x"] = G.int_valued(2, 0, (t, e), -2, 2, "bf16", "x")
    w.params["Wgu"] = G.int_valued(2, 1, (e, 2 * f), -1, 1, "bf16", "Wgu")
    ref, inter = oracle(w, None)
    dw, _ = run_gpu(ctx, w, [0, 2], binds={0: impl, 1: impl}, keep=True)
    assert_parity(to_host_f64(dw.intermediate("h")), inter["h"], "bf16", "pairing")


@pytest.mark.parametrize("dtype,impls", [("bf16", ("gemm_tc2", "gemm_tc", "gemm_simt")), ("f32", ("gemm_simt",))])
def test_exact_gelu_in_the_epilogue(ctx, dtype, impls):
    """LINEAR + bias + GELU_ERF (0.5 x (1 + erf(x / sqrt 2))) as one submodule on every GEMM kernel, and split after
    the bias so that the activation runs as an elementwise pass."""
    m, k, n = 300, 200, 264
    rng = np.random.default_rng(9)
    w = G.Workload("ge", dtype)
    w.inputs["x"] = G.make("x", dtype, rng.standard_normal((m, k)).astype(np.float32))
    w.params["W"] = G.make("W", dtype, (rng.standard_normal((k, n)) * (1.0 / k) ** 0.5 * 2).astype(np.float32))
    w.params["b"] = G.make("b", dtype, (0.3 * rng.standard_normal(n)).astype(np.float32))
    w.ops = [G._op("linear", "y0", ["x"], {"w": "W"}, n=n), G._op("bias_add", "y1", ["y0"], {"b": "b"}),
             G._op("gelu_erf", "y", ["y1"])]
    ref, _ = oracle(w, [0])
    for impl in impls:
        dw, out = run_gpu(ctx, w, [0], binds={0: impl})
        assert dw.module.bound_impl(0) == impl
        assert_parity(out, ref, dtype, f"{impl} fused")
    _, out = run_gpu(ctx, w, [0, 2])
    assert_parity(out, ref, dtype, "activation as its own pass")
