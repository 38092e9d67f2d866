"""GEMM + elementwise tail + row norm in one tensor-core kernel with the rows held in tensor memory until their
statistics are known (a cluster of CTA pairs covers whole rows; partial sums cross CTAs through distributed shared
memory): the paper's projection + residual + norm subkernel at tensor-core shape.  Against the fp64 oracle for
LayerNorm and RMSNorm, for every cluster width (1, 2, 4 pairs; one or two column tiles per pair), ragged M and N,
rows with a mean far from zero (the statistics are merged without cancellation), the two-output form whose
pre-norm value is an fp32 residual stream, several row blocks per cluster, and repeated launches."""
import numpy as np
import pytest

import workloads as W
from workloads import generate as G
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu
IMPL = "gemm_rownorm_cl"


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


# (m, k, n): n <= 256 one pair, <= 512 two, <= 1024 four pairs with one tile each, <= 2048 four pairs with two tiles
SHAPES = [(256, 64, 256), (300, 128, 512), (512, 256, 1024), (1024, 256, 2048), (129, 72, 328), (2000, 512, 1000),
          (700, 136, 776), (260, 64, 1544), (5000, 192, 1024), (6000, 128, 2048), (40000, 64, 256)]


@pytest.mark.parametrize("m,k,n", SHAPES)
def test_linear_bias_relu_layernorm(ctx, m, k, n):
    w = W.c1(3, M=m, K=k, N=n, dtype="bf16")
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, w.partitions["fused"], binds={0: IMPL})
    assert dw.module.bound_impl(0) == IMPL
    assert dw.module.launch_count() == 1
    assert_parity(out, ref, "bf16", f"fused {m}x{k}x{n}")
    # normalised rows: mean 0, variance 1 (gamma = 1, beta = 0 in this workload)
    assert np.abs(out.mean(axis=1)).max() < 2e-2 and np.abs(out.var(axis=1) - 1).max() < 5e-2


@pytest.mark.parametrize("m,k,n", [(512, 128, 512), (1000, 64, 1024), (384, 256, 2048)])
def test_rows_with_a_large_mean(ctx, m, k, n):
    """A bias of 40 puts every row's mean forty standard deviations from zero: E[x^2] - mean^2 in fp32 would lose
    the variance; the per-warp (mean, M2) partials merged with Chan's formula do not."""
    w = W.c1(5, M=m, K=k, N=n, dtype="bf16")
    w.params["b"] = G.make("b", "bf16", w.params["b"].f64().astype(np.float32) + 40.0)
    w.ops = [o for o in w.ops if o["kind"] != "relu"]
    w.ops[2]["in"] = ["y1"]
    w.partitions = {"fused": [0]}
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: IMPL})
    assert_parity(out, ref, "bf16", f"offset rows {m}x{k}x{n}")


@pytest.mark.parametrize("shape", [dict(B=2, H=4, S=384, D=128), dict(B=3, H=8, S=256, D=128), dict(B=1, H=16, S=640, D=128)])
def test_projection_residual_rmsnorm(ctx, shape):
    """C4's tail at reduced sizes (E = 512, 1024, 2048), run several times on the same buffers."""
    w = W.c4(2, **shape)
    ref, _ = oracle(w, None)
    dw, out = run_gpu(ctx, w, [0, 1], binds={1: IMPL})     # {attention}, {projection, residual, RMSNorm}
    assert dw.module.bound_impl(1) == IMPL
    assert_parity(out, ref, "bf16", "first call")
    from paper_2607_20501_b200.runner import to_host_f64
    for _ in range(3):
        again = to_host_f64(dw.forward())
        assert np.array_equal(again, out)


def test_prenorm_value_that_is_needed_later_is_written_too(ctx):
    """One decoder layer: the output projection's submodule {linear, residual add (fp32 stream), RMSNorm} has two
    outputs, the stream and its normalised copy; both come out of the one kernel."""
    w = W.c5(1, B=2, S=256, E=1024, H=8, F=512, L=1)
    ref, inter = oracle(w, None)
    # ops: 0 rmsnorm, 1 linear qkv, 2 attention, 3 linear o, 4 residual (x1), 5 rmsnorm (n2), 6 gu, 7 swiglu, 8 d, 9 residual, 10 rmsnorm
    cuts = [0, 1, 2, 3, 6, 8]
    dw, out = run_gpu(ctx, w, cuts, binds={3: IMPL, 5: IMPL}, keep=True)
    assert dw.module.bound_impl(3) == IMPL and dw.module.bound_impl(5) == IMPL
    assert_parity(out, ref, "bf16", "decoder layer through two fused projection + residual + norm kernels")
    from paper_2607_20501_b200.runner import to_host_f64
    x1 = to_host_f64(dw.intermediate("x1_0"))
    n2 = to_host_f64(dw.intermediate("n2_0"))
    assert dw.intermediate("x1_0").dtype.is_floating_point and dw.intermediate("x1_0").element_size() == 4
    assert_parity(x1, inter["x1_0"], "bf16", "the fp32 stream written beside the norm")
    assert_parity(n2, inter["n2_0"], "bf16", "the normalised copy")


def test_the_composer_does_not_pick_it_unasked(ctx):
    w = W.c1(3, M=512, K=128, N=512, dtype="bf16")
    dw, _ = run_gpu(ctx, w, w.partitions["fused"])
    assert dw.module.bound_impl(0) == "gemm_tc2+rowop"
