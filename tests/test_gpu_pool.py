"""Pooling subkernels (mean / maximum / p-norm) against the fp64 oracle, and the transfer story they stand for: the
same module with its pooling operator exchanged keeps every other binding."""
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


def _pool_only(dtype, shape, pool, k, stride, p=2.0, seed=0):
    w = G.Workload("pool", dtype)
    w.inputs["x"] = G.make("x", dtype, G._normal(seed, 0, shape))
    attrs = {"k": k, "stride": stride}
    if pool == "lp":
        attrs["p"] = p
    w.ops = [G._op(pool + "pool", "y", ["x"], **attrs)]
    w.partitions = {"fused": [0]}
    return w


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("pool", ["avg", "max", "lp"])
@pytest.mark.parametrize("shape,k,stride", [((2, 8, 8, 16), 2, 2), ((1, 7, 9, 24), 3, 2), ((3, 14, 14, 128), 7, 7), ((2, 9, 9, 5), 3, 1),
                                             ((1, 5, 6, 1), 5, 1), ((2, 56, 56, 64), 7, 7), ((1, 4, 4, 8), 1, 1), ((1, 10, 10, 40), 4, 3)])
def test_pooling_matches_the_oracle(ctx, dtype, pool, shape, k, stride):
    w = _pool_only(dtype, shape, pool, k, stride)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0])
    assert dw.module.bound_impl(0) == "pool_nhwc"
    assert out.shape == ref.shape
    assert_parity(out, ref, dtype, f"{pool} {dtype} {shape} k{k} s{stride}")


@pytest.mark.parametrize("p", [1.0, 2.0, 3.0, 6.0])
def test_p_norm_pooling_for_several_p(ctx, p):
    for dtype in ("bf16", "f32"):
        w = _pool_only(dtype, (2, 12, 12, 32), "lp", 3, 3, p=p, seed=1)
        ref, _ = oracle(w, [0])
        _, out = run_gpu(ctx, w, [0])
        assert_parity(out, ref, dtype, f"p{p} {dtype}")


def test_closed_forms(ctx):
    # a constant image: mean and maximum return the constant, the 2-norm k times it
    for pool, want in (("avg", 1.5), ("max", 1.5), ("lp", 4.5)):
        w = _pool_only("f32", (1, 6, 6, 8), pool, 3, 3)
        w.inputs["x"] = G.make("x", "f32", np.full((1, 6, 6, 8), 1.5, np.float32))
        _, out = run_gpu(ctx, w, [0])
        assert np.allclose(out, want, rtol=1e-6)
    # maximum pooling of integer-valued data is exact, and never below the mean
    w = _pool_only("bf16", (2, 8, 8, 16), "max", 2, 2)
    w.inputs["x"] = G.int_valued(3, 0, (2, 8, 8, 16), -4, 4, "bf16", "x")
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0])
    assert np.array_equal(out, ref)


def test_exchanging_the_pooling_subkernel_leaves_the_rest_alone(ctx):
    """The paper's transfer study: the module with mean pooling, then the same module with the pooling
    operator exchanged.  Each variant matches its oracle, and the convolution submodule keeps its kernel."""
    outs = {}
    for pool in ("avg", "max", "lp"):
        w = W.c7(0, NB=2, H=28, W=28, C=64, CO=128, pool=pool, k=7, stride=7)
        ref, _ = oracle(w, [0])
        for part in ("split2", "fused", "per_op"):
            dw, out = run_gpu(ctx, w, w.partitions[part])
            assert_parity(out, ref, "bf16", f"c7 {pool} {part}")
        dw, out = run_gpu(ctx, w, w.partitions["split2"])
        assert [dw.module.bound_impl(i) for i in range(2)] == ["conv3x3_tc2", "pool_nhwc"]
        outs[pool] = out
    assert (outs["max"] >= outs["avg"] - 1e-6).all()
    assert (outs["lp"] >= outs["max"] - 2e-2 * np.abs(outs["max"]) - 2e-2).all()      # 2-norm >= largest magnitude (inputs are post-ReLU)


def test_c7_full_size(ctx):
    w = W.c7(0)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, w.partitions["fused"])
    assert dw.module.bound_impl(0) == "conv3x3_tc2+pool_nhwc"
    assert_parity(out, ref, "bf16", "c7 full")
