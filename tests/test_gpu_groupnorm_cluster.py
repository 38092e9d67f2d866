"""GroupNorm with the image resident in a thread-block cluster's shared memory (one launch, one pass over HBM)
against the fp64 oracle and against the two-launch form: cluster sizes 1, 2, 4 and 8, both storage types, an
elementwise prefix inside the submodule, groups far from zero mean, pixel counts that do not divide by the
cluster size, and shapes the cluster form must refuse (they fall back to the two launches)."""
import os

import numpy as np
import pytest

from workloads import generate as G
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def _gn(x, dtype, groups, prefix=False, seed=0):
    rng = np.random.default_rng(seed)
    c = x.shape[-1]
    w = G.Workload("gn", dtype)
    w.inputs["x"] = G.make("x", dtype, x)
    w.params["gamma"] = G.make("gamma", dtype, (1 + 0.1 * rng.standard_normal(c)).astype(np.float32))
    w.params["beta"] = G.make("beta", dtype, (0.1 * rng.standard_normal(c)).astype(np.float32))
    w.ops = []
    src = "x"
    if prefix:
        w.params["b"] = G.make("b", dtype, (0.2 * rng.standard_normal(c)).astype(np.float32))
        w.ops += [G._op("bias_add", "x1", ["x"], {"b": "b"}), G._op("relu", "x2", ["x1"])]
        src = "x2"
    w.ops.append(G._op("groupnorm", "y", [src], {"gamma": "gamma", "beta": "beta"}, groups=groups, eps=1e-5))
    return w


def _run(ctx, w, two_pass):
    if two_pass:
        os.environ["MK_GN_TWO_PASS"] = "1"
    else:
        os.environ.pop("MK_GN_TWO_PASS", None)
    try:
        dw, out = run_gpu(ctx, w, [0])
        return dw.module.launch_count(), out
    finally:
        os.environ.pop("MK_GN_TWO_PASS", None)


# (shape, groups, launches in bf16, launches in fp32): images of 6 KB (cluster of 8 on a near-empty GPU), 100 KB,
# 400 KB, 800 KB and 1.5 MB in bf16; the last but two fits eight CTAs in bf16 and not in fp32
CASES = [((3, 7, 7, 64), 8, 1, 1), ((2, 20, 20, 128), 32, 1, 1), ((5, 40, 40, 128), 4, 1, 1), ((40, 56, 56, 128), 32, 1, 1),
         ((2, 57, 53, 256), 16, 1, 2), ((1, 33, 31, 32), 1, 1, 1), ((150, 8, 8, 64), 16, 1, 1)]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("shape,groups,n_bf16,n_f32", CASES)
def test_cluster_form_matches_the_oracle_and_the_two_launch_form(ctx, dtype, shape, groups, n_bf16, n_f32):
    rng = np.random.default_rng(sum(shape))
    x = (rng.standard_normal(shape) * 1.5 + 0.3).astype(np.float32)
    w = _gn(x, dtype, groups)
    ref, _ = oracle(w, [0])
    n1, out1 = _run(ctx, w, two_pass=False)
    n2, out2 = _run(ctx, w, two_pass=True)
    assert n2 == 2
    assert n1 == (n_bf16 if dtype == "bf16" else n_f32)
    assert_parity(out1, ref, dtype, "cluster form")
    assert_parity(out2, ref, dtype, "two launches")
    _, again = _run(ctx, w, two_pass=False)
    assert np.array_equal(out1, again)            # fixed order of every sum: the same bits from launch to launch


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_cluster_form_with_an_elementwise_prefix(ctx, dtype):
    rng = np.random.default_rng(5)
    x = rng.standard_normal((4, 24, 24, 64)).astype(np.float32)
    w = _gn(x, dtype, 8, prefix=True)
    ref, _ = oracle(w, [0])
    n1, out1 = _run(ctx, w, two_pass=False)
    assert n1 == 1
    assert_parity(out1, ref, dtype, "bias + relu + groupnorm in one launch")


def test_cluster_form_far_from_zero_mean(ctx):
    """fp32, groups fifty standard deviations from zero: the per-CTA sums are taken about a pivot and merged as
    (mean, M2) pairs, so the fp32 tolerance holds."""
    rng = np.random.default_rng(11)
    shape, groups = (2, 30, 30, 64), 8
    offs = np.repeat(rng.choice([-50.0, 50.0, 37.5], groups), shape[-1] // groups)
    x = (rng.standard_normal(shape) + offs).astype(np.float32)
    w = _gn(x, "f32", groups)
    ref, _ = oracle(w, [0])
    n1, out1 = _run(ctx, w, two_pass=False)
    assert n1 == 1
    assert_parity(out1, ref, "f32", "far mean")


def test_shapes_the_cluster_form_refuses(ctx):
    """An image too large for eight CTAs' shared memory and a channel count that does not vectorise take the two
    launches; the result is the oracle's either way."""
    rng = np.random.default_rng(2)
    for shape, groups, dtype in (((1, 100, 100, 128), 32, "bf16"), ((2, 9, 7, 24), 3, "bf16")):
        x = rng.standard_normal(shape).astype(np.float32)
        w = _gn(x, dtype, groups)
        ref, _ = oracle(w, [0])
        n1, out1 = _run(ctx, w, two_pass=False)
        assert n1 == 2
        assert_parity(out1, ref, dtype, str(shape))
