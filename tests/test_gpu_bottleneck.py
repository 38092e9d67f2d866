"""The residual bottleneck block (1 x 1, 3 x 3, 1 x 1 convolutions with a skip connection): a LINEAR over the channel
dimension of an NHWC tensor is the 1 x 1 convolution, so the block is three tensor-core launches.  Against the fp64
oracle under every decomposition, on image widths of one and of several tile segments."""
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


@pytest.mark.parametrize("nb,h,w,c,cm", [(2, 12, 12, 128, 64), (3, 9, 70, 256, 64), (1, 20, 20, 64, 128), (2, 56, 56, 256, 64)])
def test_bottleneck_block_matches_the_oracle(ctx, nb, h, w, c, cm):
    wl = W.c9(1, NB=nb, H=h, W=w, C=c, CM=cm)
    ref, _ = oracle(wl, [0])
    for part in ("fused", "split3", "per_op"):
        dw, out = run_gpu(ctx, wl, wl.partitions[part])
        if part == "split3":
            impls = [dw.module.bound_impl(i) for i in range(3)]
            assert impls[1] == "conv3x3_tc2" and all(i in ("gemm_tc2", "gemm_tc") for i in (impls[0], impls[2])), impls
        assert_parity(out, ref, "bf16", f"{part} [{nb},{h},{w},{c}] via {cm}")


def test_one_by_one_convolution_is_exact_on_integers(ctx):
    """LINEAR on a rank-4 input, integer-valued operands: every product and sum is exact, so any mismatch is an
    indexing error in the way the leading dimensions are flattened into GEMM rows."""
    nb, h, w, c, n = 3, 7, 9, 64, 96
    wl = G.Workload("pw", "bf16")
    wl.inputs["x"] = G.int_valued(3, 0, (nb, h, w, c), -2, 2, "bf16", "x")
    wl.params["W"] = G.int_valued(3, 1, (c, n), -2, 2, "bf16", "W")
    wl.ops = [G._op("linear", "y", ["x"], {"w": "W"}, n=n)]
    ref, _ = oracle(wl, [0])
    for impl in ("gemm_tc2", "gemm_tc", "gemm_simt"):
        dw, out = run_gpu(ctx, wl, [0], binds={0: impl})
        assert out.shape == (nb, h, w, n)
        assert np.array_equal(out, ref), impl


def test_bottleneck_block_full_size_sampled_images(ctx):
    """The benchmark's configuration ([32, 56, 56, 256] via 64 channels, default decomposition).  Images are independent
    through every operator of the block, so the oracle checks whole images exactly."""
    from oracle import modules as OM
    wl = W.c9(0)
    dw, out = run_gpu(ctx, wl, wl.partitions["fused"])
    assert dw.module.n_sub() == 1 and dw.module.bound_impl(0) == "gemm_tc2+conv3x3_tc2+gemm_tc2"   # one submodule, three launches
    assert out.shape == (32, 56, 56, 256) and np.isfinite(out).all()
    params = {k: t.f64() for k, t in wl.params.items()}
    x = wl.inputs["x"].f64()
    for n in (0, 13, 31):
        ref, _ = OM.run_module(wl.ops, {"x": x[n:n + 1]}, params, [0])
        assert_parity(out[n:n + 1], ref, "bf16", f"c9 image {n}")
