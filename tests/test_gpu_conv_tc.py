"""tcgen05 implicit-GEMM convolution (K2) against the fp64 oracle: exact on integer inputs (any
mismatch is an indexing bug: tap offsets, padding, row wrap, channel blocks), within tolerance on
random inputs with every fused tail, swap against the plain-ALU kernel."""
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


# the last two: more tiles than CTA pairs with a last wave of at most half the pairs, which runs as units of half the
# output channels each (320 and 150 tiles on 74 pairs; C_out 128 and 256)
# ... and image rows wider than one tile's 62 pixels: 63 (a second segment of one pixel), 124 (two full segments), 125,
# 200 (a ragged fourth), 112 x 112 feature maps
SHAPES = [(1, 4, 4, 64, 32), (2, 8, 8, 64, 64), (3, 9, 7, 128, 128), (2, 13, 62, 64, 96), (1, 56, 56, 128, 128),
          (5, 6, 10, 64, 256), (20, 64, 20, 64, 128), (25, 24, 9, 64, 256),
          (1, 8, 63, 64, 64), (2, 5, 124, 64, 32), (1, 9, 125, 128, 128), (1, 6, 200, 64, 96), (2, 112, 112, 64, 64)]


@pytest.mark.parametrize("nb,h,w,c,co", SHAPES)
def test_integer_inputs_are_exact(ctx, nb, h, w, c, co):
    wl = G.c3(0, NB=nb, H=h, W=w, C=c, CO=co, G=4)
    wl.inputs["x"] = G.int_valued(1, 0, (nb, h, w, c), -2, 2, "bf16", "x")
    wl.params["Wc"] = G.int_valued(1, 1, (co, 3, 3, c), -2, 2, "bf16", "Wc")
    wl.ops = wl.ops[:1]
    ref, _ = oracle(wl, [0])
    dw, out = run_gpu(ctx, wl, [0], binds={0: "conv3x3_tc2"})
    want = _bf16_round(ref)
    bad = np.argwhere(out != want)
    assert bad.size == 0, f"{len(bad)} of {out.size} mismatches, first at {bad[:6].tolist()}: got {out[tuple(bad[0])]}, want {want[tuple(bad[0])]}"


@pytest.mark.parametrize("nb,h,w,c,co", [(3, 9, 7, 128, 128), (2, 56, 56, 128, 128)])
def test_conv_chain_matches_the_oracle(ctx, nb, h, w, c, co):
    for seed in range(2):
        wl = W.c3(seed, NB=nb, H=h, W=w, C=c, CO=co, G=32)
        ref, _ = oracle(wl, [0])
        for part in ("fused", "split2", "split3"):
            dw, out = run_gpu(ctx, wl, wl.partitions[part])
            want = "conv3x3_gn_tc2" if part == "fused" else "conv3x3_tc2"
            assert dw.module.bound_impl(0).startswith(want), dw.module.bound_impl(0)
            assert_parity(out, ref, "bf16", f"{part} seed {seed}")


@pytest.mark.parametrize("nb,h,w,c,co,g", [(2, 8, 8, 64, 64, 16), (3, 9, 7, 128, 128, 32), (2, 13, 62, 64, 128, 16), (1, 6, 10, 64, 256, 16),
                                           (2, 5, 33, 64, 32, 1), (4, 56, 56, 128, 128, 32), (20, 64, 20, 64, 128, 32), (25, 24, 9, 64, 256, 8),
                                           (1, 8, 63, 64, 64, 16), (2, 7, 130, 128, 128, 32), (1, 112, 112, 64, 64, 8),
                                           (3, 10, 10, 64, 64, 32), (2, 9, 70, 128, 32, 16)])
def test_groupnorm_statistics_from_the_conv_epilogue(ctx, nb, h, w, c, co, g):
    """The fused form: the convolution's epilogue leaves per-(image, group) partial sums of what it stores
    and the normalisation reads only those (2, 4, 8, 16 and 32 channels per group; image heights that do not
    fill the last tile; widths that leave junk rows in the tile; image rows of several segments).  Swapped against the two-pass GroupNorm."""
    wl = W.c3(2, NB=nb, H=h, W=w, C=c, CO=co, G=g)
    ref, _ = oracle(wl, [0])
    dw, out = run_gpu(ctx, wl, wl.partitions["fused"])
    assert dw.module.bound_impl(0) == "conv3x3_gn_tc2"
    assert_parity(out, ref, "bf16", "fused")
    dw2, out2 = run_gpu(ctx, wl, wl.partitions["split2"])
    assert dw2.module.bound_impl(1) == "groupnorm_nhwc"
    assert np.abs(out - out2).max() <= 4e-2


@pytest.mark.parametrize("nb,h,w,c,co,g", [(2, 8, 8, 64, 64, 16), (3, 9, 7, 128, 128, 32), (2, 13, 62, 64, 128, 4)])
def test_conv_epilogue_statistics_far_from_zero_mean(ctx, nb, h, w, c, co, g):
    """Groups whose mean is some forty standard deviations from zero.  Inputs in {0, 1}, sparse weights in {-1, 0, 1}
    and a bias of 40 to 56 per group make every value the convolution stores a small integer, exact in bf16, so the
    only error left is that of the statistics: the epilogue's partial sums are taken about zero in fp32 (relative
    error of the variance about 2^-24 * mean^2 / var), the two-pass form's about a pivot.  Both must meet the oracle."""
    wl = W.c3(5, NB=nb, H=h, W=w, C=c, CO=co, G=g)
    rng = np.random.default_rng(17)
    wl.inputs["x"] = G.make("x", "bf16", (rng.random((nb, h, w, c)) < 0.5).astype(np.float32))
    sparse = rng.random((co, 3, 3, c)) < 2.0 / (9 * c)
    wl.params["Wc"] = G.make("Wc", "bf16", (sparse * rng.choice([-1.0, 1.0], (co, 3, 3, c))).astype(np.float32))
    wl.params["bias"] = G.make("bias", "bf16", np.repeat(rng.choice([40.0, 48.0, 56.0], g), co // g).astype(np.float32))
    ref, bnd = oracle(wl, list(range(len(wl.ops))))
    y2 = bnd["y2"]
    assert np.array_equal(y2, np.round(y2)) and y2.max() < 256 and y2.min() > 8     # exact in bf16, above the ReLU's cut
    grp = y2.reshape(nb, h * w, g, co // g)
    sd = grp.std(axis=(1, 3))
    assert sd.min() > 0.3 and (np.abs(grp.mean(axis=(1, 3))) / sd).min() > 15.0
    dw, out = run_gpu(ctx, wl, wl.partitions["fused"])
    assert dw.module.bound_impl(0) == "conv3x3_gn_tc2"
    assert_parity(out, ref, "bf16", "fused, far mean")
    dw2, out2 = run_gpu(ctx, wl, wl.partitions["split2"])
    assert dw2.module.bound_impl(1) == "groupnorm_nhwc"
    assert_parity(out2, ref, "bf16", "two-pass, far mean")


def test_swap_conv_kernels(ctx):
    wl = W.c3(0, NB=2, H=12, W=12, C=64, CO=64, G=8)
    ref, _ = oracle(wl, [0])
    for impl in ("conv3x3_tc2", "conv3x3_simt"):
        dw, out = run_gpu(ctx, wl, wl.partitions["split2"], binds={0: impl})
        assert dw.module.bound_impl(0) == impl
        assert_parity(out, ref, "bf16", impl)
