"""LINEAR_FP8, the block-scaled fp8 GEMM (tcgen05 kind::f8f6f4 with the per-K-block promotion in the epilogue, and
the plain-ALU kernel beside it) against the fp64 oracle: ragged M and N, one to many K blocks, tiles that straddle
weight scale blocks, integer operands with power-of-two scales (bit-exact), a fused elementwise tail, both weight
layouts, Swap between the two kernels, and the benchmark's shape on every element.

Tolerance: the module's activations are bf16, so the bf16 tolerance of every other parity test applies (rtol 2e-2,
atol 2e-2): the fp8 codes and the fp32 scales are inputs, read exactly by both sides; products of two e4m3 values
are exact in fp32, and the fp32 accumulation error over K <= 8192 terms is far below one bf16 ulp of the result."""
import numpy as np
import pytest

import workloads as W
from workloads import generate as G
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu
IMPLS = ("gemm_fp8_tc2", "gemm_fp8_simt")


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


SHAPES = [(256, 128, 128), (300, 256, 200), (128, 384, 136), (1000, 512, 520), (64, 128, 8), (1, 256, 256), (513, 1024, 384),
          (2048, 2048, 1024)]


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("m,k,n", SHAPES)
def test_block_scaled_gemm_matches_the_oracle(ctx, impl, m, k, n):
    w = W.c8(1, M=m, K=k, N=n)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: impl})
    assert dw.module.bound_impl(0) == impl and dw.module.launch_count() == 1
    assert_parity(out, ref, "bf16", f"{impl} {m}x{k}x{n}")


@pytest.mark.parametrize("impl", IMPLS)
def test_integer_operands_and_power_of_two_scales_are_exact(ctx, impl):
    """Every product, every block sum and every scaled partial sum is an integer multiple of a power of two that
    fp32 holds exactly, so the only rounding is the final one to bf16: the kernels must reproduce it bit for bit
    (a wrong scale index, a missed K block or a transposed scale table cannot hide in a tolerance)."""
    m, k, n = 384, 640, 392
    rng = np.random.default_rng(3)
    w = W.c8(0, M=m, K=k, N=n)
    w.inputs["xq"] = G.make("xq", "fp8", rng.integers(-3, 4, (m, k)).astype(np.float32))
    w.params["Wq"] = G.make("Wq", "fp8", rng.integers(-3, 4, (k, n)).astype(np.float32))
    w.inputs["sx"] = G.Tensor("sx", "f32", (2.0 ** rng.integers(-3, 2, (m, k // 128))).astype(np.float32))
    w.params["sw"] = G.Tensor("sw", "f32", (2.0 ** rng.integers(-3, 2, (-(-n // 128), k // 128))).astype(np.float32))
    ref, _ = oracle(w, [0])
    want = W.bf16_bits_to_f64(W.f32_to_bf16_bits(ref.astype(np.float32)))
    dw, out = run_gpu(ctx, w, [0], binds={0: impl})
    bad = np.argwhere(out != want)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:4].tolist()}"


def test_fused_tail_and_decompositions(ctx):
    w = W.c8(2, M=520, K=512, N=264, bias=True)                   # linear_fp8 -> + bias -> SiLU
    ref, _ = oracle(w, None)
    dw, out = run_gpu(ctx, w, w.partitions["fused"])
    assert dw.module.bound_impl(0) == "gemm_fp8_tc2" and dw.module.launch_count() == 1
    assert_parity(out, ref, "bf16", "fused")
    dw2, out2 = run_gpu(ctx, w, w.partitions["per_op"])
    assert [dw2.module.bound_impl(s) for s in range(3)] == ["gemm_fp8_tc2", "eltwise", "eltwise"]
    assert_parity(out2, ref, "bf16", "per operator")


def test_row_major_weights_go_to_the_plain_kernel(ctx):
    from paper_2607_20501_b200 import binding as B
    w = W.c8(0, M=96, K=256, N=72)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], weight_layout=B.MK_LAYOUT_ROW_MAJOR)
    assert dw.module.bound_impl(0) == "gemm_fp8_simt"
    assert_parity(out, ref, "bf16", "row-major weights")


def test_fp8_values_feed_nothing_else(ctx):
    from paper_2607_20501_b200 import MkError
    w = W.c8(0, M=64, K=128, N=64)
    w.ops = [G._op("relu", "y", ["xq"])]
    with pytest.raises(MkError):
        run_gpu(ctx, w, [0])


def test_c8_full_size_every_element(ctx):
    w = W.c8(0)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, w.partitions["fused"])
    assert dw.module.bound_impl(0) == "gemm_fp8_tc2"
    r = assert_parity(out, ref, "bf16", "c8")
    assert r["size"] == 4096 * 4096
