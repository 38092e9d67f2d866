"""Swap on the GPU: submodules bound to slow implementations are found by timing and rebound, the rest
of the composition and the result stay as they were (paper: the Swap step, threshold 0.9)."""
import pytest

import workloads as W
from paper_2607_20501_b200.runner import to_host_f64
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def test_slow_bindings_are_swapped_and_fast_ones_kept(ctx):
    w = W.c4(0, B=2, H=4, S=512, D=128)
    ref, _ = oracle(w, None)
    dw, out = run_gpu(ctx, w, w.partitions["split3"], binds={0: "attention_simt", 1: "gemm_simt"})
    assert [dw.module.bound_impl(s) for s in range(3)] == ["attention_simt", "gemm_simt", "rowop"]
    n, times = dw.swap(iters=3, tau=0.9)
    assert n == 2
    assert dw.module.bound_impl(0) in ("attention_tc2", "attention_tc")
    assert dw.module.bound_impl(1) in ("gemm_tc2", "gemm_tc")
    assert dw.module.bound_impl(2) == "rowop"
    for before, after in times[:2]:
        assert after < 0.9 * before
    assert times[2][0] == times[2][1]
    assert_parity(to_host_f64(dw.forward()), ref, "bf16", "after swap")
    # a second pass may still trade one tensor-core form for another (at this size they are within noise of
    # each other), but never goes back to the slow kernels, and the result stays right
    dw.swap(iters=3, tau=0.9)
    assert not any("simt" in dw.module.bound_impl(s) for s in range(3))
    assert_parity(to_host_f64(dw.forward()), ref, "bf16", "after the second swap")


def test_single_submodule_is_left_alone(ctx):
    w = W.c2(0, 256, 128, 256)
    dw, out = run_gpu(ctx, w, w.partitions["fused"], binds={0: "gemm_simt"})
    n, times = dw.swap(iters=2)
    assert n == 0 and dw.module.bound_impl(0) == "gemm_simt"


def test_composer_chosen_chains_survive(ctx):
    """A fused submodule that no single kernel accepts is bound to a chain of pieces; Swap finds no single
    alternative for it and must put the chain back."""
    w = W.c4(1, B=1, H=2, S=256, D=128)
    ref, _ = oracle(w, None)
    cuts = [0, 3]            # {attention, projection, residual} as one submodule, RMSNorm as another
    dw, out = run_gpu(ctx, w, cuts)
    chain = dw.module.bound_impl(0)
    assert "+" in chain
    n, _ = dw.swap(iters=2)
    assert n == 0 and dw.module.bound_impl(0) == chain
    assert_parity(to_host_f64(dw.forward()), ref, "bf16", "chain kept")


def test_swap_on_the_encoder_block(ctx):
    """The unmasked attention bound to the plain-ALU kernel and two residual GEMMs bound to the plain-ALU GEMM are
    found and rebound; the pooling-free, single-implementation submodules (LayerNorm) are left as they are."""
    w = W.c6(0, B=2, S=256, E=256, H=2, F=512, L=1)
    ref, _ = oracle(w, None)
    cuts = w.partitions["fused_tails"]
    dw, out = run_gpu(ctx, w, cuts, binds={1: "attention_simt", 2: "gemm_simt", 5: "gemm_simt"})
    before = [dw.module.bound_impl(s) for s in range(7)]
    assert before[1] == "attention_simt" and before[2] == "gemm_simt" and before[5] == "gemm_simt"
    n, times = dw.swap(iters=3, tau=0.9)
    after = [dw.module.bound_impl(s) for s in range(7)]
    # at this size either tensor-core attention kernel may measure fastest (four work items on 148 SMs)
    assert n >= 3 and after[1] in ("attention_tc2", "attention_tc") and not any("simt" in a for a in after)
    assert after[3] == before[3] == "rowop" and after[6] == before[6] == "rowop"
    assert_parity(to_host_f64(dw.forward()), ref, "bf16", "encoder block after swap")
