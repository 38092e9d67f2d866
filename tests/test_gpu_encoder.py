"""Unmasked (encoder) attention and the post-norm encoder block against the fp64 oracle: every key
visible, ragged last key tiles at every 32-key chunk boundary and inside a chunk, invariances that
only the unmasked operator has, the plain-ALU kernel beside the tensor-core one, and the composed
block (packed-QKV view, residual GEMMs, LayerNorm) at a reduced size and at the benchmark's size."""
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


def _attn_only(b, h, s, seed=0):
    """q, k, v [B, H, S, 128] -> unmasked attention, nothing else."""
    w = W.c4(seed, B=b, H=h, S=s, D=128)
    w.ops = [dict(w.ops[0], kind="attention")]
    return w


@pytest.mark.parametrize("impl", ("attention_tc2", "attention_simt"))
@pytest.mark.parametrize("b,h,s", [(1, 1, 128), (1, 2, 256), (2, 3, 384), (1, 2, 200), (1, 1, 1000), (2, 2, 64), (1, 1, 1),
                                   (1, 2, 96), (1, 1, 33), (1, 1, 129), (1, 2, 160), (1, 1, 255), (1, 1, 257),
                                   (1, 4, 2048), (3, 5, 640)])
def test_unmasked_attention_matches_the_oracle(ctx, impl, b, h, s):
    if impl == "attention_simt" and s > 640:
        pytest.skip("the plain-ALU kernel is covered at the smaller sizes")
    w = _attn_only(b, h, s)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: impl})
    assert dw.module.bound_impl(0) == impl
    assert_parity(out, ref, "bf16", f"{impl} B{b} H{h} S{s}")


def test_the_one_tile_kernel_takes_the_unmasked_operator_too(ctx):
    w = _attn_only(1, 1, 128)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: "attention_tc"})
    assert dw.module.bound_impl(0) == "attention_tc"
    assert_parity(out, ref, "bf16", "one-tile kernel, unmasked")
    dw, _ = run_gpu(ctx, w, [0])
    assert dw.module.bound_impl(0) == "attention_tc2"          # the default cover takes the two-tile kernel


@pytest.mark.parametrize("s", [100 + 3 * i for i in range(12)] + [515, 640, 777])
def test_ragged_key_tails(ctx, s):
    """Keys past S in the last key tile are hidden from every query: every remainder class modulo 32."""
    w = _attn_only(1, 2, s, seed=1)
    ref, _ = oracle(w, [0])
    for impl in ("attention_tc2", "attention_tc"):
        _, out = run_gpu(ctx, w, [0], binds={0: impl})
        assert_parity(out, ref, "bf16", f"{impl} S{s}")


def test_persistent_ctas_walk_several_items(ctx):
    w = _attn_only(2, 80, 512, seed=3)
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0], binds={0: "attention_tc2"})
    assert_parity(out, ref, "bf16", "B2 H80 S512")


def test_invariances_of_the_unmasked_operator(ctx):
    b, h, s, d = 1, 2, 300, 128
    w = _attn_only(b, h, s)
    _, out = run_gpu(ctx, w, [0], binds={0: "attention_tc2"})
    # identical keys -> uniform weights -> every query gets the mean of V
    k = w.inputs["k"].store
    w1 = _attn_only(b, h, s)
    w1.inputs["k"] = G.Tensor("k", "bf16", np.broadcast_to(k[:, :, :1], k.shape).copy())
    v = w.inputs["v"].f64()
    mean_v = np.broadcast_to(v.mean(axis=2, keepdims=True), v.shape).transpose(0, 2, 1, 3).reshape(b * s, h * d)
    _, out1 = run_gpu(ctx, w1, [0], binds={0: "attention_tc2"})
    assert_parity(out1, mean_v, "bf16", "uniform weights")
    # keys and values permuted together: the same output up to the summation order
    perm = np.random.default_rng(7).permutation(s)
    w2 = _attn_only(b, h, s)
    w2.inputs["k"] = G.Tensor("k", "bf16", np.ascontiguousarray(w.inputs["k"].store[:, :, perm]))
    w2.inputs["v"] = G.Tensor("v", "bf16", np.ascontiguousarray(w.inputs["v"].store[:, :, perm]))
    _, out2 = run_gpu(ctx, w2, [0], binds={0: "attention_tc2"})
    assert np.abs(out2 - out).max() <= 2e-2
    # the causal operator's last query sees every key: that row agrees with the unmasked operator
    wc = W.c4(0, B=b, H=h, S=s, D=d)
    wc.ops = wc.ops[:1]
    _, outc = run_gpu(ctx, wc, [0], binds={0: "attention_tc2"})
    assert np.abs(outc[s - 1] - out[s - 1]).max() <= 2e-2
    assert np.abs(outc[: s - 1] - out[: s - 1]).max() > 0.1


@pytest.mark.parametrize("step", [3.0, 100.0])
def test_row_maximum_growing_from_key_tile_to_key_tile(ctx, step):
    """Keys whose magnitude grows by a large factor every 128 positions: the stale reference maximum has to
    be raised, and the running output rescaled, at every tile boundary, for every query."""
    b, h, s = 1, 2, 600
    w = _attn_only(b, h, s, seed=5)
    k = w.inputs["k"].f64()
    gain = 1.0 + step * (np.arange(s) // 128)
    w.inputs["k"] = G.make("k", "bf16", (k * gain[None, None, :, None]).astype(np.float32))
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0], binds={0: "attention_tc2"})
    assert np.isfinite(out).all()
    assert_parity(out, ref, "bf16", f"step {step}")


def test_scores_far_below_zero_at_the_start_of_a_row(ctx):
    """The first 64 keys score about -100 log2 units against every query: the guessed reference maximum (0)
    makes the first partial row sum underflow, and the maximum must then come from the data."""
    b, h, s = 1, 2, 500
    w = _attn_only(b, h, s, seed=9)
    q = 2.5 + 0.25 * w.inputs["q"].f64()
    k = w.inputs["k"].f64()
    k[:, :, :64, :] = -2.5
    w.inputs["q"] = G.make("q", "bf16", q.astype(np.float32))
    w.inputs["k"] = G.make("k", "bf16", k.astype(np.float32))
    ref, _ = oracle(w, [0])
    _, out = run_gpu(ctx, w, [0], binds={0: "attention_tc2"})
    assert np.isfinite(out).all()
    assert_parity(out, ref, "bf16", "underflowing first half")


def test_encoder_block_at_reduced_size(ctx):
    w = W.c6(0, B=2, S=200, E=256, H=2, F=512, L=2)
    for part in ("fused_tails", "per_op", "fused"):
        ref, _ = oracle(w, [0])
        dw, out = run_gpu(ctx, w, w.partitions[part])
        assert_parity(out, ref, "bf16", f"c6 reduced {part}")
    dw, _ = run_gpu(ctx, w, w.partitions["fused_tails"])
    names = [dw.module.bound_impl(i) for i in range(dw.module.n_sub())]
    assert names[:7] == ["gemm_tc2", "attention_tc2", "gemm_tc2", "rowop", "gemm_tc2", "gemm_tc2", "rowop"]


def test_encoder_block_full_size_sampled_batch_elements(ctx):
    """The benchmark's configuration; batch elements are independent through every operator, so the
    oracle checks whole batch elements exactly."""
    w = W.c6(0)
    attn = [o for o in w.ops if o["kind"] == "attention"][0]["attrs"]
    B, S = attn["batch"], attn["seq"]
    dw, out = run_gpu(ctx, w, w.partitions["fused_tails"])
    assert {dw.module.bound_impl(s) for s in range(dw.module.n_sub())} == {"rowop", "gemm_tc2", "attention_tc2"}
    assert np.isfinite(out).all()
    ops1 = [dict(o, attrs=dict(o["attrs"])) for o in w.ops]
    for o in ops1:
        if o["kind"] == "attention":
            o["attrs"]["batch"] = 1
    from oracle import modules as OM
    params = {k: t.f64() for k, t in w.params.items()}
    for b in (0, B - 1):
        x = {"x": w.inputs["x"].f64()[b * S:(b + 1) * S]}
        ref, _ = OM.run_module(ops1, x, params, [0])
        assert_parity(out[b * S:(b + 1) * S], ref, "bf16", f"c6 batch element {b}")
