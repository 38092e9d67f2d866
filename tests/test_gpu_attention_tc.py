"""tcgen05 causal attention (K7) against the fp64 oracle: one tile, several key tiles, ragged
sequence lengths, several heads and batches, the packed-QKV view, closed forms, swap against the
plain-ALU kernel."""
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


def _attn_only(w):
    w.ops = w.ops[:1]
    return w


TC_IMPLS = ("attention_tc2", "attention_tc")


@pytest.mark.parametrize("impl", TC_IMPLS)
@pytest.mark.parametrize("b,h,s", [(1, 1, 128), (1, 2, 256), (2, 3, 384), (1, 2, 200), (1, 1, 1000), (2, 2, 64), (1, 1, 1),
                                   (1, 4, 2048), (3, 5, 640)])
def test_attention_matches_the_oracle(ctx, impl, b, h, s):
    for seed in range(2 if s <= 512 else 1):
        w = _attn_only(W.c4(seed, B=b, H=h, S=s, D=128))
        ref, _ = oracle(w, [0])
        dw, out = run_gpu(ctx, w, [0], binds={0: impl})
        assert dw.module.bound_impl(0) == impl
        assert_parity(out, ref, "bf16", f"{impl} B{b} H{h} S{s} seed{seed}")


def _unmasked(w):
    w.ops[0]["kind"] = "attention"
    return w


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("b,h,s", [(1, 1, 128), (2, 3, 384), (1, 2, 200), (1, 1, 1000), (2, 2, 64), (1, 1, 1), (1, 6, 1024), (3, 5, 197)])
def test_head_dim_64_on_the_tensor_cores(ctx, causal, b, h, s):
    """Head dimension 64 (the Transformer block of the paper's ConvolutionalVisionTransformer example has 6 heads of
    64): the composer's own pick must be the one-tile tensor-core kernel, masked and unmasked, ragged lengths
    included (197 = 14 x 14 patches + a class token)."""
    w = _attn_only(W.c4(1, B=b, H=h, S=s, D=64))
    if not causal:
        _unmasked(w)
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0])
    assert dw.module.bound_impl(0) == "attention_tc"
    assert_parity(out, ref, "bf16", f"D64 causal={causal} B{b} H{h} S{s}")
    dw2, out2 = run_gpu(ctx, w, [0], binds={0: "attention_simt"})
    assert np.abs(out - out2).max() <= 4e-2


@pytest.mark.parametrize("b,h,s", [(1, 2, 256), (2, 3, 200), (1, 1, 1000)])
def test_unmasked_one_tile_kernel_at_head_dim_128(ctx, b, h, s):
    w = _unmasked(_attn_only(W.c4(2, B=b, H=h, S=s, D=128)))
    ref, _ = oracle(w, [0])
    for impl in TC_IMPLS:
        dw, out = run_gpu(ctx, w, [0], binds={0: impl})
        assert dw.module.bound_impl(0) == impl
        assert_parity(out, ref, "bf16", f"{impl} unmasked B{b} H{h} S{s}")


def test_encoder_block_with_heads_of_64(ctx):
    """The encoder block at the ConvolutionalVisionTransformer example's head shape: E = 384, 6 heads of 64, packed
    QKV, unmasked attention; every attention of the default decomposition runs on the tensor cores."""
    w = W.c6(0, B=2, S=197, E=384, H=6, F=1536, L=1)
    part = w.partitions["fused_tails"]
    ref, _ = oracle(w, part)
    dw, out = run_gpu(ctx, w, part)
    impls = [dw.module.bound_impl(i) for i in range(dw.module.n_sub())]
    assert impls.count("attention_tc") == 1 and "attention_simt" not in impls, impls
    assert_parity(out, ref, "bf16", "encoder block, heads of 64")


@pytest.mark.parametrize("b,h,s", [(4, 48, 256), (2, 80, 512), (1, 150, 384)])
def test_persistent_ctas_walk_several_items(ctx, b, h, s):
    """More work items than SMs: a CTA of the two-tile kernel then runs several (batch, head, query
    block) items back to back, with the next item's loads and first MMA issued under the current one."""
    w = _attn_only(W.c4(3, B=b, H=h, S=s, D=128))
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: "attention_tc2"})
    assert_parity(out, ref, "bf16", f"B{b} H{h} S{s}")


def test_closed_forms(ctx):
    b, h, s, d = 1, 2, 300, 128
    w = _attn_only(W.c4(0, B=b, H=h, S=s, D=d))
    k = w.inputs["k"].store
    w.inputs["k"] = G.Tensor("k", "bf16", np.broadcast_to(k[:, :, :1], k.shape).copy())   # identical keys
    v = w.inputs["v"].f64()
    pm = np.cumsum(v, axis=2) / np.arange(1, s + 1)[None, None, :, None]     # prefix means of V
    for impl in TC_IMPLS:
        dw, out = run_gpu(ctx, w, [0], binds={0: impl})
        assert_parity(out, pm.transpose(0, 2, 1, 3).reshape(b * s, h * d), "bf16", f"{impl} uniform weights")
        # first query sees only the first key (the diagonal is kept): O = p V / p with p rounded to bf16 in the
        # numerator only, so equal up to one bf16 rounding of a single probability
        assert np.abs(out[0].reshape(h, d) - v[0, :, 0, :]).max() <= 2.0 ** -7 * np.abs(v[0, :, 0, :]).max()


def test_packed_qkv_view_and_swap(ctx):
    w = W.c5(0, B=2, S=160, E=256, H=2, F=64, L=1)
    w.ops = w.ops[:3]            # rmsnorm -> qkv linear -> attention on the packed tensor
    ref, _ = oracle(w, [0])
    outs = {}
    for impl in ("attention_tc2", "attention_tc", "attention_simt"):
        dw, out = run_gpu(ctx, w, [0, 1, 2], binds={2: impl})
        assert dw.module.bound_impl(2) == impl
        assert_parity(out, ref, "bf16", impl)
        outs[impl] = out
    assert np.abs(outs["attention_tc"] - outs["attention_simt"]).max() <= 4e-2
    assert np.abs(outs["attention_tc2"] - outs["attention_simt"]).max() <= 4e-2


def test_c4_block_at_reduced_size(ctx):
    w = W.c4(0, B=2, H=4, S=512, D=128)
    ref, inter = oracle(w, None)
    for part in ("split3", "per_op", "fused"):
        dw, out = run_gpu(ctx, w, w.partitions[part])
        assert "attention_tc" in dw.module.bound_impl(0)
        assert_parity(out, ref, "bf16", part)


@pytest.mark.parametrize("impl", TC_IMPLS)
@pytest.mark.parametrize("step", [3.0, 100.0])
def test_row_maximum_growing_from_key_tile_to_key_tile(ctx, impl, step):
    """Keys whose magnitude grows by a large factor every 128 positions, so the running row maximum
    jumps at every tile boundary.  With step 3 the jumps are some tens of log2 units; with step 100 they
    exceed the whole fp32 exponent range, so a kernel that keeps a stale reference maximum must notice
    and rescale its running output and row sum (the two-tile kernel does so only then)."""
    b, h, s, d = 1, 2, 640, 128
    w = _attn_only(W.c4(5, B=b, H=h, S=s, D=d))
    k = w.inputs["k"].f64()
    gain = 1.0 + step * (np.arange(s) // 128)
    w.inputs["k"] = G.make("k", "bf16", (k * gain[None, None, :, None]).astype(np.float32))
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: impl})
    assert_parity(out, ref, "bf16", impl)


@pytest.mark.parametrize("impl", TC_IMPLS)
def test_scores_far_below_zero_at_the_start_of_a_row(ctx, impl):
    """The first 64 keys score about -100 log2 units against every query: a kernel that starts from a guessed
    reference maximum (0) sees its first partial row sum underflow and has to take the maximum from the data;
    the early queries see ONLY those keys, so nothing later can hide a zero row sum."""
    b, h, s, d = 1, 2, 512, 128
    w = _attn_only(W.c4(9, B=b, H=h, S=s, D=d))
    q = 2.5 + 0.25 * w.inputs["q"].f64()
    k = w.inputs["k"].f64()
    k[:, :, :64, :] = -2.5
    w.inputs["q"] = G.make("q", "bf16", q.astype(np.float32))
    w.inputs["k"] = G.make("k", "bf16", k.astype(np.float32))
    ref, _ = oracle(w, [0])
    dw, out = run_gpu(ctx, w, [0], binds={0: impl})
    assert np.isfinite(out).all()
    assert_parity(out, ref, "bf16", impl)
