"""Parity at the full workload sizes, in the launch configuration bench.py times (default
decomposition, default bindings, tensor-core kernels): every element where the fp64 oracle
finishes in seconds (C2, C3), and batch element by batch element — they are independent through
every operator, so the oracle of one element is exact for its rows — for C4 and C5, where the
oracle of the whole tensor at once would need tens of GB.  Every batch element is compared, i.e.
every element of every output."""
import numpy as np
import pytest

import workloads as W
from workloads.generate import Tensor
from oracle import modules as OM
from tests.parity import assert_parity, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def test_c2_full_every_element(ctx):
    w = W.c2(0)
    ref, _ = OM.run_workload(w, [0])
    for part in ("fused", "split"):
        dw, out = run_gpu(ctx, w, w.partitions[part])
        assert dw.module.bound_impl(0) == "gemm_tc2"
        r = assert_parity(out, ref, "bf16", f"c2 {part}")
        assert r["size"] == 4096 * 4096


def test_c3_full_every_element(ctx):
    w = W.c3(0)
    ref, _ = OM.run_workload(w, [0])
    for part in ("fused", "split2"):
        dw, out = run_gpu(ctx, w, w.partitions[part])
        assert dw.module.bound_impl(0) == ("conv3x3_gn_tc2" if part == "fused" else "conv3x3_tc2")
        assert_parity(out, ref, "bf16", f"c3 {part}")
    # per (image, group) statistics of the output before the affine: mean 0, variance 1
    g, b = w.params["gamma"].f64(), w.params["beta"].f64()
    z = ((out - b) / g).reshape(32, 56 * 56, 32, 4)
    assert np.abs(z.mean(axis=(1, 3))).max() < 2e-2 and np.abs(z.var(axis=(1, 3)) - 1).max() < 5e-2


def test_c4_full_every_element(ctx):
    w = W.c4(0)
    B, H, S, D = w.inputs["q"].shape
    dw, out = run_gpu(ctx, w, w.partitions["fused"])
    assert dw.module.bound_impl(0) == "attention_tc2+gemm_tc2+rowop"
    assert np.isfinite(out).all()
    assert np.abs((out * out).mean(axis=1) - 1).max() < 2e-2          # RMSNorm, gamma = 1, holds at any size
    for b in range(B):
        sub = W.c4(0, B=1, H=1, S=1, D=D)                              # a shell to carry the slices
        sub.ops, sub.params = w.ops, w.params
        sub.inputs = {k: Tensor(k, "bf16", w.inputs[k].store[b:b + 1]) for k in ("q", "k", "v")}
        sub.inputs["r"] = Tensor("r", "bf16", w.inputs["r"].store[b * S:(b + 1) * S])
        ref, _ = OM.run_workload(sub, [0])
        assert_parity(out[b * S:(b + 1) * S], ref, "bf16", f"c4 batch element {b}")


def test_c5_full_every_element(ctx):
    w = W.c5(0)
    attn = [o for o in w.ops if o["kind"] == "attention_causal"][0]["attrs"]
    B, S = attn["batch"], attn["seq"]
    dw, out = run_gpu(ctx, w, w.partitions["fused_tails"])
    impls = {dw.module.bound_impl(s) for s in range(dw.module.n_sub())}
    assert impls == {"rowop", "gemm_tc2", "attention_tc2"}
    assert np.isfinite(out).all()
    assert np.abs((out * out).mean(axis=1) - 1).max() < 2e-2
    ops1 = [dict(o, attrs=dict(o["attrs"])) for o in w.ops]
    for o in ops1:
        if o["kind"] == "attention_causal":
            o["attrs"]["batch"] = 1
    params = {k: t.f64() for k, t in w.params.items()}
    for b in range(B):
        x = {"x": w.inputs["x"].f64()[b * S:(b + 1) * S]}
        ref, _ = OM.run_module(ops1, x, params, [0])
        assert_parity(out[b * S:(b + 1) * S], ref, "bf16", f"c5 batch element {b}")
