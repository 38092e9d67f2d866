"""Host-side logic through the C ABI (no GPU): exported symbols, shape inference, decomposition
edits and their transactional behaviour, contracts, implementation listing / binding,
workspace planning."""
import ctypes as C
import os
import re

import pytest

import workloads as W
from paper_2607_20501_b200 import binding as B
from paper_2607_20501_b200 import Context, MkError, Module

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _mod(ctx, w, **kw):
    return Module(ctx, w.ops, {k: (w.dtype, t.shape) for k, t in w.inputs.items()}, **kw)


@pytest.fixture(scope="module")
def ctx():
    return Context(-1)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "mk.h")).read()
    declared = set(re.findall(r"^MK_API [^;(]*?\b(mk_[a-z_]+)\(", header, flags=re.M))
    assert len(declared) >= 27
    lib = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)
    assert B.mk_status_str(0) == b"MK_OK" and B.mk_status_str(-3) == b"MK_ERR_NO_IMPL"


def test_a_result_nobody_reads_is_rejected(ctx):
    w = W.c2(0, 16, 8, 8)
    ops = [dict(o) for o in w.ops]
    ops[3] = dict(ops[3], **{"in": ["y1"]})              # the scale now skips the GELU: y2 is dead
    with pytest.raises(MkError):
        Module(ctx, ops, {k: (w.dtype, t.shape) for k, t in w.inputs.items()})


def test_struct_layouts_match_the_header():
    assert C.sizeof(B.mk_tensor_spec) == 4 + 4 + 8 * 4 + 4 + 4
    assert C.sizeof(B.mk_op_desc) == 4 + 12 + 16 + 16


def test_shape_inference(ctx):
    w = W.c5(0, B=2, S=8, E=16, H=2, F=24, L=1)
    m = _mod(ctx, w)
    assert m.n_ops() == 11
    assert m.value_spec("qkv_0") == (B.MK_BF16, (16, 48), 0)
    assert m.value_spec("att_0") == (B.MK_BF16, (16, 16), 0)
    assert m.value_spec("gu_0") == (B.MK_BF16, (16, 48), 0)
    assert m.value_spec("hid_0") == (B.MK_BF16, (16, 24), 0)
    assert m.value_spec("y") == (B.MK_BF16, (16, 16), 0)
    w4 = W.c4(0, B=2, H=2, S=12, D=8)
    assert _mod(ctx, w4).value_spec("a") == (B.MK_BF16, (24, 16), 0)
    w3 = W.c3(0, NB=2, H=6, W=5, C=8, CO=12, G=4)
    assert _mod(ctx, w3).value_spec("y0") == (B.MK_BF16, (2, 6, 5, 12), 0)


def test_bad_descriptions_are_rejected(ctx):
    w = W.c2(0, 16, 8, 8)
    ops = [dict(o, attrs=dict(o["attrs"])) for o in w.ops]
    ops[4]["attrs"] = {"lo": 1.0, "hi": -1.0}
    with pytest.raises(MkError) as e:
        Module(ctx, ops, {"x": ("bf16", (16, 8))})
    assert e.value.status == B.MK_ERR_INVALID_ARG
    # residual operands of different shape
    w5 = W.c5(0, B=1, S=4, E=8, H=2, F=8, L=1)
    ops = [dict(o) for o in w5.ops]
    ops[4] = dict(ops[4], **{"in": ["o_0", "qkv_0"]})
    with pytest.raises(MkError) as e:
        Module(ctx, ops, {"x": ("bf16", (4, 8))})
    assert e.value.status == B.MK_ERR_SHAPE_MISMATCH
    # groups must divide channels
    w3 = W.c3(0, NB=1, H=4, W=4, C=8, CO=8, G=3)
    with pytest.raises(MkError) as e:
        _mod(ctx, w3)
    assert e.value.status == B.MK_ERR_SHAPE_MISMATCH
    # packed attention with the wrong width
    ops = [dict(o, attrs=dict(o["attrs"])) for o in w5.ops]
    ops[2]["attrs"]["heads"] = 3
    with pytest.raises(MkError):
        Module(ctx, ops, {"x": ("bf16", (4, 8))})


def test_decomposition_edits_are_transactional(ctx):
    w = W.c2(0, 16, 8, 8)
    m = _mod(ctx, w)
    assert m.decomposition() == [0, 1, 2, 3, 4]
    m.set_decomposition([0, 2, 3, 4])
    for bad in ([1, 2], [0, 0], [0, 3, 2], [0, 5], []):
        with pytest.raises((MkError, ValueError)) as e:
            m.set_decomposition(bad)
        assert m.decomposition() == [0, 2, 3, 4]
    assert e.value.status in (B.MK_ERR_CONTRACT_VIOLATION, B.MK_ERR_INVALID_ARG)
    m.fuse(1, 3)
    assert m.decomposition() == [0, 2]
    with pytest.raises(MkError):
        m.fuse(1, 2)                       # runs off the end
    with pytest.raises(MkError):
        m.fuse(0, 1)                       # fusing one submodule is not a fusion
    assert m.decomposition() == [0, 2]
    m.split(1, 3)                          # exactly two pieces
    assert m.decomposition() == [0, 2, 3]
    for sub, at in ((0, 0), (0, 2), (2, 3), (5, 1)):
        with pytest.raises(MkError):
            m.split(sub, at)               # empty half or bad index
    assert m.decomposition() == [0, 2, 3]
    m.total_fuse()
    assert m.decomposition() == [0] and m.n_sub() == 1


def test_contracts(ctx):
    w = W.c5(0, B=2, S=8, E=16, H=2, F=24, L=2)
    m = _mod(ctx, w)
    m.set_decomposition(w.partitions["fused_tails"])
    vid = m.value_id
    ins, outs = m.contract(3)              # out-proj + residual
    assert [i for i, _ in ins] == [vid["att_0"], vid["x"]]
    assert [o for o, _ in outs] == [vid["x1_0"]]
    ins, outs = m.contract(5)              # gate/up GEMM + SwiGLU
    assert [i for i, _ in ins] == [vid["n2_0"]] and [o for o, _ in outs] == [vid["hid_0"]]
    assert outs[0][1] == (B.MK_BF16, (16, 24), 0)
    ins, outs = m.contract(6)              # down-proj + residual, skip edge from x1
    assert [i for i, _ in ins] == [vid["hid_0"], vid["x1_0"]]
    m.total_fuse()
    ins, outs = m.contract(0)
    assert [i for i, _ in ins] == [vid["x"]] and [o for o, _ in outs] == [vid["y"]]
    # a cut that leaves a value read by two later submodules still exports it once
    m.set_decomposition([0, 5, 6])
    ins, outs = m.contract(0)
    assert [o for o, _ in outs] == [vid["x1_0"]]


def test_binding_and_swap(ctx):
    w = W.c2(0, 16, 8, 8)
    m = _mod(ctx, w)
    m.set_decomposition([0, 2, 3, 4])
    before = [m.bound_impl(s) for s in range(4)]
    assert "gemm_simt" in m.impls(0) and m.impls(1) == ["eltwise"]
    with pytest.raises(MkError) as e:
        m.bind(1, "gemm_simt")             # a GEMM kernel cannot run a GELU submodule
    assert e.value.status == B.MK_ERR_NO_IMPL
    with pytest.raises(MkError):
        m.bind(0, "no_such_kernel")
    assert [m.bound_impl(s) for s in range(4)] == before
    m.bind(0, "gemm_simt")
    m.fuse(1, 3)                           # neighbours change, the explicit binding of sub 0 stays
    assert m.bound_impl(0) == "gemm_simt" and m.bound_impl(1) == "eltwise"
    m.bind(0, None)                        # back to the composer's choice
    # a fully fused C4 has no single kernel: the composer covers it with a chain
    w4 = W.c4(0, B=1, H=2, S=8, D=8)
    m4 = _mod(ctx, w4)
    m4.total_fuse()
    assert m4.impls(0) == []
    assert m4.bound_impl(0).count("+") == 2
    with pytest.raises(MkError):
        m4.bind(0, "rowop")


def test_workspace_planning(ctx):
    w = W.c2(0, 64, 32, 48)
    m = _mod(ctx, w)
    m.total_fuse()
    assert m.workspace_size() == 0         # fused: no intermediate reaches memory
    m.set_decomposition([0, 2, 3, 4])
    reuse = m.workspace_size()
    m.keep_intermediates(True)
    keep = m.workspace_size()
    one = 64 * 48 * 2
    assert keep >= 3 * one and reuse <= keep and reuse >= 2 * one
    # GroupNorm needs scratch for its partial sums even when it is the only submodule
    w3 = W.c3(0, NB=2, H=8, W=8, C=16, CO=16, G=4)
    m3 = _mod(ctx, w3)
    m3.set_decomposition([0, 3])
    assert m3.workspace_size() >= 2 * 8 * 8 * 16 * 2 + 2 * 4 * 2 * 4


def test_host_only_context_cannot_launch(ctx):
    w = W.c2(0, 16, 8, 8)
    m = _mod(ctx, w)
    with pytest.raises(MkError) as e:
        m.forward([1 << 20], 1 << 21, None, 0, 0)
    assert e.value.status == B.MK_ERR_NO_DEVICE


def test_fp32_residual_stream_dtypes(ctx):
    """RESIDUAL_ADD with an fp32 store produces an fp32 value next to bf16 activations: the row norm that
    reads it writes the module dtype again, the next residual may read the fp32 value as its second
    operand, and a contraction refuses an fp32 operand in a bf16 module."""
    w = W.c5(0, B=1, S=4, E=8, H=2, F=8, L=1)
    m = _mod(ctx, w)
    assert m.value_spec("x1_0")[0] == B.MK_F32 and m.value_spec("x2_0")[0] == B.MK_F32
    assert m.value_spec("n2_0")[0] == B.MK_BF16 and m.value_spec("y")[0] == B.MK_BF16
    assert m.value_spec("x1_0")[1] == (4, 8)
    # the same module with a bf16 stream: every value is bf16
    wb = W.c5(0, B=1, S=4, E=8, H=2, F=8, L=1, stream="bf16")
    mb = _mod(ctx, wb)
    assert mb.value_spec("x1_0")[0] == B.MK_BF16 and mb.value_spec("x2_0")[0] == B.MK_BF16
    # a linear fed directly from the fp32 stream (no norm in between) is rejected
    ops = [dict(o) for o in w.ops]
    ops[6] = dict(ops[6], **{"in": ["x1_0"]})            # gu_0 = linear(x1_0) instead of linear(n2_0)
    with pytest.raises(MkError):
        Module(ctx, ops, {"x": ("bf16", (4, 8))})
    # contracts carry the dtype across a split at the stream
    m.set_decomposition([0, 5])
    ins, outs = m.contract(1)
    assert any(dt == B.MK_F32 for _, (dt, _, _) in ins)


def test_swap_needs_a_device_and_sane_arguments(ctx):
    w = W.c2(0, 16, 8, 8)
    m = _mod(ctx, w)
    m.set_decomposition(w.partitions["split"])
    n = C.c_int32(7)
    ins = (C.c_void_p * 1)(None)
    outs = (C.c_void_p * 1)(None)
    assert B.mk_module_swap(m.h, ins, outs, None, 0, None, 0, 0.9, C.byref(n), None) == B.MK_ERR_INVALID_ARG
    assert B.mk_module_swap(m.h, ins, outs, None, 0, None, 3, 1.5, C.byref(n), None) == B.MK_ERR_INVALID_ARG
    st = B.mk_module_swap(m.h, ins, outs, None, 0, None, 3, 0.9, C.byref(n), None)
    assert st != B.MK_OK and n.value == 0          # a host-only context cannot time anything
    assert m.n_sub() == 4 and m.bound_impl(1) == "eltwise"    # bindings untouched


def test_unmasked_attention_and_the_encoder_block_on_the_host(ctx):
    """Shape inference, contracts and implementation legality of MK_OP_ATTENTION and of workload C6."""
    w = W.c6(0, B=2, S=24, E=256, H=2, F=64, L=2)
    m = _mod(ctx, w)
    assert m.n_ops() == 28
    assert m.value_spec("qkv_0") == (B.MK_BF16, (48, 768), 0)
    assert m.value_spec("att_1") == (B.MK_BF16, (48, 256), 0)
    assert m.value_spec("x2_1") == (B.MK_BF16, (48, 256), 0)
    m.set_decomposition(w.partitions["fused_tails"])
    assert m.n_sub() == 14
    # the attention submodule: every attention kernel knows the unmasked operator
    assert m.impls(1) == ["attention_tc2", "attention_tc", "attention_simt"]
    ins, outs = m.contract(1)
    vid = m.value_id
    assert [n for n, _ in ins] == [vid["qkv_0"]] and [n for n, _ in outs] == [vid["att_0"]]
    # projection + bias + residual is one GEMM with its tail; the residual's source is a contract input
    ins, outs = m.contract(2)
    assert sorted(n for n, _ in ins) == sorted([vid["att_0"], vid["x"]]) and [n for n, _ in outs] == [vid["r1_0"]]
    assert m.bound_impl(2) == "gemm_tc" and m.bound_impl(3) == "rowop"      # 48 rows: the one-SM form
    # head_dim 64: the one-tile tensor-core kernel and the plain-ALU kernel; head_dim 32: the plain-ALU kernel alone
    w64 = W.c6(0, B=1, S=8, E=128, H=2, F=32, L=1)
    m64 = _mod(ctx, w64)
    m64.set_decomposition(w64.partitions["fused_tails"])
    assert m64.impls(1) == ["attention_tc", "attention_simt"]
    w32 = W.c6(0, B=1, S=8, E=128, H=4, F=32, L=1)
    m32 = _mod(ctx, w32)
    m32.set_decomposition(w32.partitions["fused_tails"])
    assert m32.impls(1) == ["attention_simt"]
    # a packed tensor of the wrong width is rejected at creation
    ops = [dict(o, attrs=dict(o["attrs"])) for o in w.ops]
    ops[2]["attrs"]["heads"] = 3
    with pytest.raises(MkError) as e:
        Module(ctx, ops, {k: (w.dtype, t.shape) for k, t in w.inputs.items()})
    assert e.value.status == B.MK_ERR_SHAPE_MISMATCH


def test_pooling_operators_on_the_host(ctx):
    for pool in ("avg", "max", "lp"):
        w = W.c7(0, NB=2, H=20, W=17, C=8, CO=16, pool=pool, k=3, stride=2)
        m = _mod(ctx, w)
        assert m.value_spec("y3") == (B.MK_BF16, (2, 9, 8, 16), 0)      # floor((20 - 3) / 2) + 1, floor((17 - 3) / 2) + 1
        m.set_decomposition(w.partitions["split2"])
        assert m.impls(1) == ["pool_nhwc"]
        m.total_fuse()
        assert m.bound_impl(0).endswith("+pool_nhwc")                   # no kernel fuses a pooling window into a producer
    bad = W.c7(0, NB=1, H=6, W=6, C=8, CO=8, pool="avg", k=7, stride=7)   # window larger than the image
    with pytest.raises(MkError) as e:
        _mod(ctx, bad)
    assert e.value.status == B.MK_ERR_SHAPE_MISMATCH
    bad = W.c7(0, NB=1, H=8, W=8, C=8, CO=8, pool="lp", k=2, stride=2, p=0.5)
    with pytest.raises(MkError) as e:
        _mod(ctx, bad)
    assert e.value.status == B.MK_ERR_INVALID_ARG
