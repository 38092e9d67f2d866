"""RMSNorm folded across two tensor-core GEMMs (`gemm_prenorm_gemm_tc2`): the GEMM that produces the norm's input
also leaves bf16(x * gamma) and per-row partial sums of x^2, the GEMM that consumes the norm's output multiplies its
accumulator rows by 1 / rms - two launches, no pass over the activation between them.  Against the fp64 oracle of
the unfused operator sequence: ragged shapes, bf16 and fp32 norm inputs, a learnable gamma, a SwiGLU consumer, and
decoder layers whose every residual GEMM -> RMSNorm -> GEMM run is bound to it."""
import numpy as np
import pytest

import workloads as W
from workloads import generate as G
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu
IMPL = "gemm_prenorm_gemm_tc2"


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def _block(seed, M, K1, N1, N2, stream, swiglu=False, gamma=True, bias=True):
    """x -> linear W1 (+ bias) -> + r = h -> RMSNorm(gamma) -> linear W2 [-> SwiGLU] -> GELU = z; y = z + h (N2 = N1): the
    last operator, outside the fused piece, reads h again, which is what makes h an output of the piece."""
    assert N2 == N1
    w = G.Workload("pn", "bf16")
    w.inputs["x"] = G.make("x", "bf16", G._normal(seed, 0, (M, K1)))
    w.inputs["r"] = G.make("r", "bf16", G._normal(seed, 1, (M, N1)))
    w.params["W1"] = G.make("W1", "bf16", G._normal(seed, 2, (K1, N1), std=(1.0 / K1) ** 0.5))
    w.params["b1"] = G.make("b1", "bf16", G._normal(seed, 3, (N1,), std=0.1))
    w.params["g"] = G.make("g", "bf16", G._normal(seed, 4, (N1,), mean=1.0, std=0.2))
    n2w = 2 * N2 if swiglu else N2
    w.params["W2"] = G.make("W2", "bf16", G._normal(seed, 5, (N1, n2w), std=(1.0 / N1) ** 0.5))
    ops = [G._op("linear", "y0", ["x"], {"w": "W1"}, n=N1)]
    if bias:
        ops.append(G._op("bias_add", "y1", [ops[-1]["out"]], {"b": "b1"}))
    ops.append(G._op("residual_add", "h", [ops[-1]["out"], "r"], **({"store": "f32"} if stream == "f32" else {})))
    ops.append(G._op("rmsnorm", "n", ["h"], {"gamma": "g"} if gamma else {}, eps=1e-6))
    ops.append(G._op("linear", "z0", ["n"], {"w": "W2"}, n=n2w))
    if swiglu:
        ops.append(G._op("swiglu", "z1", ["z0"]))
    ops.append(G._op("gelu_tanh", "z", [ops[-1]["out"]]))
    piece_end = len(ops)
    ops.append(G._op("residual_add", "y", ["z", "h"]))
    w.ops = ops
    return w, piece_end


@pytest.mark.parametrize("stream", ["bf16", "f32"])
@pytest.mark.parametrize("M,K1,N1,N2,swiglu", [(256, 64, 256, 256, False), (300, 136, 328, 328, False), (1000, 256, 1024, 1024, True),
                                                (513, 512, 2048, 2048, False), (2048, 128, 512, 512, True)])
def test_folded_rmsnorm_between_two_gemms(ctx, stream, M, K1, N1, N2, swiglu):
    w, end = _block(7, M, K1, N1, N2, stream, swiglu)
    ref, inter = oracle(w, None)
    dw, out = run_gpu(ctx, w, [0, end], binds={0: IMPL}, keep=True)
    assert dw.module.bound_impl(0) == IMPL
    assert dw.module.launch_count() == 3                        # two GEMMs and the trailing addition
    from paper_2607_20501_b200.runner import to_host_f64
    assert_parity(to_host_f64(dw.intermediate("h")), inter["h"], "bf16", "the norm's input, written by the first GEMM")
    assert_parity(to_host_f64(dw.intermediate("z")), inter["z"], "bf16", "the second GEMM's output")
    # the module's output adds two tensors that were each rounded to their storage type at a submodule boundary
    # (z + h can cancel): judged against the boundary values the GPU itself produced, as the local checks do
    got_h, got_z = to_host_f64(dw.intermediate("h")), to_host_f64(dw.intermediate("z"))
    assert_parity(out, got_z + got_h, "bf16", "module output from its own boundary values")
    assert np.abs(out - ref).max() < 0.1
    # the composer's own cover of the same submodule is the three-kernel chain; both agree
    dw2, out2 = run_gpu(ctx, w, [0, end], keep=True)
    assert dw2.module.bound_impl(0) == "gemm_tc2+rowop+gemm_tc2"
    assert_parity(to_host_f64(dw.intermediate("z")), to_host_f64(dw2.intermediate("z")), "bf16", "fused against the chain")


def test_without_gamma_and_without_bias(ctx):
    w, end = _block(3, 384, 128, 768, 768, "f32", gamma=False, bias=False)
    ref, inter = oracle(w, None)
    dw, out = run_gpu(ctx, w, [0, end], binds={0: IMPL}, keep=True)
    from paper_2607_20501_b200.runner import to_host_f64
    assert_parity(to_host_f64(dw.intermediate("z")), inter["z"], "bf16")


def test_decoder_layers_with_every_norm_folded(ctx):
    w = W.c5(1, B=2, S=256, E=1024, H=8, F=1024, L=2)
    ref, inter = oracle(w, None)
    # layer l: ops 10l + (0 n1, 1 qkv, 2 att, 3 o, 4 x1, 5 n2, 6 gu, 7 swiglu, 8 d, 9 x2); op 20: the final norm
    cuts = [0, 1, 2, 3, 8, 12, 13, 18]
    dw, out = run_gpu(ctx, w, cuts, binds={3: IMPL, 4: IMPL, 6: IMPL}, keep=True)
    names = [dw.module.bound_impl(s) for s in range(dw.module.n_sub())]
    assert names == ["rowop", "gemm_tc2", "attention_tc2", IMPL, IMPL, "attention_tc2", IMPL, "gemm_tc2+rowop"]
    assert_parity(out, ref, "bf16", "two decoder layers")
    from paper_2607_20501_b200.runner import to_host_f64
    for name in ("x1_0", "hid_0", "x2_0", "qkv_1", "hid_1"):
        assert_parity(to_host_f64(dw.intermediate(name)), inter[name], "bf16", name)
    # repeated launches give the same bits
    again = to_host_f64(dw.forward())
    assert np.array_equal(again, out)


def test_it_declines_what_it_cannot_fold(ctx):
    from paper_2607_20501_b200 import MkError
    # LayerNorm has a mean: not a per-row scale
    w, end = _block(1, 256, 64, 256, 256, "bf16")
    for o in w.ops:
        if o["out"] == "n":
            o["kind"] = "layernorm"
            o["attrs"]["eps"] = 1e-5
    with pytest.raises(MkError):
        run_gpu(ctx, w, [0, end], binds={0: IMPL})
    # the norm's input is not needed later: the plain chain is the right composition
    w2, end2 = _block(1, 256, 64, 256, 256, "bf16")
    w2.ops = w2.ops[:end2]
    with pytest.raises(MkError):
        run_gpu(ctx, w2, [0], binds={0: IMPL})
