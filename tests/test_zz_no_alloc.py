"""The allocation-free GroupNorm entry point, for callers that cannot give the library a workspace
because they cannot allocate device memory where they call it (inside a framework's planned
memory region, from a plugin that only receives its input/output buffers, in a loop that must not
synchronise on cudaMalloc).  It must give what the composed path's GroupNorm gives - and, judged
on its own, what the fp64 oracle's GroupNorm gives - on two calls in a row that share its built-in
scratch array, must leave the device's free memory as it found it, and must refuse problems that
array cannot hold.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test."""
import gc

import numpy as np
import pytest
import torch

from workloads import generate as G
from oracle import ops as O
from oracle.compare import check_close

pytestmark = pytest.mark.gpu


def _module_groupnorm(ctx, x, gamma, beta, groups, eps, dtype):
    """The existing entry point: a one-operator module run through mk_module_forward."""
    from paper_2607_20501_b200.runner import DeviceWorkload
    w = G.Workload("gn", dtype)
    w.inputs["x"] = G.make("x", dtype, x)
    w.params["gamma"] = G.make("gamma", dtype, gamma)
    w.params["beta"] = G.make("beta", dtype, beta)
    w.ops = [G._op("groupnorm", "y", ["x"], {"gamma": "gamma", "beta": "beta"}, groups=groups, eps=eps)]
    dw = DeviceWorkload(ctx, w)
    out = dw.forward().clone()
    torch.cuda.synchronize()
    return dw, out


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_groupnorm_matches_the_workspace_path_twice_in_a_row(dtype):
    from paper_2607_20501_b200 import Context, binding as B
    ctx = Context(0)
    rng = np.random.default_rng(11)
    shapes = [((4, 14, 14, 128), 32), ((3, 9, 7, 24), 3)]     # second call: other shape, stale scratch
    stream = torch.cuda.current_stream().cuda_stream
    for shape, groups in shapes:
        c = shape[-1]
        x = (rng.standard_normal(shape) + 0.3).astype(np.float32)
        gamma = (1 + 0.1 * rng.standard_normal(c)).astype(np.float32)
        beta = (0.1 * rng.standard_normal(c)).astype(np.float32)
        dw, ref = _module_groupnorm(ctx, x, gamma, beta, groups, 1e-5, dtype)
        y = torch.full_like(ref, float("nan"))
        g, b = dw.params["gamma"][0], dw.params["beta"][0]
        gc.collect()            # tensors left over from earlier tests must not be freed between the two readings
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        st = B.mk_groupnorm_nhwc_noalloc(B.DTYPE[dtype], dw.inputs["x"].data_ptr(), y.data_ptr(), g.data_ptr(),
                                         b.data_ptr(), *shape, groups, 1e-5, stream)
        assert st == B.MK_OK, B.STATUS.get(st, st)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        rtol, atol = (2e-2, 2e-2) if dtype == "bf16" else (1e-4, 1e-5)
        a, r = y.double().cpu().numpy(), ref.double().cpu().numpy()
        assert np.isfinite(a).all()
        assert (np.abs(a - r) <= atol + rtol * np.abs(r)).all()
        # and against the definition itself, on the bytes the device was given
        w = dw.w
        want = O.groupnorm_nhwc(w.inputs["x"].f64(), w.params["gamma"].f64(), w.params["beta"].f64(), groups, 1e-5)
        res = check_close(a, want, dtype)
        assert res["ok"], res
        # a warm call (the set-up of this device is done) must not move the device's free memory:
        # torch's allocator cannot see a cudaMalloc made inside the library, the driver's own count can
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        st = B.mk_groupnorm_nhwc_noalloc(B.DTYPE[dtype], dw.inputs["x"].data_ptr(), y.data_ptr(), g.data_ptr(),
                                         b.data_ptr(), *shape, groups, 1e-5, stream)
        assert st == B.MK_OK
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, (free0, free1)
        assert check_close(y.double().cpu().numpy(), want, dtype)["ok"]
    ctx.check()


def test_noalloc_groupnorm_rejects_what_its_scratch_cannot_hold():
    from paper_2607_20501_b200 import binding as B
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    p = x.data_ptr()
    # 4096 images x up to 64 chunks x 512 groups x 8 bytes is far beyond 1 MiB: refused before any launch
    st = B.mk_groupnorm_nhwc_noalloc(B.MK_BF16, p, p, None, None, 4096, 64, 64, 512, 512, 1e-5, 0)
    assert st == B.MK_ERR_WORKSPACE_TOO_SMALL
    assert B.mk_groupnorm_nhwc_noalloc(B.MK_BF16, p, p, None, None, 1, 4, 4, 10, 3, 1e-5, 0) == B.MK_ERR_SHAPE_MISMATCH
    assert B.mk_groupnorm_nhwc_noalloc(B.MK_BF16, None, p, None, None, 1, 4, 4, 8, 2, 1e-5, 0) == B.MK_ERR_INVALID_ARG
    assert B.mk_groupnorm_nhwc_noalloc(B.MK_BF16, p, p, None, None, 1, 4, 4, 8, 2, -1.0, 0) == B.MK_ERR_INVALID_ARG
    assert B.mk_groupnorm_nhwc_noalloc(B.MK_BF16, p, p, None, None, 1, 4, 4, 8, 2, float("nan"), 0) == B.MK_ERR_INVALID_ARG
    # more images than a grid dimension holds (the scratch check alone would let groups = 1 through), and
    # extents whose product leaves 64 bits: refused as shapes, not launched
    assert B.mk_groupnorm_nhwc_noalloc(B.MK_BF16, p, p, None, None, 70000, 1, 1, 8, 1, 1e-5, 0) == B.MK_ERR_SHAPE_MISMATCH
    assert B.mk_groupnorm_nhwc_noalloc(B.MK_BF16, p, p, None, None, 1, 2 ** 40, 2 ** 40, 8, 1, 1e-5, 0) == B.MK_ERR_SHAPE_MISMATCH
    torch.cuda.synchronize()
