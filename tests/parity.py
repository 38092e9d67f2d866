"""Shared helpers of the GPU parity tests: run a workload through the C ABI on the device and
through the fp64 oracle on the host, compare element by element."""
import numpy as np

from oracle import modules as OM
from oracle.compare import check_close


def run_gpu(ctx, w, partition=None, binds=None, keep=False, weight_layout=None):
    from paper_2607_20501_b200 import binding as B
    from paper_2607_20501_b200.runner import DeviceWorkload, to_host_f64
    import torch
    dw = DeviceWorkload(ctx, w, B.MK_LAYOUT_TRANSPOSED if weight_layout is None else weight_layout)
    if partition is not None:
        dw.module.set_decomposition(partition)
    for sub, name in (binds or {}).items():
        dw.module.bind(sub, name)
    if keep:
        dw.module.keep_intermediates(True)
    out = dw.forward()
    torch.cuda.synchronize()
    ctx.check()
    return dw, to_host_f64(out)


def assert_parity(out, ref, dtype, what=""):
    r = check_close(out, ref, dtype)
    assert r["ok"], f"{what}: {r}"
    return r


def oracle(w, partition=None):
    return OM.run_workload(w, partition)
