"""One submodule evaluated in isolation on the inputs the composition gives it (mk_module_forward_sub)."""
import pytest

import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def test_a_submodule_runs_alone_on_what_the_composition_left_it(ctx):
    """mk_module_forward_sub: after a whole forward with the boundary tensors kept, any submodule can be re-run in
    isolation and reproduces its part bit for bit; a range outside the decomposition is refused."""
    import torch
    from paper_2607_20501_b200 import MkError
    from paper_2607_20501_b200.runner import DeviceWorkload, to_host_f64
    w = W.c4(0, B=1, H=2, S=256, D=128)
    dw = DeviceWorkload(ctx, w)
    dw.module.set_decomposition(w.partitions["split3"])
    dw.module.keep_intermediates(True)
    full = to_host_f64(dw.forward().clone())
    h = dw.intermediate("h").clone()
    # wipe the last two submodules' results, then run them alone
    dw.intermediate("h").zero_()
    dw.out.zero_()
    dw.forward_sub(1, 2)
    torch.cuda.synchronize()
    assert torch.equal(dw.intermediate("h"), h)
    assert (to_host_f64(dw.out) == full).all()
    # the last one alone
    dw.out.zero_()
    dw.forward_sub(2)
    torch.cuda.synchronize()
    assert (to_host_f64(dw.out) == full).all()
    for bad in ((3, 1), (-1, 1), (1, 3), (0, 0)):
        with pytest.raises(MkError):
            dw.forward_sub(*bad)
    ctx.check()
