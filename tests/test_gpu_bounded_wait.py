"""The exit a bounded wait takes when it runs out: MK_ERR_DEVICE_TIMEOUT reaches the host, the flag clears,
and the device goes on working.

Nothing here hangs or faults the GPU: the self-test kernel is one small CTA that waits, through the wait
routine of the tensor-core kernels, on a barrier nothing arrives at, gives up after about a millisecond
and returns normally (no copies in flight, no tensor memory held)."""
import pytest
import torch

import workloads as W
from tests.parity import assert_parity, oracle, run_gpu

pytestmark = pytest.mark.gpu

LIMIT = 2_000_000          # SM cycles: about a millisecond


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def test_an_expired_wait_is_reported_once_and_the_device_stays_usable(ctx):
    from paper_2607_20501_b200 import MkError, binding as B
    ctx.check()                                                     # clean before
    out = torch.full((6,), -1, dtype=torch.int64, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    st = B.mk_selftest_bounded_wait(ctx.h, LIMIT, out.data_ptr(), stream)
    assert st == B.MK_OK, B.STATUS.get(st, st)
    with pytest.raises(MkError) as e:
        ctx.check()
    assert e.value.status == B.MK_ERR_DEVICE_TIMEOUT
    assert "code 99" in str(e.value)                                # the waiter's code reached the host
    gave_up, released, t_first, t_second, late, t_late = out.cpu().tolist()
    assert gave_up == 0 and released == 0 and late == 0             # every wait returned "not completed"
    assert LIMIT < t_first < 20 * LIMIT                             # after its limit, not at the second waiter's
    assert t_second < 20 * LIMIT                                    # released by the abort flag, far before its own limit
    assert t_late < LIMIT // 10                                     # a wait after the expiry returns at once
    ctx.check()                                                     # reported once: the flag is clear again
    # and a normal forward afterwards is still oracle-parity
    w = W.c2(0, M=384, K=512, N=512)
    ref, _ = oracle(w, [0])
    dw, got = run_gpu(ctx, w, w.partitions["fused"])
    assert dw.module.bound_impl(0) == "gemm_tc2"
    assert_parity(got, ref, "bf16", "c2 after an expired wait")


def test_the_selftest_refuses_unreasonable_limits(ctx):
    from paper_2607_20501_b200 import binding as B
    out = torch.zeros(6, dtype=torch.int64, device="cuda")
    for bad in (0, 10, 10 ** 10):
        assert B.mk_selftest_bounded_wait(ctx.h, bad, out.data_ptr(), 0) == B.MK_ERR_INVALID_ARG
    assert B.mk_selftest_bounded_wait(ctx.h, LIMIT, None, 0) == B.MK_ERR_INVALID_ARG
    ctx.check()
