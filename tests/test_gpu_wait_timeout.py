"""Failure path of the device-side waits.

Every wait inside the library's kernels gives up after a time limit, raises the device status and
lets the kernel return.  Here a wait is made to run out on purpose -- a barrier that nothing
signals, 1 ms limit, the library's own wait routine -- and the host side is checked: the error
code, the site, the sticky state, and that the context stays readable and the device usable.
Nothing faults or hangs: the kernel ends by itself after the limit.
"""
import numpy as np
import pytest

from helpers import to_device
from paper_2301_08895_b200 import abs as gpu
from paper_2301_08895_b200 import inputs

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_context_stays_readable():
    import time
    import torch
    cfg = inputs.config(1)
    X, y, _ = inputs.make_data(cfg)
    w0 = inputs.make_w0(cfg)
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=40)
    ctx.run_rounds(10)
    before = ctx.get_params()
    t0 = time.perf_counter()
    with pytest.raises(gpu.AbsError) as e:
        ctx.selftest_wait_timeout(1000)
    assert time.perf_counter() - t0 < 5.0             # gave up after about a millisecond
    assert e.value.code == gpu.ETIMEOUT and "site 900" in str(e.value)
    # sticky: no more rounds on this context
    with pytest.raises(gpu.AbsError) as e2:
        ctx.run_rounds(1)
    assert e2.value.code == gpu.ETIMEOUT
    done, rc = ctx.rounds_done()
    assert done == 10 and rc == gpu.ETIMEOUT
    # what ran before is intact and readable
    assert np.array_equal(ctx.get_params(), before)
    assert len(gpu.trace_rows(ctx.get_trace(0, 10))) == 10
    ctx.close()
    # the device is fine: a fresh context runs
    ctx2 = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=40)
    ctx2.run_rounds(10)
    assert np.array_equal(ctx2.get_params(), before)
    ctx2.close()
    torch.cuda.synchronize()


def test_selftest_rejects_bad_limits():
    cfg = inputs.config(1)
    X, y, _ = inputs.make_data(cfg)
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, inputs.make_w0(cfg), max_rounds=4)
    for bad in (0, -5, 2_000_000):
        with pytest.raises(gpu.AbsError) as e:
            ctx.selftest_wait_timeout(bad)
        assert e.value.code == gpu.EINVAL
    ctx.run_rounds(2)                                  # an argument error is not sticky
    ctx.close()
