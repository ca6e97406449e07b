"""Checkpoint / resume through the C ABI: a run that is saved after n rounds and continued in a
fresh context must be bit-identical (trace and parameters) to the uninterrupted run, which the
parity tests compare with the oracle."""
import numpy as np
import pytest

from paper_2301_08895_b200 import inputs
from helpers import gpu, to_device
from test_gpu_parity import _small_cfg, _problem, EXP, GAMMA3, PARETO

pytestmark = pytest.mark.gpu


def _ctx(cfg, X, y, w0, rounds, **kw):
    Xd, yd = to_device(cfg, X, y)
    return gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=rounds, **kw), (Xd, yd)


@pytest.mark.parametrize("kind,dims,dtype,W,B,K0,S,time,kw", [
    (inputs.LSQ, (32, 1), inputs.FP32, 16, 8, 4, 6, EXP, {}),                                 # all rounds in one kernel
    (inputs.LSQ, (4096, 1), inputs.BF16, 64, 16, 8, 9, PARETO, {}),                           # bulk-copy pipeline
    (inputs.SOFTMAX, (40, 6), inputs.FP32, 12, 16, 3, 5, GAMMA3, {}),
    (inputs.MLP, (64, 128, 128, 10), inputs.BF16, 24, 32, 4, 7, EXP, {}),                     # tensor cores, two streams
    (inputs.MLP, (64, 128, 10), inputs.BF16, 8, 16, 3, 5, GAMMA3, {"local_steps": 3}),        # local steps
    (inputs.SOFTMAX, (24, 5), inputs.FP32, 10, 8, 2, 4, EXP, {"restart_rule": gpu.RESTART_EQ6}),
])
def test_resume_is_bit_identical(kind, dims, dtype, W, B, K0, S, time, kw):
    cfg = _small_cfg(kind, dims, dtype, W, B, K0, S, time, lr=0.02)
    X, y, w0 = _problem(cfg)
    n1, n2 = 13, 17
    a, keep_a = _ctx(cfg, X, y, w0, n1 + n2, **kw)
    a.run_rounds(n1 + n2)
    rows_a, params_a = gpu.trace_rows(a.get_trace()), a.get_params()
    a.close()

    b, keep_b = _ctx(cfg, X, y, w0, n1 + n2, **kw)
    b.run_rounds(n1)
    image = b.save_state()
    b.run_rounds(3)                      # the saving context may go on; the image is a copy
    b.close()

    c, keep_c = _ctx(cfg, X, y, w0, n1 + n2, **kw)
    c.restore_state(image)
    assert c.rounds_done()[0] == n1
    c.run_rounds(n2)
    rows_c, params_c = gpu.trace_rows(c.get_trace()), c.get_params()
    c.close()
    assert rows_c == rows_a
    assert np.array_equal(params_c.view(np.uint32), params_a.view(np.uint32))


def test_restore_rejects_an_image_of_another_run():
    cfg = _small_cfg(inputs.LSQ, (32, 1), inputs.FP32, 16, 8, 4, 6, EXP, lr=0.02)
    X, y, w0 = _problem(cfg)
    a, keep = _ctx(cfg, X, y, w0, 20)
    a.run_rounds(5)
    image = a.save_state()
    a.close()
    import dataclasses
    other = dataclasses.replace(cfg, run_seed=cfg.run_seed + 1)
    b, keep_b = _ctx(other, X, y, w0, 20)
    with pytest.raises(gpu.AbsError) as e:
        b.restore_state(image)
    assert e.value.code == gpu.EINVAL
    with pytest.raises(gpu.AbsError) as e:
        b.restore_state(image[:100])
    assert e.value.code == gpu.EINVAL
    b.run_rounds(4)                      # the refused restore left the context usable
    assert b.rounds_done()[0] == 4
    b.close()
    c, keep_c = _ctx(cfg, X, y, w0, 30)  # other trace capacity
    with pytest.raises(gpu.AbsError) as e:
        c.restore_state(image)
    assert e.value.code == gpu.EINVAL
    c.close()
    # same sizes, other hyper-parameters: the image carries the model description and the modes
    for kw_other, cfg_other in (({}, dataclasses.replace(cfg, lr=0.03)),               # step size
                                ({"local_steps": 3}, cfg),                               # U (the upload block keeps its size)
                                ({"sa_penalty": 1}, cfg),                                # staleness-aware step size
                                ({"restart_rule": gpu.RESTART_NONE}, cfg),               # no forced restarts
                                ({"flags": gpu.FLAG_NO_PERSISTENT}, cfg)):               # another kernel path
        d, keep_d = _ctx(cfg_other, X, y, w0, 20, **kw_other)
        with pytest.raises(gpu.AbsError) as e:
            d.restore_state(image)
        assert e.value.code == gpu.EINVAL, kw_other
        d.close()
