"""The comparison systems of the paper's evaluation (Sec. II-B, Sec. V) in the CUDA round loop:
the staleness-aware step size (SA), runs without Eq. 6's forced restarts (AdaSync, K-async SGD),
and both together (SA-AdaSync), against the oracle's runs with the same switches.
"""
import numpy as np
import pytest

from conftest import make_oracle
from helpers import compare_with_oracle, first_integer_mismatch, gpu_run, to_device
from paper_2301_08895_b200 import abs as gpu
from paper_2301_08895_b200 import inputs
from test_gpu_parity import GAMMA3, PARETO, TOL_BF16, TOL_FP32, _problem, _small_cfg

pytestmark = pytest.mark.gpu

# (kind, dims, dtype, W, B, K0, S, flags, local_steps): one case per kernel that applies the weight
CASES = [
    (inputs.LSQ, (24, 1), inputs.FP32, 12, 6, 3, 6, 0, 1),                        # all rounds in one persistent kernel
    (inputs.LSQ, (77, 1), inputs.FP32, 13, 19, 3, 6, 0, 1),                       # one CTA per worker (odd width)
    (inputs.LSQ, (72, 1), inputs.FP32, 13, 19, 3, 6, gpu.FLAG_NO_PERSISTENT, 1),  # persistent 16-byte-load kernel
    (inputs.LSQ, (1000, 1), inputs.BF16, 40, 19, 5, 8, 0, 1),                     # bulk-copy pipeline
    (inputs.SOFTMAX, (131, 7), inputs.FP32, 13, 24, 3, 6, 0, 1),                  # plain output-layer kernels
    (inputs.SOFTMAX, (784, 10), inputs.FP32, 16, 64, 4, 8, 0, 1),                 # fused ten-class kernel
    (inputs.SOFTMAX, (40, 6), inputs.FP32, 11, 16, 3, 6, 0, 1),                   # fused kernel, other class counts
    (inputs.MLP, (200, 136, 72, 10), inputs.FP32, 13, 40, 3, 6, 0, 1),            # FP32-FMA hidden layers
    (inputs.MLP, (24, 40, 24), inputs.FP32, 6, 12, 2, 5, 0, 1),                   # 24 classes: stand-alone loss kernel
    (inputs.MLP, (320, 520, 256, 10), inputs.BF16, 13, 40, 3, 6, 0, 1),           # tensor-core layers + mma output layer
    (inputs.LSQ, (24, 1), inputs.FP32, 8, 6, 3, 6, 0, 4),                         # local steps, single-layer kernel
    (inputs.SOFTMAX, (48, 10), inputs.BF16, 16, 12, 3, 6, 0, 3),
    (inputs.MLP, (64, 128, 10), inputs.BF16, 8, 16, 3, 6, 0, 3),                  # local steps on a network: uploads weighted in Eq. 3
    (inputs.MLP, (20, 32, 10), inputs.FP32, 8, 16, 3, 6, 0, 3),
]


def _run(case, rounds=40, **kw):
    kind, dims, dtype, W, B, K0, S, flags, U = case
    cfg = _small_cfg(kind, dims, dtype, W, B, K0, S, GAMMA3, lr=0.02 if kind == inputs.LSQ else 0.05)
    X, y, w0 = _problem(cfg)
    bf16 = dtype == inputs.BF16
    if U > 1:
        kw["local_steps"] = U
    return compare_with_oracle(cfg, X, y, w0, rounds, TOL_BF16 if bf16 else TOL_FP32, forced=True,
                               loss_tol=5e-2 if bf16 else None, flags=flags, **kw)


@pytest.mark.parametrize("case", CASES)
def test_staleness_aware_step_size(case):
    """SA on top of ABS: upload k enters Eq. 3 divided by max(1, tau_k)."""
    rows, orows, err, o = _run(case, sa_penalty=1, k_mode=gpu.K_FIXED)
    assert max(max(r["tau"]) for r in rows) >= 2            # the penalty really acts


@pytest.mark.parametrize("case", [CASES[0], CASES[3], CASES[5], CASES[9], CASES[12]])
def test_staleness_aware_step_size_differs_from_plain_runs(case):
    """Same integer trace (fixed K), other parameters: the switch is not a no-op on the GPU."""
    kind, dims, dtype, W, B, K0, S, flags, U = case
    cfg = _small_cfg(kind, dims, dtype, W, B, K0, S, GAMMA3, lr=0.02 if kind == inputs.LSQ else 0.05)
    X, y, w0 = _problem(cfg)
    rows_a, params_a = gpu_run(cfg, X, y, w0, 40, flags=flags, k_mode=gpu.K_FIXED, local_steps=U)
    rows_b, params_b = gpu_run(cfg, X, y, w0, 40, flags=flags, k_mode=gpu.K_FIXED, local_steps=U, sa_penalty=1)
    assert [(r["sel"], r["tau"], r["restart"]) for r in rows_a] == [(r["sel"], r["tau"], r["restart"]) for r in rows_b]
    assert not np.array_equal(params_a, params_b)


@pytest.mark.parametrize("case,sa", [(CASES[0], 0), (CASES[3], 1), (CASES[5], 0), (CASES[5], 1), (CASES[9], 1),
                                     (CASES[12], 1)])
def test_no_forced_restarts(case, sa):
    """AdaSync (adaptive K, no restarts) and SA-AdaSync: staleness beyond the threshold is consumed."""
    kind, dims, dtype, W, B, K0, S, flags, U = case
    case = (kind, dims, dtype, W, B, K0, 60, flags, U)       # room in the version ring for every age that occurs
    rows, orows, err, o = _run(case, rounds=60, restart_rule=gpu.RESTART_NONE, sa_penalty=sa,
                               bound_mode=gpu.BOUND_OFFSET, bound_offset=-2)
    assert all(r["restart"] == [] for r in rows)
    assert any(max(r["tau"]) > r["theta"] for r in rows[1:])         # older than Eq. 4 would have allowed


def test_upload_older_than_the_version_ring_ends_the_run():
    """Without forced restarts a straggler's upload can be older than the staleness bound + 1 model
    versions the context keeps: the run stops at that round with ABS_ESTALE, everything before it
    stays valid and equals the oracle's run."""
    time = inputs.TimeSpec(inputs.T_CONST, shift=1.0, slow_mod=5, slow_rem=4, slow_factor=9.5)
    cfg = _small_cfg(inputs.SOFTMAX, (40, 6), inputs.FP32, 5, 16, 2, 3, time)
    X, y, w0 = _problem(cfg)
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=60, k_mode=gpu.K_FIXED,
                                  restart_rule=gpu.RESTART_NONE)
    with pytest.raises(gpu.AbsError) as e:
        ctx.run_rounds(60)
    assert e.value.code == gpu.ESTALE
    done, rc = ctx.rounds_done()
    assert rc == gpu.ESTALE
    rows = gpu.trace_rows(ctx.get_trace(0, done))
    params = ctx.get_params()
    ctx.close()
    o = make_oracle(cfg, X, y, w0, k_mode=gpu.K_FIXED, restarts=False)
    orows = o.run(done + 1)
    # the oracle keeps every version: its round `done` is the first that consumes an age above the bound
    assert max(orows[done]["tau"]) > cfg.S and all(max(r["tau"]) <= cfg.S for r in orows[:done])
    assert first_integer_mismatch(rows, orows[:done]) is None and done > 5
    o2 = make_oracle(cfg, X, y, w0, k_mode=gpu.K_FIXED, restarts=False)
    o2.run(done)
    assert np.linalg.norm(params - o2.w) <= TOL_FP32 * np.linalg.norm(o2.w)
