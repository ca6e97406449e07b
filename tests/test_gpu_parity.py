"""Parity of the CUDA round loop (through the C ABI) with the CPU oracle.

Integer trace (K, selected ids in arrival order, staleness, restarts, end tick,
threshold, communication counter): bit-exact.  Parameters: relative L2 within
1e-5 for fp32 storage and 2e-2 for bf16 storage with fp32 master.
"""
import numpy as np
import pytest

from helpers import compare_with_oracle, gpu_run, rel_l2, to_device
from conftest import make_oracle
from paper_2301_08895_b200 import abs as gpu
from paper_2301_08895_b200 import inputs

pytestmark = pytest.mark.gpu

TOL_FP32, TOL_BF16 = 1e-5, 2e-2


def _problem(cfg):
    X, y, _ = inputs.make_data(cfg)
    return X, y, inputs.make_w0(cfg)


# ------------------------------------------------------------------ the benchmark configurations
def test_config1_lsq_fp32_full():
    cfg = inputs.config(1)
    X, y, w0 = _problem(cfg)
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, cfg.rounds, TOL_FP32)
    assert rows[-1]["K"] == cfg.W and rows[0]["K"] == cfg.K0
    assert any(r["restart"] for r in rows)


def test_config2_softmax_fp32_full():
    cfg = inputs.config(2)
    X, y, w0 = _problem(cfg)
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, cfg.rounds, TOL_FP32)
    assert rows[-1]["K"] == cfg.W


def test_config3_mlp_bf16_prefix():
    cfg = inputs.config(3).scaled(n_samples=16384)
    X, y, w0 = _problem(cfg)
    # forced: the oracle's K rule reads the GPU's uploaded losses (bf16 activations make the two
    # loss streams differ in the 3rd digit, enough to move an Eq. 5 decision by a round)
    compare_with_oracle(cfg, X, y, w0, 100, TOL_BF16, forced=True, loss_tol=5e-2)


def test_config3_free_running_prefix():
    cfg = inputs.config(3).scaled(n_samples=16384)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 25, TOL_BF16, loss_tol=5e-2)


def test_config4_mlp_bf16_prefix():
    cfg = inputs.config(4).scaled(n_samples=8192)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 10, TOL_BF16, forced=True, loss_tol=5e-2)


@pytest.mark.parametrize("W", [256, 1024])
def test_config5_lsq_bf16_reduced(W):
    cfg = inputs.config(5, W).scaled(n_samples=32768)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 40 if W == 256 else 12, TOL_BF16, forced=True, loss_tol=1e-3)


# ------------------------------------------------------------------ ragged shapes and modes
def _small_cfg(kind, dims, dtype, W, B, K0, S, time, n=3000, lr=0.05, seed=5):
    data = "lsq" if kind == inputs.LSQ else "mixture"
    c = inputs.Config("small", kind, tuple(dims), dtype, W, B, K0, S, 60, lr, n, time, data,
                      sigma=1.0, w0="he" if kind == inputs.MLP else "zeros")
    c.data_seed, c.run_seed, c.w0_seed = seed, seed + 1, seed + 2
    return c


EXP = inputs.TimeSpec(inputs.T_EXP, rate=1.0)
SEXP = inputs.TimeSpec(inputs.T_SHIFTED_EXP, shift=0.5, rate=2.0)
PARETO = inputs.TimeSpec(inputs.T_PARETO2, scale=1.0)


@pytest.mark.parametrize("dtype,tol", [(inputs.FP32, TOL_FP32), (inputs.BF16, TOL_BF16)])
@pytest.mark.parametrize("kind,dims,B", [
    (inputs.LSQ, (77, 1), 19),
    (inputs.SOFTMAX, (131, 7), 24),
    (inputs.MLP, (50, 37, 5), 24),
    (inputs.MLP, (200, 136, 72, 10), 40),
])
def test_ragged_shapes(kind, dims, B, dtype, tol):
    cfg = _small_cfg(kind, dims, dtype, 13, B, 3, 5, PARETO)
    X, y, w0 = _problem(cfg)
    forced = dtype == inputs.BF16
    compare_with_oracle(cfg, X, y, w0, 60, tol, forced=forced, loss_tol=5e-2 if forced else None)


@pytest.mark.parametrize("k_mode,bound_mode,K0,S", [
    (gpu.K_FIXED, gpu.BOUND_FIXED, 1, 40),      # ASGD
    (gpu.K_FIXED, gpu.BOUND_ADAPTIVE, 4, 0),    # K-sync: everything restarts
    (gpu.K_FIXED, gpu.BOUND_FIXED, 3, 2),       # K-async with a tight fixed bound
    (gpu.K_ADAPTIVE, gpu.BOUND_FIXED, 2, 3),
    (gpu.K_ADAPTIVE, gpu.BOUND_ADAPTIVE, 11, 0),  # K = N, bound 0: synchronous SGD
])
def test_modes_fixed_k_traces_are_pure_integer(k_mode, bound_mode, K0, S):
    cfg = _small_cfg(inputs.SOFTMAX, (40, 6), inputs.FP32, 11, 16, K0, S, SEXP)
    X, y, w0 = _problem(cfg)
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, 80, TOL_FP32, k_mode=k_mode,
                                              bound_mode=bound_mode)
    if S == 0 and k_mode == gpu.K_FIXED:
        assert all(len(r["restart"]) == 11 - K0 and set(r["tau"]) == {0} for r in rows)
    if K0 == 1:
        assert max(max(r["tau"]) for r in rows) > 11


GAMMA3 = inputs.TimeSpec(inputs.T_GAMMA, shift=0.25, rate=1.5, shape=3)
GAMMA6 = inputs.TimeSpec(inputs.T_GAMMA, shift=0.0, rate=4.0, shape=6)


@pytest.mark.parametrize("kind,dims,dtype,W,B,time", [
    (inputs.LSQ, (24, 1), inputs.FP32, 12, 6, GAMMA3),          # persistent least-squares kernel
    (inputs.SOFTMAX, (40, 6), inputs.FP32, 20, 16, GAMMA6),     # shape 6: second Philox block
    (inputs.MLP, (64, 128, 10), inputs.BF16, 40, 16, GAMMA3),
])
def test_gamma_execution_times(kind, dims, dtype, W, B, time):
    """Gamma-distributed job times (Sec. V-A): the arrival order, ticks and everything downstream
    must match the oracle exactly."""
    cfg = _small_cfg(kind, dims, dtype, W, B, 3, 5, time)
    X, y, w0 = _problem(cfg)
    bf16 = dtype == inputs.BF16
    rows, _, _, _ = compare_with_oracle(cfg, X, y, w0, 50, TOL_BF16 if bf16 else TOL_FP32, forced=bf16,
                                        loss_tol=5e-2 if bf16 else None)
    assert len({r["T_end"] for r in rows}) > 40


@pytest.mark.parametrize("a", [0, -2, -3])
def test_threshold_offset_sweep(a):
    """Eq. 4 with the constant a given, in the setting of the paper's sweep (Sec. V-B: N = 20,
    K0 = 5, a in {0, -2, -3}): traces identical to the oracle's; a smaller a restarts more."""
    cfg = _small_cfg(inputs.SOFTMAX, (40, 6), inputs.FP32, 20, 16, 5, 6, GAMMA3)
    X, y, w0 = _problem(cfg)
    rows, _, _, _ = compare_with_oracle(cfg, X, y, w0, 60, TOL_FP32, bound_mode=gpu.BOUND_OFFSET, bound_offset=a)
    assert rows[0]["theta"] == max(1, 20 // 5 + a)
    assert all(r["theta"] == max(1, 20 // r2["K"] + a) for r, r2 in zip(rows, rows[1:]))
    assert all(max(r["tau"]) <= r0["theta"] for r0, r in zip(rows, rows[1:]))


@pytest.mark.parametrize("kind,dims,dtype,W,B,K0,S,mode", [
    (inputs.SOFTMAX, (40, 6), inputs.FP32, 20, 16, 5, 3, gpu.BOUND_ADAPTIVE),
    (inputs.LSQ, (24, 1), inputs.FP32, 12, 6, 2, 2, gpu.BOUND_FIXED),          # persistent least-squares kernel
    (inputs.MLP, (64, 128, 10), inputs.BF16, 40, 16, 4, 4, gpu.BOUND_ADAPTIVE),
    (inputs.LSQ, (64, 1), inputs.BF16, 300, 8, 30, 1, gpu.BOUND_FIXED),         # bulk-copy pipeline
])
def test_restart_rule_of_eq6_as_printed(kind, dims, dtype, W, B, K0, S, mode):
    """Eq. 6 tests the age before its increment; Algorithm 1 (the default) after it.  With the
    printed rule a worker restarts one round later, so gradients of staleness S + 1 are consumed
    and the model ring holds one more version; the trace must match the oracle's `literal_eq6` run."""
    cfg = _small_cfg(kind, dims, dtype, W, B, K0, S, GAMMA3)
    X, y, w0 = _problem(cfg)
    bf16 = dtype == inputs.BF16
    rows, _, _, _ = compare_with_oracle(cfg, X, y, w0, 50, TOL_BF16 if bf16 else TOL_FP32, forced=bf16,
                                        loss_tol=5e-2 if bf16 else None, bound_mode=mode,
                                        k_mode=gpu.K_FIXED, restart_rule=gpu.RESTART_EQ6)
    assert max(max(r["tau"]) for r in rows) == S + 1          # one round older than Algorithm 1 allows
    assert sum(len(r["restart"]) for r in rows) > 0
    rows_b, _ = gpu_run(cfg, X, y, w0, 50, bound_mode=mode, k_mode=gpu.K_FIXED)
    assert max(max(r["tau"]) for r in rows_b) <= S


def test_threshold_offset_needs_a_large_enough_bound():
    cfg = _small_cfg(inputs.SOFTMAX, (40, 6), inputs.FP32, 20, 16, 5, 3, EXP)
    X, y, w0 = _problem(cfg)
    Xd, yd = to_device(cfg, X, y)
    with pytest.raises(gpu.AbsError) as e:
        gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=5, bound_mode=gpu.BOUND_OFFSET, bound_offset=0)
    assert e.value.code == gpu.EINVAL


@pytest.mark.parametrize("kind,dims,dtype,W,B,U,forced", [
    (inputs.LSQ, (24, 1), inputs.FP32, 8, 6, 10, False),        # the paper's U = 10, N = 8
    (inputs.LSQ, (77, 1), inputs.FP32, 13, 19, 3, True),
    (inputs.LSQ, (64, 1), inputs.BF16, 20, 8, 4, True),
    (inputs.SOFTMAX, (40, 6), inputs.FP32, 11, 16, 5, False),
    (inputs.SOFTMAX, (131, 7), inputs.FP32, 13, 24, 2, True),
    (inputs.SOFTMAX, (48, 10), inputs.BF16, 16, 12, 3, True),
])
def test_local_sgd_steps(kind, dims, dtype, W, B, U, forced):
    """Eq. 2 with U > 1: every job is U local minibatch steps on the worker's own copy of the model;
    trace and parameters must match the oracle's local-SGD runs."""
    cfg = _small_cfg(kind, dims, dtype, W, B, 3, 5, GAMMA3, lr=0.02)
    X, y, w0 = _problem(cfg)
    bf16 = dtype == inputs.BF16
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, 40, TOL_BF16 if bf16 else TOL_FP32, forced=forced,
                                              loss_tol=5e-2 if bf16 else None, local_steps=U)
    assert rows[-1]["loss_mean"] < rows[0]["loss_mean"]


@pytest.mark.parametrize("dims,W,B,U,K0,S", [
    ((64, 128, 10), 8, 16, 4, 3, 5),             # one tensor-core layer; a worker's rows are 16 of a 128-row tile
    ((72, 136, 256, 10), 12, 48, 3, 4, 6),       # two tensor-core layers, ragged widths
    ((64, 64, 128, 7), 5, 130, 2, 2, 3),         # two row tiles per worker (B > 128), odd class count
])
def test_local_sgd_steps_multi_layer_network(dims, W, B, U, K0, S):
    """Eq. 2 with U > 1 on a multi-layer bf16 network: every selected worker owns a copy of the
    model in HBM; a local step of all of them is one pass of the grouped tensor-core kernels."""
    cfg = _small_cfg(inputs.MLP, dims, inputs.BF16, W, B, K0, S, GAMMA3, lr=0.05)
    X, y, w0 = _problem(cfg)
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, 25, TOL_BF16, forced=True, loss_tol=5e-2, local_steps=U)
    assert rows[-1]["loss_mean"] < rows[0]["loss_mean"]


@pytest.mark.parametrize("dims,dtype,W,B,U,K0,S,forced", [
    ((20, 32, 10), inputs.FP32, 8, 16, 4, 3, 5, False),          # FP32-FMA hidden layer, fused output layer; free running
    ((33, 50, 17, 5), inputs.FP32, 9, 70, 3, 2, 4, True),        # odd widths (plain output-layer kernels), two row tiles per worker
    ((24, 40, 24), inputs.FP32, 6, 12, 2, 2, 3, True),           # 24 classes: output layer through the generic tiles
    ((30, 44, 10), inputs.BF16, 7, 20, 3, 3, 5, True),           # bf16 without tensor-core layers (widths not multiples of 8)
])
def test_local_sgd_steps_multi_layer_network_fma_paths(dims, dtype, W, B, U, K0, S, forced):
    """The per-worker local steps through the FP32-FMA layer kernels: fp32 at the fp32 tolerance."""
    cfg = _small_cfg(inputs.MLP, dims, dtype, W, B, K0, S, GAMMA3, lr=0.05)
    X, y, w0 = _problem(cfg)
    bf16 = dtype == inputs.BF16
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, 25, TOL_BF16 if bf16 else TOL_FP32, forced=forced,
                                              loss_tol=5e-2 if bf16 else None, local_steps=U)
    assert rows[-1]["loss_mean"] < rows[0]["loss_mean"]


def test_lock_step_constant_times():
    cfg = _small_cfg(inputs.LSQ, (16, 1), inputs.FP32, 8, 4, 2, 3,
                     inputs.TimeSpec(inputs.T_CONST, shift=3.0))
    X, y, w0 = _problem(cfg)
    rows, params = gpu_run(cfg, X, y, w0, 40, k_mode=gpu.K_FIXED, bound_mode=gpu.BOUND_FIXED)
    for t, r in enumerate(rows):
        assert r["sel"] == [(t * 2) % 8, (t * 2) % 8 + 1]
        assert r["T_end"] == 3 * 2 ** 20 * ((t * 2) // 8 + 1)
        assert r["tau"] == [min(t, 3)] * 2 and r["restart"] == []


def test_straggler_restarts_every_theta_plus_one_rounds():
    time = inputs.TimeSpec(inputs.T_CONST, shift=1.0, slow_mod=5, slow_rem=4, slow_factor=2.0 ** 20)
    cfg = _small_cfg(inputs.LSQ, (16, 1), inputs.FP32, 5, 4, 2, 3, time)
    X, y, w0 = _problem(cfg)
    rows, _ = gpu_run(cfg, X, y, w0, 41, k_mode=gpu.K_FIXED, bound_mode=gpu.BOUND_FIXED)
    for t, r in enumerate(rows):
        assert 4 not in r["sel"] and (4 in r["restart"]) == (t % 4 == 3)
    compare_with_oracle(cfg, X, y, w0, 41, TOL_FP32, k_mode=gpu.K_FIXED, bound_mode=gpu.BOUND_FIXED)


@pytest.mark.parametrize("W,B,K0,S", [(1, 1, 1, 0), (2, 1, 1, 1), (1024, 2, 128, 32), (33, 64, 5, 255)])
def test_edge_sizes(W, B, K0, S):
    cfg = _small_cfg(inputs.LSQ, (24, 1), inputs.FP32, W, B, K0, S, EXP, n=4096, lr=0.02)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 30, TOL_FP32)


def test_many_workers_network():
    cfg = _small_cfg(inputs.SOFTMAX, (32, 4), inputs.FP32, 300, 3, 20, 12, PARETO, n=6000)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 40, TOL_FP32)


# ------------------------------------------------------------------ API behaviour
def test_rounds_in_several_calls_equal_one_call():
    cfg = inputs.config(1)
    X, y, w0 = _problem(cfg)
    rows_a, params_a = gpu_run(cfg, X, y, w0, 50)
    from helpers import to_device
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=50)
    for n in (1, 0, 7, 42):
        ctx.run_rounds(n)
    rows_b = gpu.trace_rows(ctx.get_trace())
    assert rows_a == rows_b and np.array_equal(params_a, ctx.get_params())
    part = gpu.trace_rows(ctx.get_trace(10, 5))
    assert part == rows_a[10:15]
    with pytest.raises(gpu.AbsError) as e:
        ctx.run_rounds(1)
    assert e.value.code == gpu.ENOSPACE
    with pytest.raises(gpu.AbsError) as e:
        ctx.get_trace(45, 10)
    assert e.value.code == gpu.EINVAL
    assert ctx.launch_count() >= 3          # at least one launch per non-empty call
    ctx.close()


def test_host_dataset_entry_gives_same_result():
    cfg = inputs.config(1)
    X, y, w0 = _problem(cfg)
    rows_a, params_a = gpu_run(cfg, X, y, w0, 30)
    ctx = gpu.context_from_config(cfg, X, y, w0, max_rounds=30, data_on_host=True)
    ctx.run_rounds(30)
    assert gpu.trace_rows(ctx.get_trace()) == rows_a
    assert np.array_equal(ctx.get_params(), params_a)
    ctx.close()


def test_divergence_is_reported_and_state_stays_readable():
    cfg = _small_cfg(inputs.LSQ, (16, 1), inputs.FP32, 4, 8, 4, 0, EXP, lr=1e4)
    X, y, w0 = _problem(cfg)
    from helpers import to_device
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd * 100, yd, w0, max_rounds=200)
    with pytest.raises(gpu.AbsError) as e:
        ctx.run_rounds(200)
    assert e.value.code == gpu.EDIVERGED
    done, rc = ctx.rounds_done()
    assert rc == gpu.EDIVERGED and 0 < done < 200
    rows = gpu.trace_rows(ctx.get_trace(0, done))
    assert len(rows) == done and np.all(np.isfinite(ctx.get_params()))
    o = make_oracle(cfg, X * 100, y, w0)
    from oracle import abs_sim
    with pytest.raises(abs_sim.Diverged):
        o.run(200)
    assert abs(len(o.trace) - done) <= 1
    ctx.close()


def test_tick_range_error():
    time = inputs.TimeSpec(inputs.T_CONST, shift=2.0 ** 31)
    cfg = _small_cfg(inputs.LSQ, (16, 1), inputs.FP32, 4, 8, 2, 2, time)
    X, y, w0 = _problem(cfg)
    from helpers import to_device
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=20)
    with pytest.raises(gpu.AbsError) as e:
        ctx.run_rounds(20)
    assert e.value.code == gpu.ERANGE
    ctx.close()


@pytest.mark.parametrize("idx,rounds,n", [(3, 40, 8192), (4, 12, 8192)])
def test_side_stream_overlap_changes_nothing(idx, rounds, n):
    """The server-side kernels of round t+1 run next to the backward pass of round t; switching
    that off (everything on the caller's stream) must give the same bits."""
    cfg = inputs.config(idx).scaled(n_samples=n)
    X, y, w0 = _problem(cfg)
    rows_a, params_a = gpu_run(cfg, X, y, w0, rounds)
    rows_b, params_b = gpu_run(cfg, X, y, w0, rounds, flags=gpu.FLAG_NO_OVERLAP)
    assert rows_a == rows_b
    assert np.array_equal(params_a, params_b)


@pytest.mark.parametrize("dims,W,B", [((3072, 1024, 512, 10), 32, 64), ((320, 520, 264, 10), 13, 40),
                                      ((256, 512, 512, 256, 10), 24, 32)])
def test_merged_backward_launch_matches_separate_launches(dims, W, B):
    """A hidden layer's delta back-propagation and weight gradient share one GEMM launch (two
    problems, tiles dealt to disjoint CTAs); the flag gives each its own launch.  Every output
    element is accumulated over the same rows in the same order either way: identical bits."""
    cfg = _small_cfg(inputs.MLP, dims, inputs.BF16, W, B, 3, 5, PARETO)
    X, y, w0 = _problem(cfg)
    rows_a, params_a = gpu_run(cfg, X, y, w0, 25)
    rows_b, params_b = gpu_run(cfg, X, y, w0, 25, flags=gpu.FLAG_NO_FUSED_BACKWARD)
    assert rows_a == rows_b
    assert np.array_equal(params_a, params_b)
    compare_with_oracle(cfg, X, y, w0, 25, TOL_BF16, forced=True, loss_tol=5e-2)


def test_bf16_network_without_tensor_cores():
    """ABS_FLAG_NO_TENSOR_CORES: the hidden layers of a bf16 network on the FP32-FMA tile kernels
    (same storage points, other summation order)."""
    cfg = _small_cfg(inputs.MLP, (320, 520, 264, 10), inputs.BF16, 13, 40, 3, 5, PARETO)
    X, y, w0 = _problem(cfg)
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=1, flags=gpu.FLAG_NO_TENSOR_CORES)
    assert ctx.plan()["path"] == [0, 0, 2]        # no layer on the tensor-core path
    ctx.close()
    compare_with_oracle(cfg, X, y, w0, 25, TOL_BF16, forced=True, loss_tol=5e-2, flags=gpu.FLAG_NO_TENSOR_CORES)


@pytest.mark.parametrize("d,W,B,K0,S", [(4096, 200, 32, 25, 32), (1000, 160, 19, 7, 6), (2056, 300, 8, 300, 0)])
def test_lsq_bulk_copy_pipeline_and_plain_load_kernels(d, W, B, K0, S):
    """bf16 least squares streams the minibatch rows through shared memory with bulk copies (one
    persistent CTA per SM, items of 8 rows); the flag keeps the kernel that reads rows with plain
    16-byte loads.  Summation orders differ, so the two agree to rounding, and each agrees with
    the oracle (integer trace exactly, with the oracle's K rule fed the uploaded losses)."""
    cfg = _small_cfg(inputs.LSQ, (d, 1), inputs.BF16, W, B, K0, S, EXP, n=20000, lr=0.002)
    X, y, w0 = _problem(cfg)
    rows_a, _, err_a, _ = compare_with_oracle(cfg, X, y, w0, 30, TOL_BF16, forced=True)
    rows_b, _, err_b, _ = compare_with_oracle(cfg, X, y, w0, 30, TOL_BF16, forced=True, flags=gpu.FLAG_NO_BULK_PIPELINE)
    la = np.concatenate([r["sel_loss"] for r in rows_a])
    lb = np.concatenate([r["sel_loss"] for r in rows_b])
    if [r["sel"] for r in rows_a] == [r["sel"] for r in rows_b]:
        assert np.allclose(la, lb, rtol=1e-4, atol=1e-6)


@pytest.mark.parametrize("d,W,B,K0,S", [(8, 300, 1, 40, 3), (40, 280, 7, 280, 0), (4096, 260, 9, 20, 5),
                                         (1032, 1024, 33, 128, 2), (4088, 257, 16, 257, 1)])
def test_lsq_bulk_copy_pipeline_edge_shapes(d, W, B, K0, S):
    """Ragged row groups (B not a multiple of 8, B = 1), one 16-byte vector per row, the widest row,
    more workers than SMs, K = N from the first round."""
    cfg = _small_cfg(inputs.LSQ, (d, 1), inputs.BF16, W, B, K0, S, EXP, n=12000, lr=0.001)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 12, TOL_BF16, forced=True)


@pytest.mark.parametrize("dims,B", [((64, 128, 2), 24), ((200, 256, 16), 40), ((96, 1024, 10), 16),
                                    ((72, 128, 128, 3), 64)])
def test_output_layer_tensor_core_kernel_shapes(dims, B):
    """The mma.sync output-layer kernel at each supported width of the last hidden layer, with 2, 3,
    10 and 16 classes (class rows are padded to 16 inside the kernel)."""
    cfg = _small_cfg(inputs.MLP, dims, inputs.BF16, 13, B, 3, 5, PARETO)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 30, TOL_BF16, forced=True, loss_tol=5e-2)


# Small least-squares problems run all enqueued rounds inside one persistent kernel; the flag
# keeps the one-launch-per-step path in use, and both must agree with the oracle.
@pytest.mark.parametrize("flags", [0, gpu.FLAG_NO_PERSISTENT])
@pytest.mark.parametrize("dims,W,B,K0,S,dtype,tol", [
    ((8, 1), 3, 5, 1, 2, inputs.FP32, TOL_FP32),
    ((24, 1), 40, 7, 6, 9, inputs.BF16, TOL_BF16),
    ((256, 1), 256, 16, 32, 12, inputs.FP32, TOL_FP32),
    ((136, 1), 64, 64, 8, 40, inputs.BF16, TOL_BF16),
])
def test_small_lsq_persistent_and_stepwise_paths(dims, W, B, K0, S, dtype, tol, flags):
    cfg = _small_cfg(inputs.LSQ, dims, dtype, W, B, K0, S, SEXP, n=5000, lr=0.02)
    X, y, w0 = _problem(cfg)
    compare_with_oracle(cfg, X, y, w0, 40, tol, forced=True, flags=flags)
    # one launch covers all rounds of a call on the persistent path
    from helpers import to_device
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=40, flags=flags)
    n0 = ctx.launch_count()
    ctx.run_rounds(17)
    ctx.run_rounds(23)
    launched = ctx.launch_count() - n0
    assert (launched == 2) == (flags == 0)
    ctx.close()
