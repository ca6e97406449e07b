"""The paper's model class in the CUDA round loop (ABS_CNN: two convolution + ReLU + max-pool
blocks in front of fully connected layers, Sec. V-A) against the oracle's CNN runs."""
import numpy as np
import pytest

from helpers import compare_with_oracle, gpu_run, to_device
from paper_2301_08895_b200 import abs as gpu
from paper_2301_08895_b200 import inputs
from test_gpu_parity import GAMMA3, PARETO, TOL_BF16, TOL_FP32, _problem

pytestmark = pytest.mark.gpu

# fp32 storage, long runs: every ReLU and every max-pool is a decision on a binary32 sum.  A
# pre-activation closer to zero (or to its rival in the pool window) than the accumulation error of
# its 75 .. 150 products can fall on the other side than in the binary64 oracle, and then one delta
# is routed differently: an O(1) change of one term of a gradient that, with a few hundred rows per
# round, has only ~1e4 terms per element.  Until the first such flip the two runs agree to binary32
# rounding (measured on the benchmark-shaped network: 7e-8 after 10 rounds, every block below
# 2e-7); a flip between rounds 10 and 30 then leaves 5e-5 on the whole vector and up to 5e-4 of the
# path length on single blocks, without either side being wrong.  So the long fp32 run is compared
# at 1e-3, and the same network is also compared at the plain fp32 tolerance over its first 10 rounds.
TOL_CNN_FP32_LONG = 1e-3


def _cnn_cfg(conv, fc, dtype, W, B, K0, S, time, n=3000, lr=0.01, seed=11):
    H, Wd, c_in, k, c1, c2 = conv
    h2, w2 = ((H - k + 1) // 2 - k + 1) // 2, ((Wd - k + 1) // 2 - k + 1) // 2
    dims = (h2 * w2 * c2,) + tuple(fc)
    c = inputs.Config("cnn_small", inputs.CNN, dims, dtype, W, B, K0, S, 40, lr, n, time, "mixture",
                      sigma=0.5, w0="he", conv=tuple(conv))
    c.data_seed, c.run_seed, c.w0_seed = seed, seed + 1, seed + 2
    return c


@pytest.mark.parametrize("conv,fc,dtype,W,B,rounds,tol", [
    ((14, 14, 2, 3, 3, 4), (7, 6, 5), inputs.FP32, 9, 12, 30, TOL_FP32),            # tiny maps, odd widths everywhere
    ((18, 14, 1, 3, 5, 8), (24, 10), inputs.FP32, 13, 19, 30, TOL_FP32),            # non-square image, two affine layers
    ((32, 32, 3, 5, 6, 16), (120, 84, 10), inputs.FP32, 8, 32, 10, TOL_FP32),       # the benchmark network in fp32
    ((32, 32, 3, 5, 6, 16), (120, 84, 10), inputs.FP32, 8, 32, 30, TOL_CNN_FP32_LONG),
    ((14, 14, 2, 3, 3, 4), (7, 6, 5), inputs.BF16, 9, 12, 30, TOL_BF16),
    ((32, 32, 3, 5, 6, 16), (120, 84, 10), inputs.BF16, 8, 32, 20, TOL_BF16),       # first affine layer on tensor cores (400 -> 120)
    ((22, 22, 3, 3, 8, 16), (128, 64, 10), inputs.BF16, 20, 24, 30, TOL_BF16),      # 256 features -> 128 -> 64 on tensor cores
    ((14, 14, 2, 3, 16, 24), (12, 5), inputs.FP32, 6, 10, 10, TOL_FP32),            # wide blocks: 16 and 24 channels, 3480 parameters in the second one
])
def test_cnn_matches_oracle(conv, fc, dtype, W, B, rounds, tol):
    cfg = _cnn_cfg(conv, fc, dtype, W, B, 3, 5, GAMMA3)
    X, y, w0 = _problem(cfg)
    bf16 = dtype == inputs.BF16
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, rounds, tol, forced=True,
                                              loss_tol=5e-2 if bf16 else 10 * tol)
    assert max(max(r["tau"]) for r in rows) >= 1          # several model versions in play
    assert rows[-1]["loss_mean"] < rows[0]["loss_mean"]


@pytest.mark.parametrize("conv,fc,W,B", [((14, 14, 2, 3, 3, 4), (7, 6, 5), 6, 10),
                                          ((32, 32, 3, 5, 6, 16), (120, 84, 10), 8, 32)])
def test_cnn_gradient_of_one_round_block_by_block(conv, fc, W, B):
    """One synchronous round (K = N, bound 0) from w^0: w^1 - w^0 is -eta/N times the summed
    gradient, so every block of the oracle's gradient (both convolutions, every affine layer,
    weights and biases) is compared on its own, at the plain fp32 tolerance."""
    cfg = _cnn_cfg(conv, fc, inputs.FP32, W, B, W, 0, PARETO)
    X, y, w0 = _problem(cfg)
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, 1, TOL_FP32)
    # the comparison above is of w^1; make it one of the step itself (w^1 - w^0), block by block
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=1)
    ctx.run_rounds(1)
    step_gpu = ctx.get_params().astype(np.float64) - w0
    ctx.close()
    step_ref = o.w - w0
    from helpers import layer_blocks
    for name, sl in layer_blocks(cfg.kind, cfg.dims, cfg.conv):
        e = np.linalg.norm(step_gpu[sl] - step_ref[sl]) / np.linalg.norm(step_ref[sl])
        assert e < 2e-5, (name, e)        # binary32 master: the step is a difference of rounded numbers


def test_cnn_benchmark_configuration_prefix():
    cfg = inputs.config(6).scaled(n_samples=8192)
    X, y, w0 = _problem(cfg)
    rows, orows, err, o = compare_with_oracle(cfg, X, y, w0, 40, TOL_BF16, forced=True, loss_tol=5e-2)
    assert rows[-1]["K"] > rows[0]["K"]


def test_cnn_with_staleness_aware_step_size_and_without_restarts():
    cfg = _cnn_cfg((14, 14, 2, 3, 3, 4), (7, 6, 5), inputs.FP32, 9, 12, 3, 40, GAMMA3)
    X, y, w0 = _problem(cfg)
    rows, _, _, _ = compare_with_oracle(cfg, X, y, w0, 40, TOL_FP32, forced=True, sa_penalty=1,
                                        restart_rule=gpu.RESTART_NONE, k_mode=gpu.K_FIXED)
    assert max(max(r["tau"]) for r in rows) >= 2


def test_cnn_rejects_bad_shapes():
    cfg = _cnn_cfg((14, 14, 2, 3, 3, 4), (7, 6, 5), inputs.FP32, 4, 8, 2, 2, PARETO)
    X, y, w0 = _problem(cfg)
    Xd, yd = to_device(cfg, X, y)
    with pytest.raises(gpu.AbsError) as e:                      # 13 rows after the first convolution: no 2 x 2 pool
        gpu.context_from_config(cfg.scaled(conv=(15, 14, 2, 3, 3, 4)), Xd, yd, w0, max_rounds=2)
    assert e.value.code == gpu.EINVAL
    with pytest.raises(gpu.AbsError) as e:                      # the second block would deliver 2 x 3 x 4 features, not dims[0]
        gpu.context_from_config(cfg.scaled(conv=(14, 18, 2, 3, 3, 4)), Xd, yd, w0, max_rounds=2)
    assert e.value.code == gpu.EINVAL
    with pytest.raises(gpu.AbsError) as e:
        gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=2, local_steps=2)
    assert e.value.code == gpu.EUNSUPPORTED
