import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def oracle_dist(ts):
    """inputs.TimeSpec -> oracle TimeDist (plain field copy)."""
    from oracle import timing
    return timing.TimeDist(ts.kind, ts.shift, ts.rate, ts.scale, ts.slow_mod, ts.slow_rem,
                           ts.slow_factor, ts.shape)


def make_oracle(cfg, X, y, w0, **kw):
    from oracle import abs_sim
    from paper_2301_08895_b200 import inputs
    bf16 = cfg.dtype == inputs.BF16
    return abs_sim.ABSOracle(cfg.kind, cfg.dims, X, y, w0, cfg.batch, cfg.lr, cfg.W, cfg.K0, cfg.S,
                             oracle_dist(cfg.time), cfg.run_seed, quant=bf16,
                             x_is_bf16_bits=bf16, conv=getattr(cfg, "conv", None), **kw)
