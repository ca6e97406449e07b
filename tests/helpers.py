"""Shared helpers of the parity tests: run the CUDA library and the oracle on
the same seeded inputs and compare."""
import numpy as np

from conftest import make_oracle
from paper_2301_08895_b200 import abs as gpu
from paper_2301_08895_b200 import inputs

INT_FIELDS = ("K", "sel", "tau", "restart", "T_end", "theta", "comm")


def to_device(cfg, X, y):
    import torch
    if cfg.dtype == inputs.BF16:
        Xd = torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        Xd = torch.from_numpy(X).cuda()
    return Xd, torch.from_numpy(y).cuda()


def gpu_run(cfg, X, y, w0, rounds, **kw):
    Xd, yd = to_device(cfg, X, y)
    ctx = gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=rounds, **kw)
    ctx.run_rounds(rounds)
    rows = gpu.trace_rows(ctx.get_trace())
    params = ctx.get_params()
    ctx.close()
    return rows, params


def first_integer_mismatch(rows_a, rows_b):
    for t, (a, b) in enumerate(zip(rows_a, rows_b)):
        for f in INT_FIELDS:
            if a[f] != b[f]:
                return t, f, a[f], b[f]
    if len(rows_a) != len(rows_b):
        return min(len(rows_a), len(rows_b)), "length", len(rows_a), len(rows_b)
    return None


def rel_l2(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def layer_blocks(kind, dims, conv=None):
    """(name, slice) of every W_l and b_l inside the flat parameter vector (layout of w0)."""
    if kind == inputs.LSQ:
        return [("w", slice(0, dims[0]))]
    out, off = [], 0
    if kind == inputs.CNN:
        _, _, c_in, k, c1, c2 = conv
        for name, ci, co in (("conv1", c_in, c1), ("conv2", c1, c2)):
            n_w = k * k * ci * co
            out.append(("W_" + name, slice(off, off + n_w)))
            out.append(("b_" + name, slice(off + n_w, off + n_w + co)))
            off += n_w + co
    for l in range(len(dims) - 1):
        n_w, n_b = dims[l] * dims[l + 1], dims[l + 1]
        out.append(("W%d" % (l + 1), slice(off, off + n_w)))
        out.append(("b%d" % (l + 1), slice(off + n_w, off + n_w + n_b)))
        off += n_w + n_b
    return out


# fp32 storage: a block of a few dozen numbers sees single ReLU decisions that fall differently in
# binary32 and binary64 (a pre-activation within rounding of zero) much more than the whole vector
# does; seen: up to 1.1x the whole-vector tolerance on a 50-element bias.  Blocks of fp32 runs get
# this factor; a block that is actually wrong is off by 1e-1 or more of its movement.
BLOCK_SLACK_FP32 = 4.0


def assert_params_close(cfg, params, ref, tol, path=None):
    """Relative L2 of the whole vector within tol, and every layer block (each W_l, each b_l) within
    tol (fp32 storage: BLOCK_SLACK_FP32 * tol) of max(norm of the block, length of the path the block travelled): a wrong bias vector
    moves the norm of millions of weights by less than any tolerance, so the whole-vector figure
    alone would not see it.

    `path[name]` = sum over the rounds of the norm of the block's update in the oracle's run.  Each
    round's update is computed to a relative accuracy of about tol, and those errors add up along
    the path, whatever the block's final value is; a small bias block whose signed updates
    largely cancel ends close to where it started, and measuring its error against its final norm
    alone would ask for more than the arithmetic gives.  A block that is actually wrong (a dropped
    or doubled contribution) is off by the norm of its own movement and still fails.  Without
    `path` the block's own norm is the yardstick."""
    err = rel_l2(params, ref)
    assert err <= tol, "parameters differ: rel L2 %.3g > %.3g" % (err, tol)
    ref = np.asarray(ref, np.float64)
    got = np.asarray(params, np.float64)
    for name, sl in layer_blocks(cfg.kind, cfg.dims, getattr(cfg, "conv", None)):
        scale = max(np.linalg.norm(ref[sl]), 0.0 if path is None else path[name])
        if scale == 0.0:
            assert np.linalg.norm(got[sl]) == 0.0, "block %s should be zero" % name
            continue
        e = np.linalg.norm(got[sl] - ref[sl]) / scale
        btol = tol if cfg.dtype == inputs.BF16 else BLOCK_SLACK_FP32 * tol
        assert e <= btol, "parameter block %s differs: %.3g of max(norm, path) > %.3g" % (name, e, btol)
    return err


def oracle_run_with_paths(cfg, o, rounds, forced_losses=None):
    """o.run(rounds), also returning per layer block the summed norm of the per-round updates."""
    blocks = layer_blocks(cfg.kind, cfg.dims, getattr(cfg, "conv", None))
    path = {name: 0.0 for name, _ in blocks}
    rows = []
    for i in range(rounds):
        before = o.w.copy()
        rows.append(o.round(None if forced_losses is None else forced_losses[i]))
        for name, sl in blocks:
            path[name] += float(np.linalg.norm(o.w[sl] - before[sl]))
    return rows, path


def compare_with_oracle(cfg, X, y, w0, rounds, tol, forced=False, loss_tol=None, **kw):
    """GPU run vs oracle run.  forced=False: both run freely and the integer
    traces must be identical.  forced=True: the oracle's K rule is fed the
    GPU's uploaded losses (its own losses and parameters are still its own),
    which separates the integer machinery from last-bit loss differences."""
    gkw = {k: v for k, v in kw.items() if k in ("k_mode", "bound_mode", "bound_offset", "local_steps")}
    literal = kw.get("restart_rule", 0) == gpu.RESTART_EQ6
    sa = int(kw.get("sa_penalty", 0))
    rows, params = gpu_run(cfg, X, y, w0, rounds, flags=kw.get("flags", 0),
                           restart_rule=kw.get("restart_rule", 0), sa_penalty=sa, **gkw)
    assert len(rows) == rounds
    o = make_oracle(cfg, X, y, w0, literal_eq6=literal, sa_penalty=bool(sa),
                    restarts=kw.get("restart_rule", 0) != gpu.RESTART_NONE, **gkw)
    orows, path = oracle_run_with_paths(cfg, o, rounds, [r["sel_loss"] for r in rows] if forced else None)
    mm = first_integer_mismatch(rows, orows)
    assert mm is None, "integer trace differs at round %s field %s: gpu %s oracle %s (oracle " \
        "decision margin %.3g)" % (mm + (o.min_margin,))
    err = assert_params_close(cfg, params, o.w, tol, path)
    lt = loss_tol if loss_tol is not None else tol * 10
    for t, (a, b) in enumerate(zip(rows, orows)):
        la, lb = np.array(a["sel_loss"]), np.array(b["sel_loss"])
        assert np.all(np.abs(la - lb) <= lt * np.maximum(1.0, np.abs(lb))), \
            "uploaded losses differ in round %d" % t
    return rows, orows, err, o
