#!/usr/bin/env python
"""Benchmark of the ABS round loop on B200: worker-gradients/s and rounds/s.

A step is one complete run of the chosen configuration (all of its rounds from
w^0) through the C ABI.  `value` times the rounds with CUDA events on the
library's stream with the dataset already resident in HBM; `e2e` times the same
run from pinned host buffers (dataset + w^0 copied in, parameters + trace read
back).  One extra, untimed-for-`value` step runs with an event pair around every
kernel launch to get per-kernel durations for the roofline objects.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--rounds R]
    python bench.py --impl reference ...     # times the CPU oracle instead
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2301_08895_b200 import inputs  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (read + write) per launch at K = N on configuration 4, from ncu captures of the GEMM and the
# Eq. 3 kernel (summaries under profiles/); each figure is valid only for the kernel source it was taken
# from (first 16 hex digits of the file's sha256).
TRAFFIC = {"gemm": {"config": 4, "bytes_per_launch": 44.2e6, "file": "tc.cuh", "sha256_16": "041b65e9b34f49da",
                    "source": "ncu capture of the four GEMM launches of one round, profiles/tc_gemm_kernel_cfg4.md"},
           "update": {"config": 4, "bytes_per_launch": 63.7e6, "file": "simt.cuh", "sha256_16": "c178f6ac2b11a58b",
                      "source": "ncu capture of two launches, profiles/update_kernel_cfg4.md"}}
METRIC = "worker_gradients_per_sec"
UNIT = "worker-gradients/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def measured_traffic(which, config_index, full_size):
    import hashlib
    t = TRAFFIC[which]
    path = os.path.join(ROOT, "paper_2301_08895_b200", "csrc", t["file"])
    with open(path, "rb") as f:
        sha = hashlib.sha256(f.read()).hexdigest()[:16]
    if full_size and config_index == t["config"] and sha == t["sha256_16"]:
        return t["bytes_per_launch"]
    return None            # kernel changed since the counters were taken (or another workload)


def workload_name(cfg, rounds):
    return "%s: dims %s, W=%d, B=%d, K0=%d, S=%d, %d samples, %d rounds" % (
        cfg.name, "-".join(str(d) for d in cfg.dims), cfg.W, cfg.batch, cfg.K0, cfg.S, cfg.n_samples, rounds)


# ------------------------------------------------------------------ flop / byte models
def per_wg_flops(cfg):
    """Algorithmic flops of one worker-gradient, per kernel class: 2*B*in*out per layer for the
    forward pass, the same for the weight gradient, and for back-propagated deltas of layers >= 2."""
    B, dims = cfg.batch, cfg.dims
    if cfg.kind == inputs.LSQ:
        return {"lsq": 4.0 * B * dims[0]}
    nl = len(dims) - 1
    hidden = [2.0 * B * dims[l] * dims[l + 1] for l in range(nl - 1)]
    last = 2.0 * B * dims[nl - 1] * dims[nl]
    out = {"fwd": sum(hidden), "wgrad": sum(hidden), "dgrad": sum(hidden[1:]),
           "output": last * (3 if nl > 1 else 2)}
    if cfg.kind == inputs.CNN:
        # convolution blocks: 2 k k C_in C_out flops per output pixel forward; the weight gradient only
        # sees the pooled positions (a quarter of the pixels); the second block also back-propagates
        H, W, c_in, k, c1, c2 = cfg.conv
        h1, w1 = H - k + 1, W - k + 1
        h2, w2 = h1 // 2 - k + 1, w1 // 2 - k + 1
        f1, f2 = 2.0 * k * k * c_in * c1 * h1 * w1, 2.0 * k * k * c1 * c2 * h2 * w2
        out["conv"] = B * (f1 + f2 + 0.25 * (f1 + f2) + f2)
        out["dgrad"] = sum(hidden)          # the first affine layer back-propagates into the features too
    return out


def n_params(cfg):
    return inputs.n_params(cfg.kind, cfg.dims, cfg.conv)


def padded_rows(tr, B, RB):
    """Gradient rows the kernels process per round: the arrivals are grouped by staleness (= model
    version) and every group's rows are padded to a multiple of RB, so that a row tile never
    straddles two versions.  Returns (rows with padding, real rows) summed over the rounds."""
    padded = real = 0
    off, tau = tr["sel_off"], tr["sel_tau"]
    for t in range(len(tr["K"])):
        _, counts = np.unique(tau[off[t]:off[t + 1]], return_counts=True)
        padded += int(sum((c * B + RB - 1) // RB * RB for c in counts))
        real += int(counts.sum()) * B
    return padded, real


# ------------------------------------------------------------------ clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6),
                              ("sw_thermal_slowdown", 7), ("sw_power_cap", 8)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------ oracle (CPU) arm
def oracle_for(cfg, X, y, w0, local_steps=1, k_fixed=False):
    from oracle import abs_sim, timing
    ts = cfg.time
    bf16 = cfg.dtype == inputs.BF16
    return abs_sim.ABSOracle(cfg.kind, cfg.dims, X, y, w0, cfg.batch, cfg.lr, cfg.W, cfg.K0, cfg.S,
                             timing.TimeDist(ts.kind, ts.shift, ts.rate, ts.scale, ts.slow_mod,
                                             ts.slow_rem, ts.slow_factor, ts.shape),
                             cfg.run_seed, quant=bf16, x_is_bf16_bits=bf16, local_steps=local_steps,
                             k_mode=abs_sim.K_FIXED if k_fixed else abs_sim.K_ADAPTIVE, conv=cfg.conv)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [int(i.get("num_threads", 1)) for i in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def time_oracle(cfg, X, y, w0, rounds, budget_s, local_steps=1, k_fixed=False):
    """Runs the oracle on the first rounds of the workload until `budget_s` of CPU work is spent
    (at least 2 rounds, at most `rounds`)."""
    o = oracle_for(cfg, X, y, w0, local_steps, k_fixed)
    t0 = time.perf_counter()
    done = 0
    while done < rounds:
        o.round()
        done += 1
        if done >= 2 and time.perf_counter() - t0 >= budget_s:
            break
    dt = time.perf_counter() - t0
    wg = sum(r["K"] for r in o.trace)
    return {"value": wg / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": "first %d of %d rounds (%d worker-gradients) in %.1f s" % (done, rounds, wg, dt),
            "rounds_per_sec": done / dt}


# ------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--config", type=int, default=4, help="1..5: the benchmark configurations; 6: the paper's CNN")
    ap.add_argument("--workers", type=int, default=None, help="W of configuration 5")
    ap.add_argument("--rounds", type=int, default=None, help="rounds per step (default: the configuration's)")
    ap.add_argument("--flags", type=int, default=0, help="ABS_FLAG_* bits passed to abs_init")
    ap.add_argument("--local-steps", type=int, default=1,
                    help="U of Eq. 2: local minibatch steps per job (configurations 1, 2 and 5)")
    ap.add_argument("--k-fixed", type=int, default=None,
                    help="run with K^t fixed at this value (ABS_K_FIXED, K0 = K): the many-version-groups regime")
    ap.add_argument("--samples", type=int, default=None,
                    help="dataset rows (default: the configuration's; smaller for profiler captures)")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle work")
    ap.add_argument("--timeline", type=int, default=0,
                    help="instead of the benchmark: print the event-bracketed launches (class, start us, end us; both "
                         "streams) of this many rounds after 50 warm rounds, in the configured launch mode")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    cfg = inputs.config(args.config, args.workers)
    if args.samples:
        cfg = cfg.scaled(n_samples=args.samples)
    if args.k_fixed:
        cfg = cfg.scaled(K0=args.k_fixed)
    if world > 1:
        from paper_2301_08895_b200 import multi
        cfg.run_seed = multi.replica_seed(cfg.run_seed, rank)   # independent replicas, one per GPU
    rounds = args.rounds or cfg.rounds
    U = args.local_steps
    config_obj = {"workload": workload_name(cfg, rounds) + (", U=%d local steps" % U if U > 1 else "") +
                  (", K fixed" if args.k_fixed else ""), "lr": cfg.lr,
                  "parallelism": "replicas x%d (the round loop does not shard)" % world,
                  "l2": "flushed between steps (512 MiB write); per-round working set exceeds L2",
                  "reinit": "abs_init between steps, outside the device-timed region",
                  "per_kernel": "event pair around every launch in one extra step with all kernels on one stream"}

    if args.impl == "reference":
        if rank != 0:
            return
        X, y, _ = inputs.make_data(cfg)
        w0 = inputs.make_w0(cfg)
        per_step = max(2.0, min(args.cpu_budget, 150.0 / max(1, args.steps + args.warmup)))
        res = None
        for _ in range(args.warmup):
            time_oracle(cfg, X, y, w0, rounds, min(per_step, 3.0), U, bool(args.k_fixed))
        vals = [time_oracle(cfg, X, y, w0, rounds, per_step, U, bool(args.k_fixed)) for _ in range(args.steps)]
        res = vals[-1]
        value = float(np.mean([v["value"] for v in vals]))
        res["value"] = value
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_obj, "cpu_baseline": res,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}))
        return

    import torch
    from paper_2301_08895_b200 import abs as gpu
    from paper_2301_08895_b200 import build
    build.build()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    X, y, _ = inputs.make_data(cfg)
    w0 = inputs.make_w0(cfg)
    bf16 = cfg.dtype == inputs.BF16
    Xh = torch.from_numpy(X.view(np.int16) if bf16 else X).pin_memory()
    yh = torch.from_numpy(y).pin_memory()
    Xd = Xh.to(dev).view(torch.bfloat16) if bf16 else Xh.to(dev)
    yd = yh.to(dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    k_mode = gpu.K_FIXED if args.k_fixed else gpu.K_ADAPTIVE

    def new_ctx(host=False, flags=None):
        flags = args.flags if flags is None else flags
        if host:
            return gpu.context_from_config(cfg, Xh, yh, w0, max_rounds=rounds, data_on_host=True,
                                           device=str(dev), flags=flags, local_steps=U, k_mode=k_mode)
        return gpu.context_from_config(cfg, Xd, yd, w0, max_rounds=rounds, device=str(dev), flags=flags,
                                       local_steps=U, k_mode=k_mode)

    def device_step(profile=False):
        """One run; returns (ms on the stream, worker-gradients, launches, profile dict)."""
        # the per-kernel step runs every kernel on one stream, so that an event pair brackets the
        # kernel alone and not its wait for an SM held by the other stream (same kernels, same bits)
        ctx = new_ctx(flags=(args.flags | gpu.FLAG_NO_OVERLAP) if profile else None)
        flush.zero_()
        l0 = ctx.launch_count()
        if profile:
            ctx.profile_start(rounds * (24 if U == 1 else 4 + 12 * U) + 8)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        ctx.enqueue_rounds(rounds)
        e1.record(stream)
        e1.synchronize()
        done, rc = ctx.rounds_done()
        assert rc == gpu.OK and done == rounds, (rc, done, gpu.last_error())
        prof = ctx.profile_read() if profile else None
        plan = ctx.plan()
        tr = ctx.get_trace()
        wg = int(tr["K"].sum())
        launches = ctx.launch_count() - l0
        ks = tr["K"].copy()
        plan["padded_rows"] = padded_rows(tr, cfg.batch, plan["row_block"]) if cfg.kind != inputs.LSQ else None
        ctx.close()
        return e0.elapsed_time(e1), wg, launches, prof, ks, plan

    def e2e_step():
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ctx = new_ctx(host=True)
        ctx.run_rounds(rounds)
        params = ctx.get_params()
        tr = ctx.get_trace()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        wg = int(tr["K"].sum())
        d2h = params.nbytes + sum(v.nbytes for v in tr.values())
        ctx.close()
        return dt, wg, d2h

    if args.timeline:
        # measurement aid: every launch between two CUDA events (about 2.6 us each on their stream, and the
        # events break the back-to-back chaining of the kernels, so periods are longer than in the timed runs)
        ctx = new_ctx()
        warm = min(50, max(0, rounds - args.timeline))
        ctx.run_rounds(warm)
        ctx.profile_start(args.timeline * 40)
        ctx.run_rounds(args.timeline)
        tl = ctx.profile_timeline(args.timeline * 40)
        ctx.profile_read()
        ctx.close()
        upd = [i for i, (c, _, _) in enumerate(tl) if c == "update"]
        t0 = tl[0][1]
        for c, a, b in tl:
            print("%-8s start %8.1f  end %8.1f  dur %6.1f" % (c, 1e3 * (a - t0), 1e3 * (b - t0), 1e3 * (b - a)))
        if len(upd) >= 3:
            print("round period us: %.1f" % (1e3 * (tl[upd[-1]][2] - tl[upd[0]][2]) / (len(upd) - 1)))
        return

    for _ in range(args.warmup):
        device_step()
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    t_wall0 = time.perf_counter()
    ms, wg_total, launches = [], 0, 0
    for _ in range(args.steps):
        m, wg, ln, _, _, _ = device_step()
        ms.append(m)
        wg_total += wg
        launches += ln
    barrier()
    wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()

    # end to end through the public API with host buffers
    e2e_step()
    e2e_t, e2e_wg, d2h = [], 0, 0
    for _ in range(max(1, min(args.steps, 3))):
        dt, wg, d2h = e2e_step()
        e2e_t.append(dt)
        e2e_wg += wg
    h2d = Xh.numel() * Xh.element_size() + yh.numel() * yh.element_size() + w0.nbytes

    # per-kernel durations (event pair around every launch)
    _, wg_p, _, prof, ks, plan = device_step(profile=True)

    t_dev = sum(ms) / 1e3
    from paper_2301_08895_b200 import multi
    (t_dev, e2e_time), (wg_all, e2e_wg_all) = multi.aggregate_replicas(
        [t_dev, sum(e2e_t)], [wg_total, e2e_wg], device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    flops = per_wg_flops(cfg)
    d = n_params(cfg)
    out = {
        "metric": METRIC, "value": wg_all / t_dev, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_dev / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if bf16 else "f32", "data": "synthetic", "config": config_obj,
        "rounds_per_sec": world * rounds * args.steps / t_dev,
        "minibatch_gradients_per_sec": U * wg_all / t_dev,
        "worker_gradients_per_step": wg_total / args.steps,
        "wall_s_timed_region": wall,
        "clocks": clocks,
        "e2e": {"value": e2e_wg_all / e2e_time, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": 1e3 * e2e_time / len(e2e_t)},
        "gpu_launches": int(launches),
        "peaks": {"source": peaks["source"], "hbm_gbs": peaks["hbm_gbs"],
                  "bf16_tflops": peaks["bf16_tflops"],
                  "bf16_tflops_sustained": peaks.get("bf16_tflops_sustained")},
    }
    kernels = {k: {"launches": n, "ms": round(t, 4)} for k, (n, t) in prof.items() if n}
    out["kernel_ms_profiled_step"] = kernels
    tot_prof = sum(t for _, t in prof.values())
    if U > 1:
        # local steps: every worker's chain of U steps is sequential, one CTA per worker
        n_l, t_l = prof["lsq"]
        if cfg.kind == inputs.MLP and len(cfg.dims) > 2:
            # multi-layer network: the workers' copies live in HBM; after each step but the last the refresh
            # kernel streams, per selected worker, the upload sum (4 B/parameter), the model version the
            # worker started from and the new copy (storage type each)
            d_pad = plan.get("d_pad") or sum(cfg.dims[l] * cfg.dims[l + 1] + cfg.dims[l + 1] for l in range(len(cfg.dims) - 1))
            n_rounds_prof = max(1, prof["update"][0])             # rounds the recorded launches cover
            n_upd = (U - 1) * n_rounds_prof
            per_par = 4.0 + 2.0 * (2 if bf16 else 4)
            bytes_l = per_par * d_pad * float(np.mean(ks[:n_rounds_prof]))   # per refresh launch: bytes x d x K^t
            # the class also holds the begin and layout kernels (1 + U launches per round, small)
            out["roofline"] = {"bound": "hbm", "kernel": "local_step_kernel (+ local_begin launches)",
                               "launches": n_l, "avg_us": 1e3 * t_l / max(1, n_l),
                               "achieved": bytes_l * n_upd / (t_l * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                               "frac": bytes_l * n_upd / (t_l * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                               "peak_source": peaks["source"], "share_of_profiled_time": t_l / tot_prof,
                               "note": "algorithmic bytes of the U - 1 copy refreshes per round only, over the time of the "
                                       "whole class (begin and last-step launches included)"}
        else:
            out["roofline"] = {"bound": "latency", "kernel": "local_sgd_kernel", "achieved": None, "peak": None,
                               "unit": None, "frac": None, "traffic": None,
                               "avg_us": 1e3 * t_l / max(1, n_l), "share_of_profiled_time": t_l / tot_prof,
                               "note": "U sequential minibatch steps per job; see minibatch_gradients_per_sec"}
    elif cfg.kind == inputs.LSQ:
        # least squares reads each minibatch row once: B*d*esz + B*4 bytes per worker-gradient
        esz = 2 if bf16 else 4
        bytes_wg = cfg.batch * cfg.dims[0] * esz + cfg.batch * 4
        persistent = prof.get("rounds", (0, 0.0))[0] > 0
        n_l, t_l = prof["rounds"] if persistent else prof["lsq"]
        ach = wg_p * bytes_wg / (t_l * 1e-3) / 1e9
        out["roofline"] = {"bound": "hbm",
                           "kernel": "abs_lsq_rounds_kernel (whole rounds, latency-bound)" if persistent
                           else ("lsq_pipe_kernel" if bf16 and cfg.dims[0] <= 4096 and not (args.flags & 32)
                                 else "lsq_grad_v2_kernel"), "achieved": ach,
                           "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                           "traffic": None, "peak_source": peaks["source"],
                           "share_of_profiled_time": t_l / tot_prof}
    elif cfg.kind == inputs.CNN:
        # FP32-FMA kernels: 148 SMs x 128 lanes x 2 flop per clock at the maximum SM clock
        n_c, t_c = prof["conv"]
        peak = 148 * 128 * 2 * 1.965e9 / 1e12
        ach = wg_p * flops["conv"] / (t_c * 1e-3) / 1e12
        out["roofline"] = {"bound": "alu", "kernel": "conv_block_fwd_kernel + conv_block_bwd_kernel (+ chunk sums)",
                           "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak, "traffic": None,
                           "peak_source": "148 SMs x 128 FP32 lanes x 2 flop x 1.965 GHz",
                           "share_of_profiled_time": t_c / tot_prof}
    elif prof["fwd"][0] and bf16:
        t_g = prof["fwd"][1] + prof["dgrad"][1] + prof["wgrad"][1]
        fl = wg_p * (flops["fwd"] + flops["dgrad"] + flops["wgrad"])
        ach = fl / (t_g * 1e-3) / 1e12
        peak = peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"]
        out["roofline"] = {"bound": "tensor", "kernel": "tc_gemm_kernel (fwd+dgrad+wgrad launches)",
                           "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                           "traffic": measured_traffic("gemm", args.config, not args.samples and not args.k_fixed),
                           "traffic_source": TRAFFIC["gemm"]["source"], "peak_source": peaks["source"] + " (sustained bf16)",
                           "frac_of_burst_peak": ach / peaks["bf16_tflops"],
                           "share_of_profiled_time": t_g / tot_prof,
                           # a layer's delta back-propagation may share the weight gradient's launch:
                           # its flops then count in the "wgrad" class
                           "per_class_tflops": {c: wg_p * (flops[c] + (flops["dgrad"] if c == "wgrad" and
                                                                       prof["dgrad"][1] == 0 else 0.0))
                                                / (prof[c][1] * 1e-3) / 1e12
                                                for c in ("fwd", "dgrad", "wgrad") if prof[c][1] > 0}}
    else:
        out["roofline"] = {"bound": "latency", "achieved": None, "peak": None, "unit": None,
                           "frac": None, "traffic": None,
                           "note": "launch/dependency-latency bound configuration; see rounds_per_sec"}
    n_u, t_u = prof["update"]
    if n_u:
        # Eq. 3 step: read fp32 master + P fp32 partial sums, write master + storage-type ring slot
        esz = 2 if bf16 else 4
        P = plan["partials"] if plan["partials"] > 0 else float(np.mean(ks[:n_u]))
        bytes_launch = (8 + esz + 4 * P) * d
        ach = bytes_launch / (t_u / n_u * 1e-3) / 1e9
        traffic_u = measured_traffic("update", args.config, not args.samples)
        sec_u = t_u / n_u * 1e-3
        out["roofline_update"] = {"bound": "hbm", "kernel": "update_kernel", "launches": n_u,
                                  "avg_us": 1e3 * t_u / n_u, "partials": P,
                                  "bytes_per_launch": bytes_launch, "achieved": ach,
                                  "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                  "frac": ach / peaks["hbm_gbs"],
                                  # the same launch time against the bytes Eq. 3 needs at the least (one gradient
                                  # vector: P = 1) and against the DRAM bytes an ncu capture counted (the partial
                                  # sums the GEMMs just wrote are partly still in L2)
                                  "min_bytes_per_launch": (8 + esz + 4) * d,
                                  "frac_min_bytes": (8 + esz + 4) * d / sec_u / 1e9 / peaks["hbm_gbs"],
                                  "frac_dram": (traffic_u / sec_u / 1e9 / peaks["hbm_gbs"]) if traffic_u else None,
                                  "traffic": traffic_u,
                                  "traffic_source": TRAFFIC["update"]["source"] if traffic_u else None}
    if plan.get("padded_rows"):
        padded, real = plan["padded_rows"]
        out["padded_row_ratio"] = padded / max(1, real)      # rows the GEMMs process / rows of real samples
    out["plan"] = plan
    out["_profiled_worker_gradients"] = wg_p
    out["cpu_baseline"] = time_oracle(cfg, X, y, w0, rounds, args.cpu_budget, U, bool(args.k_fixed))
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
