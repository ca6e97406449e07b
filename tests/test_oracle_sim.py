"""Pins for the oracle's round loop (Algorithm 1, Eq. 3-6) against special
cases the paper names and closed forms that follow from its rules."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import abs_sim, models, timing
from oracle.abs_sim import ABSOracle, K_FIXED, BOUND_FIXED

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _lsq_problem(M=512, d=6, seed=0, noise=0.1):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, d))
    w_star = rng.standard_normal(d)
    y = X @ w_star + noise * rng.standard_normal(M)
    return X, y, w_star


def _check_invariants(o, rows, W, S):
    jobs_started = 0
    prev_T, prev_K = 0, 0
    comm = W
    for row in rows:
        assert len(row["sel"]) == row["K"] == len(row["tau"])          # |K^t| = K^t
        assert len(set(row["sel"])) == row["K"]
        assert not (set(row["sel"]) & set(row["restart"]))
        assert row["restart"] == sorted(row["restart"])
        assert 0 <= row["theta"] <= S
        assert all(0 <= tau <= S for tau in row["tau"])                # bounded staleness
        assert row["T_end"] >= prev_T and row["K"] >= prev_K and row["K"] <= W
        prev_T, prev_K = row["T_end"], row["K"]
        jobs_started += row["K"] + len(row["restart"])
        comm += row["K"] + len(row["restart"])
        assert row["comm"] == comm                                     # +1 per worker that communicates
    assert sum(o.job) == jobs_started
    assert all(v <= o.t for v in o.version)
    assert all(o.t - v <= max(S, 0) for v in o.version) or S == 0


# ---------------------------------------------------------------- reductions
def test_sync_sgd_reduction():
    """K = N and bound 0 is synchronous minibatch SGD (Sec. II-B): the model
    follows a plain loop that averages the N minibatch gradients."""
    X, y, _ = _lsq_problem()
    W, B, lr, seed = 4, 8, 0.05, 42
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), B, lr, W, W, 0, dist, seed)
    rows = o.run(25)
    w = np.zeros(6)
    for t in range(25):
        idx = np.concatenate([abs_sim.minibatch_indices(seed, n, t, B, W, X.shape[0])
                              for n in range(W)])
        r = X[idx] @ w - y[idx]
        w = w - lr * (X[idx].T @ r) / (W * B)
    assert np.allclose(o.w, w, rtol=1e-12, atol=1e-14)
    for t, row in enumerate(rows):
        assert sorted(row["sel"]) == list(range(W)) and set(row["tau"]) == {0}
        assert row["restart"] == []
    assert o.job == [25] * W
    _check_invariants(o, rows, W, 0)


def test_k_sync_reduction():
    """Bound 0 with fixed K < N: the stragglers' work is thrown away every
    round (K-sync SGD, Sec. I): all ages 0, N - K restarts per round."""
    X, y, _ = _lsq_problem()
    W, K = 6, 2
    dist = timing.TimeDist(timing.SHIFTED_EXP, shift=1.0, rate=1.0)
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, W, K, 0, dist, 7, k_mode=K_FIXED)
    rows = o.run(30)
    for row in rows:
        assert row["K"] == K and set(row["tau"]) == {0}
        assert len(row["restart"]) == W - K and row["theta"] == 0
    _check_invariants(o, rows, W, 0)


def test_asgd_reduction_statistics():
    """Fixed K = 1 is ASGD (Sec. II-B).  With i.i.d. exponential job times the
    arriving worker is uniform over the N workers in every round (memoryless),
    so the age of a consumed gradient is geometric with mean N - 1."""
    X, y, _ = _lsq_problem(d=3)
    W, rounds = 5, 6000
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    o = ABSOracle(models.LSQ, [3, 1], X, y, np.zeros(3), 2, 0.01, W, 1, 200, dist, 3,
                  k_mode=K_FIXED, bound_mode=BOUND_FIXED)
    rows = o.run(rounds)
    ids = np.array([row["sel"][0] for row in rows])
    taus = np.array([row["tau"][0] for row in rows[200:]])
    assert all(row["K"] == 1 and row["restart"] == [] for row in rows)
    counts = np.bincount(ids, minlength=W) / rounds
    assert np.all(np.abs(counts - 1 / W) < 4 * math.sqrt(0.16 / rounds))
    # geometric(p = 1/W) on {0,1,...}: mean W-1, variance (1-p)/p^2 = W(W-1)
    assert abs(taus.mean() - (W - 1)) < 5 * math.sqrt(W * (W - 1) / len(taus))


def test_lock_step_constant_times():
    """Equal deterministic times: arrivals go round-robin in id order."""
    X, y, _ = _lsq_problem()
    W, K, D = 8, 2, 3.0
    dist = timing.TimeDist(timing.CONST, shift=D)
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.01, W, K, W // K - 1, dist, 1,
                  k_mode=K_FIXED, bound_mode=BOUND_FIXED)
    rows = o.run(40)
    for t, row in enumerate(rows):
        first = (t * K) % W
        assert row["sel"] == list(range(first, first + K))
        assert row["T_end"] == int(D * 2 ** 20) * ((t * K) // W + 1)
        assert row["tau"] == [min(t, W // K - 1)] * K
        assert row["restart"] == []
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.01, W, W, 0, dist, 1)
    for t, row in enumerate(o.run(10)):
        assert row["sel"] == list(range(W)) and row["T_end"] == (t + 1) * int(D * 2 ** 20)
        assert set(row["tau"]) == {0}


def test_straggler_is_restarted_every_theta_plus_one_rounds():
    """One worker whose jobs take 2^40 ticks never arrives; Eq. 6 (in Algorithm
    1's order) sends it the fresh model whenever its age would exceed theta."""
    X, y, _ = _lsq_problem()
    W, K, S = 5, 2, 3
    dist = timing.TimeDist(timing.CONST, shift=1.0, slow_mod=W, slow_rem=4, slow_factor=2.0 ** 20)
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.01, W, K, S, dist, 1,
                  k_mode=K_FIXED, bound_mode=BOUND_FIXED)
    rows = o.run(41)
    for t, row in enumerate(rows):
        assert 4 not in row["sel"]
        assert (4 in row["restart"]) == (t % (S + 1) == S)
    _check_invariants(o, rows, W, S)
    # literal reading of Eq. 6 (pre-increment age) fires one round later
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.01, W, K, S, dist, 1,
                  k_mode=K_FIXED, bound_mode=BOUND_FIXED, literal_eq6=True)
    for t, row in enumerate(o.run(41)):
        assert (4 in row["restart"]) == (t % (S + 2) == S + 1)


def test_printed_eq6_equals_algorithm_order_with_threshold_plus_one():
    """Testing the age before the increment against theta is the same as testing the incremented
    age against theta + 1: with a fixed threshold the two readings play identical rounds."""
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.01, 9, 2, 2, dist, 3,
                  k_mode=K_FIXED, bound_mode=BOUND_FIXED, literal_eq6=True)
    b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.01, 9, 2, 3, dist, 3,
                  k_mode=K_FIXED, bound_mode=BOUND_FIXED)
    ra, rb = a.run(80), b.run(80)
    assert sum(len(r["restart"]) for r in ra) > 0
    for x, z in zip(ra, rb):
        assert x["theta"] + 1 == z["theta"]
        assert {k: v for k, v in x.items() if k != "theta"} == {k: v for k, v in z.items() if k != "theta"}
    assert max(max(r["tau"]) for r in ra) == 3          # one more than the bound of 2


# ------------------------------------------------------------------- rules
def test_selection_is_the_k_smallest_with_ties_to_lower_id():
    X, y, _ = _lsq_problem(d=2)
    dist = timing.TimeDist(timing.CONST, shift=1.0)
    for ticks in itertools.product([3, 5, 7], repeat=5):
        for K in (1, 2, 4):
            o = ABSOracle(models.LSQ, [2, 1], X, y, np.zeros(2), 2, 0.0, 5, K, 9, dist, 0,
                          k_mode=K_FIXED, bound_mode=BOUND_FIXED)
            o.c = list(ticks)
            row = o.round()
            pending = list(range(5))
            brute = []
            for _ in range(K):            # repeated extraction of the minimum
                best = min(pending, key=lambda n: ticks[n] * 10 + n)
                brute.append(best)
                pending.remove(best)
            assert row["sel"] == brute
            assert row["T_end"] == ticks[brute[-1]]


def test_k_rule_hand_cases():
    f = np.float32
    assert abs_sim.next_k(4, 4, 64, f(2.0), f(2.0)) == 4          # same loss -> K0
    assert abs_sim.next_k(4, 4, 64, f(2.0), f(0.5)) == 8          # loss / 4 -> K doubles
    assert abs_sim.next_k(4, 4, 64, f(2.0), f(0.5000001)) == 7    # just above the boundary
    assert abs_sim.next_k(4, 4, 64, f(1.0), f(1.0 / 9.0)) == 11   # 1/9 rounds up in binary32: 144*f(1/9) > 16
    assert abs_sim.next_k(4, 4, 64, f(1.0), f(0.0625)) == 16
    assert abs_sim.next_k(9, 4, 64, f(2.0), f(8.0)) == 9          # never decreases
    assert abs_sim.next_k(4, 4, 10, f(2.0), f(1e-6)) == 10        # capped at N
    assert abs_sim.next_k(4, 4, 10, f(2.0), f(0.0)) == 10
    with pytest.raises(abs_sim.Diverged):
        abs_sim.next_k(4, 4, 10, f(2.0), f(np.inf))
    # agrees with the real-valued formula K0 sqrt(L0/Lt) away from boundaries
    rng = np.random.default_rng(1)
    for _ in range(300):
        l0, lt = f(rng.uniform(0.5, 3)), f(rng.uniform(0.01, 3))
        real = 5 * math.sqrt(float(l0) / float(lt))
        if abs(real - round(real)) > 1e-6:
            assert abs_sim.next_k(5, 5, 1000, l0, lt) == max(5, min(1000, math.floor(real)))


def test_first_round_keeps_k0():
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 8, 3, 4, dist, 5)
    rows = o.run(2)
    assert rows[0]["K"] == 3 and rows[1]["K"] == 3     # L_0 / L_0 = 1  ->  K^1 = K^0


def test_theta_table():
    with open(os.path.join(GOLDEN, "theta_table.txt")) as f:
        rows = [tuple(int(v) for v in line.split()) for line in f
                if line.strip() and not line.startswith("#")]
    assert len(rows) >= 20
    for W, K0, S, K, theta in rows:
        assert abs_sim.theta_rule(W, K0, S, K) == theta
    assert abs_sim.theta_rule(8, 8, 0, 8) == 0           # bound 0 overrides the floor of 1


def test_theta_offset_table():
    """Eq. 4 with the constant a given (values of the paper's sweep, Sec. V-B)."""
    with open(os.path.join(GOLDEN, "theta_offset_table.txt")) as f:
        rows = [tuple(int(v) for v in line.split()) for line in f
                if line.strip() and not line.startswith("#")]
    assert len(rows) >= 20
    for W, S, K, a, theta in rows:
        assert abs_sim.theta_offset_rule(W, S, K, a) == theta


def test_offset_mode_equals_derived_offset_when_k0_divides_n():
    """BOUND_ADAPTIVE derives a = S - N/K0 from the staleness bound; when K0 divides N that a is
    an integer and BOUND_OFFSET with it must play the very same rounds."""
    X, y, _ = _lsq_problem(400, 6, seed=3)
    dist = timing.TimeDist(timing.GAMMA, shift=0.25, rate=1.0, shape=2)
    W, K0, S = 12, 3, 6                      # N/K0 = 4, a = 2
    a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, W, K0, S, dist, 5)
    b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, W, K0, S, dist, 5,
                  bound_mode=abs_sim.BOUND_OFFSET, bound_offset=S - W // K0)
    ra, rb = a.run(60), b.run(60)
    assert ra == rb
    assert any(r["restart"] for r in ra)
    # a smaller offset discards more: restarts cannot decrease (qualitative claim of Sec. V-B)
    c = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, W, K0, S, dist, 5,
                  k_mode=abs_sim.K_FIXED, bound_mode=abs_sim.BOUND_OFFSET, bound_offset=2)
    d = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, W, K0, S, dist, 5,
                  k_mode=abs_sim.K_FIXED, bound_mode=abs_sim.BOUND_OFFSET, bound_offset=-1)
    n_c = sum(len(r["restart"]) for r in c.run(60))
    n_d = sum(len(r["restart"]) for r in d.run(60))
    assert n_d >= n_c and n_d > 0
    with pytest.raises(ValueError):
        ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, W, K0, 3, dist, 5,
                  bound_mode=abs_sim.BOUND_OFFSET, bound_offset=2)


def test_loss_estimate_order_and_rounding():
    f = np.float32
    assert abs_sim.tree_sum([1.0, 2.0, 3.0]) == 6.0
    # ((a+b)+(c+0)) in binary32: with a = 1, b = c = 2^-24 the pairing decides the bits
    a, b = f(1.0), f(2.0 ** -24)
    assert abs_sim.tree_sum([a, b, b]) == f(f(a + b) + f(b + f(0))) == f(1.0)
    assert abs_sim.tree_sum([b, b, a]) == f(f(b + b) + f(a + f(0))) == f(1.0 + 2.0 ** -23)
    vals = [f(x) for x in (0.1, 0.2, 0.3, 0.4, 0.5)]
    est = abs_sim.loss_estimate(vals)
    assert isinstance(est, np.float32)
    assert abs(float(est) - 0.3) < 1e-7
    # every intermediate is a binary32 value: a sum that binary64 would keep exact gets rounded
    assert abs_sim.tree_sum([f(16777216.0), f(1.0)]) == f(16777216.0)
    assert float(abs_sim.loss_estimate([f(1.0), f(2.0)])) == 1.5


# ---------------------------------------------------------- whole-run behaviour
def test_lsq_run_reaches_normal_equation_solution():
    X, y, w_star = _lsq_problem(M=2048, d=8, seed=3, noise=0.1)
    w_ls = np.linalg.solve(X.T @ X, X.T @ y)
    dist = timing.TimeDist(timing.SHIFTED_EXP, shift=1.0, rate=1.0)
    o = ABSOracle(models.LSQ, [8, 1], X, y, np.zeros(8), 32, 0.05, 8, 2, 4, dist, 2001)
    rows = o.run(400)
    assert np.linalg.norm(o.w - w_ls) / np.linalg.norm(w_ls) < 0.03
    assert np.linalg.norm(o.w - w_star) / np.linalg.norm(w_star) < 0.05
    assert rows[-1]["loss_mean"] < 0.02 and rows[0]["loss_mean"] > 1.0
    assert rows[-1]["K"] == 8                   # K has grown to N as the loss fell
    _check_invariants(o, rows, 8, 4)


@pytest.mark.parametrize("kind,dims,quant", [(models.SOFTMAX, [12, 4], False),
                                             (models.MLP, [12, 9, 4], True)])
def test_invariants_on_classifier_runs(kind, dims, quant):
    rng = np.random.default_rng(5)
    means = rng.standard_normal((4, 12))
    lab = rng.integers(0, 4, size=600)
    X = models.round_bf16(means[lab] + rng.standard_normal((600, 12)))
    w0 = rng.standard_normal(models.n_params(kind, dims)) * 0.3
    dist = timing.TimeDist(timing.PARETO2, scale=1.0)
    o = ABSOracle(kind, dims, X, lab, w0, 8, 0.1, 12, 3, 6, dist, 77, quant=quant)
    rows = o.run(120)
    _check_invariants(o, rows, 12, 6)
    assert rows[-1]["loss_mean"] < rows[0]["loss_mean"]
    assert any(row["restart"] for row in rows)
    assert max(max(row["tau"]) for row in rows) >= 2


def test_restarts_do_not_increase_with_the_bound():
    """Sanity of the qualitative claim of Sec. V-B: a larger threshold offset
    discards fewer computations."""
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.PARETO2, scale=1.0)
    totals = []
    for S in (1, 2, 4, 8):
        o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.02, 12, 2, S, dist, 9,
                      k_mode=K_FIXED, bound_mode=BOUND_FIXED)
        totals.append(sum(len(r["restart"]) for r in o.run(150)))
    assert totals == sorted(totals, reverse=True) and totals[0] > totals[-1]


def test_forced_losses_only_steer_k():
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 8, 2, 4, dist, 5)
    rows = a.run(30)
    b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 8, 2, 4, dist, 5)
    rows_b = b.run(30, forced_losses=[r["sel_loss"] for r in rows])
    assert [r["sel"] for r in rows] == [r["sel"] for r in rows_b]
    assert np.array_equal(a.w, b.w)


def test_divergence_is_reported():
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    o = ABSOracle(models.LSQ, [6, 1], X * 1e3, y, np.zeros(6), 4, 10.0, 4, 4, 0, dist, 5)
    with pytest.raises(abs_sim.Diverged):
        o.run(200)
    assert 0 < len(o.trace) < 200


def test_integer_only_mode_replays_the_same_trace():
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.PARETO2, scale=1.0)
    a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 9, 2, 3, dist, 5)
    rows = a.run(60)
    b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 9, 2, 3, dist, 5, integer_only=True)
    rows_b = b.run(60, forced_losses=[r["sel_loss"] for r in rows])
    for ra, rb in zip(rows, rows_b):
        for f in ("K", "sel", "tau", "restart", "T_end", "theta", "comm"):
            assert ra[f] == rb[f]
    assert np.array_equal(b.w, np.zeros(6))


# ---------------------------------------------------------------- local SGD steps (U > 1)
def test_local_steps_follow_the_affine_recursion_of_least_squares():
    """For f = 1/2 (x.w - y)^2 one local step is w <- (I - eta A_u) w + eta b_u with
    A_u = X_u^T X_u / B, b_u = X_u^T y_u / B; the upload is (w^0 - w^U) / eta (Eq. 2, Algorithm 1)."""
    X, y, _ = _lsq_problem(M=300, d=5, seed=7)
    W, B, lr, U, seed = 3, 6, 0.07, 4, 21
    dist = timing.TimeDist(timing.CONST, shift=1.0)
    w0 = np.linspace(-1.0, 1.0, 5)
    o = ABSOracle(models.LSQ, [5, 1], X, y, w0, B, lr, W, W, 0, dist, seed, local_steps=U)
    for n in range(W):
        w = w0.copy()
        losses = []
        for u in range(U):
            idx = abs_sim.minibatch_indices(seed, n, 0, B, W, X.shape[0], step=u)
            Xu, yu = X[idx], y[idx]
            losses.append(0.5 * np.mean((Xu @ w - yu) ** 2))
            A, b = Xu.T @ Xu / B, Xu.T @ yu / B
            w = (np.eye(5) - lr * A) @ w + lr * b
        loss, grad_sum = o.upload(n)
        assert np.allclose(w0 - lr * grad_sum, w, rtol=0, atol=1e-12)
        assert abs(loss - np.mean(losses)) < 1e-12


def test_local_step_minibatches_use_consecutive_philox_blocks():
    from oracle import philox
    seed, n, j, B = 9, 2, 5, 10                       # ceil(10 / 4) = 3 blocks per step
    for u in (0, 1, 3):
        words = philox.minibatch_words(seed, n, j, B, step=u)
        for b in range(B):
            blk = philox.philox4x32_10((n, j, philox.TAG_MINIBATCH, 3 * u + b // 4), philox.seed_key(seed))
            assert int(words[b]) == blk[b % 4]
    a = abs_sim.minibatch_indices(seed, n, j, B, 4, 1000, step=0)
    b = abs_sim.minibatch_indices(seed, n, j, B, 4, 1000, step=1)
    assert not np.array_equal(a, b)
    assert np.array_equal(a, abs_sim.minibatch_indices(seed, n, j, B, 4, 1000))


def test_synchronous_local_sgd_reduction():
    """K = N and bound 0 with U local steps is synchronous local SGD (Sec. II-B): every round each
    worker moves U steps from the global model and the server averages the N displacements."""
    X, y, _ = _lsq_problem(M=400, d=6, seed=1)
    W, B, lr, U, seed = 4, 8, 0.05, 3, 42
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), B, lr, W, W, 0, dist, seed, local_steps=U)
    rows = o.run(12)
    w = np.zeros(6)
    for t in range(12):
        moved = np.zeros(6)
        for n in range(W):
            wl = w.copy()
            for u in range(U):
                idx = abs_sim.minibatch_indices(seed, n, t, B, W, X.shape[0], step=u)
                wl = wl - lr * X[idx].T @ (X[idx] @ wl - y[idx]) / B
            moved += w - wl
        w = w - moved / W
    assert np.allclose(o.w, w, rtol=0, atol=1e-12)
    assert all(r["K"] == W and not r["restart"] and set(r["tau"]) == {0} for r in rows)


def test_zero_step_size_makes_every_local_step_see_the_same_model():
    """With eta = 0 the U local steps are U minibatch evaluations at one model: the uploaded loss is
    the mean sample loss over all U B draws and the uploaded sum is U times their mean gradient."""
    X, y, _ = _lsq_problem(M=200, d=4, seed=2)
    W, B, U, seed = 2, 5, 3, 8
    w0 = np.array([0.3, -0.2, 0.1, 0.5])
    o = ABSOracle(models.LSQ, [4, 1], X, y, w0, B, 0.0, W, 1, 2, timing.TimeDist(timing.EXP), seed,
                  local_steps=U)
    loss, grad_sum = o.upload(1)
    idx = np.concatenate([abs_sim.minibatch_indices(seed, 1, 0, B, W, 200, step=u) for u in range(U)])
    per_sample = [models.sample_loss(models.LSQ, [4, 1], w0, X[i], y[i]) for i in idx]
    assert abs(loss - np.mean(per_sample)) < 1e-12
    assert np.allclose(grad_sum, U * (X[idx].T @ (X[idx] @ w0 - y[idx])) / len(idx), atol=1e-12)


def test_local_steps_soft_max_against_finite_differences_of_the_chain():
    """The uploaded sum of a soft-max job equals (w^0 - w^U) / eta of a chain built from numerical
    gradients of the mean sample loss (independent of the analytic gradient code)."""
    rng = np.random.default_rng(4)
    M, d_in, C, W, B, U, lr, seed = 120, 5, 3, 2, 4, 2, 0.1, 3
    X = rng.standard_normal((M, d_in))
    y = rng.integers(0, C, size=M).astype(np.int32)
    w0 = 0.1 * rng.standard_normal(d_in * C + C)
    o = ABSOracle(models.SOFTMAX, [d_in, C], X, y, w0, B, lr, W, 1, 2, timing.TimeDist(timing.EXP), seed,
                  local_steps=U)
    _, grad_sum = o.upload(0)

    def mean_loss(w, idx):
        return np.mean([models.sample_loss(models.SOFTMAX, [d_in, C], w, X[i], y[i]) for i in idx])

    w = w0.copy()
    total = np.zeros_like(w0)
    for u in range(U):
        idx = abs_sim.minibatch_indices(seed, 0, 0, B, W, M, step=u)
        g = np.zeros_like(w)
        for k in range(w.shape[0]):
            e = np.zeros_like(w)
            e[k] = 1e-6
            g[k] = (mean_loss(w + e, idx) - mean_loss(w - e, idx)) / 2e-6
        total += g
        w = w - lr * g
    assert np.allclose(grad_sum, total, atol=1e-7)


def test_bf16_local_steps_round_the_evaluation_point_not_the_copy():
    """Eq. 2 with 16-bit stored models, three local steps worked by hand.

    One worker, one sample x = 1, y = 0, so f(w) = w^2 / 2, the minibatch gradient is the
    model value the step is evaluated at, and every minibatch is that sample.  eta = 3/1024,
    w^{.,0} = 1.  bfloat16 has spacing 2^-8 just below 1.
      step 0: evaluated at 1                      -> g0 = 1,          copy -> 1 - 3/1024
      step 1: the copy 1 - 0.75 * 2^-8 is evaluated at its rounding 1 - 2^-8 = 0.99609375
              -> g1 = 0.99609375, copy (kept unrounded) -> 1 - 3/1024 - (3/1024) * 0.99609375
      step 2: that copy is 1 - 1.497 * 2^-8 and rounds to 1 - 2^-8 again -> g2 = 0.99609375
    Without the rounding g1 would be 1 - 3/1024; with the copy itself rounded after step 1,
    step 2 would start from 0.99609375 * (1 - 3/1024) = 1 - 1.747 * 2^-8, which rounds to
    1 - 2^-7, so g2 would be 0.9921875.
    """
    lr = 3.0 / 1024.0
    X, y = np.array([[1.0]]), np.array([0.0], dtype=np.float32)
    o = abs_sim.ABSOracle(models.LSQ, (1, 1), X, y, np.array([1.0]), 1, lr, 1, 1, 0,
                          timing.TimeDist(timing.CONST, shift=1.0), 3, quant=True, local_steps=3)
    loss, g = o.upload(0)
    g0, g1, g2 = 1.0, 0.99609375, 0.99609375
    assert g[0] == g0 + g1 + g2 == 2.9921875
    assert loss == (0.5 * g0 * g0 + 0.5 * g1 * g1 + 0.5 * g2 * g2) / 3.0
    # the two other readings give other numbers (the pin has teeth)
    assert g[0] != 1.0 + (1.0 - lr) + 0.99609375
    assert g[0] != 1.0 + 0.99609375 + 0.9921875
    # Eq. 3 with the upload: w^1 = w^0 - eta * (g0 + g1 + g2)
    o.round()
    assert o.w[0] == 1.0 - lr * 2.9921875
    # full precision (fp32 configurations): plain chained steps
    o2 = abs_sim.ABSOracle(models.LSQ, (1, 1), X, y, np.array([1.0]), 1, lr, 1, 1, 0,
                           timing.TimeDist(timing.CONST, shift=1.0), 3, quant=False, local_steps=3)
    _, gf = o2.upload(0)
    assert gf[0] == 1.0 + (1.0 - lr) + (1.0 - lr) * (1.0 - lr)


# ---------------------------------------------------------------- comparison systems (Sec. II-B, Sec. V)
def test_staleness_aware_step_size_by_hand():
    """SA penalises a stale gradient's step size linearly in its delay (Sec. I).  Three workers in
    lock step (constant times, K = 1): the arriving gradient has staleness min(t, 2).  One sample
    x = 1, y = 0, so f = w^2 / 2 and a gradient is the model value it was computed at; eta = 1/4.
      w^1 = 1 - 1/4 (tau 0) = 3/4;  w^2 = 3/4 - 1/4 * w^0 (tau 1) = 1/2;
      w^3 = 1/2 - 1/4 * w^0 / 2 (tau 2) = 3/8;  w^4 = 3/8 - 1/4 * w^1 / 2 (tau 2) = 9/32.
    Without the penalty the last two steps are whole: w^3 = 1/4, w^4 = 1/16."""
    X, y = np.ones((3, 1)), np.zeros(3)
    dist = timing.TimeDist(timing.CONST, shift=1.0)
    kw = dict(k_mode=K_FIXED, bound_mode=BOUND_FIXED)
    o = ABSOracle(models.LSQ, [1, 1], X, y, np.array([1.0]), 1, 0.25, 3, 1, 2, dist, 5, sa_penalty=True, **kw)
    seen = []
    for row in (o.round() for _ in range(4)):
        seen.append(o.w[0])
        assert row["restart"] == []
    assert [r["tau"] for r in o.trace] == [[0], [1], [2], [2]]
    assert seen == [0.75, 0.5, 0.375, 0.28125]
    o = ABSOracle(models.LSQ, [1, 1], X, y, np.array([1.0]), 1, 0.25, 3, 1, 2, dist, 5, **kw)
    o.run(4)
    assert o.w[0] == 0.0625


def test_staleness_aware_step_size_changes_nothing_without_staleness():
    """With bound 0 every consumed gradient has age 0 and with bound 1 at most 1: the penalty
    1 / max(1, tau) is then 1 and the run is ABS bit for bit."""
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.SHIFTED_EXP, shift=1.0, rate=1.0)
    for S in (0, 1):
        a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 6, 2, S, dist, 9)
        b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 6, 2, S, dist, 9, sa_penalty=True)
        assert a.run(40) == b.run(40) and np.array_equal(a.w, b.w)
    # and with real staleness it does change the model, never the integer decisions of a fixed-K run
    a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 6, 2, 4, dist, 9, k_mode=K_FIXED)
    b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 6, 2, 4, dist, 9, k_mode=K_FIXED, sa_penalty=True)
    ra, rb = a.run(40), b.run(40)
    assert max(max(r["tau"]) for r in ra) >= 2
    assert [(r["sel"], r["tau"], r["restart"]) for r in ra] == [(r["sel"], r["tau"], r["restart"]) for r in rb]
    assert not np.array_equal(a.w, b.w)


def test_without_restarts_equals_abs_while_no_restart_would_fire():
    """AdaSync is the loop without Eq. 6's forced restarts.  With a bound so large that Eq. 6 never
    fires, both runs are the same; with a small bound they part at the first restart."""
    X, y, _ = _lsq_problem()
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 8, 2, 200, dist, 4, bound_mode=BOUND_FIXED)
    b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 8, 2, 200, dist, 4, bound_mode=BOUND_FIXED, restarts=False)
    ra, rb = a.run(60), b.run(60)
    assert all(r["restart"] == [] for r in ra) and ra == rb and np.array_equal(a.w, b.w)
    a = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 8, 2, 2, dist, 4, k_mode=K_FIXED)
    b = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.05, 8, 2, 2, dist, 4, k_mode=K_FIXED, restarts=False)
    ra, rb = a.run(60), b.run(60)
    first = next(t for t, r in enumerate(ra) if r["restart"])
    assert ra[:first] == rb[:first]
    assert all(r["restart"] == [] for r in rb)
    assert max(max(r["tau"]) for r in rb) > 2 >= max(max(r["tau"]) for r in ra)     # unbounded vs bounded
    # communication counter: only the K uploads per round (Sec. V-B)
    assert rb[-1]["comm"] == 8 + 2 * 60


def test_without_restarts_a_straggler_arrives_with_its_full_age():
    """One worker 50 times slower than the others, K = 2 of 5, constant times: with restarts it
    would be sent the fresh model every theta + 1 rounds; without, it keeps computing on w^0 and
    its upload is consumed with the age it has then (K-async SGD, Sec. I)."""
    X, y, _ = _lsq_problem()
    W, K = 5, 2
    dist = timing.TimeDist(timing.CONST, shift=1.0, slow_mod=W, slow_rem=4, slow_factor=50.0)
    o = ABSOracle(models.LSQ, [6, 1], X, y, np.zeros(6), 4, 0.01, W, K, 3, dist, 1,
                  k_mode=K_FIXED, bound_mode=BOUND_FIXED, restarts=False)
    rows = o.run(120)
    hits = [(t, r["tau"][r["sel"].index(4)]) for t, r in enumerate(rows) if 4 in r["sel"]]
    # the four fast workers finish one job per time unit: two rounds per unit, so the slow job
    # (50 units) arrives in round 100 at the latest, with staleness equal to the round index
    assert hits and hits[0][1] == hits[0][0] and 96 <= hits[0][0] <= 100
    assert all(r["restart"] == [] for r in rows)


def test_k_async_without_restarts_statistics():
    """K = 1, no restarts, i.i.d. exponential times: the arriving worker is uniform (memoryless),
    so the consumed staleness is geometric with mean N - 1 whatever the bound says."""
    X, y, _ = _lsq_problem(d=3)
    W, rounds = 5, 6000
    dist = timing.TimeDist(timing.EXP, rate=1.0)
    o = ABSOracle(models.LSQ, [3, 1], X, y, np.zeros(3), 2, 0.01, W, 1, 1, dist, 3,
                  k_mode=K_FIXED, restarts=False, sa_penalty=True)
    rows = o.run(rounds)
    taus = np.array([row["tau"][0] for row in rows[200:]])
    assert abs(taus.mean() - (W - 1)) < 5 * math.sqrt(W * (W - 1) / len(taus))
    assert taus.max() > 10
