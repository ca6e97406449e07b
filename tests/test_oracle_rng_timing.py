"""Pins for the oracle's random streams and simulated execution times."""
import math
import os

import numpy as np
import pytest

from oracle import abs_sim, philox, timing

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v = [int(x, 16) for x in line.split()]
            rows.append((v[0:4], v[4:6], v[6:10]))
    return rows


def test_philox_known_answers():
    rows = _kat_rows()
    assert len(rows) == 3
    for ctr, key, out in rows:
        assert list(philox.philox4x32_10(ctr, key)) == out


def test_philox_vector_form_matches_scalar():
    rng = np.random.default_rng(7)
    ctr = rng.integers(0, 2 ** 32, size=(64, 4), dtype=np.uint64)
    key = (0x89ABCDEF, 0x01234567)
    vec = philox.philox4x32_10_blocks(ctr[:, 0], ctr[:, 1], ctr[:, 2], ctr[:, 3], key)
    for i in range(64):
        assert list(vec[i]) == list(philox.philox4x32_10(ctr[i], key))
    for ctr_k, key_k, out in _kat_rows():
        v = philox.philox4x32_10_blocks(*[[c] for c in ctr_k], key_k)
        assert list(v[0]) == out


def test_stream_addressing():
    seed = 0x123456789ABCDEF0
    key = philox.seed_key(seed)
    assert key == (0x9ABCDEF0, 0x12345678)
    assert philox.duration_word(seed, 5, 9) == philox.philox4x32_10((5, 9, 0, 0), key)[0]
    words = philox.minibatch_words(seed, 3, 2, 10)
    for b in range(10):
        assert int(words[b]) == philox.philox4x32_10((3, 2, 1, b // 4), key)[b % 4]


def test_words_look_uniform():
    # crude equidistribution check: mean and variance of 2^16 words
    blk = np.arange(1 << 14)
    w = philox.philox4x32_10_blocks(blk, blk * 0, blk * 0, blk * 0, (1, 2)).reshape(-1)
    u = (w.astype(np.float64) + 0.5) / 2 ** 32
    assert abs(u.mean() - 0.5) < 0.005
    assert abs(u.var() - 1 / 12) < 0.002


def test_ln_spec_close_to_libm():
    rng = np.random.default_rng(3)
    samples = list(rng.integers(0, 2 ** 32, size=4000)) + [0, 1, 2 ** 32 - 1, 2 ** 31, 2 ** 31 - 1]
    for r in samples:
        u = timing.uniform_from_word(int(r))
        assert 0.0 < u < 1.0
        ref = math.log(u)
        assert abs(timing.ln_spec(u) - ref) <= 1e-14 * max(1.0, abs(ref))
    for x in [1.0, 2.0, 0.5, math.sqrt(2.0), 1.4142135623730949, 3.0, 1e-9, 123456.789]:
        assert abs(timing.ln_spec(x) - math.log(x)) <= 1e-14 * max(1.0, abs(math.log(x)))
    assert timing.ln_spec(1.0) == 0.0


def test_ticks_monotone_in_u():
    exp = timing.TimeDist(timing.EXP, rate=1.0)
    par = timing.TimeDist(timing.PARETO2, scale=1.0)
    words = sorted(set(int(x) for x in np.random.default_rng(5).integers(0, 2 ** 32, size=3000)))
    for dist in (exp, par):
        ticks = [timing.duration_from_word(dist, 0, r) for r in words]
        # larger u  <=>  shorter job for both laws
        assert all(a >= b for a, b in zip(ticks, ticks[1:]))
        assert min(ticks) >= 1


def test_const_shift_and_slow_class():
    d = timing.TimeDist(timing.CONST, shift=1.5, slow_mod=4, slow_rem=3, slow_factor=2.0 ** 20)
    assert timing.duration_from_word(d, 0, 12345) == int(1.5 * 2 ** 20)
    assert timing.duration_from_word(d, 3, 999) == int(1.5 * 2 ** 40)
    assert timing.duration_from_word(d, 7, 0) == int(1.5 * 2 ** 40)
    e0 = timing.TimeDist(timing.EXP, rate=2.0)
    e1 = timing.TimeDist(timing.SHIFTED_EXP, shift=1.0, rate=2.0)
    for r in (0, 17, 2 ** 31, 2 ** 32 - 1):
        # the shift adds exactly 2^20 ticks up to the rounding of one addition
        assert abs(timing.duration_from_word(e1, 0, r) - timing.duration_from_word(e0, 0, r)
                   - 2 ** 20) <= 1
    with pytest.raises(OverflowError):
        timing.duration_from_word(timing.TimeDist(timing.CONST, shift=2.0 ** 40), 0, 0)


def test_exponential_law():
    d = timing.TimeDist(timing.EXP, rate=1.0)
    n = 20000
    t = np.array([timing.duration_ticks(d, 99, i, 0) for i in range(n)], dtype=np.float64) / 2 ** 20
    assert abs(t.mean() - 1.0) < 4 / math.sqrt(n)
    # memoryless tail: P(T > 1) = e^-1
    assert abs((t > 1.0).mean() - math.exp(-1)) < 4 * math.sqrt(0.23 / n)


def test_pareto_tail():
    d = timing.TimeDist(timing.PARETO2, scale=1.0)
    n = 20000
    t = np.array([timing.duration_ticks(d, 5, i, 3) for i in range(n)], dtype=np.float64) / 2 ** 20
    assert t.min() >= 1.0 - 2 ** -20
    for x in (1.5, 2.0, 4.0):
        p = x ** -2.0                    # P(dur > x) for shape 2, scale 1
        assert abs((t > x).mean() - p) < 4 * math.sqrt(p * (1 - p) / n)


def test_first_round_time_matches_order_statistic():
    """Round 0 ends at the K-th smallest of W i.i.d. Exp(1) times; its mean is
    sum_{i<K} 1/(W-i) (Renyi's representation)."""
    W, K = 12, 5
    d = timing.TimeDist(timing.EXP, rate=1.0)
    ends = []
    for seed in range(3000):
        c = sorted(timing.duration_ticks(d, seed, n, 0) for n in range(W))
        ends.append(c[K - 1] / 2 ** 20)
    expect = sum(1.0 / (W - i) for i in range(K))
    var = sum(1.0 / (W - i) ** 2 for i in range(K))
    assert abs(np.mean(ends) - expect) < 4 * math.sqrt(var / len(ends))


def test_minibatch_indices_stay_in_shard():
    W, M = 7, 1000
    covered = []
    for n in range(W):
        lo, hi = abs_sim.shard_bounds(n, W, M)
        covered += list(range(lo, hi))
        for j in range(5):
            idx = abs_sim.minibatch_indices(11, n, j, 33, W, M)
            assert idx.shape == (33,)
            assert idx.min() >= lo and idx.max() < hi
            words = philox.minibatch_words(11, n, j, 33)
            assert [int(i) for i in idx] == [lo + (int(r) * (hi - lo) >> 32) for r in words]
    assert covered == list(range(M))          # disjoint shards whose union is the dataset
    # draws spread over the whole shard
    idx = np.concatenate([abs_sim.minibatch_indices(1, 0, j, 64, 2, 1000) for j in range(200)])
    assert idx.min() < 10 and idx.max() >= 490 and abs(idx.mean() - 249.5) < 5


def test_gamma_shape_one_is_shifted_exponential():
    """Gamma(1, rate) = Exp(rate): the same Philox word, the same operations, the same ticks."""
    g1 = timing.TimeDist(timing.GAMMA, shift=0.5, rate=2.0, shape=1)
    se = timing.TimeDist(timing.SHIFTED_EXP, shift=0.5, rate=2.0)
    for n in range(12):
        for j in range(12):
            assert timing.duration_ticks(g1, 9, n, j) == timing.duration_ticks(se, 9, n, j)


def test_gamma_is_a_sum_of_exponentials_of_distinct_words():
    """Shape k adds k exponential draws taken from k different Philox words of the job (words
    0..3 of block 0, then block 1, ...); a repeated or skipped word would break the sum below."""
    seed, n, j, k, rate = 77, 3, 11, 6, 1.25
    words = philox.duration_words(seed, n, j, k)
    assert len(set(words)) == k and words[0] == philox.duration_word(seed, n, j)
    blk1 = philox.philox4x32_10((n, j, philox.TAG_DURATION, 1), philox.seed_key(seed))
    assert words[4] == blk1[0] and words[5] == blk1[1]
    exp1 = timing.TimeDist(timing.EXP, rate=rate)
    parts = [timing.duration_from_word(exp1, n, w) for w in words]           # ticks of each draw
    g = timing.TimeDist(timing.GAMMA, shift=0.0, rate=rate, shape=k)
    total = timing.duration_ticks(g, seed, n, j)
    assert abs(total - sum(parts)) <= k            # each part was floored on its own


def test_gamma_moments_and_cdf():
    """Mean k/rate, variance k/rate^2, and the distribution function against scipy's."""
    from scipy import stats
    k, rate = 3, 1.5
    g = timing.TimeDist(timing.GAMMA, shift=0.0, rate=rate, shape=k)
    v = np.array([timing.duration_ticks(g, 5, n, j) for n in range(150) for j in range(100)]) / 2.0 ** 20
    assert abs(v.mean() - k / rate) < 0.03
    assert abs(v.var() - k / rate ** 2) < 0.06
    for x in (0.5, 1.0, 2.0, 4.0):
        assert abs((v < x).mean() - stats.gamma.cdf(x, a=k, scale=1.0 / rate)) < 0.015
    with pytest.raises(ValueError):
        timing.duration_ticks(timing.TimeDist(timing.GAMMA, shape=0), 1, 0, 0)
