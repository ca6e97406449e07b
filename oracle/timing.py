"""Simulated execution time of one worker job, in integer ticks.

Test infrastructure (see the package header).  The paper draws each worker's
execution time from a distribution that produces stragglers (Sec. V-A) and the
server waits for the fastest arrivals (Sec. II-A, Algorithm 1 "server
executes").  Here a job's duration is a deterministic function of
(seed, worker n, job index j) so that the arrival order is reproducible
bit for bit:

    r    = Philox word of (n, j)                          (32 bits)
    u    = (r + 1/2) * 2**-32                             in (0, 1), exact
    dur  = shift                                          CONST
           -ln_spec(u) / rate                             EXP
           shift + (-ln_spec(u) / rate)                   SHIFTED_EXP
           scale / sqrt(u)                                PARETO2 (shape 2)
           shift + (e_0 + e_1 + ... + e_{k-1}) / rate     GAMMA, integer shape k >= 1:
               e_i = -ln_spec(u_i), u_i from word i mod 4 of Philox block
               (n, j, 0, i div 4); the sum runs left to right.  A sum of k
               independent Exp(rate) times is Gamma(k, rate), the law the paper
               draws its execution times from (Sec. V-A); k = 1 is SHIFTED_EXP
    dur *= slow_factor   if slow_mod > 0 and n mod slow_mod == slow_rem
    ticks = floor(dur * 2**20), at least 1, and below 2**53

Every floating-point step is one IEEE-754 binary64 operation rounded to
nearest (Python floats are exactly that; nothing is fused), so any other
implementation built from correctly rounded add/mul/div/sqrt reproduces the
same integers.  `ln_spec` is *defined* by the series below; how close it is to
the true logarithm only matters for the distribution's shape.
"""
import math
import struct

from . import philox

CONST, EXP, SHIFTED_EXP, PARETO2, GAMMA = 0, 1, 2, 3, 4
MAX_SHAPE = 64
TICKS_PER_UNIT = 2.0 ** 20
MAX_TICKS = 1 << 53

LN2 = 0.6931471805599453      # binary64 nearest to ln 2 (0x3FE62E42FEFA39EF)
SQRT2 = 1.4142135623730951    # binary64 nearest to sqrt 2 (0x3FF6A09E667F3BCD)


class TimeDist:
    """Plain record of the distribution parameters."""

    def __init__(self, kind, shift=0.0, rate=1.0, scale=1.0,
                 slow_mod=0, slow_rem=0, slow_factor=1.0, shape=1):
        self.kind = int(kind)
        self.shift = float(shift)
        self.rate = float(rate)
        self.scale = float(scale)
        self.slow_mod = int(slow_mod)
        self.slow_rem = int(slow_rem)
        self.slow_factor = float(slow_factor)
        self.shape = int(shape)


def ln_spec(u):
    """Series logarithm of a positive, normal binary64 number.

    u = m * 2**e with sqrt(1/2) <= m < sqrt(2) (taken from the bit pattern),
    s = (m - 1) / (m + 1),
    ln u = e*LN2 + 2 s (1 + s^2/3 + s^4/5 + ... + s^22/23), Horner from the
    highest term, coefficients 1/(2k+1) formed by one division each.
    """
    bits = struct.unpack("<Q", struct.pack("<d", u))[0]
    e = ((bits >> 52) & 0x7FF) - 1023
    m = struct.unpack("<d", struct.pack("<Q", (bits & ((1 << 52) - 1)) | (1023 << 52)))[0]
    if m >= SQRT2:          # m in [1,2) -> fold the upper part down (exact halving)
        m = m * 0.5
        e += 1
    s = (m - 1.0) / (m + 1.0)
    s2 = s * s
    p = 1.0 / 23.0
    for k in range(10, -1, -1):           # 1/21, 1/19, ..., 1/3, 1/1
        p = p * s2
        p = p + 1.0 / float(2 * k + 1)
    head = float(e) * LN2
    tail = (2.0 * s) * p
    return head + tail


def uniform_from_word(r):
    """(r + 1/2) * 2**-32: never 0, never 1, exact in binary64."""
    return (float(r) + 0.5) * (2.0 ** -32)


def duration_from_word(dist, n, r, more_words=None):
    """Ticks of a job of worker n whose Philox word is r (GAMMA: `more_words`
    are the words 1 .. shape-1 of the job)."""
    u = uniform_from_word(r)
    if dist.kind == GAMMA:
        if not (1 <= dist.shape <= MAX_SHAPE):
            raise ValueError("gamma shape out of range")
        total = -ln_spec(u)
        for i in range(1, dist.shape):
            total = total + (-ln_spec(uniform_from_word(more_words[i - 1])))
        dur = dist.shift + total / dist.rate
    elif dist.kind == CONST:
        dur = dist.shift
    elif dist.kind == EXP:
        dur = (-ln_spec(u)) / dist.rate
    elif dist.kind == SHIFTED_EXP:
        dur = dist.shift + (-ln_spec(u)) / dist.rate
    elif dist.kind == PARETO2:
        dur = dist.scale / math.sqrt(u)
    else:
        raise ValueError("unknown time distribution")
    if dist.slow_mod > 0 and n % dist.slow_mod == dist.slow_rem:
        dur = dur * dist.slow_factor
    scaled = dur * TICKS_PER_UNIT
    if not (scaled < float(MAX_TICKS)):
        raise OverflowError("job duration out of tick range")
    ticks = int(math.floor(scaled))
    return max(ticks, 1)


def duration_ticks(dist, seed, n, j):
    """Ticks of job j of worker n under `seed`."""
    if dist.kind == GAMMA and dist.shape > 1:
        words = philox.duration_words(seed, n, j, dist.shape)
        return duration_from_word(dist, n, words[0], words[1:])
    return duration_from_word(dist, n, philox.duration_word(seed, n, j))
