"""Philox4x32-10 as published by Salmon, Moraes, Dror and Shaw (SC'11).

Test infrastructure (see the package header).  Written from the published
description of the generator: a 4x32-bit counter is passed through ten rounds,
each round multiplying two counter words by fixed odd constants, exchanging
high and low product halves and mixing in a 2x32-bit key that is advanced by
Weyl constants between rounds.

The method uses it for two things (random execution times of Sec. V-A and the
independent minibatch draws of Eq. 2); both are addressed by counter, so the
draw of (worker n, job j) never depends on evaluation order.
"""
import numpy as np

MASK32 = 0xFFFFFFFF
MUL_A = 0xD2511F53   # multiplier applied to counter word 0
MUL_B = 0xCD9E8D57   # multiplier applied to counter word 2
WEYL_A = 0x9E3779B9  # key word 0 increment (golden ratio)
WEYL_B = 0xBB67AE85  # key word 1 increment (sqrt(3) - 1)


def philox4x32_10(counter, key):
    """One Philox block on Python integers.

    counter: 4 words, key: 2 words (each 0 <= x < 2**32).  Returns 4 words.
    """
    c0, c1, c2, c3 = (int(x) & MASK32 for x in counter)
    k0, k1 = (int(x) & MASK32 for x in key)
    for _ in range(10):
        prod_a = MUL_A * c0
        prod_b = MUL_B * c2
        hi_a, lo_a = prod_a >> 32, prod_a & MASK32
        hi_b, lo_b = prod_b >> 32, prod_b & MASK32
        c0, c1, c2, c3 = hi_b ^ c1 ^ k0, lo_b, hi_a ^ c3 ^ k1, lo_a
        k0 = (k0 + WEYL_A) & MASK32
        k1 = (k1 + WEYL_B) & MASK32
    return c0, c1, c2, c3


def philox4x32_10_blocks(c0, c1, c2, c3, key):
    """Vectorised form: counter words are equal-length arrays.

    Returns a uint32 array of shape (len, 4).  Same arithmetic as the scalar
    routine, on uint64 lanes masked to 32 bits.
    """
    m = np.uint64(MASK32)
    sh = np.uint64(32)
    c0 = np.asarray(c0, dtype=np.uint64) & m
    c1 = np.asarray(c1, dtype=np.uint64) & m
    c2 = np.asarray(c2, dtype=np.uint64) & m
    c3 = np.asarray(c3, dtype=np.uint64) & m
    k0 = np.uint64(int(key[0]) & MASK32)
    k1 = np.uint64(int(key[1]) & MASK32)
    for _ in range(10):
        prod_a = np.uint64(MUL_A) * c0
        prod_b = np.uint64(MUL_B) * c2
        hi_a, lo_a = prod_a >> sh, prod_a & m
        hi_b, lo_b = prod_b >> sh, prod_b & m
        c0, c1, c2, c3 = hi_b ^ c1 ^ k0, lo_b, hi_a ^ c3 ^ k1, lo_a
        k0 = (k0 + np.uint64(WEYL_A)) & m
        k1 = (k1 + np.uint64(WEYL_B)) & m
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def seed_key(seed):
    """64-bit seed -> (low word, high word) Philox key."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    return seed & MASK32, seed >> 32


TAG_DURATION = 0   # counter word 2 for the job-duration stream
TAG_MINIBATCH = 1  # counter word 2 for the minibatch-index stream


def duration_word(seed, n, j):
    """The 32-bit word that decides the duration of job j of worker n:
    word 0 of block (n, j, TAG_DURATION, 0)."""
    return philox4x32_10((n, j, TAG_DURATION, 0), seed_key(seed))[0]


def duration_words(seed, n, j, count):
    """`count` words of the job-duration stream of job j of worker n: word i is
    word (i mod 4) of block (n, j, TAG_DURATION, i // 4); word 0 is
    `duration_word`."""
    out = []
    for blk in range((count + 3) // 4):
        out.extend(int(x) for x in philox4x32_10((n, j, TAG_DURATION, blk), seed_key(seed)))
    return out[:count]


def minibatch_words(seed, n, j, batch, step=0):
    """`batch` 32-bit words for the minibatch of local step `step` of job j of
    worker n: sample b uses word (b mod 4) of block
    (n, j, TAG_MINIBATCH, step * ceil(batch / 4) + b // 4)."""
    nblk = (batch + 3) // 4
    blk = np.arange(nblk, dtype=np.uint64) + np.uint64(step * nblk)
    out = philox4x32_10_blocks(np.full(nblk, n), np.full(nblk, j),
                               np.full(nblk, TAG_MINIBATCH), blk, seed_key(seed))
    return out.reshape(-1)[:batch]
