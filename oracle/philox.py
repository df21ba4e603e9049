"""Philox4x32-10 counter-based generator -- CPU oracle copy (test infrastructure).

Written from the published definition (Salmon, Moraes, Dror, Shaw, "Parallel
random numbers: as easy as 1, 2, 3", SC'11, Section 3.3 and Table 2): a
4-word counter and a 2-word key go through ten rounds; each round multiplies
counter words 0 and 2 by two fixed odd constants, keeps high and low halves,
xors the high halves with the other counter words and the key, and permutes;
the key is bumped by two Weyl constants between rounds.

Pinned in tests against the known-answer vectors distributed with the authors'
Random123 library (tests/golden/philox4x32_10_kat.txt).

Counter convention of this project (Algorithm 1's random choices must be
reproducible from (seed, member, round)):
    counter = (member, round_or_step, stream, block), key = (seed_lo, seed_hi)
    stream 0: exploit donor draw     stream 1: explore perturbation bits
    stream 2: training-batch window  stream 3: weight initialisation
"""
from __future__ import annotations

import numpy as np

M0 = 0xD2511F53
M1 = 0xCD9E8D57
W0 = 0x9E3779B9
W1 = 0xBB67AE85
MASK = 0xFFFFFFFF

STREAM_EXPLOIT = 0
STREAM_EXPLORE = 1
STREAM_BATCH = 2
STREAM_INIT = 3
STREAM_INTERP = 4  # interpolation coefficients of the gradient penalty


def philox4x32_10(counter, key):
    """Scalar reference: counter = 4 ints, key = 2 ints (each < 2**32) -> 4 ints."""
    c0, c1, c2, c3 = (int(c) & MASK for c in counter)
    k0, k1 = (int(k) & MASK for k in key)
    for r in range(10):
        if r > 0:
            k0 = (k0 + W0) & MASK
            k1 = (k1 + W1) & MASK
        p0 = M0 * c0
        p1 = M1 * c2
        hi0, lo0 = p0 >> 32, p0 & MASK
        hi1, lo1 = p1 >> 32, p1 & MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0), lo1, (hi0 ^ c3 ^ k1), lo0
    return c0, c1, c2, c3


def philox4x32_10_np(c0, c1, c2, c3, seed: int):
    """Vectorised over counter arrays (broadcastable); returns 4 uint32 arrays."""
    c0, c1, c2, c3 = np.broadcast_arrays(*(np.asarray(c, dtype=np.uint64) for c in (c0, c1, c2, c3)))
    c0, c1, c2, c3 = (c.copy() for c in (c0, c1, c2, c3))
    k0 = int(seed) & MASK
    k1 = (int(seed) >> 32) & MASK
    m = np.uint64(MASK)
    s32 = np.uint64(32)
    for r in range(10):
        if r > 0:
            k0 = (k0 + W0) & MASK
            k1 = (k1 + W1) & MASK
        p0 = np.uint64(M0) * c0
        p1 = np.uint64(M1) * c2
        hi0, lo0 = p0 >> s32, p0 & m
        hi1, lo1 = p1 >> s32, p1 & m
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def draw(seed: int, member: int, round_or_step: int, stream: int, block: int = 0):
    """The project's keyed draw: 4 words for (seed; member, round/step, stream, block)."""
    return philox4x32_10((member, round_or_step, stream, block),
                         (int(seed) & MASK, (int(seed) >> 32) & MASK))
