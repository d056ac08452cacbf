"""Philox4x32-10 (test infrastructure; see oracle/__init__.py).

The paper only says r ~ U[0,1] (Eq. 1).  To make the randomised procedure
reproducible on any device, every uniform is a pure function of
(seed, absolute position, step index, sequence id, stream tag) through the
counter-based generator Philox4x32 with ten rounds as defined by Salmon,
Moraes, Dror and Shaw, "Parallel random numbers: as easy as 1, 2, 3" (SC'11):
a 128-bit counter, a 64-bit key, two 32x32->64 multiplications per round and a
Weyl key schedule.

Plain Python integers: slow, obviously correct.  `philox4x32_10_np` is the
same round function over numpy uint64 arrays for bulk draws.
"""
from __future__ import annotations

import numpy as np

_M0 = 0xD2511F53  # multiplier applied to counter word 0
_M1 = 0xCD9E8D57  # multiplier applied to counter word 2
_W0 = 0x9E3779B9  # key word 0 increment (golden ratio)
_W1 = 0xBB67AE85  # key word 1 increment (sqrt(3) - 1)
_MASK = 0xFFFFFFFF

STREAM_VERIFY = 0   # words 0,1,2 = acceptance / residual / re-draft uniforms
STREAM_INIT = 1     # word 0 = fresh random-token initialisation
STEP_INITIAL_WINDOW = 0xFFFFFFFF  # step index used for the very first window


def philox4x32_10(counter, key):
    """Ten Philox rounds.  counter: 4 words, key: 2 words -> 4 output words."""
    c0, c1, c2, c3 = (int(x) & _MASK for x in counter)
    k0, k1 = (int(x) & _MASK for x in key)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK
        hi1, lo1 = p1 >> 32, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK, lo1, (hi0 ^ c3 ^ k1) & _MASK, lo0
    return (c0, c1, c2, c3)


def philox4x32_10_np(c0, c1, c2, c3, k0, k1):
    """Vectorised form: all arguments broadcastable integer arrays."""
    c0, c1, c2, c3 = (np.asarray(x, dtype=np.uint64) & np.uint64(_MASK) for x in (c0, c1, c2, c3))
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = np.uint64(int(k0) & _MASK)
    k1 = np.uint64(int(k1) & _MASK)
    mask = np.uint64(_MASK)
    s32 = np.uint64(32)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + np.uint64(_W0)) & mask
            k1 = (k1 + np.uint64(_W1)) & mask
        p0 = np.uint64(_M0) * c0
        p1 = np.uint64(_M1) * c2
        hi0, lo0 = p0 >> s32, p0 & mask
        hi1, lo1 = p1 >> s32, p1 & mask
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & mask, lo1, (hi0 ^ c3 ^ k1) & mask, lo0
    return c0, c1, c2, c3


def split_seed(seed: int):
    """64-bit seed -> Philox key (low word, high word)."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    return (seed & _MASK, seed >> 32)


def u24(word: int) -> float:
    """Top 24 bits of a 32-bit word as a uniform in [0, 1).

    k / 2^24 is exactly representable in fp32 and fp64, so an fp32 device and
    this fp64 oracle compare against the identical number."""
    return float(int(word) >> 8) * (1.0 / 16777216.0)


def verify_uniforms(seed: int, position: int, step: int, seq: int):
    """(u_acc, u_res, u_draft) for one window position of one step.

    One Philox call per (sequence, step, absolute position): word 0 decides
    acceptance (Eq. 1), word 1 drives the residual resample (Eq. 2) and
    word 2 the re-draft (Eq. 3)."""
    w = philox4x32_10((position, step, seq, STREAM_VERIFY), split_seed(seed))
    return u24(w[0]), u24(w[1]), u24(w[2])


def init_uniform(seed: int, position: int, step: int, seq: int) -> float:
    """The uniform a freshly initialised slot is drawn with when its token comes from a neighbour's
    predicted distribution (Sec. 4.2 (c), (d)): the same Philox word as init_token, as a 24-bit uniform."""
    w = philox4x32_10((position, step, seq, STREAM_INIT), split_seed(seed))
    return u24(w[0])


def init_token(seed: int, position: int, step: int, seq: int, vocab: int) -> int:
    """Uniform token in [0, vocab) for a freshly initialised window slot
    (Sec. 4.2: candidates drawn from a uniform distribution): floor(word*V/2^32)."""
    w = philox4x32_10((position, step, seq, STREAM_INIT), split_seed(seed))
    return (w[0] * int(vocab)) >> 32
