"""Test-side exact arithmetic for the scale of the scaled-sign compressor (Eq. 2: ||v||_1 / n), written
with Python integers and fractions only, and tensors built so that the two readings of "turn the exact
128-bit sum into a double" -- truncate to the top 53 bits, or round to nearest -- give different floats.

Nothing here is shared with the oracle or the CUDA library: both are checked against it."""
from fractions import Fraction

import numpy as np


def fixed_sum(v):
    """S = sum_i floor(|v_i| * 2^64) with exact integers."""
    total = 0
    for a in np.asarray(v, dtype=np.float32).ravel():
        if a != 0:
            total += int(Fraction(abs(float(a))) * (1 << 64))      # int() floors a non-negative fraction
    return total


def _scale(S, n, round_to_nearest):
    if S == 0:
        return np.float32(0.0)
    p = S.bit_length() - 1
    if p > 52:
        sh = p - 52
        S = (((S + (1 << (sh - 1))) if round_to_nearest else S) >> sh) << sh
    q = Fraction(S, n)
    q = q.numerator / q.denominator                                # int / int: one correctly rounded division
    return np.float32(q * 2.0 ** -64)                              # exact scaling, one rounding to float


def scale_truncating(S, n):
    """The reading taken: clear everything below the top 53 bits, divide once in double, round once to float."""
    return _scale(S, n, False)


def scale_rounding(S, n):
    """The other reading (the sum rounded to 53 bits first): where the two differ, a case discriminates."""
    return _scale(S, n, True)


def discriminating_sum(n, top_bit, rng):
    """An integer S with leading bit `top_bit` (>= 60) for which the two readings give different floats: its
    53-bit truncation divided by n lies just below the midpoint of two neighbouring floats, the dropped
    bits are all ones, and rounding them in carries the quotient to the midpoint or beyond."""
    sh = top_bit - 52
    u = 1 << sh
    for _ in range(10000):
        S0 = (1 << top_bit) | int(rng.integers(0, 1 << 52)) << sh
        q0 = S0 // n
        g = 1 << (q0.bit_length() - 1 - 24)                        # float midpoints: odd multiples of g
        Bq = ((q0 // g) | 1) * g
        S53 = ((n * Bq - 1) // u) * u                              # largest multiple of u with S53 / n < Bq
        S = S53 + u - 1
        if S53.bit_length() - 1 != top_bit:
            continue
        if scale_truncating(S, n) != scale_rounding(S, n):
            return S
    raise AssertionError("no discriminating sum found")


def tensor_with_sum(S, n, rng, mixed_signs=True):
    """n floats whose exact fixed-point L1 sum is S (< 2^96): S cut greedily into pieces of at most 24
    significant bits (each then is one float times 2^64), scattered among zeros by a seeded permutation."""
    pieces = []
    r = S
    while r:
        s = max(r.bit_length() - 24, 0)
        c = (r >> s) << s
        pieces.append(c)
        r -= c
    assert len(pieces) <= n and S < (1 << 96)
    v = np.zeros(n, dtype=np.float32)
    pos = rng.permutation(n)[:len(pieces)]
    for q, c in zip(pos, pieces):
        v[q] = np.float32(Fraction(c, 1 << 64))
        assert Fraction(float(v[q])) == Fraction(c, 1 << 64)       # exactly representable
    if mixed_signs:
        v[pos[1::2]] *= np.float32(-1.0)
    assert fixed_sum(v) == S
    return v


def discriminating_tensor(n, top_bit, seed):
    rng = np.random.default_rng(seed)
    return tensor_with_sum(discriminating_sum(n, top_bit, rng), n, rng)
