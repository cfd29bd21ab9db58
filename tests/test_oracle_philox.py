"""Pins for the checker's counter-based generator (Philox4x32-10)."""
import math
import os

import numpy as np

from oracle import jd_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_known_answer_vectors():
    rows = _kat()
    assert len(rows) >= 2
    for ctr, key, out in rows:
        assert list(O.philox4x32_10(ctr, key)) == out


def test_each_counter_and_key_word_matters():
    # a dropped word (wrong index in the round function) would leave one of these unchanged
    base = O.philox4x32_10((1, 2, 3, 4), (5, 6))
    for i in range(4):
        c = [1, 2, 3, 4]
        c[i] ^= 0x10
        assert O.philox4x32_10(c, (5, 6)) != base
    for i in range(2):
        k = [5, 6]
        k[i] ^= 0x10
        assert O.philox4x32_10((1, 2, 3, 4), k) != base


def test_uniform24_grid_and_keying():
    u = O.uniform24(7, 3, 2, O.STREAM_ACCEPT)
    assert 0.0 <= u < 1.0
    assert (u * 2 ** 24) == int(u * 2 ** 24)
    # definition: key = seed split in two words, counter = (b, slot, stream, 0), word 0, top 24 bits
    seed = (0x299f31d0 << 32) | 0xa4093822
    w0 = O.philox4x32_10((0x243f6a88, 0x85a308d3, 1, 0), (0xa4093822, 0x299f31d0))[0]
    assert O.uniform24(seed, 0x243f6a88, 0x85a308d3, 1) == (w0 >> 8) / 2 ** 24
    # the two streams at the same slot are different draws
    assert O.uniform24(7, 3, 2, O.STREAM_ACCEPT) != O.uniform24(7, 3, 2, O.STREAM_SAMPLE)
    # seed high word is part of the key
    assert O.uniform24(1, 0, 0, 0) != O.uniform24(1 | (1 << 32), 0, 0, 0)


def test_uniformity_and_lag1():
    n = 40000
    u = np.array([O.uniform24(12345, b, b % 7, 0) for b in range(n)])
    # Kolmogorov-Smirnov against U[0,1)
    s = np.sort(u)
    i = np.arange(1, n + 1)
    dstat = max(np.max(i / n - s), np.max(s - (i - 1) / n))
    assert dstat < 1.95 / math.sqrt(n)          # ~ p > 1e-3
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / n)
    # lag-1 correlation over consecutive b
    c = np.corrcoef(u[:-1], u[1:])[0, 1]
    assert abs(c) < 4 / math.sqrt(n)
