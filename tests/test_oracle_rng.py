"""Pins for the oracle's random-number layer (CPU only).

The generator is pinned to published known-answer vectors; the uniform map and the
counter layout are pinned to their written definition and to distribution tests.
"""
import math
import os

import numpy as np
import pytest
from scipy import stats

import oracle


def _kat_rows(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(t, 16) for t in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers(golden_dir):
    rows = _kat_rows(golden_dir)
    assert len(rows) == 3
    for ctr, key, want in rows:
        got = oracle.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == want


def test_philox_counter_words_matter():
    # every counter word and key word changes the output block (catches a dropped input)
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    for i in range(4):
        c = [1, 2, 3, 4]
        c[i] += 1
        assert not np.array_equal(oracle.philox4x32_10(c, [5, 6]), base)
    for i in range(2):
        k = [5, 6]
        k[i] += 1
        assert not np.array_equal(oracle.philox4x32_10([1, 2, 3, 4], k), base)


@pytest.mark.parametrize("level", [0, 1, 2])
def test_uniform_follows_the_counter_layout(level):
    # counter = (index>>2, step, slot, (batch<<2)|level), key = seed halves, word = index&3,
    # u = (2*(word>>9)+1) / 2^24
    seed, batch, slot, step = 0x1234_5678_9ABC_DEF0, 7, 11, 1234
    for index in [0, 1, 2, 3, 4, 5, 1023, 152063, 2**31 + 5]:
        ctr = [(index >> 2) & 0xFFFFFFFF, step, slot, (batch << 2) | level]
        key = [seed & 0xFFFFFFFF, seed >> 32]
        word = int(oracle.philox4x32_10(ctr, key)[index & 3])
        want = (2 * (word >> 9) + 1) / 2**24
        assert oracle.uniform(seed, batch, slot, step, level, index) == want


def test_uniform_is_open_interval_and_float32_exact():
    us = np.array([oracle.uniform(3, 0, s, t, 0, i) for s in range(4) for t in range(4) for i in range(512)])
    assert us.min() >= 2.0**-24 and us.max() <= 1 - 2.0**-24
    assert np.array_equal(us.astype(np.float32).astype(np.float64), us)
    # the extremes of the map give finite Gumbel noise
    for u in (2.0**-24, 1 - 2.0**-24):
        g = -math.log(-math.log(u))
        assert math.isfinite(g) and -2.82 < g < 16.65


def test_uniform_is_uniform():
    us = np.array([oracle.uniform(99, 1, 0, t, 0, i) for t in range(20) for i in range(5000)])
    assert stats.kstest(us, "uniform").pvalue > 1e-3
    assert abs(us.mean() - 0.5) < 0.005
    # Gumbel noise built from it: mean = Euler-Mascheroni constant, variance = pi^2/6
    g = -np.log(-np.log(us))
    assert abs(g.mean() - 0.5772156649) < 0.02
    assert abs(g.var() - math.pi**2 / 6) < 0.05


def test_streams_are_distinct():
    a = [oracle.uniform(5, 0, 0, 0, 0, i) for i in range(64)]
    assert a != [oracle.uniform(5, 0, 0, 0, 1, i) for i in range(64)]   # level
    assert a != [oracle.uniform(5, 0, 0, 1, 0, i) for i in range(64)]   # step
    assert a != [oracle.uniform(5, 0, 1, 0, 0, i) for i in range(64)]   # slot
    assert a != [oracle.uniform(5, 1, 0, 0, 0, i) for i in range(64)]   # batch
    assert a != [oracle.uniform(6, 0, 0, 0, 0, i) for i in range(64)]   # seed
    assert a == [oracle.uniform(5, 0, 0, 0, 0, i) for i in range(64)]   # and reproducible
