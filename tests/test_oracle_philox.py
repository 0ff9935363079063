"""Pins for oracle/philox.py: published known-answer vectors, exact end-point
values of the uniform map, Box-Muller against angles worked by hand, the counter
layout, and distribution checks on 10^6 draws."""
import math
import os

import numpy as np
import pytest
from scipy import stats

from oracle import philox

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _kat_rows():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        rows.append([int(x, 16) for x in line.split()])
    return rows


@pytest.mark.parametrize("row", _kat_rows())
def test_known_answer_vectors(row):
    out = philox.philox4x32_10(*row[:6])
    assert [int(o) for o in out] == row[6:]


def test_uniform_map_end_points_and_grid():
    # r = 0 -> 2^-24 ; r = 2^32-1 -> 1 - 2^-24 ; the low 9 bits are dropped
    assert philox.uniform_from_word(0) == 2.0 ** -24
    assert philox.uniform_from_word(0xFFFFFFFF) == 1.0 - 2.0 ** -24
    assert philox.uniform_from_word(511) == 2.0 ** -24
    assert philox.uniform_from_word(512) == 3 * 2.0 ** -24
    assert philox.uniform_from_word(1 << 31) == 0.5 + 2.0 ** -24
    # every value is representable in float32 (24-bit significand)
    r = np.arange(0, 2 ** 32, 7919 * 1009, dtype=np.uint64)
    uu = philox.uniform_from_word(r)
    assert np.all(uu.astype(np.float32).astype(np.float64) == uu)


def test_box_muller_hand_values():
    # U(r_even) = 1/2 + 2^-24 ~ radius sqrt(2 ln 2); angle from r_odd
    rad = math.sqrt(-2 * math.log(0.5 + 2.0 ** -24))
    quarter = (1 << 30)           # U = 1/4 + 2^-24 -> angle ~ pi/2
    n0, n1 = philox.box_muller(1 << 31, quarter)
    ang = 2 * math.pi * (0.25 + 2.0 ** -24)
    assert n0 == pytest.approx(rad * math.cos(ang), abs=1e-15)
    assert n1 == pytest.approx(rad * math.sin(ang), abs=1e-15)
    assert abs(n0) < 1e-6 and n1 == pytest.approx(math.sqrt(2 * math.log(2)), rel=1e-6)
    n0, n1 = philox.box_muller(1 << 31, 1 << 31)      # angle ~ pi
    assert n0 == pytest.approx(-math.sqrt(2 * math.log(2)), rel=1e-6) and abs(n1) < 1e-6


def test_counter_layout():
    seed, chain, step, d = 0x1234567811223344, 77, 5, 11
    x = philox.xi(seed, chain, [step], d)[0]
    for q in range(3):
        w = [int(v) for v in philox.philox4x32_10(q, step, chain, 0, seed & 0xFFFFFFFF, seed >> 32)]
        a, b = philox.box_muller(w[0], w[1])
        c, e = philox.box_muller(w[2], w[3])
        for j, val in enumerate((a, b, c, e)):
            if 4 * q + j < d:
                assert x[4 * q + j] == val
    w = [int(v) for v in philox.philox4x32_10(0, step, chain, 1, seed & 0xFFFFFFFF, seed >> 32)]
    assert philox.u(seed, chain, [step])[0] == philox.uniform_from_word(w[0])
    # a prefix of a longer vector is the shorter vector (dimension-block counters)
    assert np.array_equal(philox.xi(seed, chain, [step], 7)[0], x[:7])
    # step / chain / seed each select a different stream
    assert not np.allclose(philox.xi(seed, chain, [step + 1], d)[0], x)
    assert not np.allclose(philox.xi(seed, chain + 1, [step], d)[0], x)
    assert not np.allclose(philox.xi(seed + 1, chain, [step], d)[0], x)


def test_distributions():
    n = 1_000_000
    x = philox.xi(3, 9, np.arange(1, n // 8 + 1), 8).ravel()
    assert abs(x.mean()) < 4 / math.sqrt(n)
    assert abs(x.var() - 1) < 4 * math.sqrt(2 / n)
    assert abs(stats.kurtosis(x)) < 4 * math.sqrt(24 / n)
    assert stats.kstest(x[::5], "norm").pvalue > 1e-3
    # components within one Philox call are uncorrelated
    c = np.corrcoef(x.reshape(-1, 4).T)
    assert np.max(np.abs(c - np.eye(4))) < 5 / math.sqrt(n / 4)
    uu = philox.u(3, 9, np.arange(1, 200_001))
    assert stats.kstest(uu, "uniform").pvalue > 1e-3
    assert 0 < uu.min() and uu.max() < 1
    # xi and u of the same step are independent streams
    x0 = philox.xi(3, 9, np.arange(1, 200_001), 1).ravel()
    assert abs(np.corrcoef(x0, uu)[0, 1]) < 5 / math.sqrt(200_000)
