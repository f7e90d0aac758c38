"""Pins for the oracle's bit-width, shift-and-round and rounding functions (CPU only).

Every check compares the C oracle with something fixed by the paper or by mathematics:
hand-worked cases (tests/golden), closed forms over all 2^bp discarded fractions, Python's
int.bit_length, and an independent bit-string transcription of Algorithm 3."""
import os
from fractions import Fraction

import numpy as np
import pytest

import pyref

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            yield line


def test_worked_cases(oref):
    n = 0
    for line in _rows("psr_worked.txt"):
        x, bp, mbits, want = map(int, line.split())
        assert oref.psr(x, bp, mbits) == want, line
        n += 1
    assert n >= 15


def test_bitwidth_is_bit_length_of_max_magnitude(oref):
    rng = np.random.default_rng(0)
    assert oref.bitwidth(np.zeros(5, np.int64)) == 0
    for v in [1, -1, 2, 3, 4, 127, 128, -128, 255, 256, 2**31 - 1, -(2**31)]:
        assert oref.bitwidth(np.array([0, v, 0])) == abs(v).bit_length()
    for _ in range(50):
        v = rng.integers(-2**31, 2**31, size=17)
        b = oref.bitwidth(v)
        mx = int(np.abs(v).max())
        assert b == mx.bit_length()
        assert 2 ** (b - 1) <= mx < 2 ** b


def test_identity_exact_and_bp1(oref):
    for x in range(-300, 301):
        # bp = 0: nothing is discarded
        assert oref.psr(x, 0, 15) == x
        # discarded bits all zero: exact division
        for bp in range(1, 9):
            assert oref.psr(x << bp, bp, 15) == x
        # bp = 1: both halves of the fraction are empty, so never rounds up
        m = abs(x) >> 1
        assert oref.psr(x, 1, 15) == (m if x >= 0 else -m)


def test_odd_symmetry_and_error_bound(oref):
    rng = np.random.default_rng(1)
    for _ in range(4000):
        bp = int(rng.integers(0, 25))
        x = int(rng.integers(-2**31 + 1, 2**31))
        q = oref.psr(x, bp, 31)
        assert oref.psr(-x, bp, 31) == -q
        assert abs(Fraction(q) - Fraction(x, 2 ** bp)) < 1
        # base is round-toward-zero of the magnitude plus an increment of 0 or 1
        assert abs(q) - (abs(x) >> bp) in (0, 1)


@pytest.mark.parametrize("bp", range(0, 15))
def test_round_up_counts_closed_form(oref, bp):
    """Over all 2^bp fractions exactly 2^h (2^h - 1) / 2 round up (twice that for odd bp,
    where the dropped bit doubles every case); given the top half T exactly T bottoms do."""
    h = bp // 2
    ups = 0
    per_top = {}
    for f in range(2 ** bp):
        up = oref.psr((5 << bp) | f, bp, 15) - 5
        assert up in (0, 1)
        ups += up
        ff = f >> 1 if bp % 2 else f
        per_top[ff >> h] = per_top.get(ff >> h, 0) + up
    want = (2 ** h) * (2 ** h - 1) // 2 * (2 if bp % 2 else 1)
    assert ups == want
    for T, c in per_top.items():
        assert c == T * (2 if bp % 2 else 1)


@pytest.mark.parametrize("bp", [2, 4, 6, 8, 10, 12])
def test_rounding_bias_statistics(oref, bp):
    """Uniform discarded bits: pseudo-stochastic bias is (1 - 2^h) / 2^(2h+1); true stochastic
    rounding (random r uniform over [0, 2^bp)) has exactly zero bias."""
    h = bp // 2
    tot = Fraction(0)
    for f in range(2 ** bp):
        tot += oref.psr((3 << bp) | f, bp, 15) - Fraction((3 << bp) | f, 2 ** bp)
    assert tot / 2 ** bp == Fraction(1 - 2 ** h, 2 ** (2 * h + 1))
    if bp <= 8:
        tot = Fraction(0)
        for f in range(2 ** bp):
            for r in range(2 ** bp):
                tot += oref.round_stochastic((3 << bp) | f, bp, 15, r) - Fraction((3 << bp) | f,
                                                                                   2 ** bp)
        assert tot == 0


def test_saturation(oref):
    # integer part already maximal and the fraction asks for an increment
    assert oref.psr(127 * 16 + 8, 4, 7) == 127
    assert oref.psr(-(127 * 16 + 8), 4, 7) == -127
    assert oref.psr(31 * 16 + 8, 4, 5) == 31
    assert oref.psr(7 * 64 + 0b101000, 6, 3) == 7
    assert oref.round_nearest(127 * 16 + 8, 4, 7) == 127
    # without saturation pressure the increment goes through
    assert oref.psr(126 * 16 + 8, 4, 7) == 127


def test_nearest(oref):
    for x in range(-1000, 1001):
        for bp in range(0, 6):
            want = pyref.nearest_bits(x, bp, 15)
            assert oref.round_nearest(x, bp, 15) == want
            # half away from zero on the magnitude
            assert abs(Fraction(want) - Fraction(x, 2 ** bp)) <= Fraction(1, 2)


def test_against_bit_string_transcription(oref):
    rng = np.random.default_rng(2)
    for _ in range(5000):
        bp = int(rng.integers(0, 25))
        mbits = int(rng.integers(1, 8))
        x = int(rng.integers(-2**31 + 1, 2**31))
        assert oref.psr(x, bp, mbits) == pyref.psr_bits(x, bp, mbits)


@pytest.mark.parametrize("mbits", [7, 5, 3, 1])
def test_shift_round_tensor(oref, mbits):
    rng = np.random.default_rng(3)
    for scale in [1, 50, 3000, 10**6, 2**30]:
        acc = rng.integers(-scale, scale + 1, size=(7, 13))
        q, b, bp = oref.shift_round(acc, mbits)
        q2, b2, bp2 = pyref.shift_round(acc, mbits)
        assert (b, bp) == (b2, bp2) == (int(np.abs(acc).max()).bit_length(),
                                        max(0, int(np.abs(acc).max()).bit_length() - mbits))
        assert np.array_equal(q.astype(np.int64), q2)
        # the shift makes full use of the mbits magnitude bits
        if b > mbits:
            assert 2 ** (mbits - 1) <= int(np.abs(q.astype(np.int64)).max()) <= 2 ** mbits - 1
        assert q.min() >= -(2 ** mbits - 1)
    assert oref.shift_round(np.zeros((2, 2), np.int64))[1:] == (0, 0)


def test_pseudo_random_half_is_near_uniform(oref):
    """The bottom half of the discarded bits of a real accumulator acts as the random number;
    on a synthetic GEMM its histogram is close to flat (Section 3.4, histogram figure)."""
    rng = np.random.default_rng(4)
    a = rng.integers(-127, 128, size=(64, 512), dtype=np.int8)
    w = rng.integers(-127, 128, size=(64, 512), dtype=np.int8)
    acc = oref.fc_fwd_acc(a, w)
    b = oref.bitwidth(acc)
    bp = b - 7
    assert bp >= 8
    h = bp // 2
    f = np.abs(acc) & (2 ** bp - 1)
    if bp % 2:
        f >>= 1
    bot = (f & (2 ** h - 1)) >> max(0, h - 3)         # 8 coarse bins
    hist = np.bincount(bot.reshape(-1), minlength=8)[:8]
    assert hist.min() > 0.8 * hist.mean() and hist.max() < 1.2 * hist.mean()
