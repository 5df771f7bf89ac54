"""Pins for the oracle's fixed-point primitives: exact rational arithmetic, brute force, invariants."""
import math
import random
from fractions import Fraction

import numpy as np
import pytest

from oracle import qlstm_ref as R

I32_MIN, I32_MAX = -(1 << 31), (1 << 31) - 1


def round_half_away(v: Fraction) -> int:
    return math.floor(v + Fraction(1, 2)) if v >= 0 else -math.floor(-v + Fraction(1, 2))


def seeded_scales(n=12, seed=7):
    rng = random.Random(seed)
    out = [((1 << 30), 1), ((1 << 31) - 1, 0), ((1 << 30), -31), ((1 << 30), 0)]
    while len(out) < n:
        out.append((rng.randrange(1 << 30, 1 << 31), rng.randrange(-20, 4)))
    return out


def test_srdhm_matches_exact_rounding():
    rng = random.Random(1)
    edge = [0, 1, -1, 2, -2, I32_MAX, I32_MIN, I32_MIN + 1, 1 << 30, -(1 << 30), (1 << 30) + 1, 12345, -54321]
    pairs = [(a, b) for a in edge for b in edge]
    pairs += [(rng.randrange(I32_MIN, I32_MAX + 1), rng.randrange(I32_MIN, I32_MAX + 1)) for _ in range(20000)]
    for a, b in pairs:
        want = round_half_away(Fraction(a * b, 1 << 31))
        want = min(want, I32_MAX)          # only a = b = -2^31 reaches 2^31
        assert R.srdhm(a, b) == want, (a, b)


def test_srdhm_ties_go_away_from_zero():
    # a * b = +-2^30 exactly halfway between 0 and +-1
    assert R.srdhm(1 << 15, 1 << 15) == 1
    assert R.srdhm(-(1 << 15), 1 << 15) == -1
    assert R.srdhm(3 << 15, 1 << 15) == 2       # 1.5 -> 2
    assert R.srdhm(-(3 << 15), 1 << 15) == -2


def test_rdivpot_matches_exact_rounding():
    rng = random.Random(2)
    for _ in range(20000):
        x = rng.randrange(-(1 << 55), 1 << 55)
        e = rng.randrange(0, 50)
        assert R.rdivpot(x, e) == round_half_away(Fraction(x, 1 << e))
    assert R.rdivpot(5, 1) == 3 and R.rdivpot(-5, 1) == -3 and R.rdivpot(7, 0) == 7
    assert R.rdivpot(1 << 30, 40) == 0 and R.rdivpot(3, 1) == 2 and R.rdivpot(-3, 1) == -2


def test_rdiv_and_isqrt_brute_force():
    rng = random.Random(3)
    for _ in range(20000):
        n = rng.randrange(-(1 << 62), 1 << 62)
        d = rng.randrange(1, 1 << rng.randrange(1, 40))
        assert R.rdiv(n, d) == round_half_away(Fraction(n, d))
    assert R.rdiv(5, 2) == 3 and R.rdiv(-5, 2) == -3 and R.rdiv(7, 3) == 2 and R.rdiv(-8, 3) == -3
    for v in list(range(0, 5000)) + [rng.randrange(0, 1 << 63) for _ in range(20000)] + [(1 << 63) - 1, (1 << 64) - 1]:
        assert R.isqrt(v) == math.isqrt(v)
    for r in [1, 2, 3, 65535, 65536, (1 << 31) - 1, (1 << 32) - 1]:
        assert R.isqrt(r * r) == r and R.isqrt(r * r - 1) == r - 1 and R.isqrt(r * r + 2 * r) == r


@pytest.mark.parametrize("scale", seeded_scales())
def test_mbqm_exhaustive_int16_against_rational(scale):
    M, s = scale
    real = Fraction(M, 1 << 31) * (Fraction(1 << s) if s >= 0 else Fraction(1, 1 << -s))
    right = max(-s, 0)
    bound = Fraction(1, 2) + Fraction(1, 1 << (right + 1))
    prev = None
    for x in range(-32768, 32768):
        got = R.mbqm(x, scale)
        exact = real * x
        if I32_MIN < exact < I32_MAX and abs(x << max(s, 0)) < (1 << 31):
            assert abs(got - exact) <= bound, (x, scale)
            if x != -32768:
                assert R.mbqm(-x, scale) == -got          # odd away from saturation
        if prev is not None:
            assert got >= prev                            # monotone
        prev = got


def test_mbqm_random_int32_against_rational():
    rng = random.Random(4)
    for scale in seeded_scales(8, seed=9):
        M, s = scale
        real = Fraction(M, 1 << 31) * (Fraction(1 << s) if s >= 0 else Fraction(1, 1 << -s))
        right = max(-s, 0)
        bound = Fraction(1, 2) + Fraction(1, 1 << (right + 1))
        for _ in range(4000):
            x = rng.randrange(I32_MIN, I32_MAX + 1)
            if abs(x << max(s, 0)) >= (1 << 31):
                continue
            assert abs(R.mbqm(x, scale) - real * x) <= bound


def test_mbqm_identity_zero_and_two_step_definition():
    for x in [0, 1, -1, 77, -32768, 32767, (1 << 30) - 1, -(1 << 30)]:
        assert R.mbqm(x, (1 << 30, 1)) == x               # 0.5 * 2 = 1, while 2x still fits int32
        assert R.mbqm(x, (0, 0)) == 0
    # the rescale is two roundings, not one: x = 3, scale = 0.5 * 2^-1 -> round(round(1.5) / 2) = round(2 / 2) = 1
    # while a single rounding of 0.75 would also give 1; x = 5: round(round(2.5) / 2) = round(3 / 2) = 2, single: 1.25 -> 1
    assert R.mbqm(5, (1 << 30, -1)) == 2
    assert R.mbqm(-5, (1 << 30, -1)) == -2


def test_mbqm_left_shift_saturates():
    assert R.mbqm(1 << 29, (1 << 30, 4)) == R.srdhm(I32_MAX, 1 << 30)
    assert R.mbqm(-(1 << 29), (1 << 30, 4)) == R.srdhm(I32_MIN, 1 << 30)


def test_accumulator_overflow_model():
    """Section 3.1.1: 2^15 products of int8 operands fit an int32 accumulator, 2^7 fit 24 bits."""
    from tests.util import paper_values
    pv = paper_values()
    k32, k24 = int(pv["int32_safe_accumulations"]), int(pv["int24_safe_accumulations"])
    worst = 128 * 128
    assert k32 * worst < (1 << 31)
    assert k24 * worst < (1 << 23)
    # with the zero point subtracted inside the matmul the operand grows to 255; still inside int32 at K = 2^15
    assert 127 * 255 * k32 < (1 << 31)
