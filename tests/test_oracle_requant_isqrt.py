"""Pins for the oracle's requantization (Appendix C.1) and I-Sqrt (Algorithm 4)."""
import math
import random
from fractions import Fraction

import pytest

import oracle


def _exact_round_half_up(num: int, c: int) -> int:
    return math.floor(Fraction(num, 2 ** c) + Fraction(1, 2))


def test_round_shift_equals_exact_rational_rounding():
    rnd = random.Random(1)
    for _ in range(20000):
        c = rnd.randint(0, 31)
        q = rnd.randint(-2 ** 31, 2 ** 31 - 1)
        b = rnd.randint(-2 ** 31 + 1, 2 ** 31 - 1)
        assert oracle.round_shift(q * b, c) == _exact_round_half_up(q * b, c)


def test_requant_clamps_symmetrically_and_rounds_half_up():
    rnd = random.Random(2)
    for _ in range(5000):
        c = rnd.randint(0, 31)
        q = rnd.randint(-2 ** 27, 2 ** 27)
        b = rnd.randint(-2 ** 31 + 1, 2 ** 31 - 1)
        for qmax in (127, 32767):
            want = max(-qmax, min(qmax, _exact_round_half_up(q * b, c)))
            assert oracle.requant(q, b, c, qmax) == want
    # half-way cases go up: 1.5 -> 2, -1.5 -> -1, 0.5 -> 1, -0.5 -> 0
    assert [oracle.requant(v, 2 ** 30, 31, 127) for v in (3, -3, 1, -1)] == [2, -1, 1, 0]
    assert oracle.requant(10 ** 7, 1932735, 31, 127) == 127
    assert oracle.requant(-10 ** 7, 1932735, 31, 127) == -127


def test_dyadic_is_the_nearest_31_bit_multiplier():
    rnd = random.Random(3)
    for _ in range(5000):
        m = math.ldexp(rnd.uniform(0.5, 1.0), rnd.randint(-40, 30)) * rnd.choice((-1, 1))
        b, c = oracle.dyadic(m)
        assert 0 <= c <= 31 and abs(b) < 2 ** 31
        # |b / 2^c - m| <= 2^-(c+1): b is the nearest integer to m * 2^c
        assert abs(Fraction(b, 2 ** c) - Fraction(m)) <= Fraction(1, 2 ** (c + 1))
        if abs(m) >= 2.0 ** -1:      # c not capped: full 31-bit mantissa
            assert 2 ** 30 <= abs(b)
        assert (b < 0) == (m < 0) or b == 0
    assert oracle.dyadic(0.0) == (0, 0)
    assert oracle.dyadic(1.0) == (2 ** 30, 30)
    assert oracle.dyadic(0.5) == (2 ** 30, 31)
    assert oracle.dyadic(2.0 ** 30) == (2 ** 30, 0)
    assert oracle.dyadic(258.0) == (258 * 2 ** 22, 22)
    with pytest.raises(oracle.OracleError):
        oracle.dyadic(2.0 ** 31)
    with pytest.raises(oracle.OracleError):
        oracle.dyadic(float("nan"))


def test_isqrt_exact_for_all_n_below_2_20():
    for n in range(2 ** 20):
        r, _ = oracle.isqrt(n)
        assert r == math.isqrt(n), n


def test_isqrt_exact_on_random_wide_inputs_and_edges():
    rnd = random.Random(4)
    for bits in range(1, 63):
        for _ in range(300):
            n = rnd.randint(2 ** (bits - 1), 2 ** bits - 1)
            assert oracle.isqrt(n)[0] == math.isqrt(n)
    for k in range(1, 31):
        for n in (k * k - 1, k * k, k * k + 1, (2 ** k) ** 2 - 1, (2 ** k) ** 2, (2 ** k + 1) ** 2 - 1):
            assert oracle.isqrt(n)[0] == math.isqrt(n)
    assert oracle.isqrt(0) == (0, 0)


def test_isqrt_division_count_is_two_to_six_for_32_bit_inputs():
    # Sec. 3.6 says "at most four iterations" for INT32 inputs; counting the
    # terminating division the repeat-until loop of Algorithm 4 does 2..6.
    rnd = random.Random(5)
    seen = set()
    for _ in range(200000):
        n = rnd.randint(1, 2 ** 32 - 1)
        seen.add(oracle.isqrt(n)[1])
    assert oracle.isqrt(16785408) == (4096, 6)
    seen.add(6)
    assert min(seen) >= 2 and max(seen) <= 6
