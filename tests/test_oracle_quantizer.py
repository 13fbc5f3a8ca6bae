"""Pins for the oracle's quantizer (Eq. 2, Eq. 3, Appendix A), none of which re-use its formula."""
from fractions import Fraction

import numpy as np
import pytest

from conftest import to_bf16
from oracle import mixkvq_oracle as O


def _data(rng, n_groups, n, outliers=True):
    x = rng.standard_normal((n_groups, n))
    if outliers:
        x[:, 0] *= 25.0
        x[n_groups // 2:, 1] -= 40.0
    return to_bf16(x)


@pytest.mark.parametrize("bits", [2, 4])
def test_error_bound_half_scale(rng, bits):
    # Appendix A: |x - x~| <= s/2 for every element, with the scale that is actually stored
    x = _data(rng, 256, 32)
    c, s, z = O.quantize_groups(x, bits)
    err = np.abs(x.astype(np.float64) - O.dequantize(c, s, z))
    slack = np.spacing(np.abs(x).max(axis=-1).astype(np.float32)).astype(np.float64)
    assert np.all(err <= s.astype(np.float64)[:, None] / 2 + slack[:, None])
    assert O.is_bf16(s) and O.is_bf16(z)


@pytest.mark.parametrize("bits", [2, 4])
def test_extremes_hit_end_codes(rng, bits):
    # z = min(X), so the minimum gets code 0 and comes back exactly; the maximum gets 2^B - 1
    x = _data(rng, 128, 32)
    c, s, z = O.quantize_groups(x, bits)
    i_min, i_max = x.argmin(-1), x.argmax(-1)
    rows = np.arange(x.shape[0])
    assert np.all(c[rows, i_min] == 0)
    assert np.all(c[rows, i_max] == (1 << bits) - 1)
    assert np.all(O.dequantize(c, s, z)[rows, i_min] == x[rows, i_min])
    assert np.all(z == x.min(-1))
    assert c.max() <= (1 << bits) - 1


@pytest.mark.parametrize("bits", [2, 4])
def test_codes_match_exact_rational_rounding(rng, bits):
    # brute force: round-half-even of the exact rational (x - z)/s with the stored s
    x = _data(rng, 24, 32)
    c, s, z = O.quantize_groups(x, bits)
    near_tie = 0
    for g in range(x.shape[0]):
        sg, zg = Fraction(float(s[g])), Fraction(float(z[g]))
        for i in range(x.shape[1]):
            y = (Fraction(float(x[g, i])) - zg) / sg
            fl = y.numerator // y.denominator
            frac = y - fl
            if frac == Fraction(1, 2):
                expect = fl + (fl & 1)                  # exact tie: the even neighbour
            elif abs(frac - Fraction(1, 2)) < Fraction(1, 1 << 20):
                near_tie += 1                           # fp32 division may land on either side
                continue
            else:
                expect = fl + (1 if frac > Fraction(1, 2) else 0)
            expect = min(max(expect, 0), (1 << bits) - 1)
            assert int(c[g, i]) == expect
    assert near_tie <= 2


@pytest.mark.parametrize("bits", [2, 4])
def test_scale_is_range_over_levels_rounded_up_to_bf16(rng, bits):
    x = _data(rng, 64, 32)
    _, s, _ = O.quantize_groups(x, bits)
    for g in range(x.shape[0]):
        exact = (Fraction(float(x[g].max())) - Fraction(float(x[g].min()))) / ((1 << bits) - 1)
        stored = Fraction(float(s[g]))
        below = Fraction(float(np.uint32(np.float32(s[g]).view(np.uint32) - 0x10000).view(np.float32)))
        # stored scale is at least the exact quotient (up to the fp32 rounding of the quotient) ...
        assert stored >= exact * (1 - Fraction(1, 1 << 23))
        # ... and the next lower bf16 value would be too small
        assert below < exact * (1 + Fraction(1, 1 << 23))


def test_constant_group(rng):
    x = np.full((3, 32), to_bf16(np.array([1.75]))[0], np.float32)
    c, s, z = O.quantize_groups(x, 2)
    assert np.all(c == 0) and np.all(s == 0) and np.all(z == x[:, 0])
    assert np.all(O.dequantize(c, s, z) == x)


def test_two_level_group_is_lossless(rng):
    # a group that only takes the values {a, a + 3h} on a bf16 grid quantizes without error at 2 bits
    a, h = 0.5, 0.25
    x = np.where(rng.random((8, 32)) < 0.5, a, a + 3 * h).astype(np.float32)
    x[:, 0], x[:, 1] = a, a + 3 * h
    c, s, z = O.quantize_groups(x, 2)
    assert np.all(s == h) and set(np.unique(c)) == {0, 3}
    assert np.all(O.dequantize(c, s, z) == x)


def test_rounding_is_half_to_even():
    # x - z = 0.5 s and 1.5 s exactly: ties go to the even code (0 and 2)
    x = np.array([[0.0, 3.0, 0.5, 1.5, 2.5] + [0.0] * 27], np.float32)
    c, s, _ = O.quantize_groups(x, 2)
    assert s[0] == 1.0
    assert list(c[0, :5]) == [0, 3, 0, 2, 2]


def test_a_truncating_quantizer_would_break_the_bound(rng):
    # the bound is a real constraint: replacing round by floor violates it on the same data
    x = _data(rng, 64, 32)
    _, s, z = O.quantize_groups(x, 2)
    c_floor = np.floor((x - z[:, None]) / s[:, None]).clip(0, 3)
    err = np.abs(x - (c_floor * s[:, None] + z[:, None]))
    assert np.any(err > s[:, None] / 2 * 1.01)
