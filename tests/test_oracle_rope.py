"""Pins of the oracle's rotary embedding (Appendix D: scores and keys are taken after the rotation).

The oracle's `rope` is checked against what the mathematics fixes, not against itself: the identity at angle 0, the
quarter turn (which exposes a wrong sign or a wrong pairing of channels), preserved pair norms, the relative-position
property of the rotated dot product, a complex multiplication done by a library routine, and an exact rational
evaluation of the stated fp32 sequence with round-to-nearest-even on small inputs."""
from fractions import Fraction

import numpy as np
import torch

from conftest import to_bf16
from oracle import mixkvq_oracle as O

D, H = 128, 64


def tables(positions, base=10000.0):
    inv = base ** (-np.arange(H, dtype=np.float64) / H)
    ang = np.asarray(positions, np.float64)[:, None] * inv[None]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def test_angle_zero_is_the_identity(rng):
    x = to_bf16(rng.normal(size=(3, 5, D)))
    y = O.rope(x, np.ones((5, H), np.float32), np.zeros((5, H), np.float32))
    assert np.array_equal(y, x)


def test_quarter_turn_swaps_the_halves_with_one_sign(rng):
    x = to_bf16(rng.normal(size=(4, D)))
    y = O.rope(x, np.zeros((4, H), np.float32), np.ones((4, H), np.float32))
    assert np.array_equal(y[:, :H], -x[:, H:])         # y[i] = -x[i + D/2]
    assert np.array_equal(y[:, H:], x[:, :H])          # y[i + D/2] = x[i]


def test_pair_norms_are_preserved_up_to_the_bf16_rounding(rng):
    x = to_bf16(rng.normal(size=(64, D)) * 8.0)
    cos, sin = tables(np.arange(64) * 37)
    y = O.rope(x, cos, sin).astype(np.float64)
    xn = np.hypot(x[:, :H], x[:, H:]).astype(np.float64)
    yn = np.hypot(y[:, :H], y[:, H:])
    assert np.all(np.abs(yn - xn) <= 2.0 ** -7 * xn + 1e-30)


def test_rotated_dot_product_depends_on_the_distance_only(rng):
    q = to_bf16(rng.normal(size=(1, D)))
    k = to_bf16(rng.normal(size=(1, D)))
    dots = []
    for m, n in [(5, 2), (105, 102), (4003, 4000)]:
        cq, sq = tables([m])
        ck, sk = tables([n])
        dots.append(float((O.rope(q, cq, sq).astype(np.float64) @ O.rope(k, ck, sk).astype(np.float64).T)[0, 0]))
    scale = float((np.abs(q).astype(np.float64) @ np.abs(k).astype(np.float64).T)[0, 0])
    assert max(dots) - min(dots) <= 3 * 2.0 ** -8 * scale


def test_equals_a_complex_multiplication_by_a_library_routine(rng):
    x = to_bf16(rng.normal(size=(2, 9, D)) * 3.0)
    pos = np.arange(9) * 11 + 3
    cos, sin = tables(pos)
    inv = 10000.0 ** (-np.arange(H, dtype=np.float64) / H)
    ang = torch.from_numpy(pos[:, None] * inv[None])
    z = torch.complex(torch.from_numpy(x[..., :H].astype(np.float64)), torch.from_numpy(x[..., H:].astype(np.float64)))
    w = z * torch.polar(torch.ones_like(ang), ang)
    want = np.concatenate([w.real.numpy(), w.imag.numpy()], axis=-1)
    got = O.rope(x, cos, sin).astype(np.float64)
    # the table is rounded to fp32 and the result to bf16
    assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 2.0 ** -20 * np.abs(x).max())


def rne_to_bf16(fr: Fraction) -> Fraction:
    """Nearest bf16 (8 significant bits, ties to even) of a rational, exponent range not an issue here."""
    if fr == 0:
        return fr
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = 0
    while a >= 2:
        a /= 2; e += 1
    while a < 1:
        a *= 2; e -= 1
    scaled = a * 128                                # in [128, 256)
    lo = scaled.numerator // scaled.denominator
    rem = scaled - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * Fraction(lo, 128) * (Fraction(2) ** e)


def test_exact_rational_evaluation_of_the_stated_sequence():
    # dyadic inputs and table entries: every fp32 product and sum below is exact, so the only rounding is the last one
    xs = [Fraction(n, 64) for n in (-75, -3, 17, 96, 127, 201)]
    cs = [Fraction(n, 256) for n in (0, 77, 181, 256, -181)]
    ss = [Fraction(n, 256) for n in (256, 244, 181, 0, 181)]
    for x1 in xs:
        for x2 in xs[::2]:
            for c, s in zip(cs, ss):
                x = np.zeros((1, D), np.float32)
                x[0, 0], x[0, H] = float(x1), float(x2)
                cos = np.ones((1, H), np.float32); sin = np.zeros((1, H), np.float32)
                cos[0, 0], sin[0, 0] = float(c), float(s)
                y = O.rope(x, cos, sin)
                assert Fraction(float(y[0, 0])) == rne_to_bf16(x1 * c - x2 * s)
                assert Fraction(float(y[0, H])) == rne_to_bf16(x2 * c + x1 * s)


def test_intermediate_products_are_rounded_to_fp32_before_the_sum():
    # x1 c and x2 s each need more than 24 bits together: the two-step fp32 sequence differs from a fused or fp64 one
    x = np.zeros((1, D), np.float32)
    x[0, 0], x[0, H] = 1.0078125, 0.0078125            # bf16 values
    cos = np.ones((1, H), np.float32); sin = np.zeros((1, H), np.float32)
    cos[0, 0] = np.float32(1.0 + 2.0 ** -23); sin[0, 0] = np.float32(1.0 + 2.0 ** -23)
    a = np.float32(np.float32(x[0, 0]) * cos[0, 0]); b = np.float32(np.float32(x[0, H]) * sin[0, 0])
    want = O.bf16_rne(np.float32(a - b))
    assert O.rope(x, cos, sin)[0, 0] == want
    assert O.is_bf16(O.rope(x, cos, sin))
