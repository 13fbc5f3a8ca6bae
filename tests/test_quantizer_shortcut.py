"""The flush kernel's quantizer shortcut, restated in numpy float32: codes from (x - z) * RN(1 / s), with the IEEE division
only within 1e-4 of a half-integer, equal round-half-even of the IEEE quotient (x - z) / s for every input tried:
random bf16 data over many scales, and inputs placed on and next to the rounding ties."""
import numpy as np


def bf16(x):
    """Round float32 values to bf16 (round-half-even), returned as float32."""
    u = np.asarray(x, np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def exact_codes(t, s, max_code):
    y = (t / s).astype(np.float32)                      # IEEE fp32 division
    return np.clip(np.rint(y), 0, max_code).astype(np.int64)


def shortcut_codes(t, s, max_code):
    r = (np.float32(1.0) / s).astype(np.float32)        # RN(1 / s)
    y = (t * r).astype(np.float32)
    frac = y - np.floor(y)
    near = np.abs(frac - np.float32(0.5)) < np.float32(1e-4)
    fast = np.clip(np.rint(y), 0, max_code).astype(np.int64)
    return np.where(near, exact_codes(t, s, max_code), fast), near


def test_random_groups_over_many_scales():
    rng = np.random.default_rng(7)
    for max_code in (3, 15):
        # scales: every bf16 value of a few binades, and random ones over a wide range
        mant = np.arange(128, 256, dtype=np.float32) / 128.0
        scales = np.concatenate([mant * np.float32(2.0 ** e) for e in (-12, -5, -1, 0, 1, 7)])
        scales = np.concatenate([scales, bf16(np.exp(rng.uniform(-9, 9, 4000)).astype(np.float32))])
        s = np.repeat(scales, 512)
        z = bf16(rng.normal(0, 4, s.size).astype(np.float32) * s)
        x = bf16(z + rng.uniform(0, max_code, s.size).astype(np.float32) * s)
        t = (x - z).astype(np.float32)                  # one fp32 subtraction, as in the kernel
        got, near = shortcut_codes(t, s, max_code)
        assert np.array_equal(got, exact_codes(t, s, max_code))
        assert near.mean() < 0.05                       # the division is the rare path


def test_on_and_beside_the_ties():
    rng = np.random.default_rng(11)
    scales = bf16(np.exp(rng.uniform(-6, 6, 20000)).astype(np.float32))
    for max_code in (3, 15):
        for k in range(max_code):
            tie = ((k + 0.5) * scales.astype(np.float64)).astype(np.float32)
            for ulps in (-3, -2, -1, 0, 1, 2, 3):
                t = (tie.view(np.int32) + ulps).view(np.float32)
                got, _ = shortcut_codes(t, scales, max_code)
                assert np.array_equal(got, exact_codes(t, scales, max_code)), (max_code, k, ulps)
