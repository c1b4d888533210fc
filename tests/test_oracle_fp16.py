"""Pins for the checker's binary16 conversions against numpy's independent implementation
and hand-derived ties."""
import numpy as np

from oracle import executor as orc


def test_all_half_patterns_widen_like_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    got = orc.half_to_float(bits)
    want = bits.view(np.float16).astype(np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_all_half_patterns_round_trip():
    bits = np.arange(65536, dtype=np.uint16)
    f = bits.view(np.float16).astype(np.float32)
    keep = ~np.isnan(f)
    back = orc.float_to_half(f)
    assert np.array_equal(back[keep], bits[keep])
    assert np.all((back[~keep] & 0x7C00) == 0x7C00) and np.all((back[~keep] & 0x3FF) != 0)


def test_hand_checked_ties_and_limits():
    cases = [
        (1.0 + 2.0 ** -11, 1.0),                    # tie, even mantissa below
        (1.0 + 3.0 * 2.0 ** -11, 1.0 + 2.0 ** -9),  # tie, odd mantissa below -> up
        (1.0 + 2.0 ** -11 + 2.0 ** -20, 1.0 + 2.0 ** -10),
        (65504.0, 65504.0), (65519.0, 65504.0), (65520.0, np.inf), (1e9, np.inf),
        (2.0 ** -24, 2.0 ** -24), (2.0 ** -25, 0.0), (2.0 ** -25 * 1.0001, 2.0 ** -24),
        (3.0 * 2.0 ** -25, 2.0 ** -23),             # 1.5 subnormal steps: tie -> even (2)
        (2.0 ** -14 - 2.0 ** -26, 2.0 ** -14),      # rounds up into the normal range
        (-0.0, -0.0), (-2.5, -2.5), (-np.inf, -np.inf),
    ]
    vals = np.array([c[0] for c in cases], dtype=np.float32)
    want = np.array([c[1] for c in cases], dtype=np.float16)
    got = orc.float_to_half(vals)
    assert np.array_equal(got, want.view(np.uint16)), (got, want.view(np.uint16))


def test_random_floats_round_like_numpy():
    rng = np.random.default_rng(5)
    raw = rng.integers(0, 2 ** 32, size=400000, dtype=np.uint64).astype(np.uint32)
    f = raw.view(np.float32)
    f = f[np.isfinite(f)]
    scaled = np.concatenate([f, (rng.standard_normal(200000) * 10.0 ** rng.uniform(-9, 5, 200000))
                             .astype(np.float32)])
    with np.errstate(over="ignore"):
        want = scaled.astype(np.float16).view(np.uint16)
    assert np.array_equal(orc.float_to_half(scaled), want)
