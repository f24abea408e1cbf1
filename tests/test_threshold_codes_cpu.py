"""The overflow kernels take a 2-bit code as [d > s/2] + [d >= 3s/2] + [d > 5s/2] for d = x - min >= 0 and a bf16
scale s > 0, instead of rounding the quotient d / s (Eq. 1 with the rounding of the quantiser: nearest, ties to even,
clamped at 3).  This checks that identity in IEEE binary32 for EVERY positive finite bf16 scale, at the three
thresholds themselves and at the binary32 neighbours on either side (where the two could differ if they ever
did), and on random d; numpy's float32 division is the correctly rounded one the definition uses."""
import numpy as np
import pytest

pytestmark = pytest.mark.filterwarnings("ignore::RuntimeWarning")  # overflow of 4 * s at the largest scales, filtered out


def _by_division(d, s):
    with np.errstate(over="ignore", invalid="ignore"):
        q = (d / s).astype(np.float32)
    return np.clip(np.rint(q), 0, 3).astype(np.int64)   # np.rint: ties to even


def _by_thresholds(d, s):
    h = np.float32(0.5)
    t1, t2, t3 = h * s, np.float32(1.5) * s, np.float32(2.5) * s
    return (d > t1).astype(np.int64) + (d >= t2).astype(np.int64) + (d > t3).astype(np.int64)


def _all_positive_bf16():
    bits = np.arange(1, 0x7F80, dtype=np.uint32) << 16      # subnormals included, inf and NaN excluded
    return bits.view(np.float32)


def test_threshold_products_are_exact():
    s = _all_positive_bf16().astype(np.float64)
    for c in (0.5, 1.5, 2.5):
        prod = c * s
        ok = np.isfinite(prod.astype(np.float32))
        assert (prod.astype(np.float32).astype(np.float64)[ok] == prod[ok]).all()


def test_codes_by_thresholds_equal_codes_by_rounded_division_near_every_threshold():
    s = _all_positive_bf16()
    s = s[np.isfinite(np.float32(2.5) * s) & np.isfinite(np.float32(4) * s)]
    for c in (0.5, 1.5, 2.5):
        t = np.float32(c) * s
        d = t.copy()
        lo, hi = t.copy(), t.copy()
        cases = [d]
        for _ in range(3):                                   # three binary32 steps to either side
            lo = np.nextafter(lo, np.float32(0))
            hi = np.nextafter(hi, np.float32(np.inf))
            cases += [lo.copy(), hi.copy()]
        for dd in cases:
            assert np.array_equal(_by_thresholds(dd, s), _by_division(dd, s)), c
    # ties go to the even neighbour
    assert _by_thresholds(np.float32([0.5, 1.5, 2.5]), np.float32([1, 1, 1])).tolist() == [0, 2, 2]


def test_codes_by_thresholds_equal_codes_by_rounded_division_on_random_inputs():
    rng = np.random.default_rng(7)
    s = rng.choice(_all_positive_bf16(), size=2_000_000)
    s = s[np.isfinite(np.float32(4) * s)]
    d = (rng.random(len(s)) * 3.2).astype(np.float32) * s    # quotients in [0, 3.2): beyond 3 the clamp applies
    assert np.array_equal(_by_thresholds(d, s), _by_division(d, s))
    # differences of bf16 values, as the kernel forms them (x - min rounded to binary32)
    x = (rng.integers(0, 0x7F80, size=len(s)).astype(np.uint32) << 16).view(np.float32)
    mn = (rng.integers(0, 0x7F80, size=len(s)).astype(np.uint32) << 16).view(np.float32)
    x, mn = np.maximum(x, mn), np.minimum(x, mn)
    with np.errstate(over="ignore", invalid="ignore"):
        d = (x - mn).astype(np.float32)
        sc = ((d / np.float32(3)).astype(np.float32).view(np.uint32) >> 16 << 16).view(np.float32)  # some scale near d/3
    keep = (sc > 0) & np.isfinite(np.float32(4) * sc)
    for dd in (d[keep], (d[keep] * np.float32(0.5)).astype(np.float32), (d[keep] * np.float32(0.83)).astype(np.float32)):
        assert np.array_equal(_by_thresholds(dd, sc[keep]), _by_division(dd, sc[keep]))
