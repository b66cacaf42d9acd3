"""Pins for the oracle's bfloat16 rounding (mixed-precision mode: the working
parameter is the master rounded to nearest, ties to even).

The expected value comes from the *definition* (the nearest representable
value, ties to the even significand) evaluated in exact arithmetic, and from a
library routine (torch's CPU conversion), not from the bit manipulation the
oracle uses.
"""
from fractions import Fraction

import numpy as np
import torch

import oracle


def _bf16_value(h: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns, as float64."""
    return (h.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _nearest_even_by_definition(f32: np.ndarray, lo_bits: np.ndarray) -> np.ndarray:
    """f lies in [V(lo), V(lo+1)]; pick the nearer value, ties -> even pattern.
    Differences of two binary32 numbers one bf16 step apart are exact in binary64."""
    f = f32.astype(np.float64)
    lo, hi = _bf16_value(lo_bits), _bf16_value(lo_bits + 1)
    d_lo, d_hi = np.abs(f - lo), np.abs(hi - f)
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & ((lo_bits & 1) == 1))
    return np.where(pick_hi, lo_bits + 1, lo_bits).astype(np.uint16)


def test_f32_to_bf16_exhaustive_over_all_patterns_and_half_ulp_neighbours():
    # all positive finite bf16 patterns whose successor is still finite
    h = np.arange(0, 0x7F7F, dtype=np.uint32)
    base = h << np.uint32(16)
    offsets = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0xFFFF], dtype=np.uint32)
    bits = (base[:, None] + offsets[None, :]).reshape(-1)
    lo = np.repeat(h, len(offsets))
    f = bits.view(np.float32)
    want = _nearest_even_by_definition(f, lo)
    got = np.fromiter((oracle.bf16_from_f32(v) for v in f), dtype=np.uint16, count=f.size)
    assert np.array_equal(got, want)
    # library routine on the same inputs
    lib = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, lib)
    # negative half: sign symmetry
    sub = slice(0, f.size, 37)
    got_neg = np.fromiter((oracle.bf16_from_f32(-v) for v in f[sub]), dtype=np.uint16)
    assert np.array_equal(got_neg, want[sub] | 0x8000)


def test_f32_to_bf16_overflow_inf_and_nan():
    big = np.array([0x7F7FFFFF], dtype=np.uint32).view(np.float32)[0]   # max binary32
    assert oracle.bf16_from_f32(big) == 0x7F80                          # rounds to +inf
    assert oracle.bf16_from_f32(float("inf")) == 0x7F80
    assert oracle.bf16_from_f32(float("-inf")) == 0xFF80
    n = oracle.bf16_from_f32(float("nan"))
    assert (n & 0x7F80) == 0x7F80 and (n & 0x007F) != 0
    assert oracle.bf16_from_f32(0.0) == 0 and oracle.bf16_from_f32(-0.0) == 0x8000


def test_bf16_to_f32_is_exact_widening():
    for h in list(range(0, 0x7F80, 97)) + [0x7F7F, 0x0001, 0x8001]:
        got = np.float32(oracle.bf16_to_f32(h))
        assert got.view(np.uint32) == np.uint32(h << 16)


def _exact_nearest_bf16(d: float) -> int:
    """Definition in rationals: search the two neighbouring patterns."""
    a = Fraction(abs(d))
    sign = 0x8000 if d < 0 else 0
    # bisect over positive finite patterns (values increase with the pattern)
    lo, hi = 0, 0x7F7F
    val = lambda h: Fraction(float(_bf16_value(np.array([h], dtype=np.uint32))[0]))
    if a >= val(hi):
        top = val(hi) + (val(hi) - val(hi - 1)) / 2
        return sign | (0x7F80 if a >= top else hi)
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if val(mid) <= a:
            lo = mid
        else:
            hi = mid
    d_lo, d_hi = a - val(lo), val(hi) - a
    if d_hi < d_lo or (d_hi == d_lo and (lo & 1)):
        return sign | hi
    return sign | lo


def test_f64_to_bf16_single_rounding_near_midpoints():
    rng = np.random.default_rng(3)
    pats = np.concatenate([rng.integers(1, 0x7F7E, size=300), [1, 2, 0x007F, 0x0080, 0x0081, 0x3F80]])
    for h in pats:
        lo = float(_bf16_value(np.array([h], dtype=np.uint32))[0])
        hi = float(_bf16_value(np.array([h + 1], dtype=np.uint32))[0])
        mid = (lo + hi) / 2                      # exact in binary64
        for d in (lo, mid, np.nextafter(mid, np.inf), np.nextafter(mid, -np.inf),
                  np.nextafter(lo, np.inf), np.nextafter(hi, -np.inf),
                  lo + (hi - lo) * 0.3, -mid, -np.nextafter(mid, np.inf)):
            d = float(d)
            assert oracle.bf16_from_f64(d) == _exact_nearest_bf16(d), (hex(int(h)), d)


def test_f64_path_agrees_with_f32_path_on_binary32_inputs():
    rng = np.random.default_rng(5)
    f = (rng.standard_normal(20000) * 0.02).astype(np.float32)
    for v in f[:4000]:
        assert oracle.bf16_from_f64(float(v)) == oracle.bf16_from_f32(float(v))
