"""Pins for the oracle's bf16 conversions: round-to-nearest-even worked by hand from the format.

bf16 keeps the top 16 bits of a float32 (8-bit exponent, 7 stored mantissa bits). A float32 whose
low 16 bits are exactly 0x8000 lies half way between two bf16 values and must go to the one whose
last mantissa bit is 0; anything above the half-way point goes up, anything below goes down.
Every expected value here is written out as an exact sum of powers of two, not computed by the
function under test.
"""
import numpy as np

from oracle import bf16_to_f32, f32_to_bf16


def _rt(x):
    return float(bf16_to_f32(f32_to_bf16(np.array([x], dtype=np.float32)))[0])


def test_exact_ties_go_to_the_even_neighbour():
    u = 2.0 ** -7                      # spacing of bf16 values in [1, 2)
    # 1 + u/2 lies between 1 (mantissa 0, even) and 1 + u (mantissa 1, odd) -> 1
    assert _rt(1 + 2.0 ** -8) == 1.0
    # 1 + 3u/2 lies between 1 + u (odd) and 1 + 2u (even) -> 1 + 2u = 1 + 2^-6
    assert _rt(1 + 3 * 2.0 ** -8) == 1 + 2.0 ** -6
    # 1 + 5u/2: between 1 + 2u (even) and 1 + 3u (odd) -> 1 + 2u
    assert _rt(1 + 5 * 2.0 ** -8) == 1 + 2.0 ** -6
    # negative twins: rounding is symmetric in the sign
    assert _rt(-(1 + 2.0 ** -8)) == -1.0
    assert _rt(-(1 + 3 * 2.0 ** -8)) == -(1 + 2.0 ** -6)


def test_near_ties_go_to_the_nearest_neighbour():
    # just above the half-way point -> up (round-half-down or truncation would give 1)
    assert _rt(1 + 2.0 ** -8 + 2.0 ** -20) == 1 + 2.0 ** -7
    # just below the half-way point -> down (round-half-up on a biased add would still give 1)
    assert _rt(1 + 2.0 ** -8 - 2.0 ** -20) == 1.0
    # just below the upper tie of an odd value -> stays odd (1 + u), not the even 1 + 2u
    assert _rt(1 + 3 * 2.0 ** -8 - 2.0 ** -20) == 1 + 2.0 ** -7
    assert _rt(-(1 + 2.0 ** -8 + 2.0 ** -20)) == -(1 + 2.0 ** -7)


def test_tie_that_carries_into_the_exponent():
    # largest bf16 below 2 is 2 - 2^-7 (mantissa 0x7F, odd); half way to 2 is 2 - 2^-8 -> 2 (even)
    assert _rt(2 - 2.0 ** -8) == 2.0
    # and the tie below it, between 2 - 2^-6 (even mantissa 0x7E) and 2 - 2^-7 (odd) -> 2 - 2^-6
    assert _rt(2 - 3 * 2.0 ** -8) == 2 - 2.0 ** -6


def test_bit_patterns_of_hand_encoded_values():
    # 1.0 = 0x3F80, -2.0 = 0xC000, 0.15625 = 1.25 * 2^-3 -> exponent 124 (0x7C), mantissa 0x20
    x = np.array([1.0, -2.0, 0.15625, 0.0, -0.0], dtype=np.float32)
    assert f32_to_bf16(x).tolist() == [0x3F80, 0xC000, 0x3E20, 0x0000, 0x8000]
    assert bf16_to_f32(np.array([0x3F80, 0xC000, 0x3E20], dtype=np.uint16)).tolist() == [1.0, -2.0, 0.15625]


def test_every_bf16_value_round_trips_and_every_tie_is_even():
    # all finite positive bf16 patterns: widening then narrowing is the identity, and the exact
    # mid-point between neighbours b and b + 1 rounds to whichever of the two has an even pattern
    b = np.arange(0x0080, 0x7F7F, dtype=np.uint32)            # normal, finite, with a finite successor
    assert np.array_equal(f32_to_bf16(bf16_to_f32(b.astype(np.uint16))), b.astype(np.uint16))
    mid = ((b << np.uint32(16)) | np.uint32(0x8000)).view(np.float32)
    expect = np.where(b % 2 == 0, b, b + 1).astype(np.uint16)
    assert np.array_equal(f32_to_bf16(mid), expect)
