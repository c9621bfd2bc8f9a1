"""Pins of the E4M3 conversions and of quantisation-after-pruning (CPU only).

The format's constants are worked by hand from its definition (1-4-3 bits, bias 7, no infinities,
subnormals m * 2^-9, largest finite value 448 = 1.75 * 2^8); nearest-value rounding is checked by
brute force with exact rational arithmetic that shares no code with the oracle's search.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import fp8
from oracle.bf16 import f32_to_bf16, bf16_to_f32
from oracle.prune24 import prune24


def test_decode_hand_values():
    hand = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x39: 1.125, 0x3C: 1.5,
            0x40: 2.0, 0x7E: 448.0, 0x77: 240.0, 0xB8: -1.0, 0xFE: -448.0, 0x30: 0.5}
    for code, val in hand.items():
        assert float(fp8.e4m3_to_f32(np.uint8(code))) == val, hex(code)
    assert np.isnan(fp8.e4m3_to_f32(np.uint8(0x7F))) and np.isnan(fp8.e4m3_to_f32(np.uint8(0xFF)))
    v = fp8.e4m3_to_f32(np.arange(0x7F, dtype=np.uint8))
    assert np.all(np.diff(v) > 0)                                    # codes order like their values
    assert np.isfinite(fp8.e4m3_to_f32(np.arange(256, dtype=np.uint8))).sum() == 254


def test_encode_hand_cases():
    cases = [(1.0, 0x38), (-1.0, 0xB8), (448.0, 0x7E), (449.0, 0x7E), (1e9, 0x7E), (-1e9, 0xFE), (np.inf, 0x7E),
             (464.0, 0x7E),                       # would be the tie towards the NaN slot: clamped
             (1.0625, 0x38),                      # tie between 1.0 (code even) and 1.125 -> even
             (1.1875, 0x3A),                      # tie between 1.125 (0x39) and 1.25 (0x3A) -> even
             (1.0626, 0x39), (1.18749, 0x39),
             (2.0 ** -10, 0x00),                  # half the smallest subnormal: tie -> code 0
             (3 * 2.0 ** -10, 0x02),              # tie between codes 1 and 2 -> 2
             (2.0 ** -10 * 1.001, 0x01), (0.0, 0x00), (-0.0, 0x80), (-2.0 ** -11, 0x80),
             (2.0 ** -6 - 2.0 ** -10, 0x08),      # tie between the largest subnormal (0x07) and 2^-6 (0x08) -> even
             (15.5, 0x58),                        # tie between 15 (1.875 * 2^3 = 0x57) and 16 (0x58): carries into the exponent
             (0.3, 0x2A)]                         # 0.3 in [0.28125 (0x29), 0.3125 (0x2A)]: nearer 0.3125
    for x, code in cases:
        assert int(fp8.f32_to_e4m3(np.array([x], dtype=np.float32))[0]) == code, (x, hex(code))
    assert int(fp8.f32_to_e4m3(np.array([np.nan], dtype=np.float32))[0]) == 0x7F


def test_encode_roundtrip_all_codes():
    codes = np.arange(256, dtype=np.uint8)
    finite = (codes & 0x7F) != 0x7F
    back = fp8.f32_to_e4m3(fp8.e4m3_to_f32(codes[finite]))
    assert np.array_equal(back, codes[finite])


def _brute_nearest(x: float) -> int:
    """Nearest finite code by exhaustive search in exact arithmetic; ties -> even code; clamp at 448."""
    table = []
    for c in range(0x7F):
        e, m = c >> 3, c & 7
        table.append(Fraction(m, 8) * Fraction(1, 64) if e == 0 else (1 + Fraction(m, 8)) * Fraction(2) ** (e - 7))
    a = min(abs(Fraction(x)), Fraction(448))
    best = min(range(0x7F), key=lambda c: (abs(table[c] - a), c % 2))
    return best | (0x80 if np.signbit(np.float32(x)) else 0)


def test_encode_matches_exact_brute_force():
    rng = np.random.default_rng(7)
    xs = np.concatenate([rng.standard_normal(300) * 3, rng.standard_normal(100) * 200, rng.standard_normal(100) * 0.01,
                         np.ldexp(rng.integers(1, 64, 200).astype(np.float64), rng.integers(-14, 4, 200)),   # many exact ties
                         ]).astype(np.float32)
    got = fp8.f32_to_e4m3(xs)
    for x, g in zip(xs, got):
        assert int(g) == _brute_nearest(float(x)), float(x)


def test_quantize_is_one_float32_product_then_one_rounding():
    # scale 3 makes the float32 product inexact for some bf16 inputs only beyond 24 bits: never here,
    # so quantize(x, 3) must equal the exact-rational nearest code of 3x
    rng = np.random.default_rng(8)
    x = f32_to_bf16(rng.standard_normal(400).astype(np.float32))
    q = fp8.quantize_fp8(x, 3.0)
    xf = bf16_to_f32(x)
    for xi, qi in zip(xf, q):
        assert int(qi) == _brute_nearest(float(xi) * 3.0)


def test_prune24_fp8_is_quantisation_of_the_bf16_result():
    rng = np.random.default_rng(9)
    w = f32_to_bf16((rng.standard_normal((16, 64)) * 0.05).astype(np.float32)).reshape(16, 64)
    for mode in (0, 1):
        ref = prune24(w, group_dim=1, mode=mode)
        r = fp8.prune24_fp8(w, 64.0, mode=mode)
        assert np.array_equal(r.meta, ref.meta) and np.array_equal(r.pos, ref.pos)
        # a power-of-two scale commutes with decoding: decode(q) / 64 is the nearest E4M3-grid point of the value
        kept = bf16_to_f32(ref.vals).astype(np.float64)
        err = np.abs(fp8.e4m3_to_f32(r.vals).astype(np.float64) / 64.0 - kept)
        # E4M3 spacing is 2^-3 relative (normal range) and 2^-9 / 64 absolute (subnormal range): half of it bounds the error
        assert np.all(err <= np.maximum(np.abs(kept) * 2.0 ** -4, 2.0 ** -10 / 64.0) + 1e-12)
        # the dense form holds the same codes at the kept positions and +0 elsewhere
        g = r.dense.reshape(16, 16, 4)
        picked = np.take_along_axis(g, r.pos.astype(np.int64), axis=-1).reshape(16, 32)
        assert np.array_equal(picked, r.vals)
        assert (g != 0).sum(axis=-1).max() <= 2


def test_prune24_fp8_exactly_representable_weights_survive():
    # weights drawn from the E4M3 grid itself, scale 1: quantisation must be the identity on the kept values
    rng = np.random.default_rng(10)
    codes = rng.integers(0, 0x7F, size=(8, 32)).astype(np.uint8) | (rng.integers(0, 2, size=(8, 32)).astype(np.uint8) << 7)
    w = f32_to_bf16(fp8.e4m3_to_f32(codes)).reshape(8, 32)           # every E4M3 value is a bf16 value
    assert np.array_equal(bf16_to_f32(w), fp8.e4m3_to_f32(codes))
    r = fp8.prune24_fp8(w, 1.0)
    ref = prune24(w, group_dim=1, mode=0)
    assert np.array_equal(fp8.e4m3_to_f32(r.vals), bf16_to_f32(ref.vals))


def test_saturation_in_the_fused_pass():
    w = f32_to_bf16(np.array([[1000.0, -2000.0, 1.0, 2.0] * 4], dtype=np.float32)).reshape(1, 16)
    r = fp8.prune24_fp8(w, 1.0)
    assert set(r.vals.ravel().tolist()) == {0x7E, 0xFE}


def test_gemm_fp8_small_by_hand():
    a = fp8.f32_to_e4m3(np.array([[1.0, 2.0], [0.5, -4.0]], dtype=np.float32))
    b = fp8.f32_to_e4m3(np.array([[3.0, 1.0], [-1.0, 0.25]], dtype=np.float32))
    c = fp8.gemm_fp8(a, b, 0.5)
    assert np.array_equal(c, np.array([[2.5, -0.25], [-1.25, -0.75]], dtype=np.float32))


def test_prune24_fp8_strided_groups_are_the_transposed_problem():
    rng = np.random.default_rng(12)
    w = f32_to_bf16((rng.standard_normal((32, 24)) * 0.05).astype(np.float32)).reshape(32, 24)
    for mode in (0, 1):
        a = fp8.prune24_fp8(w, 100.0, mode=mode, group_dim=0)
        b = fp8.prune24_fp8(np.ascontiguousarray(w.T), 100.0, mode=mode, group_dim=1)
        assert np.array_equal(a.vals, b.vals) and np.array_equal(a.meta, b.meta)
        assert np.array_equal(a.dense, b.dense.T)
