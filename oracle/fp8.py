"""FP8 operands whose quantisation rides on the sparsification pass (Section 3.2.2, last paragraph).

Test infrastructure only (see the package docstring).

What the paper fixes
  * FP8 quantisation is independent of the sparsity recipe and can be folded into the passes that
    already scan a matrix element by element (pruning a weight, sparsifying an activation).
  * 2:4 products exist for fp8 operands as for bf16 ones (Section 1).

Readings where the paper is silent
  * Format: E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities; the all-ones
    exponent with mantissa 7 is NaN; largest finite magnitude 448; subnormals m * 2^-9).
  * Scaling: one float32 scale per tensor, chosen by the caller and passed in;
    q = e4m3(float32(x) * scale) with ONE float32 multiplication and one rounding to nearest,
    ties to the even code, magnitudes above 448 (and infinities) clamped to 448, NaN kept NaN.
  * Order: the 2:4 decision and, in soft-threshold mode, the shrinkage are those of the bf16 path
    (taken on the bf16 magnitudes, result rounded to bf16); the kept values are then quantised.
    The fp8 operand is therefore exactly "quantise(the bf16 path's output)", produced in one pass.
  * A product of quantised operands is returned as alpha * sum_k a_q b_q with alpha supplied by the
    caller (normally 1 / (scale_a * scale_b)) and rounded to bf16.
"""
from dataclasses import dataclass

import numpy as np

from .bf16 import bf16_to_f32, f32_to_bf16
from .prune24 import prune24

E4M3_MAX = 448.0


def e4m3_to_f32(code: np.ndarray) -> np.ndarray:
    """Value of an E4M3 code, from the format's definition."""
    c = np.asarray(code, dtype=np.uint8).astype(np.int64)
    s, e, m = c >> 7, (c >> 3) & 15, c & 7
    normal = np.ldexp(1.0 + m / 8.0, e - 7)
    sub = np.ldexp(m / 8.0, -6)
    v = np.where(e == 0, sub, normal)
    v = np.where((e == 15) & (m == 7), np.nan, v)
    return np.where(s == 1, -v, v).astype(np.float32)


# the 127 finite non-negative values in code order (code 0x00 .. 0x7E): strictly increasing
_POS = e4m3_to_f32(np.arange(0x7F, dtype=np.uint8)).astype(np.float64)


def f32_to_e4m3(x: np.ndarray) -> np.ndarray:
    """Nearest E4M3 code of a float32: ties to the even code, clamped at +-448, NaN -> 0x7F."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    sign = (f.view(np.uint32) >> np.uint32(31)).astype(np.uint8) << np.uint8(7)
    a = np.abs(f.astype(np.float64))
    a_c = np.minimum(np.where(np.isnan(a), 0.0, a), E4M3_MAX)
    hi = np.clip(np.searchsorted(_POS, a_c, side="left"), 0, 0x7E)       # first code with value >= a
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a_c - _POS[lo], _POS[hi] - a_c
    take_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(take_lo, lo, hi).astype(np.uint8)
    return np.where(np.isnan(a), np.uint8(0x7F), code | sign).astype(np.uint8)


def quantize_fp8(x_bits: np.ndarray, scale) -> np.ndarray:
    """bf16 bits -> E4M3 codes of float32(x) * scale (one float32 product, then one rounding)."""
    prod = (bf16_to_f32(x_bits) * np.float32(scale)).astype(np.float32)
    return f32_to_e4m3(prod).reshape(np.shape(x_bits))


@dataclass
class Prune24Fp8Result:
    vals: np.ndarray     # uint8 E4M3 codes [R, K/2]: the kept values, quantised, in position order
    meta: np.ndarray     # uint16 [R, K/16]: canonical metadata (identical to the bf16 path's)
    dense: np.ndarray    # uint8 E4M3 codes [R, K]: quantised pruned matrix (dropped -> +0)
    pos: np.ndarray      # uint8 [R, K/4, 2]


def prune24_fp8(w_bits: np.ndarray, scale, mode: int = 0, group_dim: int = 1) -> Prune24Fp8Result:
    """2:4 (groups along a row, or along a column with K-major outputs, as in `prune24`), then
    quantisation of what is kept. `dense` keeps the orientation of the input."""
    p = prune24(w_bits, group_dim=group_dim, mode=mode)
    return Prune24Fp8Result(vals=quantize_fp8(p.vals, scale), meta=p.meta, dense=quantize_fp8(p.dense, scale), pos=p.pos)


def gemm_fp8(a_codes: np.ndarray, b_codes: np.ndarray, alpha) -> np.ndarray:
    """C[m, n] = alpha * sum_k A[m, k] B[n, k] on the decoded operands, in float64; float32 out."""
    a = e4m3_to_f32(a_codes).astype(np.float64)
    b = e4m3_to_f32(b_codes).astype(np.float64)
    return ((a @ b.T) * float(np.float32(alpha))).astype(np.float32)


def gemm_fp8_bf16(a_codes: np.ndarray, b_codes: np.ndarray, alpha) -> np.ndarray:
    return f32_to_bf16(gemm_fp8(a_codes, b_codes, alpha)).reshape(a_codes.shape[0], b_codes.shape[0])
