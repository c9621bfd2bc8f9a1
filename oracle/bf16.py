"""bf16 <-> float32 conversions used by the oracle (test infrastructure only).

bf16 is the upper half of an IEEE float32. Widening is exact; narrowing is
round-to-nearest-even on the 16 discarded bits. NaNs keep a quiet payload.
"""
import numpy as np


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32)
    return (u << np.uint32(16)).view(np.float32)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    # add 0x7FFF plus the parity of the bit that becomes the new LSB: ties go to even
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    out = ((u + bias) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(f)
    if nan.any():
        out = np.where(nan, ((u >> np.uint32(16)) | np.uint32(0x0040)).astype(np.uint16), out)
    return out
