"""2:4 weight sparsification: magnitude selection, optional soft-thresholding, packing.

Test infrastructure only (see the package docstring).

What the paper fixes
  * n:m format with n = 2, m = 4: a group of four neighbours holds no more than two non-zero
    entries (Section 1's definition of n:m sparsity).
  * The mask is the magnitude-based one: the two largest magnitudes of the group stay
    (Section 2.2, first sentence); equal magnitudes are resolved towards the lower index.
  * Soft-thresholding (Section 2.2): with the group's magnitudes sorted
    |t1| <= |t2| <= |t3| <= |t4|, the threshold is t = |t2| (the second smallest, i.e. the
    larger of the two dropped magnitudes); every element moves towards zero by t and the two
    smallest become zero:  a - t for a > t,  0 for -t < a <= t,  a + t for a <= -t.
  * The packed form is "values plus sparsity metadata" (Section 3.2.1).

Readings where the paper is silent
  * Groups run along the reduction dimension of the product that consumes the matrix.
  * A group always records exactly two positions, even if fewer than two elements are non-zero.
  * Magnitudes are compared on the bf16 bit pattern with the sign cleared (monotone for finite
    values; +0 and -0 compare equal).
  * The soft-threshold subtraction is one float32 operation on the widened bf16 values and the
    result is rounded to bf16 with round-to-nearest-even. No rescaling factor is applied.

Metadata: one nibble per group, ``pos0 | pos1 << 2`` with ``pos0 < pos1`` the kept positions;
four consecutive groups of a row form one little-endian ``uint16``.
"""
from dataclasses import dataclass

import numpy as np

from .bf16 import bf16_to_f32, f32_to_bf16


@dataclass
class Prune24Result:
    dense: np.ndarray   # uint16 bf16 bits, same shape/orientation as the input, dropped -> +0
    vals: np.ndarray    # uint16 bf16 bits [R, K/2]: kept values in position order
    meta: np.ndarray    # uint16 [R, K/16]: canonical metadata
    pos: np.ndarray     # uint8 [R, K/4, 2]: kept positions (pos0 < pos1)


def _select_top2_of4(keys: np.ndarray) -> np.ndarray:
    """keys [..., 4] unsigned magnitudes -> (rank [..., 4], boolean keep mask [..., 4]).

    An element's rank is the number of elements that precede it in the order
    (magnitude descending, index ascending); ranks 0 and 1 are kept.
    """
    k = keys.astype(np.int32)
    rank = np.zeros(k.shape, dtype=np.int8)
    for i in range(4):
        for j in range(4):
            if j == i:
                continue
            before = (k[..., j] > k[..., i]) | ((k[..., j] == k[..., i]) & (j < i))
            rank[..., i] += before
    return rank, rank < 2


def prune24(w_bits: np.ndarray, group_dim: int = 1, mode: int = 0) -> Prune24Result:
    """Sparsify a bf16 matrix to 2:4.

    group_dim = 1: groups are four consecutive elements of a row (R = rows, K = cols).
    group_dim = 0: groups are four consecutive elements of a column; the packed outputs are
                   written K-major, i.e. for the transposed matrix (R = cols, K = rows).
    mode 0: hard magnitude pruning; mode 1: soft-thresholding.
    """
    w = np.asarray(w_bits, dtype=np.uint16)
    assert w.ndim == 2
    a = w if group_dim == 1 else w.T          # [R, K], groups along K
    R, K = a.shape
    assert K % 16 == 0, "K must be a multiple of 16 (four groups per metadata word)"
    g = np.ascontiguousarray(a).reshape(R, K // 4, 4)

    keys = g & np.uint16(0x7FFF)
    rank, keep = _select_top2_of4(keys)

    # kept positions in ascending order
    idx = np.broadcast_to(np.arange(4, dtype=np.int64), g.shape)
    pos = np.sort(np.where(keep, idx, 99), axis=-1)[..., :2].astype(np.uint8)   # [R, K/4, 2]

    if mode == 0:
        out = np.where(keep, g, np.uint16(0))
    else:
        # threshold = magnitude of the element of rank 2 (second smallest of the four)
        t_key = np.take_along_axis(keys, np.argmax(rank == 2, axis=-1)[..., None], axis=-1)
        t = bf16_to_f32(t_key.astype(np.uint16))                    # [R, K/4, 1] float32 >= 0
        af = bf16_to_f32(g)
        shrunk = np.where(af > 0, af - t, np.where(af < 0, af + t, np.float32(0.0))).astype(np.float32)
        out = np.where(keep, f32_to_bf16(shrunk).reshape(g.shape), np.uint16(0))

    vals = np.take_along_axis(out, pos.astype(np.int64), axis=-1).reshape(R, K // 2)
    nib = (pos[..., 0].astype(np.uint16) | (pos[..., 1].astype(np.uint16) << np.uint16(2)))   # [R, K/4]
    nib4 = nib.reshape(R, K // 16, 4)
    meta = (nib4[..., 0] | (nib4[..., 1] << np.uint16(4)) | (nib4[..., 2] << np.uint16(8))
            | (nib4[..., 3] << np.uint16(12))).astype(np.uint16)

    dense_rk = out.reshape(R, K)
    dense = dense_rk if group_dim == 1 else np.ascontiguousarray(dense_rk.T)
    return Prune24Result(dense=np.ascontiguousarray(dense), vals=np.ascontiguousarray(vals),
                         meta=meta, pos=pos)


def decompress24(vals: np.ndarray, meta: np.ndarray) -> np.ndarray:
    """Expand packed values + canonical metadata back to the dense [R, K] matrix."""
    vals = np.asarray(vals, dtype=np.uint16)
    meta = np.asarray(meta, dtype=np.uint16)
    R, Kh = vals.shape
    K = 2 * Kh
    nib = np.stack([(meta >> np.uint16(4 * i)) & np.uint16(0xF) for i in range(4)], axis=-1).reshape(R, K // 4)
    p0 = (nib & np.uint16(3)).astype(np.int64)
    p1 = ((nib >> np.uint16(2)) & np.uint16(3)).astype(np.int64)
    out = np.zeros((R, K // 4, 4), dtype=np.uint16)
    v = vals.reshape(R, K // 4, 2)
    np.put_along_axis(out, p0[..., None], v[..., 0:1], axis=-1)
    np.put_along_axis(out, p1[..., None], v[..., 1:2], axis=-1)
    return out.reshape(R, K)
