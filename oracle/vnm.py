"""SquaredReLU + V:N:M (Venom) activation sparsification.

Test infrastructure only (see the package docstring).

What the paper fixes (Section 2.3, Table 5)
  * Blocks of V rows by M columns; a block keeps four of its M columns, and every row of the
    block keeps the two larger magnitudes among those four (a 2:4 pattern chosen greedily by
    magnitude). Density is therefore N/M with N = 2 (Table 5: M = 16, 32, 64 -> 87.5, 93.75,
    96.875 % sparsity).
  * The activation is y2 = ReLU(y1)^2 (Eq. 2).

Readings where the paper is silent or garbled
  * "sub-matrices of size [nrows // V, M]" is read as nrows // V block-rows of V x M blocks
    (the cited format definition; it is what Table 5's percentages fit).
  * Which four columns stay is not stated. Reading: column score = sum over the block's V rows of
    the magnitude of the bf16 activation, accumulated sequentially from the first row to the
    last in float32 (round-to-nearest, no fused multiply-add, no re-association); the four
    columns that come first in (score descending, index ascending) stay and are recorded in
    ascending index order. This order of accumulation is part of the format contract.
  * Rounding points: the pre-activation is a bf16 value y1b; h = y1b*y1b for y1b > 0 else 0 is
    evaluated in float32 (exact for bf16 inputs) and stored as hb = bf16(h); every decision is a
    function of hb only. ReLU(y1b) is what the backward pass needs and is saved in packed form.
  * The 2:4 stage applies the same rule as weight pruning (two largest magnitudes of the four
    kept columns, ties to the lower position) row by row.

Outputs for an input [T, F] with G = F / M groups per row and B = T / V block-rows
  vals      uint16 [T, 2G]      kept activation values hb, in position order
  relu_vals uint16 [T, 2G]      max(y1b, 0) at the same positions (only with apply_sqrelu)
  meta      uint16 [T, G/4]     canonical nibbles over the condensed [T, 4G] matrix
  colidx    uint8  [B, G, 4]    kept columns of each block, ascending, each < M
  dense     uint16 [T, F]       hb on the mask, +0 elsewhere
"""
from dataclasses import dataclass
from typing import Optional

import numpy as np

from .bf16 import bf16_to_f32, f32_to_bf16
from .prune24 import _select_top2_of4


@dataclass
class VnmResult:
    vals: np.ndarray
    meta: np.ndarray
    colidx: np.ndarray
    relu_vals: Optional[np.ndarray]
    dense: np.ndarray
    mask: np.ndarray        # bool [T, F]
    hb: np.ndarray          # uint16 [T, F]: activation before masking


def squared_relu_bf16(y1b_bits: np.ndarray):
    """Eq. 2 on bf16 inputs: returns (hb bits, relu bits)."""
    y = bf16_to_f32(y1b_bits)
    pos = y > 0
    r = np.where(pos, y, np.float32(0.0)).astype(np.float32)
    h = (r * r).astype(np.float32)
    return f32_to_bf16(h).reshape(y.shape), f32_to_bf16(r).reshape(y.shape)


def vnm_sparsify(p_bits: np.ndarray, V: int, M: int, N: int = 2, apply_sqrelu: bool = True) -> VnmResult:
    p = np.asarray(p_bits, dtype=np.uint16)
    T, F = p.shape
    assert N == 2, "only N = 2 is defined (four kept columns, 2:4 inside them)"
    assert M >= 4 and T % V == 0 and F % M == 0 and (F // M) % 4 == 0
    G, B = F // M, T // V

    if apply_sqrelu:
        hb, relu = squared_relu_bf16(p)
    else:
        hb, relu = p, None

    # ---- stage 1: column scores, sequential float32 accumulation over the V rows of a block
    mag = bf16_to_f32(hb & np.uint16(0x7FFF)).reshape(B, V, G, M)
    score = np.zeros((B, G, M), dtype=np.float32)
    for r in range(V):                      # ascending row order, one float32 add per row
        score = (score + mag[:, r]).astype(np.float32)

    # the four columns first in (score descending, index ascending); scores are >= 0 so the
    # float32 bit pattern orders them exactly
    sbits = score.view(np.uint32).astype(np.int64)
    crank = np.zeros((B, G, M), dtype=np.int32)
    for i in range(M):
        for j in range(M):
            if j == i:
                continue
            before = (sbits[..., j] > sbits[..., i]) | ((sbits[..., j] == sbits[..., i]) & (j < i))
            crank[..., i] += before
    keepcol = crank < 4                                                   # [B, G, M]
    cidx = np.broadcast_to(np.arange(M, dtype=np.int64), keepcol.shape)
    colidx = np.sort(np.where(keepcol, cidx, 10 ** 6), axis=-1)[..., :4]   # ascending [B, G, 4]

    # ---- stage 2: 2:4 over the four kept columns, row by row
    hb4 = hb.reshape(B, V, G, M)
    gather = np.broadcast_to(colidx[:, None], (B, V, G, 4))
    kept = np.take_along_axis(hb4, gather, axis=-1)                        # [B, V, G, 4]
    _, keep2 = _select_top2_of4(kept & np.uint16(0x7FFF))
    pidx = np.broadcast_to(np.arange(4, dtype=np.int64), kept.shape)
    pos = np.sort(np.where(keep2, pidx, 99), axis=-1)[..., :2]             # [B, V, G, 2]

    vals = np.take_along_axis(kept, pos, axis=-1).reshape(T, 2 * G)
    relu_vals = None
    if relu is not None:
        rk = np.take_along_axis(relu.reshape(B, V, G, M), gather, axis=-1)
        relu_vals = np.ascontiguousarray(np.take_along_axis(rk, pos, axis=-1).reshape(T, 2 * G))

    nib = (pos[..., 0] | (pos[..., 1] << 2)).astype(np.uint16).reshape(T, G // 4, 4)
    meta = (nib[..., 0] | (nib[..., 1] << np.uint16(4)) | (nib[..., 2] << np.uint16(8))
            | (nib[..., 3] << np.uint16(12))).astype(np.uint16)

    # dense masked matrix and boolean mask
    mask4 = np.zeros((B, V, G, M), dtype=bool)
    cols_kept = np.take_along_axis(gather, pos, axis=-1)                   # [B, V, G, 2] column ids
    np.put_along_axis(mask4, cols_kept, True, axis=-1)
    mask = mask4.reshape(T, F)
    dense = np.where(mask, hb, np.uint16(0))

    return VnmResult(vals=np.ascontiguousarray(vals), meta=meta, colidx=colidx.astype(np.uint8),
                     relu_vals=relu_vals, dense=dense, mask=mask, hb=hb)


def decompress_vnm(vals: np.ndarray, meta: np.ndarray, colidx: np.ndarray, V: int, M: int) -> np.ndarray:
    """Expand packed V:N:M storage to the dense [T, F] matrix."""
    vals = np.asarray(vals, dtype=np.uint16)
    T, G2 = vals.shape
    G = G2 // 2
    B = T // V
    nib = np.stack([(meta >> np.uint16(4 * i)) & np.uint16(0xF) for i in range(4)], axis=-1).reshape(B, V, G)
    p0 = (nib & np.uint16(3)).astype(np.int64)
    p1 = ((nib >> np.uint16(2)) & np.uint16(3)).astype(np.int64)
    ci = np.broadcast_to(np.asarray(colidx, dtype=np.int64)[:, None], (B, V, G, 4))
    c0 = np.take_along_axis(ci, p0[..., None], axis=-1)
    c1 = np.take_along_axis(ci, p1[..., None], axis=-1)
    out = np.zeros((B, V, G, M), dtype=np.uint16)
    v = vals.reshape(B, V, G, 2)
    np.put_along_axis(out, c0, v[..., 0:1], axis=-1)
    np.put_along_axis(out, c1, v[..., 1:2], axis=-1)
    return out.reshape(T, G * M)
