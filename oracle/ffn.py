"""Masked FFN forward/backward (Algorithms 1 and 2) and the dense FFN (Eqs. 1-8).

Test infrastructure only (see the package docstring).

Layout: T tokens, D = d_model, F = d_ffn; X [T, D], W1 [F, D], W2 [D, F], Y and dY [T, D]
(the paper writes W1 [D, F], W2 [F, D] and y = x W; this is the same mathematics with the
weights stored transposed). All tensors cross this interface as bf16 bit patterns (uint16).

Algorithm 1 (forward)          y1 = X @ sparsify24(W1);  y2 = ReLU(y1)^2;  y2 -> V:N:M;  y3 = y2 @ W2
Algorithm 2 (backward)         dy2 = dy3 @ sparsify24(W2^T);  dW2 = y2^T @ dy3;
                               dy1 = 2 dy2 ReLU(y1);  dX = dy1 @ W1^T;  dW1 = dy1^T @ X
with exactly one sparse operand per product (Section 3): W2 is dense in the forward product,
W1 is dense in dX, and dW1, dW2 are gradients for the dense master weights.

Readings where the paper is silent
  * Both weight prunings run their groups along d_model (the reduction dimension of the product
    that consumes them).
  * dy1 carries the mask of y2 (Algorithm 2 colours it as V:N:M and says y1, y2 are saved from
    the forward pass); it is not re-selected.
  * Rounding points: y1, y2 (= hb), dy1 are rounded to bf16 where they are stored; dy2 is used
    in float32. Products accumulate in float64 here.
"""
from dataclasses import dataclass
from typing import Optional

import numpy as np

from .bf16 import bf16_to_f32, f32_to_bf16
from .prune24 import prune24, Prune24Result
from .vnm import vnm_sparsify, squared_relu_bf16, VnmResult


def matmul_f64(a_f32: np.ndarray, b_f32: np.ndarray) -> np.ndarray:
    """C = A @ B with float64 accumulation, returned as float32."""
    return (a_f32.astype(np.float64) @ b_f32.astype(np.float64)).astype(np.float32)


@dataclass
class SparseFwd:
    w1s: Prune24Result
    y1b: np.ndarray          # uint16 [T, F]
    act: VnmResult           # y2 in V:N:M form (+ packed ReLU(y1b))
    y3: np.ndarray           # float32 [T, D]


@dataclass
class SparseBwd:
    w2s: Prune24Result       # pruned along D: packed [F, D/2]
    dy2: np.ndarray          # float32 [T, F]
    dy1_dense: np.ndarray    # uint16 [T, F], zero off the mask
    dy1_vals: np.ndarray     # uint16 [T, 2F/M], packed with y2's metadata
    dX: np.ndarray           # float32 [T, D]
    dW1: np.ndarray          # float32 [F, D]
    dW2: np.ndarray          # float32 [D, F]


def sparse_ffn_fwd(X, W1, W2, V: int, M: int, N: int = 2, prune_mode: int = 0,
                   forced_y1b: Optional[np.ndarray] = None,
                   _all_ones_masks: bool = False) -> SparseFwd:
    """Algorithm 1. ``forced_y1b`` replaces the oracle's own bf16 pre-activations (stage-wise
    comparison). ``_all_ones_masks`` is a test hook: no pruning, no activation mask."""
    Xf = bf16_to_f32(X)
    w1s = prune24(W1, group_dim=1, mode=prune_mode)
    W1s_f = bf16_to_f32(W1 if _all_ones_masks else w1s.dense)
    if forced_y1b is None:
        y1b = f32_to_bf16(matmul_f64(Xf, W1s_f.T)).reshape(Xf.shape[0], W1s_f.shape[0])
    else:
        y1b = np.asarray(forced_y1b, dtype=np.uint16)
    act = vnm_sparsify(y1b, V=V, M=M, N=N, apply_sqrelu=True)
    if _all_ones_masks:
        act.dense = act.hb
        act.mask = np.ones_like(act.mask)
    y3 = matmul_f64(bf16_to_f32(act.dense), bf16_to_f32(W2).T)
    return SparseFwd(w1s=w1s, y1b=y1b, act=act, y3=y3)


def sparse_ffn_bwd(dY, X, W1, W2, fwd: SparseFwd, prune_mode: int = 0,
                   _all_ones_masks: bool = False) -> SparseBwd:
    """Algorithm 2 with the forward pass's saved y1b / y2 / mask."""
    dYf, Xf = bf16_to_f32(dY), bf16_to_f32(X)
    w2s = prune24(W2, group_dim=0, mode=prune_mode)           # groups along D (dim 0 of [D, F])
    W2s_f = bf16_to_f32(W2 if _all_ones_masks else w2s.dense)  # [D, F]
    dy2 = matmul_f64(dYf, W2s_f)                               # [T, F] float32
    _, relu_bits = squared_relu_bf16(fwd.y1b)
    relu = bf16_to_f32(relu_bits)
    dy1_full = (np.float32(2.0) * dy2 * relu).astype(np.float32)
    dy1_bits = f32_to_bf16(dy1_full).reshape(dy2.shape)
    dy1_dense = np.where(fwd.act.mask, dy1_bits, np.uint16(0))
    y2m = bf16_to_f32(fwd.act.dense)
    dy1m = bf16_to_f32(dy1_dense)
    dW2 = matmul_f64(dYf.T, y2m)                               # [D, F]
    dX = matmul_f64(dy1m, bf16_to_f32(W1))                     # dense W1
    dW1 = matmul_f64(dy1m.T, Xf)                               # [F, D]
    dy1_vals = _pack_like(dy1_dense, fwd.act)
    return SparseBwd(w2s=w2s, dy2=dy2, dy1_dense=dy1_dense, dy1_vals=dy1_vals, dX=dX, dW1=dW1, dW2=dW2)


def _pack_like(dense_bits: np.ndarray, act: VnmResult) -> np.ndarray:
    """Pack a [T, F] matrix with the positions recorded in ``act`` (colidx + nibbles)."""
    T, F = dense_bits.shape
    B, G, _ = act.colidx.shape
    V, M = T // B, F // G
    nib = np.stack([(act.meta >> np.uint16(4 * i)) & np.uint16(0xF) for i in range(4)], axis=-1).reshape(B, V, G)
    p0 = (nib & np.uint16(3)).astype(np.int64)
    p1 = ((nib >> np.uint16(2)) & np.uint16(3)).astype(np.int64)
    ci = np.broadcast_to(act.colidx.astype(np.int64)[:, None], (B, V, G, 4))
    c0 = np.take_along_axis(ci, p0[..., None], axis=-1)
    c1 = np.take_along_axis(ci, p1[..., None], axis=-1)
    d4 = dense_bits.reshape(B, V, G, M)
    v0 = np.take_along_axis(d4, c0, axis=-1)
    v1 = np.take_along_axis(d4, c1, axis=-1)
    return np.ascontiguousarray(np.concatenate([v0, v1], axis=-1).reshape(T, 2 * G))


@dataclass
class DenseFwd:
    y1b: np.ndarray     # uint16 [T, F]
    hb: np.ndarray      # uint16 [T, F]
    y3: np.ndarray      # float32 [T, D]


@dataclass
class DenseBwd:
    dy1: np.ndarray     # uint16 [T, F]
    dX: np.ndarray
    dW1: np.ndarray
    dW2: np.ndarray


def dense_ffn_fwd(X, W1, W2, forced_y1b: Optional[np.ndarray] = None) -> DenseFwd:
    """Eqs. 1-3 with no pruning (the closing dense phase and the speed-up baseline)."""
    Xf = bf16_to_f32(X)
    if forced_y1b is None:
        y1b = f32_to_bf16(matmul_f64(Xf, bf16_to_f32(W1).T)).reshape(Xf.shape[0], W1.shape[0])
    else:
        y1b = np.asarray(forced_y1b, dtype=np.uint16)
    hb, _ = squared_relu_bf16(y1b)
    y3 = matmul_f64(bf16_to_f32(hb), bf16_to_f32(W2).T)
    return DenseFwd(y1b=y1b, hb=hb, y3=y3)


def dense_ffn_bwd(dY, X, W1, W2, fwd: DenseFwd) -> DenseBwd:
    """Eqs. 4-8."""
    dYf, Xf = bf16_to_f32(dY), bf16_to_f32(X)
    dy2 = matmul_f64(dYf, bf16_to_f32(W2))
    _, relu_bits = squared_relu_bf16(fwd.y1b)
    dy1 = f32_to_bf16((np.float32(2.0) * dy2 * bf16_to_f32(relu_bits)).astype(np.float32)).reshape(dy2.shape)
    dy1f = bf16_to_f32(dy1)
    return DenseBwd(dy1=dy1,
                    dX=matmul_f64(dy1f, bf16_to_f32(W1)),
                    dW1=matmul_f64(dy1f.T, Xf),
                    dW2=matmul_f64(dYf.T, bf16_to_f32(fwd.hb)))
