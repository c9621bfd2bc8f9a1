"""Neuron-level experts that produce the V:N:M pattern (Section 3.1, Algorithm 3, Figure 4).

Test infrastructure only (see the package docstring).

What the paper fixes
  * Offline, the columns of W1 (one d_model-vector per hidden feature; rows of W1 [F, D] in this
    code's layout) are clustered into non-overlapping subsets, the "experts"; an expert is
    represented by its cluster centre and features join centres by L2 distance (Figure 4a).
  * Per token, `x @ ExpertMeans` decides the expert (Section 3.1 step 1); tokens of one expert are
    placed in adjacent rows (step 2); each group of tokens is multiplied with its expert's columns
    only (step 3), and the result "will be in the V:N:M format".
  * Inside the kept columns the 2:4 pattern is chosen greedily by magnitude (Section 2.3).

Readings where the paper is silent or at odds with itself
  * Number and size of experts: V:N:M keeps four of every M columns, so E = M / 4 experts of
    exactly F / E features each (M = 64 gives the 16 experts the text calls typical; Table 5's
    sparsities follow: a token keeps 2 of every 4 features of one expert, density 2 / M).
    Clustering is therefore BALANCED k-means: Lloyd iterations with L2 distance whose assignment
    step gives every expert the same number of features.
  * How an expert's column set becomes "four kept columns per block": the hidden features of an FFN
    can be renumbered freely (rows of W1 and columns of W2 together), so they are stored
    expert-major: expert e owns the contiguous block [e F/E, (e+1) F/E). Interleaving the blocks
    four features at a time (group g, column 4 e + j  <->  feature e F/E + 4 g + j) turns a block of
    V tokens of expert e into a V:N:M block whose kept columns are 4 e .. 4 e + 3 in every group;
    `vnm_view` does exactly that and is checked against the V:N:M invariants.
  * Routing score: Algorithm 3 says cosine distance, Figure 4 L2 distance, the text the product
    x @ ExpertMeans. The text is taken: the largest dot product wins (top-1), ties to the lower
    expert. The decision is taken on float64 dot products of the bf16 operands; a device that
    accumulates differently may legitimately pick another expert on a near tie, which is why the
    step functions accept the routing as an input (`forced_expert`).
  * Clustering details (Lloyd's start, the balanced assignment order, the number of iterations) are
    not in the paper; any balanced partition is a valid router. This file's choices: centres start
    as the means of E contiguous blocks of features; assignment takes (feature, expert) pairs in
    order of increasing squared distance and gives a feature to the first expert with room.

Everything downstream (SquaredReLU, rounding points, the pruned W1 / W2, which operand is dense in
which product) is exactly the masked step of `oracle.ffn`; only the activation mask differs.
"""
from dataclasses import dataclass
from typing import Optional

import numpy as np

from .bf16 import bf16_to_f32, f32_to_bf16
from .prune24 import prune24, _select_top2_of4
from .vnm import squared_relu_bf16
from .ffn import matmul_f64


def fit_experts(w1_bits: np.ndarray, E: int, iters: int = 8):
    """Balanced k-means over the rows of W1 [F, D]. Returns (expert_of_feature int32 [F],
    means bf16 bits [E, D])."""
    W = bf16_to_f32(w1_bits).astype(np.float64)
    F, D = W.shape
    assert F % E == 0
    cap = F // E
    centres = W.reshape(E, cap, D).mean(axis=1)
    assign = np.repeat(np.arange(E), cap)
    for _ in range(iters):
        d2 = ((W * W).sum(axis=1)[:, None] - 2.0 * W @ centres.T + (centres * centres).sum(axis=1)[None, :])
        order = np.lexsort((np.tile(np.arange(E), F), np.repeat(np.arange(F), E), d2.ravel()))   # distance, then f, then e
        new = np.full(F, -1, dtype=np.int64)
        room = np.full(E, cap, dtype=np.int64)
        left = F
        for idx in order:
            f, e = divmod(int(idx), E)
            if new[f] < 0 and room[e] > 0:
                new[f] = e
                room[e] -= 1
                left -= 1
                if left == 0:
                    break
        if np.array_equal(new, assign):
            break
        assign = new
        centres = np.stack([W[assign == e].mean(axis=0) for e in range(E)])
    return assign.astype(np.int32), f32_to_bf16(centres.astype(np.float32)).reshape(E, D)


def expert_major_permutation(expert_of_feature: np.ndarray) -> np.ndarray:
    """perm such that feature perm[i] of the original numbering is feature i of the expert-major one."""
    return np.argsort(expert_of_feature, kind="stable")


def route(x_bits: np.ndarray, means_bits: np.ndarray):
    """Top-1 expert per token by the dot product with the expert means. Returns (expert int32 [T],
    logits float64 [T, E])."""
    logits = bf16_to_f32(x_bits).astype(np.float64) @ bf16_to_f32(means_bits).astype(np.float64).T
    return np.argmax(logits, axis=1).astype(np.int32), logits      # argmax returns the first maximum


@dataclass
class RoutedFwd:
    expert: np.ndarray      # int32 [T]
    y1b: np.ndarray         # uint16 [T, F]: pre-activation, +0 outside the token's expert block
    mask: np.ndarray        # bool [T, F]: kept activations (two of every four features of the expert block)
    pos: np.ndarray         # uint8 [T, F/(4E), 2]: kept positions inside each group of four of the block
    y2: np.ndarray          # uint16 [T, F]: bf16(ReLU(y1b)^2) on the mask, +0 elsewhere
    relu: np.ndarray        # uint16 [T, F]: ReLU(y1b) on the mask
    y3: np.ndarray          # float32 [T, D]
    w1s_dense: np.ndarray   # uint16 [F, D] pruned W1


@dataclass
class RoutedBwd:
    dy1: np.ndarray         # uint16 [T, F], +0 off the mask
    dX: np.ndarray
    dW1: np.ndarray
    dW2: np.ndarray


def _block_mask(expert: np.ndarray, F: int, E: int) -> np.ndarray:
    return (np.arange(F)[None, :] // (F // E)) == expert[:, None]


def routed_ffn_fwd(X, W1, W2, means, E: int, prune_mode: int = 0, forced_expert: Optional[np.ndarray] = None,
                   forced_y1b: Optional[np.ndarray] = None) -> RoutedFwd:
    """Algorithm 1 with MoEToVenom as the activation sparsifier. W1 [F, D] and W2 [D, F] are given in
    expert-major feature order. `forced_y1b` [T, F/E] replaces the oracle's own pre-activations of each
    token's expert block (stage-wise comparison with a device that rounds differently)."""
    T, D = X.shape
    F = W1.shape[0]
    Fe = F // E
    expert = route(X, means)[0] if forced_expert is None else np.asarray(forced_expert, dtype=np.int32)
    w1s = prune24(W1, group_dim=1, mode=prune_mode)
    block = _block_mask(expert, F, E)
    if forced_y1b is None:
        y1 = f32_to_bf16(matmul_f64(bf16_to_f32(X), bf16_to_f32(w1s.dense).T)).reshape(T, F)
    else:
        y1 = np.zeros((T, F), dtype=np.uint16)
        cols = expert[:, None].astype(np.int64) * Fe + np.arange(Fe)[None, :]
        np.put_along_axis(y1, cols, np.asarray(forced_y1b, dtype=np.uint16), axis=1)
    y1b = np.where(block, y1, np.uint16(0))
    hb, relu = squared_relu_bf16(y1b)
    # 2:4 by magnitude inside every group of four consecutive features (Section 2.3's greedy rule)
    _, keep = _select_top2_of4((hb & np.uint16(0x7FFF)).reshape(T, F // 4, 4))
    mask = keep.reshape(T, F) & block
    idx = np.broadcast_to(np.arange(4), (T, F // 4, 4))
    pos_all = np.sort(np.where(keep, idx, 99), axis=-1)[..., :2].astype(np.uint8)       # [T, F/4, 2]
    gcols = expert[:, None].astype(np.int64) * (Fe // 4) + np.arange(Fe // 4)[None, :]
    pos = np.take_along_axis(pos_all, gcols[..., None], axis=1)
    y2 = np.where(mask, hb, np.uint16(0))
    y3 = matmul_f64(bf16_to_f32(y2), bf16_to_f32(W2).T)
    return RoutedFwd(expert=expert, y1b=y1b, mask=mask, pos=pos, y2=y2, relu=np.where(mask, relu, np.uint16(0)),
                     y3=y3, w1s_dense=w1s.dense)


def routed_ffn_bwd(dY, X, W1, W2, fwd: RoutedFwd, prune_mode: int = 0) -> RoutedBwd:
    """Algorithm 2 on the routed mask: dy2 through the pruned W2, dy1 = 2 dy2 ReLU(y1) on the mask,
    dX through the dense W1, and the two weight gradients (zero outside a token's expert block by
    construction, which is what makes them cheap)."""
    dYf, Xf = bf16_to_f32(dY), bf16_to_f32(X)
    w2s = prune24(W2, group_dim=0, mode=prune_mode)
    dy2 = matmul_f64(dYf, bf16_to_f32(w2s.dense))
    dy1_full = f32_to_bf16((np.float32(2.0) * dy2 * bf16_to_f32(fwd.relu)).astype(np.float32)).reshape(dy2.shape)
    dy1 = np.where(fwd.mask, dy1_full, np.uint16(0))
    dy1f = bf16_to_f32(dy1)
    return RoutedBwd(dy1=dy1, dX=matmul_f64(dy1f, bf16_to_f32(W1)), dW1=matmul_f64(dy1f.T, Xf),
                     dW2=matmul_f64(dYf.T, bf16_to_f32(fwd.y2)))


def token_order(expert: np.ndarray, E: int, pad: int = 1):
    """Tokens grouped by expert (stable), each expert's segment padded to a multiple of `pad` rows.
    Returns (src_of_row int64 [rows], -1 on padding rows; start [E + 1] segment boundaries)."""
    src, start = [], [0]
    for e in range(E):
        t = np.flatnonzero(expert == e)
        n = -(-len(t) // pad) * pad
        src.append(np.concatenate([t, np.full(n - len(t), -1, dtype=np.int64)]))
        start.append(start[-1] + n)
    return np.concatenate(src), np.asarray(start, dtype=np.int64)


def vnm_view(fwd: RoutedFwd, E: int, V: int):
    """The routed activation as a V:N:M matrix with M = 4 E: tokens in expert order (segments padded
    to V rows with zero rows), features interleaved four at a time across the experts. Returns
    (dense uint16 [rows, F], colidx uint8 [rows / V, F / M, 4])."""
    T, F = fwd.y2.shape
    Fe, M = F // E, 4 * E
    src, _ = token_order(fwd.expert, E, pad=V)
    rows = len(src)
    y2p = np.where((src >= 0)[:, None], fwd.y2[np.maximum(src, 0)], np.uint16(0))
    ep = np.where(src >= 0, fwd.expert[np.maximum(src, 0)], -1)
    # feature e Fe + 4 g + j  ->  column g M + 4 e + j
    f = np.arange(F)
    e_of, i_of = f // Fe, f % Fe
    col = (i_of // 4) * M + 4 * e_of + (i_of % 4)
    dense = np.zeros((rows, F), dtype=np.uint16)
    dense[:, col] = y2p
    blk_e = ep.reshape(rows // V, V)
    # a padded block may hold padding rows only at its end; its expert is that of its first row
    be = blk_e[:, 0]
    colidx = (4 * be[:, None, None] + np.arange(4)[None, None, :]).astype(np.uint8)
    return dense, np.broadcast_to(colidx, (rows // V, F // M, 4)).copy()
