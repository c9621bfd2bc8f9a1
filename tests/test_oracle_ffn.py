"""Pins for the oracle's masked FFN forward/backward and the dense FFN."""
import numpy as np
import pytest

import oracle
from oracle import bf16_to_f32, f32_to_bf16
from paper_2602_06183_b200 import synth


def _rel(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b.astype(np.float64)) / max(np.linalg.norm(b.astype(np.float64)), 1e-30))


def _inputs(T=64, D=32, F=64, seed=0, sigma=0.2):
    return synth.ffn_inputs(T, D, F, sigma, seed)


def test_matmul_f64_small_integers_by_hand():
    a = np.array([[1, 2], [3, 4]], dtype=np.float32)
    b = np.array([[5, 6], [7, 8]], dtype=np.float32)
    assert np.array_equal(oracle.matmul_f64(a, b), np.array([[19, 22], [43, 50]], dtype=np.float32))


def test_forward_equals_packed_sparse_product():
    """Pruned-dense x dense equals the product evaluated from the packed storage:
    y1 from (vals, meta) of W1, y3 from (vals, meta, colidx) of y2 with gathered rows of W2^T."""
    X, W1, W2, dY = _inputs()
    V, M = 16, 8
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M)
    T, D = X.shape
    F = W1.shape[0]
    Xf = bf16_to_f32(X).astype(np.float64)
    # y1[t, f] = sum over groups of the two kept values times the X entries at their positions
    vals = bf16_to_f32(fwd.w1s.vals).astype(np.float64).reshape(F, D // 4, 2)
    pos = fwd.w1s.pos.astype(np.int64)
    y1 = np.zeros((T, F))
    for f in range(F):
        cols = (np.arange(D // 4)[:, None] * 4 + pos[f]).reshape(-1)          # kept columns of row f
        y1[:, f] = Xf[:, cols] @ vals[f].reshape(-1)
    assert np.array_equal(f32_to_bf16(y1.astype(np.float32)).reshape(T, F), fwd.y1b)
    # y3 from the condensed V:N:M storage
    G = F // M
    W2t = bf16_to_f32(W2).astype(np.float64).T                                   # [F, D]
    av = bf16_to_f32(fwd.act.vals).astype(np.float64).reshape(T, G, 2)
    y3 = np.zeros((T, D))
    for t in range(T):
        b = t // V
        for g in range(G):
            nib = (int(fwd.act.meta[t, g // 4]) >> (4 * (g % 4))) & 0xF
            for k, p in enumerate((nib & 3, nib >> 2)):
                feat = g * M + int(fwd.act.colidx[b, g, p])
                y3[t] += av[t, g, k] * W2t[feat]
    assert _rel(y3.astype(np.float32), fwd.y3) < 1e-6


def test_dense_mode_matches_numpy_and_finite_differences():
    X, W1, W2, dY = _inputs(T=8, D=16, F=16, seed=3, sigma=0.3)
    fwd = oracle.dense_ffn_fwd(X, W1, W2)
    Xd, W1d, W2d, dYd = (bf16_to_f32(a).astype(np.float64) for a in (X, W1, W2, dY))
    y1 = Xd @ W1d.T
    assert np.array_equal(f32_to_bf16(y1.astype(np.float32)).reshape(y1.shape), fwd.y1b)

    # finite differences in float64 on the un-rounded function L = sum(dY * y3)
    def loss(Xd, W1d, W2d):
        y1 = Xd @ W1d.T
        return float((dYd * ((np.maximum(y1, 0) ** 2) @ W2d.T)).sum())

    def fd(which, i, j, h=1e-5):
        args = [Xd.copy(), W1d.copy(), W2d.copy()]
        args[which][i, j] += h
        up = loss(*args)
        args[which][i, j] -= 2 * h
        return (up - loss(*args)) / (2 * h)

    # analytic gradients per Eqs. 4-8 in float64 (no bf16 rounding) agree with finite differences
    dy2 = dYd @ W2d
    dy1 = 2 * dy2 * np.maximum(y1, 0)
    gX, gW1, gW2 = dy1 @ W1d, dy1.T @ Xd, dYd.T @ (np.maximum(y1, 0) ** 2)
    for (i, j) in [(0, 0), (3, 5), (7, 15)]:
        assert abs(fd(0, i, j) - gX[i, j]) < 1e-5 * max(1, abs(gX[i, j]))
        assert abs(fd(1, i, j) - gW1[i, j]) < 1e-5 * max(1, abs(gW1[i, j]))
        assert abs(fd(2, i, j) - gW2[i, j]) < 1e-5 * max(1, abs(gW2[i, j]))
    # and the oracle (with its bf16 rounding points) sits within bf16 accuracy of them
    bwd = oracle.dense_ffn_bwd(dY, X, W1, W2, fwd)
    assert _rel(bwd.dX, gX) < 1e-2 and _rel(bwd.dW1, gW1) < 1e-2 and _rel(bwd.dW2, gW2) < 1e-2
    assert _rel(fwd.y3, (np.maximum(y1, 0) ** 2) @ W2d.T) < 1e-2


def test_all_ones_masks_reduce_to_dense_mode():
    X, W1, W2, dY = _inputs(T=32, D=32, F=64, seed=5)
    sf = oracle.sparse_ffn_fwd(X, W1, W2, V=16, M=8, _all_ones_masks=True)
    sb = oracle.sparse_ffn_bwd(dY, X, W1, W2, sf, _all_ones_masks=True)
    df = oracle.dense_ffn_fwd(X, W1, W2)
    db = oracle.dense_ffn_bwd(dY, X, W1, W2, df)
    assert np.array_equal(sf.y1b, df.y1b) and np.array_equal(sf.y3, df.y3)
    assert np.array_equal(sb.dX, db.dX) and np.array_equal(sb.dW1, db.dW1) and np.array_equal(sb.dW2, db.dW2)


def test_sparse_backward_follows_algorithm2_operand_colouring():
    X, W1, W2, dY = _inputs(T=32, D=32, F=64, seed=7)
    V, M = 16, 8
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M)
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd)
    Xd, W1d, W2d, dYd = (bf16_to_f32(a).astype(np.float64) for a in (X, W1, W2, dY))
    mask = fwd.act.mask
    # dy2 uses W2 pruned along d_model (groups of four consecutive rows of W2 [D, F])
    W2s = bf16_to_f32(bwd.w2s.dense).astype(np.float64)
    nz = (W2s != 0).reshape(W2.shape[0] // 4, 4, W2.shape[1]).sum(axis=1)
    assert nz.max() <= 2
    assert _rel(bwd.dy2, dYd @ W2s) < 1e-6
    # dy1 lives on y2's mask only, with the factor 2 ReLU(y1)
    relu = np.maximum(bf16_to_f32(fwd.y1b).astype(np.float64), 0)
    expect = np.where(mask, 2 * bwd.dy2.astype(np.float64) * relu, 0)
    assert not bwd.dy1_dense[~mask].any()
    assert _rel(bf16_to_f32(bwd.dy1_dense), expect) < 4e-3
    dy1m = bf16_to_f32(bwd.dy1_dense).astype(np.float64)
    # dX uses the DENSE W1; dW1, dW2 are dense-shaped gradients of the master weights
    assert _rel(bwd.dX, dy1m @ W1d) < 1e-6
    assert _rel(bwd.dX, dy1m @ bf16_to_f32(fwd.w1s.dense).astype(np.float64)) > 1e-3
    assert _rel(bwd.dW1, dy1m.T @ Xd) < 1e-6
    y2m = bf16_to_f32(fwd.act.dense).astype(np.float64)
    assert _rel(bwd.dW2, dYd.T @ y2m) < 1e-6
    # packed dy1 shares y2's metadata
    assert np.array_equal(oracle.decompress_vnm(bwd.dy1_vals, fwd.act.meta, fwd.act.colidx, V, M), bwd.dy1_dense)


def test_dw2_is_true_gradient_of_masked_forward():
    X, W1, W2, dY = _inputs(T=16, D=16, F=32, seed=9, sigma=0.3)
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=8, M=8)
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd)
    y2m = bf16_to_f32(fwd.act.dense).astype(np.float64)
    dYd, W2d = bf16_to_f32(dY).astype(np.float64), bf16_to_f32(W2).astype(np.float64)

    def loss(W2d):
        return float((dYd * (y2m @ W2d.T)).sum())

    for (i, j) in [(0, 0), (5, 17), (15, 31)]:
        h = 1e-4
        Wp, Wm = W2d.copy(), W2d.copy()
        Wp[i, j] += h
        Wm[i, j] -= h
        g = (loss(Wp) - loss(Wm)) / (2 * h)
        assert abs(g - bwd.dW2[i, j]) < 1e-4 * max(1.0, abs(g))


def test_soft_threshold_mode_uses_shrunk_weights():
    X, W1, W2, dY = _inputs(T=32, D=32, F=64, seed=11)
    hard = oracle.sparse_ffn_fwd(X, W1, W2, V=16, M=8, prune_mode=0)
    soft = oracle.sparse_ffn_fwd(X, W1, W2, V=16, M=8, prune_mode=1)
    assert np.array_equal(hard.w1s.meta, soft.w1s.meta)
    W1soft = bf16_to_f32(oracle.prune24(W1, 1, 1).dense).astype(np.float64)
    y1 = bf16_to_f32(X).astype(np.float64) @ W1soft.T
    assert np.array_equal(f32_to_bf16(y1.astype(np.float32)).reshape(y1.shape), soft.y1b)
    assert not np.array_equal(hard.y1b, soft.y1b)


def test_teacher_forced_y1b_is_used():
    X, W1, W2, dY = _inputs(T=32, D=32, F=64, seed=13)
    free = oracle.sparse_ffn_fwd(X, W1, W2, V=16, M=8)
    y1b = free.y1b.copy()
    y1b[0, 0] ^= 1                                            # one-ulp perturbation
    forced = oracle.sparse_ffn_fwd(X, W1, W2, V=16, M=8, forced_y1b=y1b)
    assert np.array_equal(forced.y1b, y1b)
