"""Pins for the oracle's neuron-level router (Section 3.1, Algorithm 3, Figure 4)."""
import os

import numpy as np
import pytest

import oracle
from oracle import router as R
from oracle import bf16_to_f32, f32_to_bf16
from paper_2602_06183_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x):
    return f32_to_bf16(np.asarray(x, dtype=np.float32))


def _inputs(T, D, F, E, seed):
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, 0.05, seed)
    means = synth.normal_bf16((E, D), 0.0, 1.0, seed, 9)
    return X, W1, W2, dY, means


def test_clustering_recovers_planted_balanced_clusters():
    """Rows drawn tightly around E well-separated centres, in shuffled order: every cluster must come
    back whole, each expert gets exactly F / E features, and the means are the cluster centroids."""
    rng = np.random.default_rng(0)
    E, cap, D = 4, 24, 16
    centres = rng.integers(-4, 5, size=(E, D)).astype(np.float32) * 8.0
    label = rng.permutation(np.repeat(np.arange(E), cap))
    W = centres[label] + rng.integers(-1, 2, size=(E * cap, D)).astype(np.float32)
    assign, means = R.fit_experts(_bits(W), E)
    assert sorted(np.bincount(assign, minlength=E)) == [cap] * E                 # a balanced partition
    for e in range(E):                                                           # planted clusters stay whole
        assert len(set(label[assign == e])) == 1
    for e in range(E):
        centroid = W[assign == e].astype(np.float64).mean(axis=0)
        assert np.array_equal(means[e], _bits(centroid.astype(np.float32)))


def test_clustering_is_a_balanced_partition_on_unstructured_weights():
    W1 = synth.normal_bf16((256, 32), 0.0, 0.02, seed=3)
    for E in (2, 4, 16):
        assign, means = R.fit_experts(W1, E, iters=4)
        assert assign.shape == (256,) and means.shape == (E, 32)
        assert np.array_equal(np.bincount(assign, minlength=E), np.full(E, 256 // E))
        perm = R.expert_major_permutation(assign)
        assert sorted(perm) == list(range(256))                                   # a permutation
        assert np.array_equal(assign[perm], np.repeat(np.arange(E), 256 // E))    # expert-major, contiguous blocks


def test_hidden_unit_permutation_leaves_the_ffn_unchanged():
    """Renumbering the hidden features (rows of W1 with the matching columns of W2) is a
    reparametrisation: the dense layer computes the same function, so storing the features
    expert-major costs nothing."""
    X, W1, W2, dY = synth.ffn_inputs(32, 16, 64, 0.1, seed=5)
    perm = np.random.default_rng(1).permutation(64)
    a = oracle.dense_ffn_fwd(X, W1, W2)
    b = oracle.dense_ffn_fwd(X, W1[perm], np.ascontiguousarray(W2[:, perm]))
    assert np.array_equal(a.y1b[:, perm], b.y1b)
    np.testing.assert_allclose(a.y3, b.y3, rtol=1e-6, atol=1e-6)


def test_routing_is_the_largest_dot_product_with_ties_to_the_lower_expert():
    rng = np.random.default_rng(2)
    X = rng.integers(-3, 4, size=(64, 8)).astype(np.float32)
    means = rng.integers(-3, 4, size=(4, 8)).astype(np.float32)
    means[2] = means[1]                                       # an exact duplicate: expert 2 can never win over 1
    expert, logits = R.route(_bits(X), _bits(means))
    for t in range(64):
        best = max(range(4), key=lambda e: (float(X[t] @ means[e]), -e))          # brute force, exact integers
        assert expert[t] == best
        assert logits[t, expert[t]] == max(logits[t])
    assert not (expert == 2).any()


@pytest.mark.parametrize("E", [2, 4, 8, 16])
def test_routed_activation_is_vnm_with_m_equal_4e(E):
    """A token keeps two of every four features of ONE expert's block: density 2 / (4 E), Table 5's
    sparsities for M = 16, 32, 64; grouped by expert and interleaved, the matrix obeys the V:N:M
    structure of Section 2.3 with the expert's four columns kept in every group."""
    T, D, F, V = 96, 32, 64 * E, 16
    X, W1, W2, dY, means = _inputs(T, D, F, E, seed=10 + E)
    # strictly positive pre-activations so that every kept slot is non-zero
    fwd = R.routed_ffn_fwd(X, W1, W2, means, E, forced_y1b=_bits(np.abs(bf16_to_f32(
        synth.normal_bf16((T, F // E), 0, 1, seed=E))) + 1.0))
    M = 4 * E
    assert int(fwd.mask.sum()) == T * F * 2 // M
    table = {int(l.split()[2]): float(l.split()[3]) for l in open(os.path.join(GOLDEN, "table5_sparsity.txt"))
             if l.strip() and not l.startswith("#")}
    if M in table:
        assert 100.0 * (1 - fwd.mask.mean()) == table[M]
    block = (np.arange(F)[None, :] // (F // E)) == fwd.expert[:, None]
    assert not (fwd.y2[~block] != 0).any() and not fwd.mask[~block].any()
    dense, colidx = R.vnm_view(fwd, E, V)
    B, G = dense.shape[0] // V, F // M
    nz = ((dense & 0x7FFF) != 0).reshape(B, V, G, M)
    live = nz.any(axis=1)                                                         # [B, G, M]
    assert live.sum(axis=-1).max() <= 4 and nz.sum(axis=-1).max() <= 2
    for b in range(B):                                                            # live columns are the recorded ones
        for g in range(G):
            assert set(np.flatnonzero(live[b, g])) <= set(colidx[b, g])
    assert int(nz.sum()) == T * F * 2 // M                                        # nothing lost by the regrouping


def test_one_expert_is_plain_2to4_activation_sparsity():
    """E = 1: every token keeps two of every four features, which is the V:N:M step with M = 4."""
    X, W1, W2, dY = synth.ffn_inputs(64, 32, 128, 0.1, seed=21)
    means = synth.normal_bf16((1, 32), 0, 1, seed=21, stream=9)
    a = R.routed_ffn_fwd(X, W1, W2, means, 1)
    b = oracle.sparse_ffn_fwd(X, W1, W2, V=16, M=4)
    assert np.array_equal(a.y1b, b.y1b) and np.array_equal(a.mask, b.act.mask) and np.array_equal(a.y2, b.act.dense)
    np.testing.assert_array_equal(a.y3, b.y3)
    ab, bb = R.routed_ffn_bwd(dY, X, W1, W2, a), oracle.sparse_ffn_bwd(dY, X, W1, W2, b)
    assert np.array_equal(ab.dy1, bb.dy1_dense)
    for k in ("dX", "dW1", "dW2"):
        np.testing.assert_array_equal(getattr(ab, k), getattr(bb, k))


def test_grouped_products_equal_the_masked_products():
    """Step 3 of Section 3.1 as written: gather each expert's tokens, multiply them with that expert's
    columns only, scatter back. It must equal the masked dense formulation the oracle evaluates, for
    the forward product and for all three gradients."""
    T, D, F, E = 80, 32, 128, 4
    X, W1, W2, dY, means = _inputs(T, D, F, E, seed=31)
    fwd = R.routed_ffn_fwd(X, W1, W2, means, E)
    bwd = R.routed_ffn_bwd(dY, X, W1, W2, fwd)
    assert len(set(fwd.expert)) > 1
    Fe = F // E
    f64 = lambda b: bf16_to_f32(b).astype(np.float64)
    w2s = oracle.prune24(W2, group_dim=0).dense
    y3 = np.zeros((T, D)); dX = np.zeros((T, D)); dW1 = np.zeros((F, D)); dW2 = np.zeros((D, F))
    for e in range(E):
        t = np.flatnonzero(fwd.expert == e)
        blk = slice(e * Fe, (e + 1) * Fe)
        y1 = f32_to_bf16((f64(X[t]) @ f64(fwd.w1s_dense[blk]).T).astype(np.float32)).reshape(len(t), Fe)
        assert np.array_equal(y1, fwd.y1b[t][:, blk])
        y2 = f64(fwd.y2[t][:, blk])
        y3[t] = y2 @ f64(W2[:, blk]).T
        dy2 = (f64(dY[t]) @ f64(w2s[:, blk])).astype(np.float32)
        dy1 = f32_to_bf16((np.float32(2.0) * dy2 * bf16_to_f32(fwd.relu[t][:, blk])).astype(np.float32)).reshape(len(t), Fe)
        dy1 = np.where(fwd.mask[t][:, blk], dy1, np.uint16(0))
        assert np.array_equal(dy1, bwd.dy1[t][:, blk])
        dX[t] = f64(dy1) @ f64(W1[blk])
        dW1[blk] = f64(dy1).T @ f64(X[t])
        dW2[:, blk] = f64(dY[t]).T @ y2
    np.testing.assert_allclose(y3, fwd.y3, rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(dX, bwd.dX, rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(dW1, bwd.dW1, rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(dW2, bwd.dW2, rtol=1e-6, atol=1e-6)


def test_routed_dw2_is_the_gradient_of_the_forward_product_under_the_frozen_mask():
    T, D, F, E = 24, 16, 32, 2
    X, W1, W2, dY, means = _inputs(T, D, F, E, seed=41)
    fwd = R.routed_ffn_fwd(X, W1, W2, means, E)
    bwd = R.routed_ffn_bwd(dY, X, W1, W2, fwd)
    y2, dYf, W2f = bf16_to_f32(fwd.y2).astype(np.float64), bf16_to_f32(dY).astype(np.float64), bf16_to_f32(W2).astype(np.float64)
    loss = lambda w2: float(((y2 @ w2.T) * dYf).sum())
    rng = np.random.default_rng(0)
    for _ in range(12):
        d, f = int(rng.integers(D)), int(rng.integers(F))
        h = 1e-3
        wp, wm = W2f.copy(), W2f.copy()
        wp[d, f] += h; wm[d, f] -= h
        assert (loss(wp) - loss(wm)) / (2 * h) == pytest.approx(float(bwd.dW2[d, f]), rel=1e-4, abs=1e-5)


def test_token_order_groups_and_pads():
    expert = np.array([1, 0, 1, 1, 0, 2, 1], dtype=np.int32)
    src, start = R.token_order(expert, 3, pad=4)
    assert start.tolist() == [0, 4, 8, 12]
    assert src.tolist() == [1, 4, -1, -1, 0, 2, 3, 6, 5, -1, -1, -1]
