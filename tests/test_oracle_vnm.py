"""Pins for the oracle's SquaredReLU + V:N:M sparsification."""
import itertools
import os

import numpy as np
import pytest

from oracle import vnm_sparsify, decompress_vnm, prune24, bf16_to_f32, f32_to_bf16
from paper_2602_06183_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x):
    return f32_to_bf16(np.asarray(x, dtype=np.float32))


def _small_int_block(rng, T, F, zero_frac=0.6, hi=6):
    """Non-negative small integers: every partial sum is exact in float32 and float64."""
    x = rng.integers(0, hi, size=(T, F)).astype(np.float32)
    x[rng.random((T, F)) < zero_frac] = 0
    return x


def test_table5_sparsity_values():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table5_sparsity.txt")) if l.strip() and not l.startswith("#")]
    for V, N, M, pct in rows:
        V, N, M, pct = int(V), int(N), int(M), float(pct)
        T, F = V * 2, M * 8
        x = np.abs(synth.bf16_bits_to_f32(synth.normal_bf16((T, F), 0, 1, seed=M))) + 1.0   # no zeros
        res = vnm_sparsify(_bits(x), V=V, M=M, N=N, apply_sqrelu=False)
        kept = int(res.mask.sum())
        assert kept == T * F * N // M
        assert 100.0 * (1 - kept / (T * F)) == pct
        assert int(((res.dense & 0x7FFF) != 0).sum()) == kept


@pytest.mark.parametrize("V,M", [(64, 8), (128, 16), (64, 4), (32, 32)])
def test_structure_invariants(V, M):
    T, F = V * 3, M * 8
    p = synth.act_sweep_matrix(T, F, seed=V + M)
    res = vnm_sparsify(p, V=V, M=M)
    B, G = T // V, F // M
    nz = ((res.dense & 0x7FFF) != 0).reshape(B, V, G, M)
    assert nz.any(axis=1).sum(axis=-1).max() <= 4            # at most four live columns per block
    assert nz.sum(axis=-1).max() <= 2                        # at most two non-zeros per row of a block
    assert res.mask.reshape(B, V, G, M).sum(axis=-1).min() == 2 == res.mask.reshape(B, V, G, M).sum(axis=-1).max()
    assert np.all(np.diff(res.colidx.astype(int), axis=-1) > 0) and res.colidx.max() < M
    assert np.array_equal(decompress_vnm(res.vals, res.meta, res.colidx, V, M), res.dense)
    # masked values are the activation itself, ReLU values are max(p, 0)
    pf = bf16_to_f32(p)
    h = np.where(pf > 0, pf * pf, 0).astype(np.float32)
    assert np.array_equal(res.hb, f32_to_bf16(h).reshape(T, F))
    assert np.array_equal(np.where(res.mask, res.hb, 0), res.dense)


def test_squared_relu_values():
    p = _bits(np.array([[-2.0, -0.0, 0.0, 0.5, 1.5, 3.0, -1e-3, 256.0] * 4] * 4, dtype=np.float32))
    res = vnm_sparsify(p, V=4, M=8)
    assert np.array_equal(bf16_to_f32(res.hb[0, :8]),
                          np.array([0, 0, 0, 0.25, 2.25, 9.0, 0, 65536.0], dtype=np.float32))
    # ReLU values stored next to the kept activations are the un-squared positives
    assert set(np.unique(bf16_to_f32(res.relu_vals))) <= {0.0, 0.5, 1.5, 3.0, 256.0}
    assert np.array_equal(bf16_to_f32(res.relu_vals) ** 2, bf16_to_f32(res.vals))


def test_column_choice_brute_force_small_integers():
    rng = np.random.default_rng(1)
    V, M = 8, 8
    for trial in range(40):
        x = _small_int_block(rng, V, M * 4)
        res = vnm_sparsify(_bits(x), V=V, M=M, apply_sqrelu=False)
        for g in range(4):
            blk = x[:, g * M:(g + 1) * M].astype(np.float64)
            colmass = blk.sum(axis=0)
            # first subset in lexicographic order among those of maximal retained column mass
            best, best_set = None, None
            for s in itertools.combinations(range(M), 4):
                m = colmass[list(s)].sum()
                if best is None or m > best:
                    best, best_set = m, s
            assert tuple(res.colidx[0, g]) == best_set
            # stage 2 per row: first pair of maximal mass among the four kept columns
            for r in range(V):
                four = blk[r, list(best_set)]
                bp, bpair = None, None
                for pair in itertools.combinations(range(4), 2):
                    m = four[pair[0]] + four[pair[1]]
                    if bp is None or m > bp:
                        bp, bpair = m, pair
                nib = (int(res.meta[r, 0]) >> (4 * g)) & 0xF
                assert (nib & 3, nib >> 2) == bpair


def test_m4_reduces_to_row_wise_2to4():
    p = synth.prune_sweep_matrix(64, 64, seed=21, tie_frac=0.3)
    res = vnm_sparsify(p, V=16, M=4, apply_sqrelu=False)
    ref = prune24(p, group_dim=1, mode=0)
    assert np.array_equal(res.dense, ref.dense)
    assert np.array_equal(res.vals, ref.vals) and np.array_equal(res.meta, ref.meta)
    assert np.all(res.colidx == np.arange(4))


def test_v1_reduces_to_top2_of_m_per_row():
    rng = np.random.default_rng(2)
    M = 8
    x = _small_int_block(rng, 16, M * 4, zero_frac=0.3, hi=50)
    res = vnm_sparsify(_bits(x), V=1, M=M, apply_sqrelu=False)
    for r in range(16):
        for g in range(4):
            seg = x[r, g * M:(g + 1) * M]
            order = sorted(range(M), key=lambda j: (-seg[j], j))[:2]
            kept = np.flatnonzero(res.mask[r, g * M:(g + 1) * M])
            assert sorted(order) == list(kept)


def test_all_zero_block_defaults():
    p = _bits(np.full((8, 32), -1.0, dtype=np.float32))
    res = vnm_sparsify(p, V=8, M=8)
    assert np.all(res.colidx == np.arange(4))
    assert np.all(res.meta == (4 | 4 << 4 | 4 << 8 | 4 << 12))          # positions (0, 1) everywhere
    assert not res.vals.any() and not res.dense.any()


def test_accumulation_order_is_sequential_float32():
    # Column 0 holds 2^24 then 127 ones; column 1 holds 2^24 then one 64.
    V, M = 128, 8
    y = np.zeros((V, 32), dtype=np.float32)
    y[0, 0] = 2.0 ** 24
    y[1:, 0] = 1.0                      # 127 ones: exact sum 2^24 + 127, sequential float32 sum 2^24
    y[0, 1] = 2.0 ** 24
    y[1, 1] = 64.0                      # sequential float32 sum 2^24 + 64
    y[:, 2:5] = 2.0 ** 25
    res = vnm_sparsify(_bits(y), V=V, M=M, apply_sqrelu=False)
    # exact arithmetic would keep column 0 (127 > 64); the declared order keeps column 1
    assert tuple(res.colidx[0, 0]) == (1, 2, 3, 4)


def test_tie_between_columns_goes_to_lower_index():
    x = np.zeros((4, 32), dtype=np.float32)
    x[:, [1, 3, 5, 6, 7]] = 1.0          # five equal columns: the first four of them stay
    res = vnm_sparsify(_bits(x), V=4, M=8, apply_sqrelu=False)
    assert tuple(res.colidx[0, 0]) == (1, 3, 5, 6)
    # zero-score columns fill the remaining slots from the left
    z = np.zeros((4, 32), dtype=np.float32)
    z[:, 6] = 1.0
    res = vnm_sparsify(_bits(z), V=4, M=8, apply_sqrelu=False)
    assert tuple(res.colidx[0, 0]) == (0, 1, 2, 6)
    # within the row the single non-zero sits at position 3 and is kept with position 0
    assert (int(res.meta[0, 0]) & 0xF) == (0 | 3 << 2)


def test_column_score_is_taken_on_the_squared_activation():
    """With the activation on, the block's kept columns are ranked by the sum of h = ReLU(p)^2
    (the stored activation y2 of Eq. 2, the tensor Section 2.3 sparsifies), not by the sum of the
    un-squared ReLU(p). One column with a single 4 (sum 4, sum of squares 16) against columns of
    three 2s (sum 6, sum of squares 12): the squares rank the single-4 column first, the plain
    values would rank it last."""
    V, M = 4, 8
    p = np.full((V, 32), -1.0, dtype=np.float32)
    p[0, 0] = 4.0                         # column 0: sum 4, sum of squares 16
    for c in (1, 2, 3, 4):
        p[0:3, c] = 2.0                   # columns 1-4: sum 6, sum of squares 12
    res = vnm_sparsify(_bits(p), V=V, M=M, apply_sqrelu=True)
    # squares: 16 > 12 = 12 = 12 = 12 -> columns 0, 1, 2, 3 (ties to the lower index)
    assert tuple(res.colidx[0, 0]) == (0, 1, 2, 3)
    # (un-squared sums would give 6, 6, 6, 6 > 4 -> columns 1, 2, 3, 4)
    # row 0 keeps the 16 and the first 4 among the kept columns; the stored values are the squares
    assert (int(res.meta[0, 0]) & 0xF) == (0 | 1 << 2)
    assert bf16_to_f32(res.vals[0, :2]).tolist() == [16.0, 4.0]
    assert bf16_to_f32(res.relu_vals[0, :2]).tolist() == [4.0, 2.0]


def test_column_choice_brute_force_with_the_activation_on():
    """Brute force over all C(M, 4) column subsets and all six row pairs on small signed integers
    with SquaredReLU applied: the retained mass is the mass of max(p, 0)^2 (exact in float32)."""
    rng = np.random.default_rng(11)
    V, M = 8, 8
    for trial in range(40):
        p = rng.integers(-6, 7, size=(V, M * 4)).astype(np.float32)
        res = vnm_sparsify(_bits(p), V=V, M=M, apply_sqrelu=True)
        h = np.where(p > 0, p * p, 0.0).astype(np.float64)
        for g in range(4):
            blk = h[:, g * M:(g + 1) * M]
            colmass = blk.sum(axis=0)
            best, best_set = None, None
            for s in itertools.combinations(range(M), 4):
                m = colmass[list(s)].sum()
                if best is None or m > best:
                    best, best_set = m, s
            assert tuple(res.colidx[0, g]) == best_set
            for r in range(V):
                four = blk[r, list(best_set)]
                bp, bpair = None, None
                for pair in itertools.combinations(range(4), 2):
                    m = four[pair[0]] + four[pair[1]]
                    if bp is None or m > bp:
                        bp, bpair = m, pair
                nib = (int(res.meta[r, 0]) >> (4 * g)) & 0xF
                assert (nib & 3, nib >> 2) == bpair
