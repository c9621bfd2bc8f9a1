"""Pins for the oracle's 2:4 pruning: brute force, closed form, invariants, round trips."""
import itertools
import os

import numpy as np
import pytest

from oracle import prune24, decompress24, bf16_to_f32, f32_to_bf16
from paper_2602_06183_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x):
    return f32_to_bf16(np.asarray(x, dtype=np.float32))


def _brute_pair(group_f64):
    """Enumerate the six position pairs in lexicographic order; first pair with the largest
    exact magnitude sum wins. This equals 'two largest magnitudes, ties to the lower index'."""
    best, best_pair = None, None
    for pair in itertools.combinations(range(4), 2):
        s = abs(group_f64[pair[0]]) + abs(group_f64[pair[1]])
        if best is None or s > best:
            best, best_pair = s, pair
    return best_pair


def test_exhaustive_alphabet_matches_brute_force():
    alphabet = np.array([0.0, -0.0, 1.0, -1.0, 2.5], dtype=np.float32)
    groups = np.array(list(itertools.product(range(5), repeat=4)))
    w = alphabet[groups]                                     # [625, 4]
    w16 = np.tile(w, (1, 4))                                  # pad K to 16 (four groups per word)
    res = prune24(_bits(w16), group_dim=1, mode=0)
    for r in range(w.shape[0]):
        expect = _brute_pair(w[r].astype(np.float64))
        assert tuple(res.pos[r, 0]) == expect, (w[r], res.pos[r, 0], expect)


def test_random_matches_brute_force_with_ties():
    w = synth.prune_sweep_matrix(64, 256, seed=7, tie_frac=0.3)
    res = prune24(w, group_dim=1, mode=0)
    wf = bf16_to_f32(w).astype(np.float64).reshape(64, 64, 4)
    for r in range(64):
        for g in range(64):
            assert tuple(res.pos[r, g]) == _brute_pair(wf[r, g])


def test_nm_invariant_and_value_preservation():
    w = synth.prune_sweep_matrix(128, 512, seed=3)
    res = prune24(w, group_dim=1, mode=0)
    d = res.dense.reshape(128, 128, 4)
    assert ((d & 0x7FFF) != 0).sum(axis=-1).max() <= 2          # at most two non-zeros per group
    # kept entries are bit-identical to the input, dropped entries are +0
    same = d == w.reshape(128, 128, 4)
    assert np.all(same | (d == 0))
    assert same.sum(axis=-1).min() >= 2
    # retained magnitude is maximal: no dropped element exceeds a kept one
    mag = (w.reshape(128, 128, 4) & 0x7FFF).astype(np.int32)
    kept = np.zeros_like(same)
    np.put_along_axis(kept, res.pos.astype(np.int64), True, axis=-1)
    assert np.all(np.where(kept, mag, 1 << 20).min(axis=-1) >= np.where(kept, -1, mag).max(axis=-1))


def test_metadata_round_trip_and_nibble_format():
    w = synth.prune_sweep_matrix(32, 128, seed=11, tie_frac=0.2)
    for mode in (0, 1):
        res = prune24(w, group_dim=1, mode=mode)
        assert np.array_equal(decompress24(res.vals, res.meta), res.dense)
        nib0 = res.meta[:, 0] & 0xF                               # first group of each row
        assert np.array_equal(nib0 & 3, res.pos[:, 0, 0])
        assert np.array_equal(nib0 >> 2, res.pos[:, 0, 1])
        assert np.all(res.pos[..., 0] < res.pos[..., 1])


def test_hand_packed_example():
    # group (1, -3, 0.5, 2): keep positions 1 and 3 -> nibble 1 | 3<<2 = 13
    row = np.array([[1, -3, 0.5, 2] + [0, 0, 0, 0] + [5, 4, 3, 2] + [0, 7, 0, 7]], dtype=np.float32)
    res = prune24(_bits(row), group_dim=1, mode=0)
    # groups: (1,3) -> 13 ; all-zero -> (0,1) -> 4 ; (0,1) -> 4 ; (1,3) -> 13
    assert int(res.meta[0, 0]) == 13 | (4 << 4) | (4 << 8) | (13 << 12)
    assert np.array_equal(bf16_to_f32(res.vals[0]), np.array([-3, 2, 0, 0, 5, 4, 7, 7], dtype=np.float32))


def test_group_dim0_is_transpose_of_group_dim1():
    w = synth.prune_sweep_matrix(64, 48, seed=5, tie_frac=0.2, axis=0)       # [D=64, F=48]
    a = prune24(w, group_dim=0, mode=0)
    b = prune24(np.ascontiguousarray(w.T), group_dim=1, mode=0)
    assert np.array_equal(a.vals, b.vals) and np.array_equal(a.meta, b.meta)
    assert a.vals.shape == (48, 32)
    assert np.array_equal(a.dense, b.dense.T)
    # structure is along dim 0 of the original
    d = a.dense.reshape(16, 4, 48)
    assert ((d & 0x7FFF) != 0).sum(axis=1).max() <= 2


def test_soft_threshold_golden_cases():
    rows = []
    for line in open(os.path.join(GOLDEN, "soft_threshold_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        lhs, rhs = line.split("|")
        rows.append(([float(x) for x in lhs.split()], [float(x) for x in rhs.split()]))
    for a, fa in rows:
        res = prune24(_bits(np.array([a * 4], dtype=np.float32)), group_dim=1, mode=1)
        got = bf16_to_f32(res.dense[0, :4])
        assert np.array_equal(got, np.array(fa, dtype=np.float32)), (a, got, fa)


def test_soft_threshold_closed_form_random():
    w = synth.prune_sweep_matrix(64, 256, seed=13, tie_frac=0.2)
    res = prune24(w, group_dim=1, mode=1)
    hard = prune24(w, group_dim=1, mode=0)
    assert np.array_equal(res.pos, hard.pos) and np.array_equal(res.meta, hard.meta)
    a = bf16_to_f32(w).astype(np.float64).reshape(64, 64, 4)
    t = np.sort(np.abs(a), axis=-1)[..., 1:2]                        # second smallest magnitude
    f = np.where(a > t, a - t, np.where(a <= -t, a + t, 0.0))        # the paper's piecewise form
    expect = f32_to_bf16(f.astype(np.float32)).reshape(a.shape)
    got = res.dense.reshape(a.shape)
    # identical up to the sign of zero (the closed form can produce -0 only through a + t = 0)
    assert np.array_equal(bf16_to_f32(got), bf16_to_f32(expect))
    # two smallest magnitudes are zero, kept magnitudes shrink by exactly t (where exact in bf16)
    assert ((got & 0x7FFF) != 0).sum(axis=-1).max() <= 2


def test_soft_threshold_is_continuous_across_a_tie():
    # second and third magnitudes swap order: dense outputs must coincide on both sides
    eps = 2.0 ** -8
    lo = np.array([[4.0, 1.0, 1.0 - eps, 0.25] * 4], dtype=np.float32)
    hi = np.array([[4.0, 1.0 - eps, 1.0, 0.25] * 4], dtype=np.float32)
    tie = np.array([[4.0, 1.0, 1.0, 0.25] * 4], dtype=np.float32)
    d_lo = bf16_to_f32(prune24(_bits(lo), mode=1).dense)[0, :4]
    d_hi = bf16_to_f32(prune24(_bits(hi), mode=1).dense)[0, :4]
    d_tie = bf16_to_f32(prune24(_bits(tie), mode=1).dense)[0, :4]
    # 4 - (1 - eps) = 3 + eps rounds to 3 in bf16 (8 significant bits)
    assert np.array_equal(d_lo, np.array([3.0, eps, 0, 0], dtype=np.float32))
    assert np.array_equal(d_hi, np.array([3.0, 0, eps, 0], dtype=np.float32))
    assert np.array_equal(d_tie, np.array([3.0, 0, 0, 0], dtype=np.float32))
    # hard pruning, in contrast, jumps by a full element at the same point
    h_lo = bf16_to_f32(prune24(_bits(lo), mode=0).dense)[0, :4]
    assert h_lo[1] == 1.0


def test_negative_zero_and_sign_handling():
    row = np.array([[-0.0, 0.0, -0.0, 0.0] + [-2.0, -2.0, 2.0, 2.0] + [0.0] * 8], dtype=np.float32)
    res = prune24(_bits(row), mode=0)
    assert tuple(res.pos[0, 0]) == (0, 1) and tuple(res.pos[0, 1]) == (0, 1)
    assert res.vals[0, 0] == 0x8000 and res.vals[0, 1] == 0x0000     # kept bits pass through
