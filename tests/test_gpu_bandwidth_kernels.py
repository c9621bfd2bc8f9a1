"""Bit-exact parity of prune24_compress and vnm_sparsify_act (CUDA, through the C ABI) with the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06183_b200 import binding, synth
from util import to_dev, bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols", [(128, 256), (96, 1040), (1, 16), (513, 4112)])
@pytest.mark.parametrize("mode", [0, 1])
def test_prune24_rows_bit_exact(rows, cols, mode):
    w = synth.prune_sweep_matrix(rows, cols, seed=1000 + rows + mode, tie_frac=0.1)
    ref = oracle.prune24(w, group_dim=1, mode=mode)
    vals, meta, dense = binding.sf_prune24_compress(to_dev(w), 1, mode, want_dense=True)
    torch.cuda.synchronize()
    assert np.array_equal(bits(meta), ref.meta)
    assert np.array_equal(bits(vals), ref.vals)
    assert np.array_equal(bits(dense), ref.dense)


@pytest.mark.parametrize("rows,cols", [(128, 64), (256, 1000), (16, 8), (4112, 520)])
@pytest.mark.parametrize("mode", [0, 1])
def test_prune24_cols_bit_exact(rows, cols, mode):
    w = synth.prune_sweep_matrix(rows, cols, seed=2000 + rows + mode, tie_frac=0.1, axis=0)
    ref = oracle.prune24(w, group_dim=0, mode=mode)
    vals, meta, dense = binding.sf_prune24_compress(to_dev(w), 0, mode, want_dense=True)
    torch.cuda.synchronize()
    assert vals.shape == (cols, rows // 2)
    assert np.array_equal(bits(meta), ref.meta)
    assert np.array_equal(bits(vals), ref.vals)
    assert np.array_equal(bits(dense), ref.dense)


def test_prune24_strided_input_and_special_values():
    w = synth.prune_sweep_matrix(64, 512, seed=5, tie_frac=0.5)
    w[:, :16] = 0                       # all-zero groups
    w[0, 16:32] = 0x8000                # negative zeros
    big = to_dev(np.concatenate([w, w], axis=1))        # ld = 1024, logical cols = 512
    view = big[:, :512]
    ref = oracle.prune24(w, 1, 0)
    vals, meta, _ = binding.sf_prune24_compress(view, 1, 0)
    torch.cuda.synchronize()
    assert np.array_equal(bits(meta), ref.meta) and np.array_equal(bits(vals), ref.vals)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("group_dim", [1, 0])
def test_prune24_special_values_both_modes(group_dim, mode):
    """Infinities, NaNs, subnormals, signed zeros and exact ties in every position of a group, hard and soft:
    the order is the one of the magnitude bit patterns, a NaN that is kept becomes zero under soft-thresholding
    (it is neither above nor below the threshold), an infinite threshold makes NaN of infinite kept values."""
    rng = np.random.default_rng(40 + group_dim + 2 * mode)
    special = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x0080, 0x7F80, 0xFF80, 0x7FC0, 0xFFC0, 0x7F7F, 0xFF7F,
                        0x3F80, 0xBF80, 0x3F81, 0x4000], dtype=np.uint16)
    w = synth.prune_sweep_matrix(128, 256, seed=41, tie_frac=0.3)
    pick = rng.random(w.shape) < 0.35
    w[pick] = special[rng.integers(0, len(special), size=int(pick.sum()))]
    ref = oracle.prune24(w, group_dim, mode)
    vals, meta, dense = binding.sf_prune24_compress(to_dev(w), group_dim, mode, want_dense=True)
    torch.cuda.synchronize()
    assert np.array_equal(bits(meta), ref.meta)

    def same(a, b):                                   # NaN payloads are not part of the contract
        fa, fb = oracle.bf16_to_f32(a), oracle.bf16_to_f32(b)
        return np.array_equal(np.isnan(fa), np.isnan(fb)) and np.array_equal(a[~np.isnan(fa)], b[~np.isnan(fb)])
    assert same(bits(vals), ref.vals)
    assert same(bits(dense), ref.dense)


@pytest.mark.parametrize("T,F,V,M", [(128, 512, 64, 8), (256, 1024, 128, 16), (128, 320, 64, 4),
                                     (64, 256, 32, 32), (128, 256, 64, 64), (192, 832, 64, 8)])
def test_vnm_bit_exact(T, F, V, M):
    p = synth.act_sweep_matrix(T, F, seed=3000 + T + M)
    ref = oracle.vnm_sparsify(p, V=V, M=M)
    vals, meta, colidx, relu, dense = binding.sf_vnm_sparsify_act(to_dev(p), V, M, want_dense=True)
    torch.cuda.synchronize()
    assert np.array_equal(colidx.cpu().numpy(), ref.colidx)
    assert np.array_equal(bits(meta), ref.meta)
    assert np.array_equal(bits(vals), ref.vals)
    assert np.array_equal(bits(relu), ref.relu_vals)
    assert np.array_equal(bits(dense), ref.dense)


@pytest.mark.parametrize("T,F,V,M,apply", [
    (128, 512, 64, 8, True), (256, 1024, 128, 8, True), (192, 832, 64, 8, True),       # ragged last strip (832 = 3 x 256 + 64)
    (96, 1088, 32, 8, False), (256, 1024, 128, 16, True), (128, 1600, 64, 16, True),   # 1600 = 6 x 256 + 64
    (128, 1152, 32, 32, True), (256, 1152, 128, 32, False), (128, 1280, 64, 64, True), (256, 768, 128, 64, True),
    (48, 576, 16, 8, True), (4096, 2048, 64, 8, True)])                                 # many strips per persistent CTA
def test_vnm_streaming_kernel_bit_exact(T, F, V, M, apply):
    """Without a dense copy the call runs the streaming kernel (TMA-fed strip ring, overlapped scoring and
    emitting warps); every output must equal the oracle's bit for bit, also through a strided view."""
    p = synth.act_sweep_matrix(T, F, seed=4000 + T + F + M)
    ref = oracle.vnm_sparsify(p, V=V, M=M, apply_sqrelu=apply)
    wide = torch.zeros((T, F + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :F] = to_dev(p)
    for src in (to_dev(p), wide[:, :F]):
        vals, meta, colidx, relu, dense = binding.sf_vnm_sparsify_act(src, V, M, apply_sqrelu=apply)
        torch.cuda.synchronize()
        assert dense is None
        assert np.array_equal(colidx.cpu().numpy(), ref.colidx)
        assert np.array_equal(bits(meta), ref.meta)
        assert np.array_equal(bits(vals), ref.vals)
        if apply:
            assert np.array_equal(bits(relu), ref.relu_vals)


def test_vnm_no_activation_and_ties():
    # raw magnitudes with many exact ties, negative values, apply_sqrelu = 0
    p = synth.prune_sweep_matrix(128, 512, seed=9, tie_frac=0.5)
    p[:64, :64] = 0
    ref = oracle.vnm_sparsify(p, V=64, M=8, apply_sqrelu=False)
    vals, meta, colidx, relu, dense = binding.sf_vnm_sparsify_act(to_dev(p), 64, 8, apply_sqrelu=False, want_dense=True)
    torch.cuda.synchronize()
    assert relu is None
    assert np.array_equal(colidx.cpu().numpy(), ref.colidx)
    assert np.array_equal(bits(meta), ref.meta) and np.array_equal(bits(vals), ref.vals)
    assert np.array_equal(bits(dense), ref.dense)


def test_vnm_accumulation_order_case():
    y = np.zeros((128, 256), dtype=np.float32)
    y[0, 0] = 2.0 ** 24
    y[1:, 0] = 1.0
    y[0, 1] = 2.0 ** 24
    y[1, 1] = 64.0
    y[:, 2:5] = 2.0 ** 25
    p = synth.f32_to_bf16_bits(y)
    ref = oracle.vnm_sparsify(p, V=128, M=8, apply_sqrelu=False)
    _, _, colidx, _, _ = binding.sf_vnm_sparsify_act(to_dev(p), 128, 8, apply_sqrelu=False)
    assert tuple(colidx.cpu().numpy()[0, 0]) == (1, 2, 3, 4) == tuple(ref.colidx[0, 0])


def test_empty_inputs_are_noops():
    w = torch.empty((0, 256), dtype=torch.bfloat16, device="cuda")
    vals, meta, _ = binding.sf_prune24_compress(w, 1, 0)
    assert vals.numel() == 0 and meta.numel() == 0


def test_vnm_special_values_bit_exact():
    """-0, subnormal squares, overflow to inf, exact ties at zero: packed arithmetic must match."""
    rng = np.random.default_rng(3)
    base = np.array([-0.0, 0.0, 1e-20, 3e-20, 1e-19, 1.5e19, 3e19, 1e-30, 0.5, -0.5, 2.0, 1e-10], dtype=np.float32)
    x = base[rng.integers(0, base.size, size=(128, 512))]
    p = synth.f32_to_bf16_bits(x)
    for V in (64, 128):
        ref = oracle.vnm_sparsify(p, V=V, M=8)
        vals, meta, colidx, relu, dense = binding.sf_vnm_sparsify_act(to_dev(p), V, 8, want_dense=True)
        torch.cuda.synchronize()
        assert np.array_equal(colidx.cpu().numpy(), ref.colidx)
        assert np.array_equal(bits(meta), ref.meta)
        assert np.array_equal(bits(vals), ref.vals)
        assert np.array_equal(bits(relu), ref.relu_vals)
        assert np.array_equal(bits(dense), ref.dense)


def _random_prune_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        group_dim = int(rng.integers(0, 2))
        k = int(rng.integers(1, 40)) * 16                      # reduction length: whole metadata words
        r = int(rng.integers(1, 60)) * 8
        rows, cols = (r, k) if group_dim == 1 else (k, r)
        out.append((rows, cols, group_dim, int(rng.integers(0, 2)), int(rng.integers(0, 3)) * 8, int(rng.integers(1, 1 << 20))))
    return out


@pytest.mark.parametrize("rows,cols,group_dim,mode,pad,seed", _random_prune_shapes(24, seed=20260207))
def test_prune24_random_shapes(rows, cols, group_dim, mode, pad, seed):
    """Seeded draw of legal shapes (ragged panels, single rows, padded leading dimension), both directions and modes."""
    w = synth.prune_sweep_matrix(rows, cols, seed=seed, tie_frac=0.2)
    ref = oracle.prune24(w, group_dim, mode)
    wide = torch.zeros((rows, cols + pad), dtype=torch.bfloat16, device="cuda")
    wide[:, :cols] = to_dev(w)
    vals, meta, dense = binding.sf_prune24_compress(wide[:, :cols], group_dim, mode, want_dense=True)
    torch.cuda.synchronize()
    assert np.array_equal(bits(meta), ref.meta)
    assert np.array_equal(bits(vals), ref.vals)
    assert np.array_equal(bits(dense), ref.dense)
    vals2, meta2, _ = binding.sf_prune24_compress(wide[:, :cols], group_dim, mode)
    assert torch.equal(vals2, vals) and torch.equal(meta2, meta)


def _random_vnm_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        M = int(rng.choice([4, 8, 16, 32, 64]))
        V = int(rng.choice([16, 32, 48, 64, 96, 128]))
        T = V * int(rng.integers(1, 5))
        F = 64 * int(rng.integers(1, 30))
        if F % (4 * M):
            continue
        out.append((T, F, V, M, bool(rng.integers(0, 2)), int(rng.integers(0, 3)) * 8, int(rng.integers(1, 1 << 20))))
    return out


@pytest.mark.parametrize("T,F,V,M,apply,pad,seed", _random_vnm_shapes(24, seed=20260208))
def test_vnm_random_shapes(T, F, V, M, apply, pad, seed):
    """Seeded draw of legal (T, F, V, M): whichever kernel the call picks (streaming or strip-staged) must give the
    oracle's bits, with and without the dense copy, through a strided view."""
    p = synth.act_sweep_matrix(T, F, seed=seed)
    ref = oracle.vnm_sparsify(p, V=V, M=M, apply_sqrelu=apply)
    wide = torch.zeros((T, F + pad), dtype=torch.bfloat16, device="cuda")
    wide[:, :F] = to_dev(p)
    for want_dense in (False, True):
        vals, meta, colidx, relu, dense = binding.sf_vnm_sparsify_act(wide[:, :F], V, M, apply_sqrelu=apply, want_dense=want_dense)
        torch.cuda.synchronize()
        assert np.array_equal(colidx.cpu().numpy(), ref.colidx)
        assert np.array_equal(bits(meta), ref.meta)
        assert np.array_equal(bits(vals), ref.vals)
        if apply:
            assert np.array_equal(bits(relu), ref.relu_vals)
        if want_dense:
            assert np.array_equal(bits(dense), ref.dense)
