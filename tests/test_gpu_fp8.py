"""Parity of the E4M3 path with the oracle: the quantiser on every bf16 pattern, pruning with quantisation in
one pass (bit-exact), and the dense / 2:4 tensor-core products on codes (the oracle's packed operands go in,
so a metadata-order mistake cannot hide behind the GPU's own packer)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import fp8
from paper_2602_06183_b200 import binding, synth
from util import to_dev, bits, f32, rel_fro, assert_close_elementwise, Guarded

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _u8(t):
    return t.detach().contiguous().cpu().numpy()


def _dev8(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("scale", [1.0, 0.37, 64.0, 2.0 ** -9, 3.0e38, 448.0])
def test_quantize_every_bf16_pattern(scale):
    x = np.arange(65536, dtype=np.uint16).reshape(256, 256)
    got = _u8(binding.sf_fp8_quantize(to_dev(x), scale))
    ref = fp8.quantize_fp8(x, scale)
    nan = np.isnan(oracle.bf16_to_f32(x))
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.all((got[nan] & 0x7F) == 0x7F)                  # a NaN stays a NaN code; its sign is not specified


def test_quantize_strided_rows_and_guards():
    x = synth.normal_bf16((96, 160), 0, 1, seed=11)
    wide = torch.zeros((96, 200), dtype=torch.bfloat16, device="cuda")
    wide[:, :160] = to_dev(x)
    assert np.array_equal(_u8(binding.sf_fp8_quantize(wide[:, :160], 16.0)), fp8.quantize_fp8(x, 16.0))
    assert binding.sf_fp8_quantize(torch.empty((0, 64), dtype=torch.bfloat16, device="cuda"), 1.0).numel() == 0


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("rows,cols,scale", [(8, 32, 1.0), (130, 96, 24.0), (256, 1024, 300.0), (77, 4096, 0.5)])
def test_prune24_fp8_bit_exact(rows, cols, scale, mode):
    w = synth.prune_sweep_matrix(rows, cols, seed=rows + cols + mode, tie_frac=0.15)
    ref = fp8.prune24_fp8(w, scale, mode=mode)
    vals, meta, dense = binding.sf_prune24_compress_fp8(to_dev(w), mode, scale, want_dense=True)
    torch.cuda.synchronize()
    assert np.array_equal(bits(meta), ref.meta)
    assert np.array_equal(_u8(vals), ref.vals)
    assert np.array_equal(_u8(dense), ref.dense)
    # strided source, no dense copy
    wide = torch.zeros((rows, cols + 24), dtype=torch.bfloat16, device="cuda")
    wide[:, :cols] = to_dev(w)
    vals2, meta2, none = binding.sf_prune24_compress_fp8(wide[:, :cols], mode, scale)
    assert none is None and torch.equal(vals2, vals) and torch.equal(meta2, meta)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("rows,cols,scale", [(16, 8, 1.0), (128, 64, 30.0), (400, 136, 500.0), (1024, 512, 2.0), (272, 1000, 64.0)])
def test_prune24_fp8_strided_groups_bit_exact(rows, cols, scale, mode):
    """Groups along a column, outputs K-major (the W2 direction): ragged panels, strided source."""
    w = synth.prune_sweep_matrix(rows, cols, seed=3 * rows + cols + mode, tie_frac=0.15)
    ref = fp8.prune24_fp8(w, scale, mode=mode, group_dim=0)
    wide = torch.zeros((rows, cols + 16), dtype=torch.bfloat16, device="cuda")
    wide[:, :cols] = to_dev(w)
    for src in (to_dev(w), wide[:, :cols]):
        vals, meta, none = binding.sf_prune24_compress_fp8(src, mode, scale, group_dim=0)
        torch.cuda.synchronize()
        assert none is None
        assert np.array_equal(bits(meta), ref.meta)
        assert np.array_equal(_u8(vals), ref.vals)
    with pytest.raises(binding.SparseFFNError):
        binding.sf_prune24_compress_fp8(to_dev(w), mode, scale, want_dense=True, group_dim=0)


def test_prune24_fp8_saturates_and_keeps_signed_zero():
    w = synth.f32_to_bf16_bits(np.array([[1000.0, -2000.0, 1.0, 2.0, -0.0, 0.0, -1e-30, 1e-30] * 4], dtype=np.float32))
    ref = fp8.prune24_fp8(w.reshape(1, 32), 1.0)
    vals, meta, dense = binding.sf_prune24_compress_fp8(to_dev(w.reshape(1, 32)), 0, 1.0, want_dense=True)
    assert np.array_equal(_u8(vals), ref.vals) and np.array_equal(bits(meta), ref.meta) and np.array_equal(_u8(dense), ref.dense)


def _codes(shape, seed, lim=0x60):
    """Random finite E4M3 codes with magnitudes below 2^5 (code < lim) and random signs."""
    rng = np.random.default_rng(seed)
    return (rng.integers(0, lim, size=shape).astype(np.uint8) | (rng.integers(0, 2, size=shape).astype(np.uint8) << 7))


@pytest.mark.parametrize("M,N,K", [(256, 256, 128), (512, 768, 1152), (256, 512, 4096)])
def test_dense_fp8_gemm(M, N, K):
    A, B = _codes((M, K), 1 + K), _codes((N, K), 2 + K)
    out = Guarded((M, N), torch.bfloat16)
    C, ws = binding.sf_gemm_fp8_dense(_dev8(A), _dev8(B), 2.0 ** -6, C_out=out.t)
    assert binding.sf_check_status(ws) == binding.SF_OK
    out.check("fp8 dense product")
    ref = fp8.gemm_fp8(A, B, 2.0 ** -6)
    assert rel_fro(f32(C), ref) < TOL
    assert_close_elementwise(f32(C), ref, K, "fp8 dense product")


def test_fp8_gemms_exact_on_small_integers():
    # codes of small integers and halves: every product and partial sum is exact in float32
    rng = np.random.default_rng(5)
    table = fp8.f32_to_e4m3(np.array([-3, -2, -1, -0.5, 0, 0.5, 1, 2, 3], dtype=np.float32))
    A = table[rng.integers(0, 9, size=(256, 512))]
    B = table[rng.integers(0, 9, size=(256, 512))]
    C, ws = binding.sf_gemm_fp8_dense(_dev8(A), _dev8(B), 0.25)
    assert np.array_equal(bits(C), fp8.gemm_fp8_bf16(A, B, 0.25))          # exact sum, one rounding to bf16
    # the same through the 2:4 route: prune A's decoded values, keep the codes
    w = oracle.f32_to_bf16(fp8.e4m3_to_f32(A)).reshape(A.shape)
    p = fp8.prune24_fp8(w, 1.0)
    Cs, ws = binding.sf_gemm_fp8_sparse24(_dev8(p.vals), torch.from_numpy(p.meta.view(np.int16)).cuda(), _dev8(B), 0.25)
    assert binding.sf_check_status(ws) == binding.SF_OK
    assert np.array_equal(bits(Cs), fp8.gemm_fp8_bf16(p.dense, B, 0.25))


@pytest.mark.parametrize("M,N,K", [(256, 256, 256), (512, 768, 1280), (768, 256, 4096), (1024, 1024, 2048)])
def test_sparse24_fp8_gemm_against_oracle_packing(M, N, K):
    w = synth.prune_sweep_matrix(M, K, seed=M + K, tie_frac=0.1)
    p = fp8.prune24_fp8(w, 2000.0)                             # weights ~ N(0, 0.02): codes of O(10)
    B = _codes((N, K), 9 + N)
    out = Guarded((M, N), torch.bfloat16)
    C, ws = binding.sf_gemm_fp8_sparse24(_dev8(p.vals), torch.from_numpy(p.meta.view(np.int16)).cuda(), _dev8(B),
                                         2.0 ** -8, C_out=out.t)
    assert binding.sf_check_status(ws) == binding.SF_OK
    out.check("fp8 2:4 product")
    ref = fp8.gemm_fp8(p.dense, B, 2.0 ** -8)
    assert rel_fro(f32(C), ref) < TOL
    assert_close_elementwise(f32(C), ref, K, "fp8 2:4 product")


def test_sparse24_fp8_metadata_probe_one_hot():
    """One stored value per row at a time, B = identity: the output row shows where the tensor core put it.
    Every (row mod 128, 16-column word) position class of the metadata order is visited."""
    M, N, K = 256, 256, 256
    rng = np.random.default_rng(3)
    pos = np.sort(np.stack([rng.permutation(4)[:2] for _ in range(M * K // 4)]), axis=1).reshape(M, K // 4, 2)
    nib = (pos[..., 0] | (pos[..., 1] << 2)).astype(np.uint16).reshape(M, K // 16, 4)
    meta = (nib[..., 0] | (nib[..., 1] << 4) | (nib[..., 2] << 8) | (nib[..., 3] << 12)).astype(np.uint16)
    vals = np.tile(np.array([0x38, 0x40], dtype=np.uint8), (M, K // 4))           # slot 0 = 1.0, slot 1 = 2.0
    eye = np.zeros((N, K), dtype=np.uint8)
    eye[np.arange(N), np.arange(K)] = 0x38
    C, ws = binding.sf_gemm_fp8_sparse24(_dev8(vals), torch.from_numpy(meta.view(np.int16)).cuda(), _dev8(eye), 1.0)
    want = np.zeros((M, K // 4, 4), dtype=np.float32)
    np.put_along_axis(want, pos[..., 0:1].astype(np.int64), 1.0, axis=-1)
    np.put_along_axis(want, pos[..., 1:2].astype(np.int64), 2.0, axis=-1)
    assert np.array_equal(f32(C), want.reshape(M, K))


def test_fp8_pipeline_prune_quantise_multiply():
    """The whole route on the GPU's own packer: W pruned and quantised in one pass, X quantised, product
    compared with the oracle run on the same bf16 inputs."""
    M, N, K = 512, 512, 1024
    w = synth.prune_sweep_matrix(M, K, seed=21, tie_frac=0.05)
    x = synth.normal_bf16((N, K), 0, 1, seed=22)
    sw, sx = 4000.0, 32.0
    vals, meta, _ = binding.sf_prune24_compress_fp8(to_dev(w), 0, sw)
    xq = binding.sf_fp8_quantize(to_dev(x), sx)
    alpha = 1.0 / (sw * sx)
    C, ws = binding.sf_gemm_fp8_sparse24(vals, meta, xq, alpha)
    assert binding.sf_check_status(ws) == binding.SF_OK
    p = fp8.prune24_fp8(w, sw)
    ref = fp8.gemm_fp8(p.dense, fp8.quantize_fp8(x, sx), alpha)
    assert rel_fro(f32(C), ref) < TOL
    assert_close_elementwise(f32(C), ref, K, "fp8 pipeline")
    # and the quantised product tracks the bf16 one to fp8 accuracy (two 2^-4 relative roundings per term)
    exact = oracle.bf16_to_f32(oracle.prune24(w, 1, 0).dense).astype(np.float64) @ oracle.bf16_to_f32(x).astype(np.float64).T
    assert rel_fro(f32(C), exact) < 0.06


def test_fp8_argument_checks():
    a = torch.zeros((256, 128), dtype=torch.uint8, device="cuda")
    m = torch.zeros((256, 16), dtype=torch.int16, device="cuda")
    b = torch.zeros((256, 256), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.SparseFFNError):
        binding.sf_gemm_fp8_sparse24(a[:128], m[:128], b, 1.0)                # Mr % 256
    with pytest.raises(binding.SparseFFNError):
        binding.sf_gemm_fp8_dense(a, b[:, :128].contiguous()[:100], 1.0)      # Nc % 256
    with pytest.raises(binding.SparseFFNError):
        binding.sf_prune24_compress_fp8(torch.zeros((4, 48), dtype=torch.bfloat16, device="cuda"), 0, 1.0)   # cols % 32
    with pytest.raises(binding.SparseFFNError):
        binding.sf_prune24_compress_fp8(torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda"), 2, 1.0)   # mode
