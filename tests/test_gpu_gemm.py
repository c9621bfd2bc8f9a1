"""Parity of the tensor-core products (dense, 2:4-sparse, Venom-gathered) with float64 products of
the oracle's masked matrices. Inputs to the sparse kernels are the ORACLE's packed operands, so a
metadata-layout or gather mistake in the kernel cannot hide behind the GPU's own packer."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06183_b200 import binding, synth
from util import to_dev, bits, f32, rel_fro, assert_close_elementwise, Guarded

pytestmark = pytest.mark.gpu
TOL = 1e-2      # relative Frobenius error, bf16 outputs vs float64-accumulated reference


def _f64(b):
    return oracle.bf16_to_f32(b).astype(np.float64)


@pytest.mark.parametrize("a_k,b_k", [(True, True), (True, False), (False, True), (False, False)])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (384, 512, 448), (256, 256, 128), (512, 768, 1024)])
def test_dense_gemm_layouts(a_k, b_k, M, N, K):
    A = synth.normal_bf16((M, K) if a_k else (K, M), 0, 1, seed=1, stream=M + K)
    B = synth.normal_bf16((N, K) if b_k else (K, N), 0, 1, seed=2, stream=N + K)
    C, ws = binding.sf_gemm_dense(to_dev(A), a_k, to_dev(B), b_k)
    assert binding.sf_check_status(ws) == binding.SF_OK
    Af = _f64(A) if a_k else _f64(A).T
    Bf = _f64(B) if b_k else _f64(B).T
    assert rel_fro(f32(C), Af @ Bf.T) < TOL
    assert_close_elementwise(f32(C), Af @ Bf.T, K, "dense product")


def test_dense_gemm_exact_small_integers():
    # integer data: every product and partial sum is exact, so the result must match exactly
    rng = np.random.default_rng(0)
    A = synth.f32_to_bf16_bits(rng.integers(-3, 4, size=(128, 128)).astype(np.float32))
    B = synth.f32_to_bf16_bits(rng.integers(-3, 4, size=(256, 128)).astype(np.float32))
    C, ws = binding.sf_gemm_dense(to_dev(A), True, to_dev(B), True)
    assert binding.sf_check_status(ws) == binding.SF_OK
    assert np.array_equal(f32(C), (_f64(A) @ _f64(B).T).astype(np.float32))


@pytest.mark.parametrize("Mr,Nc,K", [(128, 256, 128), (256, 512, 640), (384, 256, 1024), (1024, 768, 2048)])
def test_sparse24_gemm_against_oracle_packing(Mr, Nc, K):
    W = synth.prune_sweep_matrix(Mr, K, seed=Mr + K, tie_frac=0.1)
    W = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(W) * 50.0)       # O(1) magnitudes
    X = synth.normal_bf16((Nc, K), 0, 1, seed=3, stream=K)
    p = oracle.prune24(W, group_dim=1, mode=0)
    meta = torch.from_numpy(p.meta.view(np.int16)).cuda()
    Ct, ws = binding.sf_gemm_sparse24(to_dev(p.vals), meta, to_dev(X))
    assert binding.sf_check_status(ws) == binding.SF_OK
    ref = _f64(X) @ _f64(p.dense).T                                     # [Nc, Mr] = X W_s^T
    assert Ct.shape == (Nc, Mr)
    assert rel_fro(f32(Ct), ref) < TOL
    assert_close_elementwise(f32(Ct), ref, K, "2:4 product")


@pytest.mark.parametrize("b_k", [True, False])
@pytest.mark.parametrize("Mr,Nc,K", [(256, 256, 128), (512, 768, 1152)])
def test_sparse24_gemm_row_major_output(b_k, Mr, Nc, K):
    W = synth.prune_sweep_matrix(Mr, K, seed=Mr + K + 1, tie_frac=0.1)
    W = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(W) * 50.0)
    B = synth.normal_bf16((Nc, K) if b_k else (K, Nc), 0, 1, seed=4, stream=K)
    p = oracle.prune24(W, group_dim=1, mode=0)
    meta = torch.from_numpy(p.meta.view(np.int16)).cuda()
    C, ws = binding.sf_gemm_sparse24_rm(to_dev(p.vals), meta, to_dev(B), b_k)
    assert binding.sf_check_status(ws) == binding.SF_OK
    Bf = _f64(B) if b_k else _f64(B).T
    assert rel_fro(f32(C), _f64(p.dense) @ Bf.T) < TOL
    assert_close_elementwise(f32(C), _f64(p.dense) @ Bf.T, K, "2:4 product, row-major output")


def test_sparse24_gemm_one_hot_metadata_probe():
    """Each kept value is a distinct power of two in an otherwise zero row and B is an identity
    slice, so the output says which K position every stored value was multiplied with."""
    Mr, Nc, K = 128, 256, 128
    rng = np.random.default_rng(5)
    W = np.zeros((Mr, K), dtype=np.float32)
    for r in range(Mr):
        for g in range(K // 4):
            pos = sorted(rng.choice(4, size=2, replace=False))
            W[r, 4 * g + pos[0]] = 1.0 + (g % 7)
            W[r, 4 * g + pos[1]] = -(1.0 + (g % 5))
    Wb = synth.f32_to_bf16_bits(W)
    p = oracle.prune24(Wb, 1, 0)
    assert np.array_equal(p.dense, Wb)
    X = np.zeros((Nc, K), dtype=np.float32)
    X[np.arange(K), np.arange(K)] = 1.0                                  # first K rows: identity
    Ct, ws = binding.sf_gemm_sparse24(to_dev(p.vals), torch.from_numpy(p.meta.view(np.int16)).cuda(),
                                      to_dev(synth.f32_to_bf16_bits(X)))
    assert binding.sf_check_status(ws) == binding.SF_OK
    got = f32(Ct)                                                        # [Nc, Mr]; rows < K give W^T
    assert np.array_equal(got[:K].T, W)
    assert not got[K:].any()


@pytest.mark.parametrize("T,F,Nc,V,M", [(128, 256, 256, 128, 8), (256, 1024, 512, 128, 8), (256, 512, 256, 64, 8),
                                        (128, 1024, 256, 128, 16), (128, 512, 256, 64, 4),
                                        # Table 5's group widths: 93.75 % and 96.875 % sparse
                                        (256, 2048, 512, 128, 32), (256, 2048, 256, 64, 32),
                                        (256, 4096, 512, 128, 64), (128, 4096, 256, 64, 64), (384, 2048, 768, 128, 64)])
def test_venom_gemm_against_oracle_packing(T, F, Nc, V, M):
    P = synth.normal_bf16((T, F), 0.2, 1.0, seed=T + F + M)
    Bt = synth.normal_bf16((F, Nc), 0, 1, seed=7, stream=F)
    a = oracle.vnm_sparsify(P, V=V, M=M)
    meta = torch.from_numpy(a.meta.view(np.int16)).cuda()
    colidx = torch.from_numpy(a.colidx).cuda()
    out = Guarded((T, Nc), torch.bfloat16)
    C, ws = binding.sf_gemm_venom(to_dev(a.vals), meta, colidx, to_dev(Bt), V, M, C_out=out.t)
    assert binding.sf_check_status(ws) == binding.SF_OK
    out.check("Venom product output")
    ref = _f64(a.dense) @ _f64(Bt)
    assert rel_fro(f32(C), ref) < TOL
    assert_close_elementwise(f32(C), ref, 4 * F // M, "Venom product")


def test_gemm_shape_errors():
    A = torch.zeros((100, 64), dtype=torch.bfloat16, device="cuda")
    B = torch.zeros((256, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SparseFFNError) as e:
        binding.sf_gemm_dense(A, True, B, True)
    assert e.value.status == binding.SF_ERR_SHAPE


def test_bounded_wait_runs_out_and_is_reported():
    """A wait on a barrier that nothing completes gives up after its clock budget, the kernel sets
    the status word and returns; the host reads SF_ERR_TIMEOUT once, then SF_OK again, and the
    context keeps working."""
    ws = torch.zeros((256,), dtype=torch.uint8, device="cuda")
    assert binding.sf_check_status(ws) == binding.SF_OK
    binding.sf_selftest_wait_expiry(ws, budget_clocks=1_000_000)
    assert binding.sf_check_status(ws) == binding.SF_ERR_TIMEOUT
    assert binding.sf_check_status(ws) == binding.SF_OK              # reported once, then cleared
    A = synth.normal_bf16((128, 64), 0, 1, seed=1)
    B = synth.normal_bf16((256, 64), 0, 1, seed=2)
    Cm, ws2 = binding.sf_gemm_dense(to_dev(A), True, to_dev(B), True)
    assert binding.sf_check_status(ws2) == binding.SF_OK
    assert rel_fro(f32(Cm), _f64(A) @ _f64(B).T) < TOL
