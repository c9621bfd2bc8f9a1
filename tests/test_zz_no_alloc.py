"""The no-allocation variant of the 2:4-sparse product against the regular entry point.

Some users of this library cannot allocate device memory at the point where they need the product
(they run inside another framework's allocator callback, or are plugins that only receive input and
output tensors). sf_gemm_sparse24_noalloc serves them from a scratch array built into the library.
This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06183_b200 import binding, synth
from util import to_dev, f32, rel_fro, assert_close_elementwise

pytestmark = pytest.mark.gpu


def _operands(Mr, Nc, K, seed):
    W = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(synth.prune_sweep_matrix(Mr, K, seed=seed, tie_frac=0.1)) * 50.0)
    X = synth.normal_bf16((Nc, K), 0, 1, seed=seed, stream=7)
    p = oracle.prune24(W, group_dim=1, mode=0)
    ref = oracle.bf16_to_f32(X).astype(np.float64) @ oracle.bf16_to_f32(p.dense).astype(np.float64).T   # [Nc, Mr]
    return to_dev(p.vals), torch.from_numpy(p.meta.view(np.int16)).cuda(), to_dev(X), ref


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    # two calls back to back on different shapes: the second must not see the first one's scratch
    for (Mr, Nc, K, seed) in [(384, 512, 1024, 31), (128, 256, 256, 32)]:
        vals, meta, X, oracle_ref = _operands(Mr, Nc, K, seed)
        ref, ws = binding.sf_gemm_sparse24(vals, meta, X)
        assert binding.sf_check_status(ws) == binding.SF_OK
        out = torch.empty((Nc, Mr), dtype=torch.bfloat16, device="cuda")     # caller-owned output
        binding.sf_gemm_sparse24_noalloc(vals, meta, X, out)                   # first call on a device: looks up the array
        torch.cuda.synchronize()
        out.zero_()
        allocs = lambda: torch.cuda.memory_stats().get("allocation.all.allocated", 0)   # cumulative count
        before, free_before = allocs(), torch.cuda.mem_get_info()[0]
        binding.sf_gemm_sparse24_noalloc(vals, meta, X, out)
        torch.cuda.synchronize()
        assert allocs() == before                                              # nothing through torch's allocator
        assert torch.cuda.mem_get_info()[0] == free_before                     # and nothing from the driver either
        assert binding.sf_check_status(None) == binding.SF_OK                  # the built-in status word: no expired wait
        assert torch.cuda.mem_get_info()[0] == free_before
        # against the float64 product of the oracle's pruned matrix, then against the regular entry point
        assert rel_fro(f32(out), oracle_ref) < 1e-2
        assert_close_elementwise(f32(out), oracle_ref, K, "no-allocation 2:4 product")
        assert torch.equal(out, ref)                                           # same kernel, same bits


def test_noalloc_rejects_shapes_beyond_the_builtin_scratch():
    Mr, K, Nc = 8192, 8192, 256            # Mr*K/8 = 8 MiB > 4 MiB
    vals = torch.empty((Mr, K // 2), dtype=torch.bfloat16, device="cuda")
    meta = torch.empty((Mr, K // 16), dtype=torch.int16, device="cuda")
    X = torch.empty((Nc, K), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((Nc, Mr), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SparseFFNError) as e:
        binding.sf_gemm_sparse24_noalloc(vals, meta, X, out)
    assert e.value.status == binding.SF_ERR_WORKSPACE
