"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments before launching anything (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2602_06183_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "sparseffn.h")).read()
    declared = set(re.findall(r"SF_API\s+(?:const\s+char\*|int)\s+(sf_\w+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTED_SYMBOLS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert binding.status_string(0) == "SF_OK"
    for code in range(-8, 0):
        assert binding.status_string(code).startswith("SF_ERR_")


def test_size_queries_and_shape_errors(lib):
    assert binding.sf_prune24_sizes(128, 256, 1) == (128 * 256, 128 * 256 // 8)
    a, b = C.c_size_t(), C.c_size_t()
    assert lib.sf_prune24_sizes(128, 250, 1, C.byref(a), C.byref(b)) == binding.SF_ERR_SHAPE
    assert lib.sf_prune24_sizes(128, 256, 2, C.byref(a), C.byref(b)) == binding.SF_ERR_SHAPE
    assert lib.sf_prune24_sizes(128, 256, 1, None, C.byref(b)) == binding.SF_ERR_NULL
    assert binding.sf_vnm_sizes(128, 256, 64, 2, 8) == (128 * 64 * 2, 128 * 8 * 2, 2 * 32 * 4)
    c = C.c_size_t()
    assert lib.sf_vnm_sizes(128, 256, 64, 1, 8, C.byref(a), C.byref(b), C.byref(c)) == binding.SF_ERR_UNSUPPORTED
    assert lib.sf_vnm_sizes(100, 256, 64, 2, 8, C.byref(a), C.byref(b), C.byref(c)) == binding.SF_ERR_SHAPE
    assert lib.sf_vnm_sizes(128, 256, 64, 2, 12, C.byref(a), C.byref(b), C.byref(c)) == binding.SF_ERR_SHAPE


def test_null_and_alignment_rejected_before_launch(lib):
    # shapes fine, pointers NULL -> SF_ERR_NULL without touching a device
    assert lib.sf_prune24_compress(None, 128, 256, 256, 1, 0, None, None, None, None) == binding.SF_ERR_NULL
    fake = C.c_void_p(0x1008)   # 8-byte aligned only
    ok = C.c_void_p(0x1000)
    assert lib.sf_prune24_compress(fake, 128, 256, 256, 1, 0, ok, ok, None, None) == binding.SF_ERR_ALIGN
    assert lib.sf_prune24_compress(ok, 128, 256, 100, 1, 0, ok, ok, None, None) == binding.SF_ERR_ALIGN
    assert lib.sf_vnm_sparsify_act(None, 128, 256, 256, 64, 2, 8, 1, None, None, None, None, None, None) == binding.SF_ERR_NULL
    # empty inputs are a no-op
    assert lib.sf_prune24_compress(None, 0, 256, 256, 1, 0, None, None, None, None) == binding.SF_OK


def test_schedule_logic_matches_the_oracle(lib):
    """The schedule functions are host arithmetic, so they are compared with the oracle here."""
    from oracle import schedule as S
    for warm, sparse, total in [(0, 0, 1), (0, 5, 5), (3, 4, 12), (1000, 30000, 60000), (2, 0, 9)]:
        sc = binding.make_schedule(warm, sparse, total)
        probe = sorted({0, max(warm - 1, 0), warm, min(warm + sparse, total - 1), max(warm + sparse - 1, 0), total - 1})
        for step in probe:
            assert binding.sf_schedule_step_kind(sc, step) == S.step_kind(step, warm, sparse, total)
        for s in (1.0, 1.22, 2.2, 7.0):
            assert binding.sf_schedule_speedup(sc, s) == pytest.approx(S.schedule_speedup(sparse, total, s), rel=1e-14)
    for args in [(2048, 8192, 32, 8, 64), (4096, 16384, 32, 8, 128), (16384, 53248, 128, 8, 128)]:
        assert binding.sf_ffn_flop_fraction(*args) == pytest.approx(S.ffn_flop_fraction(*args), rel=1e-14)
    for f, s in [(0.0, 3.0), (0.5, 2.0), (0.82, 1.22), (1.0, 7.0)]:
        assert binding.sf_end_to_end_speedup(f, s) == pytest.approx(S.end_to_end_speedup(f, s), rel=1e-14)


def test_schedule_rejects_bad_arguments(lib):
    kind, out = C.c_int(), C.c_double()
    sc = binding.make_schedule(3, 4, 12)
    assert lib.sf_schedule_step_kind(None, 0, C.byref(kind)) == binding.SF_ERR_NULL
    assert lib.sf_schedule_step_kind(C.byref(sc), 0, None) == binding.SF_ERR_NULL
    assert lib.sf_schedule_step_kind(C.byref(sc), 12, C.byref(kind)) == binding.SF_ERR_SHAPE
    assert lib.sf_schedule_step_kind(C.byref(sc), -1, C.byref(kind)) == binding.SF_ERR_SHAPE
    for bad in [(-1, 4, 12), (3, -4, 12), (3, 4, 0), (9, 4, 12)]:
        b = binding.make_schedule(*bad)
        assert lib.sf_schedule_step_kind(C.byref(b), 0, C.byref(kind)) == binding.SF_ERR_SHAPE
        assert lib.sf_schedule_speedup(C.byref(b), 2.0, C.byref(out)) == binding.SF_ERR_SHAPE
    assert lib.sf_schedule_speedup(C.byref(sc), 0.0, C.byref(out)) == binding.SF_ERR_SHAPE
    assert lib.sf_end_to_end_speedup(1.5, 2.0, C.byref(out)) == binding.SF_ERR_SHAPE
    assert lib.sf_ffn_flop_fraction(0, 8, 1, 1, 1, C.byref(out)) == binding.SF_ERR_SHAPE
    # a step outside the schedule is rejected before any pointer is looked at
    assert lib.sf_ffn_fwd_scheduled(C.byref(sc), 99, None, None, None, None, None, None, 0, None, 0, None) == binding.SF_ERR_SHAPE


def test_step_calls_reject_short_buffers_before_launching(lib):
    """Every step call is told how large its context and workspace are and refuses, on the host,
    buffers smaller than sf_ffn_workspace_size reports (no device is touched: the pointers are fake)."""
    desc = binding.make_desc(1024, 256, 1024, 64, 8)
    need_ctx, need_ws = binding.sf_ffn_workspace_size(desc)
    assert need_ctx > 0 and need_ws > 256
    ok = C.c_void_p(0x10000)
    d = C.byref(desc)
    W = binding.SF_ERR_WORKSPACE
    # (the size query reports the larger of the sparse and the dense step's needs, so "short" here
    # means well below either)
    assert lib.sf_sparse_ffn_fwd(d, ok, ok, ok, ok, ok, need_ctx // 2, ok, need_ws, None) == W
    assert lib.sf_sparse_ffn_fwd(d, ok, ok, ok, ok, ok, need_ctx, ok, need_ws // 2, None) == W
    assert lib.sf_sparse_ffn_bwd(d, ok, ok, ok, ok, ok, need_ctx, ok, ok, ok, ok, 0, None) == W
    assert lib.sf_dense_ffn_fwd(d, ok, ok, ok, ok, ok, 16, ok, need_ws, None) == W
    assert lib.sf_dense_ffn_bwd(d, ok, ok, ok, ok, ok, need_ctx, ok, ok, ok, ok, 255, None) == W
    assert lib.sf_ffn_step_host(d, 0, ok, ok, ok, ok, ok, ok, ok, ok, ok, ok, need_ctx // 2, ok, need_ws, None) == W
    sc = binding.make_schedule(0, 1, 2)
    assert lib.sf_ffn_fwd_scheduled(C.byref(sc), 0, d, ok, ok, ok, ok, ok, need_ctx, ok, need_ws // 2, None) == W
    # NULL and alignment still come first
    assert lib.sf_sparse_ffn_fwd(d, None, ok, ok, ok, ok, need_ctx, ok, need_ws, None) == binding.SF_ERR_NULL
    # unknown flag bits are refused
    bad = binding.make_desc(1024, 256, 1024, 64, 8, flags=32)
    a, b = C.c_size_t(), C.c_size_t()
    assert lib.sf_ffn_workspace_size(C.byref(bad), C.byref(a), C.byref(b)) == binding.SF_ERR_UNSUPPORTED


def test_context_size_of_the_d4096_layer(lib):
    """M = 8 keeps ReLU(y1) and the operands of the sparse products in packed forms only: the context of
    the d_model = 4096 layer with 8192 tokens is about 0.7 GB with the one masked [T, F] copy the
    weight-gradient product reads, and below 0.6 GB when that product expands its operand itself
    (three masked [T, F] copies alone would be 0.8 GB)."""
    desc = binding.make_desc(8192, 4096, 16384, 128, 8)
    ctx, ws = binding.sf_ffn_workspace_size(desc)
    assert ctx < 0.75e9
    lean = binding.make_desc(8192, 4096, 16384, 128, 8, flags=binding.SF_FFN_PACKED_GRAD_OPERANDS)
    lctx, lws = binding.sf_ffn_workspace_size(lean)
    assert lctx < 0.6e9 and lws < ws


def test_router_fit_matches_the_oracle(lib):
    """The offline clustering is host code, so it is compared with the oracle here: planted clusters
    come back whole, the partition is balanced, the permutation is expert-major and stable, the means
    are the centroids, and on unstructured weights the assignment agrees with the oracle's."""
    import numpy as np
    from oracle import router as R
    from oracle import f32_to_bf16, bf16_to_f32
    from paper_2602_06183_b200 import synth
    rng = np.random.default_rng(0)
    E, cap, D = 4, 24, 16
    centres = rng.integers(-4, 5, size=(E, D)).astype(np.float32) * 8.0
    label = rng.permutation(np.repeat(np.arange(E), cap))
    W = f32_to_bf16(centres[label] + rng.integers(-1, 2, size=(E * cap, D)).astype(np.float32)).reshape(E * cap, D)
    expert, perm, means = binding.sf_router_fit_host(W, E)
    o_expert, o_means = R.fit_experts(W, E)
    assert np.array_equal(expert, o_expert) and np.array_equal(means, o_means)
    assert np.array_equal(perm, R.expert_major_permutation(o_expert))
    for e in range(E):
        assert len(set(label[expert == e])) == 1
    W1 = synth.normal_bf16((512, 64), 0.0, 0.02, seed=3)
    for E in (2, 16):
        expert, perm, means = binding.sf_router_fit_host(W1, E, iters=1)
        o_expert, o_means = R.fit_experts(W1, E, iters=1)
        assert np.array_equal(np.bincount(expert, minlength=E), np.full(E, 512 // E))
        assert np.array_equal(expert[perm], np.repeat(np.arange(E), 512 // E))
        assert (expert == o_expert).mean() > 0.99
        for e in range(E):
            c = bf16_to_f32(W1[expert == e]).astype(np.float64).mean(axis=0).astype(np.float32)
            assert np.array_equal(means[e], f32_to_bf16(c))
    a, b = C.c_void_p(0x1000), None
    assert lib.sf_router_fit_host(a, 10, 4, 3, 1, a, a, a) == binding.SF_ERR_SHAPE
    assert lib.sf_router_fit_host(b, 12, 4, 3, 1, a, a, a) == binding.SF_ERR_NULL


def test_routed_step_argument_checks_on_the_host(lib):
    desc = binding.make_router_desc(1024, 256, 1024, 4)
    need_ctx, need_ws = binding.sf_routed_ffn_workspace_size(desc)
    assert need_ctx > 0 and need_ws > 256
    ok = C.c_void_p(0x10000)
    d = C.byref(desc)
    assert lib.sf_routed_ffn_fwd(d, ok, ok, ok, ok, None, ok, ok, need_ctx - 1, ok, need_ws, None) == binding.SF_ERR_WORKSPACE
    assert lib.sf_routed_ffn_bwd(d, ok, ok, ok, ok, ok, need_ctx, ok, ok, ok, ok, need_ws - 1, None) == binding.SF_ERR_WORKSPACE
    assert lib.sf_routed_ffn_fwd(d, None, ok, ok, ok, None, ok, ok, need_ctx, ok, need_ws, None) == binding.SF_ERR_NULL
    assert lib.sf_routed_ffn_fwd(d, C.c_void_p(0x10008), ok, ok, ok, None, ok, ok, need_ctx, ok, need_ws, None) == binding.SF_ERR_ALIGN
    bad = binding.make_router_desc(1024, 256, 1024, 4, flags=binding.SF_FFN_UNFUSED_ACT)
    a, b = C.c_size_t(), C.c_size_t()
    assert lib.sf_routed_ffn_workspace_size(C.byref(bad), C.byref(a), C.byref(b)) == binding.SF_ERR_UNSUPPORTED
    assert lib.sf_router_route(ok, ok, 128, 100, 4, ok, None, None) == binding.SF_ERR_SHAPE
    assert lib.sf_router_route(ok, ok, 0, 256, 4, ok, None, None) == binding.SF_OK
    p, n = C.c_void_p(), C.c_size_t()
    assert lib.sf_routed_ctx_view(d, ok, binding.SF_RCTX_Y1, C.byref(p), C.byref(n)) == binding.SF_ERR_UNSUPPORTED
    assert lib.sf_routed_ctx_view(d, ok, 99, C.byref(p), C.byref(n)) == binding.SF_ERR_SHAPE
