"""Parity of the sparse and dense FFN step (CUDA, through the C ABI) with the oracle.

Protocol: stage-wise, teacher-forced. The oracle re-runs the selection on the GPU's own bf16
pre-activations (a one-ulp difference in y1 may legitimately flip a near-tie), so masks, metadata
and packed values must be bit-identical; products are compared in relative Frobenius norm against
float64-accumulated references evaluated with those masks. The free-running oracle is compared too.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06183_b200 import binding, synth
from util import to_dev, bits, f32, rel_fro, assert_close_elementwise, Guarded

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _run_sparse(cfg, prune_mode=0, act_shift=0.0, flags=binding.SF_FFN_SAVE_Y1):
    """One sparse step through the C ABI. Context, workspace and every output sit between guard
    zones that are checked after the step (nothing may be written outside a buffer)."""
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"], act_shift=act_shift)
    desc = binding.make_desc(T, D, F, V, M, prune_mode=prune_mode, flags=flags)
    nctx, nws = binding.sf_ffn_workspace_size(desc)
    gctx, gws = Guarded(nctx, zero=True), Guarded(nws, zero=True)
    ctx, ws = gctx.t, gws.t
    w2_fd = bool(flags & binding.SF_FFN_W2_FD)                # W2 handed over (and dW2 returned) as [F, D]
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, np.ascontiguousarray(W2.T) if w2_fd else W2, dY))
    gY, ggX = Guarded((T, D), torch.bfloat16), Guarded((T, D), torch.bfloat16)
    ggW1, ggW2 = Guarded((F, D), torch.bfloat16), Guarded((F, D) if w2_fd else (D, F), torch.bfloat16)
    Y, gX, gW1, gW2 = gY.t, ggX.t, ggW1.t, ggW2.t
    binding.sf_sparse_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    binding.sf_sparse_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    for g, name in ((gctx, "context"), (gws, "workspace"), (gY, "Y"), (ggX, "dX"), (ggW1, "dW1"), (ggW2, "dW2")):
        g.check(name)
    G = F // M
    view = lambda buf, field: binding.sf_ctx_view(desc, buf, field)
    out = dict(
        y2_vals=bits(view(ctx, binding.SF_CTX_Y2_VALS)).reshape(T, 2 * G),
        relu_vals=bits(view(ctx, binding.SF_CTX_RELU_VALS)).reshape(T, 2 * G),
        meta=bits(view(ctx, binding.SF_CTX_META)).reshape(T, G // 4),
        colidx=view(ctx, binding.SF_CTX_COLIDX).cpu().numpy().reshape(T // V, G, 4),
        Y=f32(Y), dX=f32(gX), dW1=f32(gW1), dW2=f32(gW2).T if w2_fd else f32(gW2))
    if flags & binding.SF_FFN_SAVE_Y1:
        out["y1"] = bits(view(ctx, binding.SF_CTX_Y1)).reshape(T, F)
    if M == 8:
        # the activation and dy1 live in their 2:4 layout over all F columns
        m24 = bits(view(ctx, binding.SF_CTX_Y2_META24)).reshape(T, F // 16)
        out["meta24"] = m24
        out["vals24"] = bits(view(ctx, binding.SF_CTX_Y2_VALS24)).reshape(T, F // 2)
        out["relu24"] = bits(view(ctx, binding.SF_CTX_RELU_VALS24)).reshape(T, F // 2)
        out["dy1_dense"] = oracle.decompress24(bits(view(ws, binding.SF_CTX_DY1_VALS24)).reshape(T, F // 2), m24)
    else:
        dy1_vals = bits(view(ws, binding.SF_CTX_DY1_VALS)).reshape(T, 2 * G)
        out["dy1_dense"] = oracle.decompress_vnm(dy1_vals, out["meta"], out["colidx"], V=V, M=M)
    return (X, W1, W2, dY), out


def _check_against_oracle(inputs, g, cfg, prune_mode=0):
    """Stage-wise, teacher-forced comparison of one step with the oracle (needs the saved y1)."""
    X, W1, W2, dY = inputs
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, prune_mode=prune_mode, forced_y1b=g["y1"])
    assert np.array_equal(g["colidx"], fwd.act.colidx)
    assert np.array_equal(g["meta"], fwd.act.meta)
    assert np.array_equal(g["y2_vals"], fwd.act.vals)
    assert np.array_equal(g["relu_vals"], fwd.act.relu_vals)
    if M == 8:
        nib = np.stack([(g["meta24"] >> np.uint16(4 * i)) & np.uint16(0xF) for i in range(4)], axis=-1)
        assert ((nib & 3) < (nib >> 2)).all()                    # legal position pairs everywhere
        assert np.array_equal(oracle.decompress24(g["vals24"], g["meta24"]), fwd.act.dense)
        relu_dense = np.where(fwd.act.mask, oracle.vnm.squared_relu_bf16(g["y1"])[1], np.uint16(0))
        assert np.array_equal(oracle.decompress24(g["relu24"], g["meta24"]), relu_dense)
    assert rel_fro(g["Y"], fwd.y3) < TOL
    assert_close_elementwise(g["Y"], fwd.y3, F, "Y")
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd, prune_mode=prune_mode)
    assert not (g["dy1_dense"][~fwd.act.mask] != 0).any()        # nothing outside y2's mask
    assert rel_fro(oracle.bf16_to_f32(g["dy1_dense"]), oracle.bf16_to_f32(bwd.dy1_dense)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(g["dy1_dense"]), oracle.bf16_to_f32(bwd.dy1_dense), D, "dy1")
    # The remaining products are compared with the oracle evaluated on the GPU's own dy1 (a one-ulp
    # difference in dy1 is legitimate and would otherwise be charged to dX and dW1 as well).
    dy1m = oracle.bf16_to_f32(g["dy1_dense"]).astype(np.float64)
    refs = dict(dX=dy1m @ oracle.bf16_to_f32(W1).astype(np.float64),
                dW1=dy1m.T @ oracle.bf16_to_f32(X).astype(np.float64), dW2=bwd.dW2)
    for k, Kred in (("dX", F), ("dW1", T), ("dW2", T)):
        assert rel_fro(g[k], refs[k]) < TOL, k
        assert_close_elementwise(g[k], refs[k], Kred, k)
    for k, ref in (("dX", bwd.dX), ("dW1", bwd.dW1)):
        assert rel_fro(g[k], ref) < TOL, k
    return fwd, bwd


@pytest.mark.parametrize("prune_mode,act_shift", [(0, 0.0), (1, 0.0), (0, -1.3)])
def test_sparse_ffn_c1_teacher_forced(prune_mode, act_shift):
    cfg = synth.FFN_CONFIGS["c1_small"]
    (X, W1, W2, dY), g = _run_sparse(cfg, prune_mode, act_shift)
    V, M = cfg["V"], cfg["M"]
    # stage 1: the GPU's y1 against the oracle's own product with the pruned W1
    free = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, prune_mode=prune_mode)
    assert rel_fro(oracle.bf16_to_f32(g["y1"]), oracle.bf16_to_f32(free.y1b)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(g["y1"]), oracle.bf16_to_f32(free.y1b), cfg["D"], "y1")
    # stages 2 and 3: selection on the GPU's y1 bit for bit, products with those masks
    _check_against_oracle((X, W1, W2, dY), g, cfg, prune_mode)
    # free-running comparison: masks may differ in a few near-tie blocks only
    disagree = float((free.act.colidx != g["colidx"]).any(axis=-1).mean())
    assert disagree < 0.05
    assert rel_fro(g["Y"], free.y3) < 5e-2


@pytest.mark.parametrize("cfg", [
    dict(T=1024, D=256, F=1024, V=64, N=2, M=8, sigma_w=0.02, seed=0),      # fused epilogue, three 64-token blocks per tile
    dict(T=512, D=256, F=512, V=128, N=2, M=8, sigma_w=0.05, seed=3),       # two-kernel path (the default for V = 128)
    dict(T=512, D=256, F=2048, V=128, N=2, M=16, sigma_w=0.05, seed=17),    # condensed Venom products
], ids=["m8_v64", "m8_v128", "m16_v128"])
def test_step_without_saved_y1_is_the_same_step(cfg):
    """The benchmarked configuration keeps no y1 (flags = 0), which moves buffers inside the context and
    the workspace. Everything it produces must equal, bit for bit, the teacher-forced run that saves
    y1 and is checked against the oracle; what the context exposes is compared with the oracle too."""
    inputs, g1 = _run_sparse(cfg, flags=binding.SF_FFN_SAVE_Y1)
    fwd, _ = _check_against_oracle(inputs, g1, cfg)
    _, g0 = _run_sparse(cfg, flags=0)
    assert "y1" not in g0
    for k in g0:
        assert np.array_equal(g0[k], g1[k]), k
    assert np.array_equal(g0["colidx"], fwd.act.colidx) and np.array_equal(g0["y2_vals"], fwd.act.vals)


@pytest.mark.parametrize("V,act_shift", [(64, 0.0), (128, 0.0), (64, -1.3)])
def test_fused_activation_epilogue_equals_the_two_kernel_path(V, act_shift):
    """SquaredReLU + V:N:M inside the y1 product's epilogue against the stand-alone kernel on a stored
    y1: same accumulation, same selection rule, so every output must agree bit for bit. T is not a
    multiple of the fused kernel's 192-token tile, so the last tile is ragged."""
    cfg = dict(T=1280, D=512, F=768, V=V, N=2, M=8, sigma_w=0.05, seed=41)
    Y1 = binding.SF_FFN_SAVE_Y1
    inputs, fused = _run_sparse(cfg, act_shift=act_shift, flags=Y1 | binding.SF_FFN_FUSED_ACT)
    _, two = _run_sparse(cfg, act_shift=act_shift, flags=Y1 | binding.SF_FFN_UNFUSED_ACT)
    for k in fused:
        assert np.array_equal(fused[k], two[k]), k
    _check_against_oracle(inputs, fused, cfg)
    # and with the weight-gradient products reading the packed operands instead of masked [T, F] copies
    _, packed = _run_sparse(cfg, act_shift=act_shift, flags=Y1 | binding.SF_FFN_FUSED_ACT | binding.SF_FFN_PACKED_GRAD_OPERANDS)
    for k in fused:
        assert np.array_equal(fused[k], packed[k]), k


@pytest.mark.parametrize("flags", [0, binding.SF_FFN_UNFUSED_ACT], ids=["fused", "two_kernel"])
def test_all_zero_activation_takes_the_default_pattern(flags):
    """Degenerate input: X = 0 makes every pre-activation +0, so every column score ties at zero. The
    block keeps columns 0-3 (ties to the lower column), every row positions (0, 1), all values are zero
    and every output of the step is exactly zero."""
    cfg = dict(T=512, D=256, F=512, V=64, N=2, M=8, sigma_w=0.05, seed=5)
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    _, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"])
    X = np.zeros((T, D), dtype=np.uint16)
    desc = binding.make_desc(T, D, F, V, M, flags=flags | binding.SF_FFN_SAVE_Y1)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, W2, dY))
    Y = torch.full((T, D), 7.0, dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.full_like(dX_, 7.0), torch.full_like(dW1_, 7.0), torch.full_like(dW2_, 7.0)
    binding.sf_sparse_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
    binding.sf_sparse_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    G = F // M
    colidx = binding.sf_ctx_view(desc, ctx, binding.SF_CTX_COLIDX).cpu().numpy().reshape(T // V, G, 4)
    assert np.all(colidx == np.arange(4))
    assert np.all(bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_META)) == 0x4444)
    assert not bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_Y2_VALS)).any()
    assert not bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_Y1)).any()
    ref = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M)
    assert np.array_equal(colidx, ref.act.colidx) and np.all(ref.act.meta == 0x4444)
    for t in (Y, gX, gW1, gW2):
        assert not bits(t).any()


def test_plain_24_view_of_m4_activations_is_exact():
    """M = 4 is 2:4 activation sparsity: the packed V:N:M form is itself the 2:4 operand the products
    consume. Decompressed with its own metadata it must be the oracle's masked dense y2 bit for bit,
    and dy1 packed by the dy1 product's epilogue must sit at the same positions."""
    cfg = dict(synth.FFN_CONFIGS["c1_small"], M=4)
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], 4
    inputs, g = _run_sparse(cfg)
    fwd, bwd = _check_against_oracle(inputs, g, cfg)
    desc = binding.make_desc(T, D, F, V, M, flags=binding.SF_FFN_SAVE_Y1)
    assert np.all(g["colidx"] == np.arange(4))
    assert np.array_equal(oracle.decompress24(g["y2_vals"], g["meta"]), fwd.act.dense)


@pytest.mark.parametrize("cfg", [
    dict(T=512, D=256, F=2048, V=128, N=2, M=16, sigma_w=0.05, seed=17),
    dict(T=512, D=256, F=2048, V=64, N=2, M=4, sigma_w=0.05, seed=27),      # 2:4 activation sparsity
    dict(T=512, D=256, F=2048, V=128, N=2, M=32, sigma_w=0.05, seed=55),    # condensed, gathered Venom product
    dict(T=256, D=256, F=4096, V=128, N=2, M=64, sigma_w=0.05, seed=87),    # Table 5's widest group
    dict(T=256, D=256, F=2048, V=64, N=2, M=64, sigma_w=0.05, seed=88),
], ids=["m16", "m4", "m32", "m64_v128", "m64_v64"])
def test_sparse_ffn_other_group_widths(cfg):
    inputs, g = _run_sparse(cfg)
    _check_against_oracle(inputs, g, cfg)


@pytest.mark.parametrize("T,D,F,V,M", [(256, 256, 256, 128, 8), (256, 256, 256, 64, 8), (512, 512, 512, 128, 16),
                                       (768, 256, 1280, 128, 8), (768, 256, 1280, 64, 8)])
def test_sparse_ffn_smallest_and_odd_tile_counts(T, D, F, V, M):
    """One tile per product, fewer k-blocks than pipeline stages, tile counts that are not a
    multiple of the raster band."""
    cfg = dict(T=T, D=D, F=F, V=V, N=2, M=M, sigma_w=0.05, seed=T + F + V)
    inputs, g = _run_sparse(cfg)
    _check_against_oracle(inputs, g, cfg)


@pytest.mark.parametrize("T,D,F,V,M", [(384, 384, 640, 64, 8), (640, 384, 384, 128, 8), (896, 640, 384, 64, 8),
                                       (384, 640, 896, 64, 4), (384, 384, 1152, 128, 8)])
@pytest.mark.parametrize("flags", [binding.SF_FFN_SAVE_Y1, binding.SF_FFN_SAVE_Y1 | binding.SF_FFN_UNFUSED_ACT],
                         ids=["default", "two_kernel"])
def test_sparse_ffn_odd_multiples_of_128(T, D, F, V, M, flags):
    """T, D or F = 128 (mod 256): the last row of CTA pairs of a product is half empty (its second CTA works
    on zero-filled rows and must store nothing: the guard zones around every buffer check that too)."""
    cfg = dict(T=T, D=D, F=F, V=V, N=2, M=M, sigma_w=0.05, seed=T + 2 * D + 3 * F)
    for prune_mode in (0, 1):
        inputs, g = _run_sparse(cfg, prune_mode, flags=flags)
        _check_against_oracle(inputs, g, cfg, prune_mode)


@pytest.mark.parametrize("T,D,F,V,M", [(1024, 256, 1024, 64, 8), (384, 640, 896, 128, 8), (512, 512, 1024, 64, 4),
                                       (512, 256, 1024, 128, 16), (256, 512, 2048, 64, 32)])
def test_sparse_ffn_with_w2_stored_as_f_by_d(T, D, F, V, M):
    """SF_FFN_W2_FD: the same layer with W2 handed over (and dW2 returned) as [F, D]: contiguous pruning of W2,
    W2 as the MN-major operand of y3, no transposed copy for the gathered products; checked against the oracle
    like every other step, in both prune modes and with the two-kernel activation path."""
    cfg = dict(T=T, D=D, F=F, V=V, N=2, M=M, sigma_w=0.05, seed=T + D + F + M)
    for prune_mode, extra in ((0, 0), (1, binding.SF_FFN_UNFUSED_ACT if M == 8 else 0)):
        inputs, g = _run_sparse(cfg, prune_mode, flags=binding.SF_FFN_SAVE_Y1 | binding.SF_FFN_W2_FD | extra)
        _check_against_oracle(inputs, g, cfg, prune_mode)
    if M == 8:
        inputs, g = _run_sparse(cfg, 0, flags=binding.SF_FFN_SAVE_Y1 | binding.SF_FFN_W2_FD | binding.SF_FFN_PACKED_GRAD_OPERANDS) \
            if (T % 256 == 0 and D % 256 == 0 and F % 256 == 0) else (None, None)
        if g is not None:
            _check_against_oracle(inputs, g, cfg, 0)


@pytest.mark.parametrize("name", ["c1_small", "odd128"])
def test_dense_ffn_c1(name):
    cfg = synth.FFN_CONFIGS["c1_small"] if name == "c1_small" else dict(T=384, D=640, F=896, V=64, M=8, sigma_w=0.05, seed=77)
    T, D, F = cfg["T"], cfg["D"], cfg["F"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"])
    w2_fd = name == "odd128"                                   # this case also hands W2 over as [F, D]
    desc = binding.make_desc(T, D, F, cfg["V"], cfg["M"], flags=binding.SF_FFN_W2_FD if w2_fd else 0)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, np.ascontiguousarray(W2.T) if w2_fd else W2, dY))
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)
    binding.sf_dense_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
    binding.sf_dense_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    if w2_fd:
        gW2 = gW2.T
    y1 = bits(ctx[: T * F * 2].view(torch.bfloat16)).reshape(T, F)
    free = oracle.dense_ffn_fwd(X, W1, W2)
    assert rel_fro(oracle.bf16_to_f32(y1), oracle.bf16_to_f32(free.y1b)) < TOL
    fwd = oracle.dense_ffn_fwd(X, W1, W2, forced_y1b=y1)
    bwd = oracle.dense_ffn_bwd(dY, X, W1, W2, fwd)
    assert rel_fro(f32(Y), fwd.y3) < TOL
    assert rel_fro(f32(gX), bwd.dX) < TOL
    assert rel_fro(f32(gW1), bwd.dW1) < TOL
    assert rel_fro(f32(gW2), bwd.dW2) < TOL


def test_step_from_host_buffers_matches_device_path():
    cfg = synth.FFN_CONFIGS["c1_small"]
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"])
    desc = binding.make_desc(T, D, F, V, M)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    staging = torch.empty((binding.sf_ffn_host_staging_size(desc),), dtype=torch.uint8, device="cuda")
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    hX, hW1, hW2, hdY = pin(X), pin(W1), pin(W2), pin(dY)
    hY, hdX = torch.empty_like(hX, pin_memory=True), torch.empty_like(hX, pin_memory=True)
    hdW1, hdW2 = torch.empty_like(hW1, pin_memory=True), torch.empty_like(hW2, pin_memory=True)
    binding.sf_ffn_step_host(desc, False, hX, hW1, hW2, hdY, hY, hdX, hdW1, hdW2, staging, ctx, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    (_, _, _, _), g = _run_sparse(cfg)
    as_f32 = lambda t: t.view(torch.bfloat16).float().numpy()
    assert np.array_equal(as_f32(hY), g["Y"]) and np.array_equal(as_f32(hdX), g["dX"])
    assert np.array_equal(as_f32(hdW1), g["dW1"]) and np.array_equal(as_f32(hdW2), g["dW2"])


@pytest.mark.parametrize("dense", [False, True])
def test_back_to_back_host_steps_do_not_race(dense):
    """Uploads and downloads run on the library's own copy streams. Two steps with different inputs
    that share one staging area, context and workspace, enqueued without a synchronisation between
    them, must each give the result of running alone: the second step's uploads may not overtake the
    first step's kernels, and its kernels may not overtake the first step's downloads."""
    cfg = synth.FFN_CONFIGS["c1_small"]
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    desc = binding.make_desc(T, D, F, V, M)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    staging = torch.empty((binding.sf_ffn_host_staging_size(desc),), dtype=torch.uint8, device="cuda")
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    ins = [tuple(pin(a) for a in synth.ffn_inputs(T, D, F, cfg["sigma_w"], seed)) for seed in (11, 12)]
    outs = lambda i: tuple(torch.empty_like(i[k], pin_memory=True) for k in (0, 0, 1, 2))   # Y, dX, dW1, dW2

    def run(pairs):
        for i, o in pairs:
            binding.sf_ffn_step_host(desc, dense, i[0], i[1], i[2], i[3], o[0], o[1], o[2], o[3], staging, ctx, ws)
        assert binding.sf_check_status(ws) == binding.SF_OK

    alone = [outs(i) for i in ins]
    for i, o in zip(ins, alone):
        run([(i, o)])
    assert not torch.equal(alone[0][0], alone[1][0])
    for _ in range(3):
        together = [outs(i) for i in ins]
        run(list(zip(ins, together)))
        for a, b in zip(alone, together):
            for x, y in zip(a, b):
                assert torch.equal(x, y)


def test_sparse_step_replays_from_a_cuda_graph():
    """The step enqueues kernels only (no allocation, no synchronisation), so it can be captured
    once and replayed; the replay must reproduce the eager results bit for bit."""
    cfg = synth.FFN_CONFIGS["c1_small"]
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"])
    desc = binding.make_desc(T, D, F, V, M)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, W2, dY))
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)

    def step():
        binding.sf_sparse_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
        binding.sf_sparse_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)

    step()                                          # eager run (also does the one-time kernel set-up)
    torch.cuda.synchronize()
    eager = [t.clone() for t in (Y, gX, gW1, gW2)]
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    for t in (Y, gX, gW1, gW2):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert binding.sf_check_status(ws) == binding.SF_OK
    for a, b in zip(eager, (Y, gX, gW1, gW2)):
        assert torch.equal(a, b)


def test_ffn_rejects_ragged_shapes():
    for shape in [(1000, 256, 1024, 64, 8), (128, 256, 1024, 64, 8),      # not a multiple of 128; a single 128-row block
                  (384, 256, 1024, 128, 16),                                # gathered Venom products keep whole 256-row tiles
                  (512, 384, 1024, 128, 32)]:
        desc = binding.make_desc(*shape)
        with pytest.raises(binding.SparseFFNError) as e:
            binding.sf_ffn_workspace_size(desc)
        assert e.value.status == binding.SF_ERR_SHAPE
    desc = binding.make_desc(1024, 256, 1024, 64, 8, N=1)
    with pytest.raises(binding.SparseFFNError) as e:
        binding.sf_ffn_workspace_size(desc)
    assert e.value.status == binding.SF_ERR_UNSUPPORTED


def test_scheduled_steps_dispatch_to_the_right_kind():
    """A short run (2 warm-up, 3 sparse, 2 dense): every scheduled step reproduces, bit for bit,
    the direct call of the kind the schedule assigns to it."""
    cfg = synth.FFN_CONFIGS["c1_small"]
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"])
    desc = binding.make_desc(T, D, F, V, M)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, W2, dY))

    def run(fwd, bwd):
        Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
        gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)
        fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
        bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
        assert binding.sf_check_status(ws) == binding.SF_OK
        return Y, gX, gW1, gW2

    direct = {binding.SF_STEP_SPARSE: run(binding.sf_sparse_ffn_fwd, binding.sf_sparse_ffn_bwd),
              binding.SF_STEP_DENSE: run(binding.sf_dense_ffn_fwd, binding.sf_dense_ffn_bwd)}
    assert not torch.equal(direct[0][0], direct[1][0])
    sc = binding.make_schedule(2, 3, 7)
    kinds = []
    for step in range(7):
        kind = binding.sf_schedule_step_kind(sc, step)
        kinds.append(kind)
        got = run(lambda *a: binding.sf_ffn_fwd_scheduled(sc, step, *a),
                  lambda *a: binding.sf_ffn_bwd_scheduled(sc, step, *a))
        for a, b in zip(got, direct[kind]):
            assert torch.equal(a, b)
    assert kinds == [0, 0, 1, 1, 1, 0, 0]


def _legal_random_configs(n, seed):
    """Seeded draw of legal step shapes: T, D, F multiples of 128 from 256 up (of 256 for M >= 16, whose gathered
    products keep whole tiles), V in {64, 128}, M in {4..32}, whole metadata words, condensed reduction 4F/M a
    multiple of 128 for M >= 16, both prune modes, symmetric or ~90 %-negative pre-activations."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        V, M = int(rng.choice([64, 128])), int(rng.choice([4, 8, 16, 32]))
        q = 256 if M >= 16 else 128
        T, D, F = (int(rng.integers(256 // q, 1024 // q + 1)) * q for _ in range(3))
        F *= int(rng.integers(1, 3))
        if T % V or F % (4 * M) or (M >= 16 and (4 * F // M) % 128):
            continue
        out.append((T, D, F, V, M, int(rng.integers(0, 2)), float(rng.choice([0.0, -1.3])), int(rng.integers(1, 1 << 20))))
    return out


@pytest.mark.parametrize("T,D,F,V,M,prune_mode,act_shift,seed", _legal_random_configs(12, seed=20260206))
def test_sparse_ffn_random_legal_shapes(T, D, F, V, M, prune_mode, act_shift, seed):
    cfg = dict(T=T, D=D, F=F, V=V, N=2, M=M, sigma_w=0.05, seed=seed)
    inputs, g = _run_sparse(cfg, prune_mode, act_shift)
    _check_against_oracle(inputs, g, cfg, prune_mode)
