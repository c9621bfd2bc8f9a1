"""Parity at the benchmark's full sizes, on outputs the oracle can compute one sample at a time.

FFN step (the launch configuration bench.py times): whole V-blocks of tokens are checked for
y1 / masks / y2 / y3 / dy1 / dX, and whole M-groups of features (all tokens) for dW1 / dW2 — the
V:N:M selection of a block only needs its own rows, and that of a group only its own columns, so
both samples are exact restrictions of the full problem. Standalone prune / sparsify sweeps are
checked bit for bit on sampled rows / blocks of the full-size matrices.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_06183_b200 import binding, synth
from util import to_dev, bits, f32, rel_fro, assert_close_elementwise, Guarded

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _full_step(cfg, flags):
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"])
    desc = binding.make_desc(T, D, F, V, M, flags=flags)
    nctx, nws = binding.sf_ffn_workspace_size(desc)
    gctx, gws = Guarded(nctx, zero=True), Guarded(nws, zero=True)
    dX_, dW1_, dW2_, ddY = (to_dev(a) for a in (X, W1, W2, dY))
    outs = [Guarded((T, D), torch.bfloat16), Guarded((T, D), torch.bfloat16), Guarded((F, D), torch.bfloat16),
            Guarded((D, F), torch.bfloat16)]
    Y, gX, gW1, gW2 = (o.t for o in outs)
    binding.sf_sparse_ffn_fwd(desc, dX_, dW1_, dW2_, Y, gctx.t, gws.t)
    binding.sf_sparse_ffn_bwd(desc, ddY, dX_, dW1_, dW2_, gctx.t, gX, gW1, gW2, gws.t)
    assert binding.sf_check_status(gws.t) == binding.SF_OK
    for g, nm in zip([gctx, gws] + outs, ["context", "workspace", "Y", "dX", "dW1", "dW2"]):
        g.check(nm)
    return (X, W1, W2, dY), desc, gctx.t, gws.t, (Y, gX, gW1, gW2)


@pytest.mark.parametrize("name", ["c4_d4096", "c4_d4096_v128", "c4_d4096_m16", "c5_d8192"])
def test_ffn_step_full_size_sampled(name):
    cfg = synth.FFN_CONFIGS[name]
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    G = F // M
    (X, W1, W2, dY), desc, ctx, ws, (Y, gX, gW1, gW2) = _full_step(cfg, binding.SF_FFN_SAVE_Y1)
    view = lambda buf, field: binding.sf_ctx_view(desc, buf, field)
    y1_dev = view(ctx, binding.SF_CTX_Y1).view(T, F)
    vals_dev = view(ctx, binding.SF_CTX_Y2_VALS).view(T, 2 * G)
    relu_dev = view(ctx, binding.SF_CTX_RELU_VALS).view(T, 2 * G)
    meta_dev = view(ctx, binding.SF_CTX_META).view(T, G // 4)
    cidx_dev = view(ctx, binding.SF_CTX_COLIDX).view(T // V, G, 4)

    # ---- sample 1: two whole V-blocks of tokens (first and last), all features
    blocks = [0, T // V - 1]
    rows = np.concatenate([np.arange(b * V, (b + 1) * V) for b in blocks])
    rows_t = torch.from_numpy(rows).cuda()
    y1_rows = bits(y1_dev[rows_t])
    free = oracle.sparse_ffn_fwd(X[rows], W1, W2, V=V, M=M)
    assert rel_fro(oracle.bf16_to_f32(y1_rows), oracle.bf16_to_f32(free.y1b)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(y1_rows), oracle.bf16_to_f32(free.y1b), D, "y1")
    fwd = oracle.sparse_ffn_fwd(X[rows], W1, W2, V=V, M=M, forced_y1b=y1_rows)
    assert np.array_equal(cidx_dev[torch.tensor(blocks).cuda()].cpu().numpy(), fwd.act.colidx)
    assert np.array_equal(bits(meta_dev[rows_t]), fwd.act.meta)
    assert np.array_equal(bits(vals_dev[rows_t]), fwd.act.vals)
    assert np.array_equal(bits(relu_dev[rows_t]), fwd.act.relu_vals)
    assert rel_fro(f32(Y[rows_t]), fwd.y3) < TOL
    assert_close_elementwise(f32(Y[rows_t]), fwd.y3, F, "Y")
    bwd = oracle.sparse_ffn_bwd(dY[rows], X[rows], W1, W2, fwd)
    if M == 8:
        m24 = bits(view(ctx, binding.SF_CTX_Y2_META24).view(T, F // 16)[rows_t])
        assert np.array_equal(oracle.decompress24(bits(view(ctx, binding.SF_CTX_Y2_VALS24).view(T, F // 2)[rows_t]), m24),
                              fwd.act.dense)
        dy1_rows = oracle.decompress24(bits(view(ws, binding.SF_CTX_DY1_VALS24).view(T, F // 2)[rows_t]), m24)
    else:
        dy1_rows = oracle.decompress_vnm(bits(view(ws, binding.SF_CTX_DY1_VALS).view(T, 2 * G)[rows_t]),
                                         fwd.act.meta, fwd.act.colidx, V=V, M=M)
    assert rel_fro(oracle.bf16_to_f32(dy1_rows), oracle.bf16_to_f32(bwd.dy1_dense)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(dy1_rows), oracle.bf16_to_f32(bwd.dy1_dense), D, "dy1")
    assert rel_fro(f32(gX[rows_t]), bwd.dX) < TOL
    f64 = lambda b: oracle.bf16_to_f32(b).astype(np.float64)
    assert_close_elementwise(f32(gX[rows_t]), f64(dy1_rows) @ f64(W1), F, "dX")

    # ---- sample 2: four whole M-groups of features, all tokens -> columns of dW2, rows of dW1
    groups = [0, G // 3, (2 * G) // 3, G - 1]
    cols = np.concatenate([np.arange(g * M, (g + 1) * M) for g in groups])
    cols_t = torch.from_numpy(cols).cuda()
    y1_cols = bits(y1_dev[:, cols_t])
    act = oracle.vnm_sparsify(y1_cols, V=V, M=M)
    # the GPU's masks for these groups are the oracle's on the same pre-activations
    assert np.array_equal(cidx_dev[:, torch.tensor(groups).cuda()].cpu().numpy(), act.colidx)
    dW2_ref = f64(dY).T @ f64(act.dense)                                  # [D, |cols|]
    assert rel_fro(f32(gW2[:, cols_t]), dW2_ref) < TOL
    assert_close_elementwise(f32(gW2[:, cols_t]), dW2_ref, T, "dW2")
    w2s_cols = oracle.prune24(np.ascontiguousarray(W2[:, cols]), group_dim=0).dense   # groups along D
    dy2 = (f64(dY) @ f64(w2s_cols)).astype(np.float32)
    relu = np.maximum(oracle.bf16_to_f32(y1_cols), 0)
    dy1 = oracle.f32_to_bf16((np.float32(2.0) * dy2 * relu).astype(np.float32)).reshape(dy2.shape)
    dy1 = np.where(act.mask, dy1, np.uint16(0))
    dW1_ref = f64(dy1).T @ f64(X)                                          # [|cols|, D]
    assert rel_fro(f32(gW1[cols_t]), dW1_ref) < TOL

    # ---- the configuration the benchmark times keeps no y1: it must reproduce this run bit for bit
    saved = [t.clone() for t in (Y, gX, gW1, gW2)]
    saved_ctx = [view(ctx, f).clone() for f in (binding.SF_CTX_Y2_VALS, binding.SF_CTX_META, binding.SF_CTX_COLIDX)]
    del ctx, ws, Y, gX, gW1, gW2, y1_dev, vals_dev, relu_dev, meta_dev, cidx_dev
    torch.cuda.empty_cache()
    _, desc0, ctx0, ws0, outs0 = _full_step(cfg, 0)
    for a, b in zip(saved, outs0):
        assert torch.equal(a, b)
    for a, f in zip(saved_ctx, (binding.SF_CTX_Y2_VALS, binding.SF_CTX_META, binding.SF_CTX_COLIDX)):
        assert torch.equal(a, binding.sf_ctx_view(desc0, ctx0, f))


@pytest.mark.parametrize("rows,cols", synth.PRUNE_SWEEP_SHAPES)
def test_prune_sweep_full_size_sampled_rows(rows, cols):
    w = synth.prune_sweep_matrix(rows, cols, seed=1000 + rows % 97 + cols % 89, tie_frac=0.05)
    wd = to_dev(w)
    rng = np.random.default_rng(rows)
    for mode in (0, 1):
        vals, meta, _ = binding.sf_prune24_compress(wd, 1, mode)
        sample = np.sort(rng.choice(rows, size=192, replace=False))
        ref = oracle.prune24(w[sample], group_dim=1, mode=mode)
        st = torch.from_numpy(sample).cuda()
        assert np.array_equal(bits(meta[st]), ref.meta)
        assert np.array_equal(bits(vals[st]), ref.vals)
    # strided groups: sampled output rows are sampled input columns
    vals, meta, _ = binding.sf_prune24_compress(wd, 0, 0)
    sample = np.sort(rng.choice(cols, size=64, replace=False))
    ref = oracle.prune24(np.ascontiguousarray(w[:, sample]), group_dim=0, mode=0)
    st = torch.from_numpy(sample).cuda()
    assert np.array_equal(bits(meta[st]), ref.meta)
    assert np.array_equal(bits(vals[st]), ref.vals)


@pytest.mark.parametrize("V,M", [(64, 8), (128, 8), (64, 16), (128, 16)])
def test_act_sweep_full_size_sampled_blocks(V, M):
    T = F = 16384
    p = synth.act_sweep_matrix(T, F, seed=2000)
    vals, meta, colidx, relu, _ = binding.sf_vnm_sparsify_act(to_dev(p), V, M)
    torch.cuda.synchronize()
    blocks = [0, 7, T // V - 1]
    for b in blocks:
        ref = oracle.vnm_sparsify(p[b * V:(b + 1) * V], V=V, M=M)
        sl = slice(b * V, (b + 1) * V)
        assert np.array_equal(colidx[b].cpu().numpy(), ref.colidx[0])
        assert np.array_equal(bits(meta[sl]), ref.meta)
        assert np.array_equal(bits(vals[sl]), ref.vals)
        assert np.array_equal(bits(relu[sl]), ref.relu_vals)
    # the sparsity the paper quotes for trained models: about 90 % zeros before the format's own pruning
    zero_frac = float((oracle.bf16_to_f32(p[:1024]) <= 0).mean())
    assert 0.88 < zero_frac < 0.93


@pytest.mark.parametrize("E", [2, 16])
def test_routed_step_full_size_sampled(E):
    """The routed step at the d_model = 4096 layer's full size (the shape bench.py times). Sampled
    tokens give exact restrictions for Y, dy1 and dX (a token only needs its own row and its expert's
    block); sampled groups of four features give exact restrictions for dW2 / dW1 (a feature's
    gradient sums over the tokens of its expert, whose activations only need the four features)."""
    from oracle import router as R
    T, D, F = 8192, 4096, 16384
    Fe = F // E
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, 0.02, 4)
    means = synth.normal_bf16((E, D), 0.0, 1.0, 4, 9)
    desc = binding.make_router_desc(T, D, F, E, flags=binding.SF_FFN_SAVE_Y1)
    nctx, nws = binding.sf_routed_ffn_workspace_size(desc)
    gctx, gws = Guarded(nctx, zero=True), Guarded(nws, zero=True)
    dX_, dW1_, dW2_, ddY, dM = (to_dev(a) for a in (X, W1, W2, dY, means))
    outs = [Guarded((T, D), torch.bfloat16), Guarded((T, D), torch.bfloat16), Guarded((F, D), torch.bfloat16),
            Guarded((D, F), torch.bfloat16)]
    Y, gX, gW1, gW2 = (o.t for o in outs)
    binding.sf_routed_ffn_fwd(desc, dX_, dW1_, dW2_, dM, Y, gctx.t, gws.t)
    binding.sf_routed_ffn_bwd(desc, ddY, dX_, dW1_, dW2_, gctx.t, gX, gW1, gW2, gws.t)
    assert binding.sf_check_status(gws.t) == binding.SF_OK
    for g, nm in zip([gctx, gws] + outs, ["context", "workspace", "Y", "dX", "dW1", "dW2"]):
        g.check(nm)
    view = lambda buf, f: binding.sf_routed_ctx_view(desc, buf, f)
    expert = view(gctx.t, binding.SF_RCTX_EXPERT).cpu().numpy()
    row = view(gctx.t, binding.SF_RCTX_ROW_OF_TOKEN).cpu().numpy()
    ref_expert, ref_logits = R.route(X, means)
    assert (expert == ref_expert).mean() > 0.995                      # near ties may differ (float32 accumulation)
    rows_max = view(gctx.t, binding.SF_RCTX_SRC_OF_ROW).numel()
    y1_dev = view(gctx.t, binding.SF_RCTX_Y1).view(rows_max, Fe)
    vals_dev = view(gctx.t, binding.SF_RCTX_Y2_VALS).view(rows_max, Fe // 2)
    meta_dev = view(gctx.t, binding.SF_RCTX_META).view(rows_max, Fe // 16)
    dy1_dev = view(gws.t, binding.SF_RCTX_DY1_VALS).view(rows_max, Fe // 2)
    f64 = lambda b: oracle.bf16_to_f32(b).astype(np.float64)

    # ---- sample 1: 96 tokens spread over the batch
    toks = np.sort(np.random.default_rng(E).choice(T, size=96, replace=False))
    rt = torch.from_numpy(row[toks].astype(np.int64)).cuda()
    y1_rows = bits(y1_dev[rt])
    free = R.routed_ffn_fwd(X[toks], W1, W2, means, E, forced_expert=expert[toks])
    cols = expert[toks][:, None].astype(np.int64) * Fe + np.arange(Fe)[None, :]
    free_y1 = np.take_along_axis(free.y1b, cols, axis=1)
    assert rel_fro(oracle.bf16_to_f32(y1_rows), oracle.bf16_to_f32(free_y1)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(y1_rows), oracle.bf16_to_f32(free_y1), D, "y1")
    fwd = R.routed_ffn_fwd(X[toks], W1, W2, means, E, forced_expert=expert[toks], forced_y1b=y1_rows)
    m_rows = bits(meta_dev[rt])
    assert np.array_equal(oracle.decompress24(bits(vals_dev[rt]), m_rows), np.take_along_axis(fwd.y2, cols, axis=1))
    tt = torch.from_numpy(toks).cuda()
    assert rel_fro(f32(Y[tt]), fwd.y3) < TOL
    assert_close_elementwise(f32(Y[tt]), fwd.y3, Fe, "Y")
    bwd = R.routed_ffn_bwd(dY[toks], X[toks], W1, W2, fwd)
    dy1_rows = oracle.decompress24(bits(dy1_dev[rt]), m_rows)
    ref_dy1 = np.take_along_axis(bwd.dy1, cols, axis=1)
    assert rel_fro(oracle.bf16_to_f32(dy1_rows), oracle.bf16_to_f32(ref_dy1)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(dy1_rows), oracle.bf16_to_f32(ref_dy1), D, "dy1")
    dy1_full = np.zeros((len(toks), F), dtype=np.uint16)
    np.put_along_axis(dy1_full, cols, dy1_rows, axis=1)
    dX_ref = f64(dy1_full) @ f64(W1)
    assert rel_fro(f32(gX[tt]), dX_ref) < TOL
    assert_close_elementwise(f32(gX[tt]), dX_ref, Fe, "dX")

    # ---- sample 2: groups of four features of three experts, all tokens of those experts
    for e in sorted({0, E // 2, E - 1}):
        te = np.flatnonzero(expert == e)
        rte = torch.from_numpy(row[te].astype(np.int64)).cuda()
        fl = np.concatenate([np.arange(4 * g, 4 * g + 4) for g in (0, Fe // 8, Fe // 4 - 1)])     # local features
        flt = torch.from_numpy(fl).cuda()
        y1g = bits(y1_dev[rte][:, flt])
        hb, relu = oracle.vnm.squared_relu_bf16(y1g)
        _, keep = R._select_top2_of4((hb & np.uint16(0x7FFF)).reshape(len(te), -1, 4))
        keep = keep.reshape(len(te), -1)
        y2g = np.where(keep, hb, np.uint16(0))
        gf = e * Fe + fl                                                            # global features
        gft = torch.from_numpy(gf).cuda()
        dW2_ref = f64(dY[te]).T @ f64(y2g)
        assert rel_fro(f32(gW2[:, gft]), dW2_ref) < TOL
        assert_close_elementwise(f32(gW2[:, gft]), dW2_ref, len(te), "dW2")
        w2s = oracle.prune24(np.ascontiguousarray(W2[:, gf]), group_dim=0).dense
        dy2 = (f64(dY[te]) @ f64(w2s)).astype(np.float32)
        dy1g = oracle.f32_to_bf16((np.float32(2.0) * dy2 * oracle.bf16_to_f32(relu)).astype(np.float32)).reshape(dy2.shape)
        dy1g = np.where(keep, dy1g, np.uint16(0))
        dW1_ref = f64(dy1g).T @ f64(X[te])
        assert rel_fro(f32(gW1[gft]), dW1_ref) < TOL


@pytest.mark.parametrize("m,n,k", [(4096, 16384, 4096), (8192, 4096, 16384)])
def test_fp8_products_full_size_sampled(m, n, k):
    """The E4M3 route at the micro-benchmark's shapes: prune + quantise on the GPU checked bit for bit on sampled
    rows, the dense and the 2:4 product on sampled rows x sampled columns against float64 products of the
    oracle's codes."""
    from oracle import fp8
    w = synth.prune_sweep_matrix(m, k, seed=31, tie_frac=0.02)
    x = synth.normal_bf16((n, k), 0, 1, seed=32)
    sw, sx = 3000.0, 32.0
    alpha = 1.0 / (sw * sx)
    wd, xd = to_dev(w), to_dev(x)
    vals, meta, _ = binding.sf_prune24_compress_fp8(wd, 0, sw)
    wq, xq = binding.sf_fp8_quantize(wd, sw), binding.sf_fp8_quantize(xd, sx)
    outs = Guarded((m, n), torch.bfloat16), Guarded((m, n), torch.bfloat16)
    Cs, ws = binding.sf_gemm_fp8_sparse24(vals, meta, xq, alpha, C_out=outs[0].t)
    assert binding.sf_check_status(ws) == binding.SF_OK
    Cd, ws = binding.sf_gemm_fp8_dense(wq, xq, alpha, C_out=outs[1].t)
    assert binding.sf_check_status(ws) == binding.SF_OK
    for o in outs:
        o.check("fp8 product")
    rng = np.random.default_rng(m + n)
    rows = np.sort(np.concatenate([rng.choice(m, size=93, replace=False), [0, m - 129, m - 1]]))
    cols = np.sort(np.concatenate([rng.choice(n, size=381, replace=False), [0, n - 225, n - 1]]))
    rt, ct = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    p = fp8.prune24_fp8(w[rows], sw)
    assert np.array_equal(vals[rt].cpu().numpy(), p.vals) and np.array_equal(bits(meta[rt]), p.meta)
    xq_ref = fp8.quantize_fp8(x[cols], sx)
    assert np.array_equal(xq[ct].cpu().numpy(), xq_ref)
    for C, a_codes, what in ((Cs, p.dense, "fp8 2:4 product"), (Cd, fp8.quantize_fp8(w[rows], sw), "fp8 dense product")):
        got = f32(C[rt][:, ct])
        ref = fp8.gemm_fp8(a_codes, xq_ref, alpha)
        assert rel_fro(got, ref) < TOL, what
        assert_close_elementwise(got, ref, k, what)
