"""Parity of the routed FFN step (neuron-level experts, Section 3.1 / Algorithm 3) with the oracle.

Protocol. Routing takes an integer decision from floating-point logits, and the device accumulates
them in float32: the test checks that every device decision is a valid arg-max within the
accumulation error (and equal to the oracle's wherever the margin is clear), then teacher-forces the
oracle with the device's routing and the device's bf16 pre-activations. From there on everything
integer (token order, kept positions, metadata, packed values) must match bit for bit and every
product within the element-wise bound and 1e-2 relative Frobenius error.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import router as R
from paper_2602_06183_b200 import binding, synth
from util import to_dev, bits, f32, rel_fro, assert_close_elementwise, Guarded

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _nibbles(meta):
    return np.stack([(meta >> np.uint16(4 * i)) & np.uint16(0xF) for i in range(4)], axis=-1).reshape(meta.shape[0], -1)


def _run(T, D, F, E, seed, prune_mode=0, forced=None, skew=None, fit=False):
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, 0.05, seed)
    means = synth.normal_bf16((E, D), 0.0, 1.0, seed, 9)
    if fit:                                    # the whole offline recipe: cluster, renumber the hidden features
        _, perm, means = binding.sf_router_fit_host(W1, E, iters=2)
        W1, W2 = np.ascontiguousarray(W1[perm]), np.ascontiguousarray(W2[:, perm])
    if skew is not None:                       # a shared component in the tokens that one expert's mean picks up
        m, x = oracle.bf16_to_f32(means).copy(), oracle.bf16_to_f32(X).copy()
        x[:, 0] = 2.0
        m[skew, 0] = 24.0
        means, X = oracle.f32_to_bf16(m).reshape(E, D), oracle.f32_to_bf16(x).reshape(T, D)
    desc = binding.make_router_desc(T, D, F, E, prune_mode=prune_mode, flags=binding.SF_FFN_SAVE_Y1)
    nctx, nws = binding.sf_routed_ffn_workspace_size(desc)
    gctx, gws = Guarded(nctx, zero=True), Guarded(nws, zero=True)
    dX_, dW1_, dW2_, dY_, dM = (to_dev(a) for a in (X, W1, W2, dY, means))
    outs = [Guarded((T, D), torch.bfloat16), Guarded((T, D), torch.bfloat16), Guarded((F, D), torch.bfloat16),
            Guarded((D, F), torch.bfloat16)]
    Y, gX, gW1, gW2 = (o.t for o in outs)
    fe = None if forced is None else torch.from_numpy(forced.astype(np.int32)).cuda()
    binding.sf_routed_ffn_fwd(desc, dX_, dW1_, dW2_, dM, Y, gctx.t, gws.t, forced_expert=fe)
    assert binding.sf_check_status(gws.t) == binding.SF_OK
    binding.sf_routed_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, gctx.t, gX, gW1, gW2, gws.t)
    assert binding.sf_check_status(gws.t) == binding.SF_OK
    for g, nm in zip([gctx, gws] + outs, ["context", "workspace", "Y", "dX", "dW1", "dW2"]):
        g.check(nm)
    view = lambda buf, f: binding.sf_routed_ctx_view(desc, buf, f)
    Fe = F // E
    rows = view(gctx.t, binding.SF_RCTX_SRC_OF_ROW).numel()
    g = dict(expert=view(gctx.t, binding.SF_RCTX_EXPERT).cpu().numpy(),
             row_of_token=view(gctx.t, binding.SF_RCTX_ROW_OF_TOKEN).cpu().numpy(),
             src_of_row=view(gctx.t, binding.SF_RCTX_SRC_OF_ROW).cpu().numpy(),
             seg=view(gctx.t, binding.SF_RCTX_SEGMENTS).cpu().numpy(),
             logits=view(gctx.t, binding.SF_RCTX_LOGITS).view(T, E).cpu().numpy(),
             y1=bits(view(gctx.t, binding.SF_RCTX_Y1)).reshape(rows, Fe),
             vals=bits(view(gctx.t, binding.SF_RCTX_Y2_VALS)).reshape(rows, Fe // 2),
             relu=bits(view(gctx.t, binding.SF_RCTX_RELU_VALS)).reshape(rows, Fe // 2),
             meta=bits(view(gctx.t, binding.SF_RCTX_META)).reshape(rows, Fe // 16),
             dy1=bits(view(gws.t, binding.SF_RCTX_DY1_VALS)).reshape(rows, Fe // 2),
             Y=f32(Y), dX=f32(gX), dW1=f32(gW1), dW2=f32(gW2))
    return (X, W1, W2, dY, means), g


def _check(inputs, g, T, D, F, E, prune_mode=0, routed_by_device=True):
    X, W1, W2, dY, means = inputs
    Fe = F // E
    expert = g["expert"]
    # ---- step 1: the routing decision
    ref_expert, ref_logits = R.route(X, means)
    if routed_by_device:
        np.testing.assert_allclose(g["logits"], ref_logits, rtol=0, atol=2e-4 * np.abs(ref_logits).max() + 1e-3)
        top2 = np.sort(ref_logits, axis=1)[:, -2:] if E > 1 else np.stack([ref_logits[:, 0] - 1, ref_logits[:, 0]], 1)
        margin = top2[:, 1] - top2[:, 0]
        tol = 4e-4 * np.abs(ref_logits).max() + 2e-3
        assert np.array_equal(expert[margin > tol], ref_expert[margin > tol])          # clear winners agree
        chosen = ref_logits[np.arange(T), expert]
        assert (chosen >= ref_logits.max(axis=1) - tol).all()                          # near ties: still an arg-max
    # ---- step 2: stable grouping, segments padded to 256 rows
    seg, src, row = g["seg"], g["src_of_row"], g["row_of_token"]
    counts = np.bincount(expert, minlength=E)
    assert np.array_equal(seg[E + 1:], counts)
    exp_src, exp_start = R.token_order(expert, E, pad=256)
    pad_start = [0]
    for e in range(E):                                                                  # an empty expert keeps one zero tile
        pad_start.append(pad_start[-1] + max(256, -(-int(counts[e]) // 256) * 256))
    assert seg[: E + 1].tolist() == pad_start
    for e in range(E):
        t = np.flatnonzero(expert == e)
        assert np.array_equal(src[seg[e]: seg[e] + len(t)], t)                         # original order inside an expert
        assert (src[seg[e] + len(t): seg[e + 1]] == -1).all()
    assert np.array_equal(src[row], np.arange(T))
    used = seg[E]
    tok = src[:used]
    live = tok >= 0
    # ---- step 3, forward: teacher-forced on the device's routing and bf16 pre-activations
    y1_tok = np.zeros((T, Fe), dtype=np.uint16)
    y1_tok[tok[live]] = g["y1"][:used][live]
    free = R.routed_ffn_fwd(X, W1, W2, means, E, prune_mode=prune_mode, forced_expert=expert)
    cols = expert[:, None].astype(np.int64) * Fe + np.arange(Fe)[None, :]
    free_y1 = np.take_along_axis(free.y1b, cols, axis=1)
    assert rel_fro(oracle.bf16_to_f32(y1_tok), oracle.bf16_to_f32(free_y1)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(y1_tok), oracle.bf16_to_f32(free_y1), D, "y1")
    assert not g["y1"][:used][~live].any()                                              # padding rows hold zeros
    fwd = R.routed_ffn_fwd(X, W1, W2, means, E, prune_mode=prune_mode, forced_expert=expert, forced_y1b=y1_tok)
    nib = _nibbles(g["meta"][:used][live])
    assert np.array_equal(nib & 3, fwd.pos[tok[live], :, 0]) and np.array_equal(nib >> 2, fwd.pos[tok[live], :, 1])
    y2_blk = np.take_along_axis(fwd.y2, cols, axis=1)
    relu_blk = np.take_along_axis(fwd.relu, cols, axis=1)
    assert np.array_equal(oracle.decompress24(g["vals"][:used][live], g["meta"][:used][live]), y2_blk[tok[live]])
    assert np.array_equal(oracle.decompress24(g["relu"][:used][live], g["meta"][:used][live]), relu_blk[tok[live]])
    assert rel_fro(g["Y"], fwd.y3) < TOL
    assert_close_elementwise(g["Y"], fwd.y3, Fe, "Y")
    # ---- backward
    bwd = R.routed_ffn_bwd(dY, X, W1, W2, fwd, prune_mode=prune_mode)
    dy1_blk = np.take_along_axis(bwd.dy1, cols, axis=1)
    dy1_gpu = np.zeros((T, Fe), dtype=np.uint16)
    dy1_gpu[tok[live]] = oracle.decompress24(g["dy1"][:used][live], g["meta"][:used][live])
    assert rel_fro(oracle.bf16_to_f32(dy1_gpu), oracle.bf16_to_f32(dy1_blk)) < TOL
    assert_close_elementwise(oracle.bf16_to_f32(dy1_gpu), oracle.bf16_to_f32(dy1_blk), D, "dy1")
    dy1_full = np.zeros((T, F), dtype=np.uint16)
    np.put_along_axis(dy1_full, cols, dy1_gpu, axis=1)
    f64 = lambda b: oracle.bf16_to_f32(b).astype(np.float64)
    refs = dict(dX=f64(dy1_full) @ f64(W1), dW1=f64(dy1_full).T @ f64(X), dW2=bwd.dW2)
    for k, Kred in (("dX", Fe), ("dW1", T), ("dW2", T)):
        assert rel_fro(g[k], refs[k]) < TOL, k
        assert_close_elementwise(g[k], refs[k], Kred, k)
    assert rel_fro(g["dX"], bwd.dX) < TOL and rel_fro(g["dW1"], bwd.dW1) < TOL


@pytest.mark.parametrize("T,D,F,E", [(512, 256, 512, 2), (1024, 256, 1024, 4), (768, 512, 4096, 16), (256, 256, 256, 1)])
def test_routed_step_against_the_oracle(T, D, F, E):
    inputs, g = _run(T, D, F, E, seed=100 + E)
    _check(inputs, g, T, D, F, E)


def test_routed_step_soft_threshold_and_skewed_routing():
    """Most tokens on one expert, several experts nearly or entirely empty (their weight-gradient blocks
    must come out as exact zeros), soft-thresholded weights."""
    T, D, F, E = 1024, 256, 2048, 8
    inputs, g = _run(T, D, F, E, seed=7, prune_mode=1, skew=3)
    assert np.bincount(g["expert"], minlength=E)[3] > T // 2
    _check(inputs, g, T, D, F, E, prune_mode=1)
    # forcing every token onto two experts leaves the other six without tokens
    forced = (np.arange(T) % 2).astype(np.int32) * 5
    inputs, g = _run(T, D, F, E, seed=8, forced=forced)
    assert np.array_equal(g["expert"], forced)
    _check(inputs, g, T, D, F, E, routed_by_device=False)
    Fe = F // E
    for e in (1, 2, 3, 4, 6, 7):
        assert not g["dW1"][e * Fe:(e + 1) * Fe].any() and not g["dW2"][:, e * Fe:(e + 1) * Fe].any()


def test_routed_step_with_fitted_experts():
    """Offline fit on the host (balanced clusters, expert-major renumbering of W1's rows and W2's
    columns, means as the router's operand), then the step: the composition a user runs."""
    T, D, F, E = 512, 256, 1024, 4
    inputs, g = _run(T, D, F, E, seed=77, fit=True)
    _check(inputs, g, T, D, F, E)


def test_routed_step_without_saved_y1_and_repeated_is_bit_identical():
    """The benchmarked layout keeps no y1; two runs in a row on the same buffers and the run that saves
    y1 must produce the same bits everywhere (no atomics, no order-dependent accumulation)."""
    T, D, F, E = 768, 256, 1024, 4
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, 0.05, 55)
    means = synth.normal_bf16((E, D), 0.0, 1.0, 55, 9)
    dX_, dW1_, dW2_, dY_, dM = (to_dev(a) for a in (X, W1, W2, dY, means))
    results = []
    for flags in (0, 0, binding.SF_FFN_SAVE_Y1):
        desc = binding.make_router_desc(T, D, F, E, flags=flags)
        nctx, nws = binding.sf_routed_ffn_workspace_size(desc)
        if flags == 0 and results:
            pass                                   # second run re-uses the first run's dirty buffers
        else:
            ctx = torch.zeros((nctx,), dtype=torch.uint8, device="cuda")
            ws = torch.zeros((nws,), dtype=torch.uint8, device="cuda")
        Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
        gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)
        binding.sf_routed_ffn_fwd(desc, dX_, dW1_, dW2_, dM, Y, ctx, ws)
        binding.sf_routed_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
        assert binding.sf_check_status(ws) == binding.SF_OK
        results.append((Y, gX, gW1, gW2, binding.sf_routed_ctx_view(desc, ctx, binding.SF_RCTX_Y2_VALS).clone(),
                        binding.sf_routed_ctx_view(desc, ctx, binding.SF_RCTX_EXPERT).clone()))
    for other in results[1:]:
        for a, b in zip(results[0], other):
            assert torch.equal(a, b)


def test_routed_step_replays_from_a_cuda_graph():
    """Routing, grouping and the tile tables all stay on the device (no host round trip, no allocation), so the
    routed step can be captured once and replayed; a replay on different tokens must follow their routing."""
    T, D, F, E = 768, 256, 1024, 4
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, 0.05, 56)
    X2 = synth.ffn_inputs(T, D, F, 0.05, 57)[0]
    means = synth.normal_bf16((E, D), 0.0, 1.0, 56, 9)
    dXa, dXb, dW1_, dW2_, dY_, dM = (to_dev(a) for a in (X, X2, W1, W2, dY, means))
    desc = binding.make_router_desc(T, D, F, E)
    nctx, nws = binding.sf_routed_ffn_workspace_size(desc)
    ctx = torch.zeros((nctx,), dtype=torch.uint8, device="cuda")
    ws = torch.zeros((nws,), dtype=torch.uint8, device="cuda")
    Xin = dXa.clone()
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(Xin), torch.empty_like(dW1_), torch.empty_like(dW2_)

    def step():
        binding.sf_routed_ffn_fwd(desc, Xin, dW1_, dW2_, dM, Y, ctx, ws)
        binding.sf_routed_ffn_bwd(desc, dY_, Xin, dW1_, dW2_, ctx, gX, gW1, gW2, ws)

    eager = {}
    for name, src in (("a", dXa), ("b", dXb)):
        Xin.copy_(src)
        step()
        torch.cuda.synchronize()
        eager[name] = [t.clone() for t in (Y, gX, gW1, gW2)]
    assert not torch.equal(eager["a"][0], eager["b"][0])
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    for name, src in (("a", dXa), ("b", dXb), ("a", dXa)):
        Xin.copy_(src)
        for t in (Y, gX, gW1, gW2):
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert binding.sf_check_status(ws) == binding.SF_OK
        for a, b in zip(eager[name], (Y, gX, gW1, gW2)):
            assert torch.equal(a, b)


def test_routed_step_all_zero_tokens():
    """X = 0: every logit ties at zero, so every token goes to expert 0 (ties to the lower expert), the
    other experts keep one zero tile each, and all outputs are exactly zero."""
    T, D, F, E = 512, 256, 1024, 4
    _, W1, W2, dY = synth.ffn_inputs(T, D, F, 0.05, 9)
    X = np.zeros((T, D), dtype=np.uint16)
    means = synth.normal_bf16((E, D), 0.0, 1.0, 9, 9)
    desc = binding.make_router_desc(T, D, F, E)
    nctx, nws = binding.sf_routed_ffn_workspace_size(desc)
    ctx, ws = torch.zeros((nctx,), dtype=torch.uint8, device="cuda"), torch.zeros((nws,), dtype=torch.uint8, device="cuda")
    dX_, dW1_, dW2_, dY_, dM = (to_dev(a) for a in (X, W1, W2, dY, means))
    Y = torch.full((T, D), 3.0, dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.full_like(dX_, 3.0), torch.full_like(dW1_, 3.0), torch.full_like(dW2_, 3.0)
    binding.sf_routed_ffn_fwd(desc, dX_, dW1_, dW2_, dM, Y, ctx, ws)
    binding.sf_routed_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    assert not binding.sf_routed_ctx_view(desc, ctx, binding.SF_RCTX_EXPERT).any()
    seg = binding.sf_routed_ctx_view(desc, ctx, binding.SF_RCTX_SEGMENTS).cpu().numpy()
    assert seg.tolist() == [0, 512, 768, 1024, 1280, 512, 0, 0, 0]
    for t in (Y, gX, gW1, gW2):
        assert not bits(t).any()


def test_router_entry_point_alone():
    T, D, E = 2048, 512, 16
    X = synth.normal_bf16((T, D), 0, 1, seed=1)
    means = synth.normal_bf16((E, D), 0, 1, seed=2)
    expert, logits = binding.sf_router_route(to_dev(X), to_dev(means))
    ref_expert, ref_logits = R.route(X, means)
    np.testing.assert_allclose(logits.cpu().numpy(), ref_logits, rtol=0, atol=1e-3 * np.abs(ref_logits).max())
    assert (expert.cpu().numpy() == ref_expert).mean() > 0.995


def test_routed_desc_rejected_on_the_host():
    for bad in [(512, 256, 512, 3), (512, 256, 512, 32), (500, 256, 512, 2), (512, 256, 256, 2)]:
        with pytest.raises(binding.SparseFFNError) as e:
            binding.sf_routed_ffn_workspace_size(binding.make_router_desc(*bad))
        assert e.value.status == binding.SF_ERR_SHAPE
