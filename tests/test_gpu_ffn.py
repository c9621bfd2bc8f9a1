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
from util import to_dev, bits, f32, rel_fro

pytestmark = pytest.mark.gpu
TOL = 1e-2


def _run_sparse(cfg, prune_mode=0, act_shift=0.0):
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"], act_shift=act_shift)
    desc = binding.make_desc(T, D, F, V, M, prune_mode=prune_mode, flags=1)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, W2, dY))
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)
    binding.sf_sparse_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    binding.sf_sparse_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    G = F // M
    out = dict(
        y1=bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_Y1)).reshape(T, F),
        y2_vals=bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_Y2_VALS)).reshape(T, 2 * G),
        relu_vals=bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_RELU_VALS)).reshape(T, 2 * G),
        meta=bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_META)).reshape(T, G // 4),
        colidx=binding.sf_ctx_view(desc, ctx, binding.SF_CTX_COLIDX).cpu().numpy().reshape(T // V, G, 4),
        dy1_vals=bits(binding.sf_ctx_view(desc, ws, binding.SF_CTX_DY1_VALS)).reshape(T, 2 * G),
        Y=f32(Y), dX=f32(gX), dW1=f32(gW1), dW2=f32(gW2))
    return (X, W1, W2, dY), out


@pytest.mark.parametrize("prune_mode,act_shift", [(0, 0.0), (1, 0.0), (0, -1.3)])
def test_sparse_ffn_c1_teacher_forced(prune_mode, act_shift):
    cfg = synth.FFN_CONFIGS["c1_small"]
    (X, W1, W2, dY), g = _run_sparse(cfg, prune_mode, act_shift)
    V, M = cfg["V"], cfg["M"]
    # stage 1: the GPU's y1 against the oracle's own product with the pruned W1
    free = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, prune_mode=prune_mode)
    assert rel_fro(oracle.bf16_to_f32(g["y1"]), oracle.bf16_to_f32(free.y1b)) < TOL
    # stage 2: selection on the GPU's y1 must agree bit for bit
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, prune_mode=prune_mode, forced_y1b=g["y1"])
    assert np.array_equal(g["colidx"], fwd.act.colidx)
    assert np.array_equal(g["meta"], fwd.act.meta)
    assert np.array_equal(g["y2_vals"], fwd.act.vals)
    assert np.array_equal(g["relu_vals"], fwd.act.relu_vals)
    # stage 3: products with those masks
    assert rel_fro(g["Y"], fwd.y3) < TOL
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd, prune_mode=prune_mode)
    assert rel_fro(oracle.bf16_to_f32(g["dy1_vals"]), oracle.bf16_to_f32(bwd.dy1_vals)) < TOL
    assert rel_fro(g["dX"], bwd.dX) < TOL
    assert rel_fro(g["dW1"], bwd.dW1) < TOL
    assert rel_fro(g["dW2"], bwd.dW2) < TOL
    # free-running comparison: masks may differ in a few near-tie blocks only
    disagree = float((free.act.colidx != g["colidx"]).any(axis=-1).mean())
    assert disagree < 0.05
    assert rel_fro(g["Y"], free.y3) < 5e-2


@pytest.mark.parametrize("M,act_shift", [(8, 0.0), (8, -1.3), (4, 0.0)])
def test_plain_24_view_of_y2_and_dy1_is_exact(M, act_shift):
    """For M <= 8 the products consume y2 / dy1 as plain 2:4 operands over all F columns. That view,
    decompressed with its own metadata, must be the oracle's masked dense y2 bit for bit, hold at
    most two entries per four columns with ascending positions, and dy1's view must be the masked
    dense dy1 at the same positions."""
    cfg = dict(synth.FFN_CONFIGS["c1_small"], M=M)
    T, D, F, V = cfg["T"], cfg["D"], cfg["F"], cfg["V"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"], act_shift=act_shift)
    desc = binding.make_desc(T, D, F, V, M, flags=1)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, W2, dY))
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)
    binding.sf_sparse_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
    binding.sf_sparse_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
    y1 = bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_Y1)).reshape(T, F)
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, forced_y1b=y1)
    v24 = bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_Y2_VALS24)).reshape(T, F // 2)
    m24 = bits(binding.sf_ctx_view(desc, ctx, binding.SF_CTX_Y2_META24)).reshape(T, F // 16)
    nib = np.stack([(m24 >> np.uint16(4 * i)) & np.uint16(0xF) for i in range(4)], axis=-1)
    assert ((nib & 3) < (nib >> 2)).all()                        # legal position pairs everywhere
    assert np.array_equal(oracle.decompress24(v24, m24), fwd.act.dense)
    # dy1 in the same positions: compare with the masked dense dy1 the oracle derives from the GPU's masks
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd)
    d24 = bits(binding.sf_ctx_view(desc, ws, binding.SF_CTX_DY1_VALS24)).reshape(T, F // 2)
    dy1_gpu = oracle.decompress24(d24, m24)
    dy1_ref = oracle.decompress_vnm(bwd.dy1_vals, fwd.act.meta, fwd.act.colidx, V=V, M=M)
    assert not (dy1_gpu[~fwd.act.mask] != 0).any()               # nothing outside y2's mask
    assert rel_fro(oracle.bf16_to_f32(dy1_gpu), oracle.bf16_to_f32(dy1_ref)) < TOL


def test_sparse_ffn_v128_m16():
    cfg = dict(T=512, D=256, F=2048, V=128, N=2, M=16, sigma_w=0.05, seed=17)
    (X, W1, W2, dY), g = _run_sparse(cfg)
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=128, M=16, forced_y1b=g["y1"])
    assert np.array_equal(g["colidx"], fwd.act.colidx) and np.array_equal(g["meta"], fwd.act.meta)
    assert np.array_equal(g["y2_vals"], fwd.act.vals)
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd)
    for k, ref in (("Y", fwd.y3), ("dX", bwd.dX), ("dW1", bwd.dW1), ("dW2", bwd.dW2)):
        assert rel_fro(g[k], ref) < TOL, k


@pytest.mark.parametrize("V,M", [(64, 4), (128, 32)])
def test_sparse_ffn_other_group_widths(V, M):
    """M = 4 is 2:4 activation sparsity (every column kept, the plain-2:4 path); M = 32 runs the
    condensed, gathered Venom product."""
    cfg = dict(T=512, D=256, F=2048, V=V, N=2, M=M, sigma_w=0.05, seed=23 + M)
    (X, W1, W2, dY), g = _run_sparse(cfg)
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, forced_y1b=g["y1"])
    assert np.array_equal(g["colidx"], fwd.act.colidx) and np.array_equal(g["meta"], fwd.act.meta)
    assert np.array_equal(g["y2_vals"], fwd.act.vals)
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd)
    for k, ref in (("Y", fwd.y3), ("dX", bwd.dX), ("dW1", bwd.dW1), ("dW2", bwd.dW2)):
        assert rel_fro(g[k], ref) < TOL, k


@pytest.mark.parametrize("T,D,F,V,M", [(256, 256, 256, 128, 8), (256, 256, 256, 64, 8), (512, 512, 512, 128, 16),
                                       (768, 256, 1280, 128, 8)])
def test_sparse_ffn_smallest_and_odd_tile_counts(T, D, F, V, M):
    """One tile per product, fewer k-blocks than pipeline stages, tile counts that are not a
    multiple of the raster band."""
    cfg = dict(T=T, D=D, F=F, V=V, N=2, M=M, sigma_w=0.05, seed=T + F + V)
    (X, W1, W2, dY), g = _run_sparse(cfg)
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, forced_y1b=g["y1"])
    assert np.array_equal(g["colidx"], fwd.act.colidx) and np.array_equal(g["meta"], fwd.act.meta)
    assert np.array_equal(g["y2_vals"], fwd.act.vals)
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd)
    for k, ref in (("Y", fwd.y3), ("dX", bwd.dX), ("dW1", bwd.dW1), ("dW2", bwd.dW2)):
        assert rel_fro(g[k], ref) < TOL, k


def test_dense_ffn_c1():
    cfg = synth.FFN_CONFIGS["c1_small"]
    T, D, F = cfg["T"], cfg["D"], cfg["F"]
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"])
    desc = binding.make_desc(T, D, F, cfg["V"], cfg["M"])
    ctx, ws = binding.alloc_ffn_buffers(desc)
    dX_, dW1_, dW2_, dY_ = (to_dev(a) for a in (X, W1, W2, dY))
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)
    binding.sf_dense_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
    binding.sf_dense_ffn_bwd(desc, dY_, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)
    assert binding.sf_check_status(ws) == binding.SF_OK
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
    desc = binding.make_desc(1000, 256, 1024, 64, 8)
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
    """Seeded draw of legal step shapes: T, D, F multiples of 256, V in {64, 128}, M in {4..32},
    condensed reduction 4F/M a multiple of 128, both prune modes, symmetric or ~90 %-negative
    pre-activations."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        T, D, F = (int(rng.integers(1, 4)) * 256 for _ in range(3))
        F *= int(rng.integers(1, 3))
        V, M = int(rng.choice([64, 128])), int(rng.choice([4, 8, 16, 32]))
        if (4 * F // M) % 128:
            continue
        out.append((T, D, F, V, M, int(rng.integers(0, 2)), float(rng.choice([0.0, -1.3])), int(rng.integers(1, 1 << 20))))
    return out


@pytest.mark.parametrize("T,D,F,V,M,prune_mode,act_shift,seed", _legal_random_configs(10, seed=20260206))
def test_sparse_ffn_random_legal_shapes(T, D, F, V, M, prune_mode, act_shift, seed):
    cfg = dict(T=T, D=D, F=F, V=V, N=2, M=M, sigma_w=0.05, seed=seed)
    (X, W1, W2, dY), g = _run_sparse(cfg, prune_mode, act_shift)
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M, prune_mode=prune_mode, forced_y1b=g["y1"])
    assert np.array_equal(g["colidx"], fwd.act.colidx) and np.array_equal(g["meta"], fwd.act.meta)
    assert np.array_equal(g["y2_vals"], fwd.act.vals) and np.array_equal(g["relu_vals"], fwd.act.relu_vals)
    bwd = oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd, prune_mode=prune_mode)
    for k, ref in (("Y", fwd.y3), ("dX", bwd.dX), ("dW1", bwd.dW1), ("dW2", bwd.dW2)):
        assert rel_fro(g[k], ref) < TOL, k
