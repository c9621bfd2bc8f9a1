"""Stand-alone throughput sweeps of the bandwidth kernels and single products (one JSON line each).

    python -m paper_2602_06183_b200.sweeps [--which prune,act,gemm,c5,mma,power]

prune: 2:4 prune + compress on the weight shapes of the sweep configuration (both group directions,
       hard and soft), GB/s at 3.125 algorithmic bytes per element.
act:   SquaredReLU + V:N:M sparsify on 16384 x 16384 pre-activations with ~90 % negatives,
       V in {64, 128}, M in {8, 16}.
gemm:  dense vs 2:4 vs Venom products at the paper's micro-benchmark shape (m, n, k) = (4096, 16384, 4096)
       and at the FFN shapes.
c5:    sparse and dense step of the d_model = 8192 layer.
mma:   clocks per tcgen05.mma issued back to back from shared memory (dense / 2:4, one CTA / CTA pair):
       what the tensor pipe can do for the product kernels' tile shapes.
power: seconds-long loops of the dense and the 2:4 product on random and on all-zero operands with
       SM clock and board power sampled by nvidia-smi: separates the power cap from the kernel.
Inputs larger than the L2; times are CUDA-event averages over 20 launches after 3 warm-ups.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    return json.load(open(p))["hbm_gbs"] if os.path.exists(p) else 6650.0


def _time(fn, iters=20, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def prune_sweep():
    peak = _hbm_peak()
    for i, (rows, cols) in enumerate(synth.PRUNE_SWEEP_SHAPES):
        w = _dev(synth.prune_sweep_matrix(rows, cols, seed=1000 + i))
        for group_dim in (1, 0):
            for mode in (0, 1):
                out = binding.sf_prune24_compress(w, group_dim, mode)
                ms = _time(lambda: binding.sf_prune24_compress(w, group_dim, mode, out=out))
                gbs = 3.125 * rows * cols / (ms / 1e3) / 1e9
                print(json.dumps({"kernel": "prune24_compress", "rows": rows, "cols": cols, "group_dim": group_dim,
                                  "prune_mode": mode, "us": ms * 1e3, "GBps": gbs, "frac_of_measured_hbm": gbs / peak}))


def act_sweep():
    peak = _hbm_peak()
    T = F = 16384
    p = _dev(synth.act_sweep_matrix(T, F, seed=2000))
    for V in (64, 128):
        for M in (8, 16):
            out = binding.sf_vnm_sparsify_act(p, V, M)
            ms = _time(lambda: binding.sf_vnm_sparsify_act(p, V, M, out=out))
            nbytes = T * F * (2 + 4.0 / M + 4.0 / M + 0.5 / M) + (T // V) * (F // M) * 4
            gbs = nbytes / (ms / 1e3) / 1e9
            print(json.dumps({"kernel": "vnm_sparsify_act", "T": T, "F": F, "V": V, "M": M, "us": ms * 1e3,
                              "bytes_per_element": nbytes / (T * F), "GBps": gbs, "frac_of_measured_hbm": gbs / peak}))


def gemm_sweep():
    for (m, n, k) in [(4096, 16384, 4096), (16384, 8192, 4096), (8192, 4096, 16384)]:
        A = torch.randn((m, k), device="cuda").to(torch.bfloat16)
        B = torch.randn((n, k), device="cuda").to(torch.bfloat16)
        C = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
        ws = torch.zeros((binding.sf_gemm_workspace_size(m, k),), dtype=torch.uint8, device="cuda")
        ms_d = _time(lambda: binding.sf_gemm_dense(A, True, B, True, C_out=C, workspace=ws))
        vals, meta, _ = binding.sf_prune24_compress(A, 1, 0)
        ms_p = _time(lambda: binding.sf_prune24_compress(A, 1, 0, out=(vals, meta, None)))
        ms_s = _time(lambda: binding.sf_gemm_sparse24_rm(vals, meta, B, True, C_out=C, workspace=ws))
        fl = 2.0 * m * n * k
        print(json.dumps({"shape_mnk": [m, n, k], "dense_ms": ms_d, "dense_tflops": fl / ms_d / 1e9,
                          "sparse24_ms": ms_s, "sparse24_dense_equiv_tflops": fl / ms_s / 1e9,
                          "prune_ms": ms_p, "speedup_gemm_only": ms_d / ms_s,
                          "speedup_with_prune": ms_d / (ms_s + ms_p)}))
    # Venom (condensed operand, gathered B rows) at the sparsities of Table 5 and below
    T, F, N = 8192, 16384, 4096
    A = torch.randn((T, F), device="cuda").to(torch.bfloat16)
    Bd = torch.randn((N, F), device="cuda").to(torch.bfloat16)
    Cd = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    wsd = torch.zeros((binding.sf_gemm_workspace_size(T, F),), dtype=torch.uint8, device="cuda")
    ms_dense = _time(lambda: binding.sf_gemm_dense(A, True, Bd, True, C_out=Cd, workspace=wsd))
    del A, Bd, Cd
    for M in (8, 16, 32, 64):
        G = F // M
        P = _dev(synth.normal_bf16((T, F), 0.0, 1.0, seed=7))
        vals, meta, colidx, _, _ = binding.sf_vnm_sparsify_act(P, 128, M)
        Bt = torch.randn((F, N), device="cuda").to(torch.bfloat16)
        C = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
        ws = torch.zeros((binding.sf_gemm_workspace_size(T, F),), dtype=torch.uint8, device="cuda")
        ms_v = _time(lambda: binding.sf_gemm_venom(vals, meta, colidx, Bt, 128, M, C_out=C, workspace=ws))
        print(json.dumps({"kernel": "gemm_venom", "T": T, "F": F, "N": N, "V": 128, "M": M,
                          "sparsity_pct": 100.0 * (1 - 2.0 / M), "ms": ms_v, "dense_ms": ms_dense,
                          "speedup_vs_dense": ms_dense / ms_v, "dense_equiv_tflops": 2.0 * T * F * N / ms_v / 1e9}))


def c5_step():
    cfg = synth.FFN_CONFIGS["c5_d8192"]
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    X, W1, W2, dY = (_dev(a) for a in synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"]))
    desc = binding.make_desc(T, D, F, V, M)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(X), torch.empty_like(W1), torch.empty_like(W2)

    def sparse():
        binding.sf_sparse_ffn_fwd(desc, X, W1, W2, Y, ctx, ws)
        binding.sf_sparse_ffn_bwd(desc, dY, X, W1, W2, ctx, gX, gW1, gW2, ws)

    def dense():
        binding.sf_dense_ffn_fwd(desc, X, W1, W2, Y, ctx, ws)
        binding.sf_dense_ffn_bwd(desc, dY, X, W1, W2, ctx, gX, gW1, gW2, ws)

    ms_s, ms_d = _time(sparse, iters=10), _time(dense, iters=10)
    fl = 12.0 * T * D * F
    print(json.dumps({"workload": "c5_d8192", "sparse_step_ms": ms_s, "dense_step_ms": ms_d,
                      "sparse_dense_equiv_tflops": fl / ms_s / 1e9, "dense_tflops": fl / ms_d / 1e9,
                      "speedup": ms_d / ms_s, "status": binding.sf_check_status(ws)}))


def mma_rate():
    for sparse, two in [(False, False), (True, False), (False, True), (True, True)]:
        clk = binding.sf_probe_mma_rate(sparse, two)
        macs = 128 * 256 * (32 if sparse else 16)               # dense-equivalent MACs per instruction per SM
        print(json.dumps({"probe": "mma_rate", "operand": "2:4" if sparse else "dense",
                          "cta_group": 2 if two else 1, "tile_per_cta": [128, 256, 32 if sparse else 16],
                          "clk_per_mma": round(clk, 1), "dense_equiv_flop_per_clk_per_sm": round(2 * macs / clk)}))


def _sampled_loop(fn, seconds=2.5):
    """Run fn back to back for `seconds`; median SM clock / power over the last two thirds of the samples."""
    import statistics
    import subprocess
    import time
    q = "clocks.sm,power.draw,clocks_event_reasons.sw_power_cap,clocks_event_reasons.hw_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown"
    dev = str(torch.cuda.current_device())
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        dev = vis.split(",")[int(dev)]
    p = subprocess.Popen(["nvidia-smi", "-i", dev, f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "50"],
                         stdout=subprocess.PIPE, text=True)
    for _ in range(10):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n, t0 = 0, time.time()
    e0.record()
    while time.time() - t0 < seconds:
        for _ in range(50):
            fn()
        n += 50
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    p.terminate()
    rows = [l.split(", ") for l in p.communicate()[0].strip().splitlines() if l.count(",") >= 4]
    rows = rows[len(rows) // 3:] or [["0", "0", "", "", ""]]
    return {"ms": e0.elapsed_time(e1) / n,
            "sm_mhz_median": statistics.median(float(r[0]) for r in rows),
            "power_w_median": statistics.median(float(r[1]) for r in rows),
            "sw_power_cap_share": sum(r[2].strip() == "Active" for r in rows) / len(rows),
            "hw_or_thermal_slowdown_samples": sum(r[3].strip() == "Active" or r[4].strip() == "Active" for r in rows)}


def power_loops():
    m, n, k = 16384, 8192, 4096
    fl = 2.0 * m * n * k
    for data in ("randn", "zeros"):
        gen = (lambda s: torch.randn(s, device="cuda")) if data == "randn" else (lambda s: torch.zeros(s, device="cuda"))
        A, B = gen((m, k)).to(torch.bfloat16), gen((n, k)).to(torch.bfloat16)
        C = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
        ws = torch.zeros((binding.sf_gemm_workspace_size(m, k),), dtype=torch.uint8, device="cuda")
        vals, meta, _ = binding.sf_prune24_compress(A, 1, 0)
        for kind, fn in [("dense", lambda: binding.sf_gemm_dense(A, True, B, True, C_out=C, workspace=ws)),
                         ("sparse24", lambda: binding.sf_gemm_sparse24_rm(vals, meta, B, True, C_out=C, workspace=ws))]:
            r = _sampled_loop(fn)
            r.update({"probe": "sustained_loop", "data": data, "kernel": kind, "shape_mnk": [m, n, k],
                      "dense_equiv_tflops": fl / r["ms"] / 1e9,
                      "tflops_per_ghz": fl / r["ms"] / 1e9 / max(r["sm_mhz_median"] / 1e3, 1e-9)})
            print(json.dumps(r))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--which", default="prune,act,gemm,c5")
    args = ap.parse_args()
    from . import build
    build.build()
    for w in args.which.split(","):
        {"prune": prune_sweep, "act": act_sweep, "gemm": gemm_sweep, "c5": c5_step, "mma": mma_rate,
         "power": power_loops}[w]()


if __name__ == "__main__":
    main()
