#!/usr/bin/env python
"""Benchmark of the sparsified-FFN training step (fwd + bwd) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line (rank 0). A "step" is one pass of the whole hot path: 2:4 prune of W1,
sparse y1 product, SquaredReLU + V:N:M sparsify, Venom y3 product, 2:4 prune of W2, sparse dy1
product, dy1 pack, Venom dX product and the two weight-gradient products, on synthetic inputs of
the named workload (default: the d_model = 4096 FFN layer, 8192 tokens).

metric  = dense-equivalent TFLOP/s of the sparse step: 6 products x 2*T*D*F flop / step time.
N > 1   = N independent replicas of the layer (the path has no exchange step), launched by
          torchrun; the value is the aggregate over all ranks, timed as the max over ranks.
--impl reference times the CPU oracle (a deliberately plain numpy program) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "sparse_ffn_fwd_bwd_dense_equiv_tflops"
UNIT = "TFLOP/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = []
        for line in open(self.f.name):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 7:
                try:
                    rows.append((float(parts[0]), float(parts[1]), float(parts[2]), parts[3:7]))
                except ValueError:
                    pass
        os.unlink(self.f.name)
        if not rows:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        loaded = [r for r in rows if r[2] > 0.5 * max(x[2] for x in rows)] or rows
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in rows for i in range(4) if r[3][i].lower().startswith("active")})
        return dict(sm_mhz=float(np.median([r[0] for r in loaded])), sm_max_mhz=rows[0][1],
                    power_w_max=max(r[2] for r in rows), samples=len(rows), reasons=reasons)


def _oracle_step(X, W1, W2, dY, V, M):
    import oracle
    fwd = oracle.sparse_ffn_fwd(X, W1, W2, V=V, M=M)
    oracle.sparse_ffn_bwd(dY, X, W1, W2, fwd)


def _cpu_threads():
    """Threads the oracle's float64 products run on (numpy's BLAS pool); its element-wise parts
    (selection, rounding) are single-threaded numpy."""
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_06183_b200 import synth
    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    Ts, Fs = V, max(256, F // 8)                      # one V-block of tokens, a slice of the features
    X, W1, W2, dY = synth.ffn_inputs(Ts, D, Fs, cfg["sigma_w"], cfg["seed"])
    for _ in range(args.warmup):
        _oracle_step(X, W1, W2, dY, V, M)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        _oracle_step(X, W1, W2, dY, V, M)
    dt = time.perf_counter() - t0
    flops = 12.0 * Ts * D * Fs * args.steps
    val = flops / dt / 1e12
    sample = f"{Ts} tokens x d_model {D} x {Fs} of {F} features per step (full fwd+bwd incl. both weight prunings)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "T": T, "D": D, "F": F, "V": V, "N": 2, "M": M, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": _cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_2602_06183_b200 import binding, build, replicas, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback exists)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    binding.lib()

    T, D, F, V, M = cfg["T"], cfg["D"], cfg["F"], cfg["V"], cfg["M"]
    K, W = args.steps, args.warmup
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"] + rank)
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    hX, hW1, hW2, hdY = pin(X), pin(W1), pin(W2), pin(dY)
    dX_, dW1_, dW2_, ddY = (h.cuda().view(torch.bfloat16) for h in (hX, hW1, hW2, hdY))
    desc = binding.make_desc(T, D, F, V, M, prune_mode=args.prune_mode)
    ctx, ws = binding.alloc_ffn_buffers(desc)
    Y = torch.empty((T, D), dtype=torch.bfloat16, device="cuda")
    gX, gW1, gW2 = torch.empty_like(dX_), torch.empty_like(dW1_), torch.empty_like(dW2_)

    def sparse_step():
        binding.sf_sparse_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
        binding.sf_sparse_ffn_bwd(desc, ddY, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)

    def dense_step():
        binding.sf_dense_ffn_fwd(desc, dX_, dW1_, dW2_, Y, ctx, ws)
        binding.sf_dense_ffn_bwd(desc, ddY, dX_, dW1_, dW2_, ctx, gX, gW1, gW2, ws)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1), device="cuda")

    for _ in range(W if args.quick else max(W, 3)):
        sparse_step()
    if binding.sf_check_status(ws) != binding.SF_OK:
        raise SystemExit("device status: a bounded wait expired during warm-up")

    sampler = ClockSampler(local) if rank == 0 else None
    ms = timed(sparse_step, K)
    clocks = sampler.stop() if sampler else None
    flop_step = 12.0 * T * D * F
    value = replicas.aggregate_tflops(flop_step, K, ms)

    if args.quick:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
                              "ms_per_step": ms / K, "config": {"workload": args.workload}, "quick": True}))
        return
    for _ in range(2):
        dense_step()
    ms_dense = timed(dense_step, K)
    if binding.sf_check_status(ws) != binding.SF_OK:
        raise SystemExit("device status: a bounded wait expired")

    # ---- per-kernel times inside the step (events recorded by the library between its kernels)
    plain24 = (M <= 8)                       # activations multiplied as plain 2:4 operands (no row gather)
    act_gemm = "gemm_sparse24" if plain24 else "gemm_venom"
    names = ["prune24_W1", "gemm_sparse24_y1", "vnm_sparsify", "transpose_W2", f"{act_gemm}_y3",
             None, "prune24_W2", "gemm_sparse24_dy1", "pack_dy1", f"{act_gemm}_dX", "gemm_dense_dW2", "gemm_dense_dW1"]
    with binding.StageTrace(13 * K) as tr:
        for _ in range(K):
            sparse_step()
    d = tr.durations_ms()
    per = {}
    for s in range(K):
        seg = d[13 * s: 13 * s + 12]
        for n, v in zip(names, seg):
            if n:
                per.setdefault(n, []).append(v)
    kern_ms = {n: float(np.mean(v)) for n, v in per.items()}
    if plain24:
        kern_ms.pop("transpose_W2", None)    # not launched on this path (zero-length interval)
        kern_ms.pop("pack_dy1", None)        # dy1 is packed by the dy1 product's epilogue on this path
    unit = 2.0 * T * D * F                   # flop of one dense product
    peaks = _peaks()
    # Kernel groups by the device function that runs them. Algorithmic work per launch: one dense
    # product (2*T*D*F flop) for every product; the peak it is held against is the measured dense
    # bf16 GEMM peak for the dense kernel, twice that for the 2:4 kernel (nominal 2:4 ratio), and
    # M/4 times more for the condensed Venom kernel.
    groups = {
        "gemm_tc2_kernel<dense, MN-major A and B> (dW2, dW1)": (["gemm_dense_dW2", "gemm_dense_dW1"], 1.0),
        "gemm_tc2_kernel<2:4 sparse> (y1, dy1" + (", y3, dX)" if plain24 else ")"):
            (["gemm_sparse24_y1", "gemm_sparse24_dy1"] + ([f"{act_gemm}_y3", f"{act_gemm}_dX"] if plain24 else []), 2.0),
    }
    if not plain24:
        groups["gemm_tc_kernel<venom> (y3, dX)"] = ([f"{act_gemm}_y3", f"{act_gemm}_dX"], 2.0 * M / 4.0)
    tot = {g: sum(kern_ms[k] for k in ks) for g, (ks, _) in groups.items()}
    dom = max(tot, key=tot.get)
    ks, ratio = groups[dom]
    avg_ms = tot[dom] / len(ks)
    achieved = unit / (avg_ms / 1e3) / 1e12                      # dense-equivalent TFLOP/s of the kernel
    peak = peaks["bf16_tflops_sustained"] * ratio
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath):
        traffic = json.load(open(tpath)).get(dom.split(" (")[0])
    roofline = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": traffic,
                "peak_source": peaks["source"] + " sustained bf16 GEMM" + (f" x {ratio:g} (nominal sparse ratio)" if ratio != 1.0 else ""),
                "avg_launch_ms": avg_ms, "launches_per_step": len(ks),
                "share_of_step": tot[dom] / sum(kern_ms.values()),
                "other_groups": {g: {"avg_launch_ms": tot[g] / len(groups[g][0]),
                                     "frac": unit / (tot[g] / len(groups[g][0]) / 1e3) / 1e12 / (peaks["bf16_tflops_sustained"] * groups[g][1])}
                                 for g in groups if g != dom}}
    hbm = peaks["hbm_gbs"]
    prune_gbs = 3.125 * F * D / (kern_ms["prune24_W1"] / 1e3) / 1e9
    # bytes the V:N:M kernel moves in the step: input, V:N:M-packed values + ReLU values + metadata
    # (canonical and tensor-core order) + colidx, the two masked dense copies, and (M = 8) the 2:4 view
    vnm_bytes = T * F * (2 + 4.0 / M + 4.0 / M + 1.0 / M) + (T // V) * (F // M) * 4 + 2 * T * F * 2
    if plain24 and M == 8:
        vnm_bytes += T * F * (1.0 + 0.25)
    vnm_gbs = vnm_bytes / (kern_ms["vnm_sparsify"] / 1e3) / 1e9
    launches_per_step = 9 if plain24 else 11

    # ---- end to end through the host-buffer entry point (H2D of inputs and D2H of results timed)
    staging = torch.empty((binding.sf_ffn_host_staging_size(desc),), dtype=torch.uint8, device="cuda")
    # (empty_like of a pinned tensor is pageable: ask for pinned results explicitly)
    hY, hdX = torch.empty_like(hX, pin_memory=True), torch.empty_like(hX, pin_memory=True)
    hgW1, hgW2 = torch.empty_like(hW1, pin_memory=True), torch.empty_like(hW2, pin_memory=True)
    assert all(t.is_pinned() for t in (hX, hW1, hW2, hdY, hY, hdX, hgW1, hgW2))

    def host_step():
        binding.sf_ffn_step_host(desc, False, hX, hW1, hW2, hdY, hY, hdX, hgW1, hgW2, staging, ctx, ws)

    host_step()
    ms_e2e = timed(host_step, K)
    e2e_val = replicas.aggregate_tflops(flop_step, K, ms_e2e)
    h2d = 2 * T * D * 2 + 2 * F * D * 2
    d2h = h2d

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(W, 3),
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "T": T, "D": D, "F": F, "V": V, "N": 2, "M": M,
                   "prune_mode": args.prune_mode, "parallelism": f"replicas x{world}",
                   "l2": "per-step inputs (402 MB of operands, >2 GB of intermediates) exceed the 126 MB L2"},
        "dense_step_ms": ms_dense / K, "speedup_vs_dense_step": ms_dense / ms,
        "dense_step_tflops": replicas.aggregate_tflops(flop_step, K, ms_dense),
        "kernel_ms": kern_ms,
        "prune24_gbs": prune_gbs, "prune24_frac_of_hbm": prune_gbs / hbm,
        "vnm_sparsify_gbs": vnm_gbs, "vnm_frac_of_hbm": vnm_gbs / hbm,
        "roofline": roofline, "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": UNIT, "ms_per_step": ms_e2e / K, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": launches_per_step * K,
    }

    if rank == 0 and world == 1 and not args.skip_cpu_baseline:
        Ts = V
        sX, sW1, sW2, sdY = X[:Ts], W1, W2, dY[:Ts]
        t0 = time.perf_counter()
        _oracle_step(sX, sW1, sW2, sdY, V, M)
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": 12.0 * Ts * D * F / dt / 1e12, "unit": UNIT, "cores": _cpu_threads(),
                               "kind": "oracle", "seconds": dt,
                               "sample": f"first {Ts} tokens (one V-block) of the workload, full layer width, "
                                         "fwd+bwd incl. both full-size weight prunings"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4_d4096")
    ap.add_argument("--prune-mode", type=int, default=0)
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true",
                    help="sparse step only (no dense step, trace, e2e, CPU baseline): for profiler captures")
    args = ap.parse_args()
    from paper_2602_06183_b200 import synth
    cfg = synth.FFN_CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
