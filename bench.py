#!/usr/bin/env python
"""Benchmark of the sparsified-FFN training step (fwd + bwd) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line (rank 0). For the FFN workloads a "step" is one pass of the whole hot path:
2:4 prune of W1, the 2:4 y1 product with SquaredReLU + V:N:M selection (in its epilogue or as a
second kernel, see config.path), the y3 product, 2:4 prune of W2, the 2:4 dy1 product with the
dy1 epilogue, the dX product and the two weight-gradient products, on synthetic inputs of the named
workload (default: the d_model = 4096 FFN layer, 8192 tokens).

metric  = dense-equivalent TFLOP/s of the sparse step: 6 products x 2*T*D*F flop / step time.
value   = that metric over exactly K timed steps after W (>= 3) warm-up steps; per-kernel times come
          from events the library records between its kernels inside the same K steps.
sustained = the same step in K-step blocks alternating with dense-step blocks for at least
          --sustain-seconds per arm (medians): what the part delivers once it sits on its power cap.
N > 1   = N independent replicas of the layer (the path has no exchange step); `--gpus N` starts the
          N ranks itself when it is not already running under torchrun; the value is the aggregate
          over all ranks, timed as the max over ranks.
Other workloads: c2_prune (2:4 prune + compress sweep), c3_act (SquaredReLU + V:N:M sweep), gemm_micro
          (2:4 and Venom products against the dense product, the paper's micro-benchmark shapes).
--impl reference times the CPU oracle (a deliberately plain numpy program) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "sparse_ffn_fwd_bwd_dense_equiv_tflops"
UNIT = "TFLOP/s"
SWEEP_WORKLOADS = ("c2_prune", "c3_act", "gemm_micro", "fp8_micro")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def _l2_note(operand_bytes: int, activation_bytes: int) -> str:
    """Which of the two timing rules holds: inputs larger than the L2, or not (then the line says so)."""
    if operand_bytes > 126e6:
        return f"per-step operands ({operand_bytes / 1e6:.0f} MB) and intermediates exceed the 126 MB L2: no flush needed"
    return (f"per-step operands ({operand_bytes / 1e6:.1f} MB) and the [T, F] intermediates ({activation_bytes / 1e6:.1f} MB each) "
            "fit the 126 MB L2 and no flush is done: a parity-size workload, its timing is L2-resident and is not a benchmark figure")


def _traffic():
    """Per-launch DRAM traffic of the step's kernels from the committed single-pass ncu capture."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    return json.load(open(path)) if os.path.exists(path) else {}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        dev = vis.split(",")[gpu_index] if vis else str(gpu_index)
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={dev}", f"--query-gpu={self.Q}",
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


# ---- stage names in the order the library records its trace events (see sf_trace_set) ----------------
TRACE_NAMES = ["prune24_W1", "gemm_y1", "vnm_sparsify", "transpose_W2", "gemm_y3",
               None, "prune24_W2", "gemm_dy1", "pack_dy1", "gemm_dX", "gemm_dW2", "gemm_dW1"]


def _step_path(V, M):
    """Which kernels the library runs for this configuration (mirrors the rule in the step's layout)."""
    if M == 8:
        return "fused" if V == 64 else "two_kernel"
    return "plain24" if M == 4 else "venom"


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
    K, W = args.steps, max(args.warmup, 3) if not args.quick else args.warmup
    X, W1, W2, dY = synth.ffn_inputs(T, D, F, cfg["sigma_w"], cfg["seed"] + rank)
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    hX, hW1, hW2, hdY = pin(X), pin(W1), pin(W2), pin(dY)
    dX_, dW1_, dW2_, ddY = (h.cuda().view(torch.bfloat16) for h in (hX, hW1, hW2, hdY))
    desc = binding.make_desc(T, D, F, V, M, prune_mode=args.prune_mode, flags=args.flags)
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

    for _ in range(W):
        sparse_step()
    if binding.sf_check_status(ws) != binding.SF_OK:
        raise SystemExit("device status: a bounded wait expired during warm-up")

    flop_step = 12.0 * T * D * F
    if args.quick and args.quick_arm == "routed":
        E = M // 4
        rdesc = binding.make_router_desc(T, D, F, E, prune_mode=args.prune_mode)
        rc, rw = binding.sf_routed_ffn_workspace_size(rdesc)
        rctx, rws = torch.zeros((rc,), dtype=torch.uint8, device="cuda"), torch.zeros((rw,), dtype=torch.uint8, device="cuda")
        means = torch.from_numpy(synth.normal_bf16((E, D), 0.0, 1.0, cfg["seed"], 9).view(np.int16)).cuda().view(torch.bfloat16)

        def sparse_step():                     # the quick path below times whatever this name holds
            binding.sf_routed_ffn_fwd(rdesc, dX_, dW1_, dW2_, means, Y, rctx, rws)
            binding.sf_routed_ffn_bwd(rdesc, ddY, dX_, dW1_, dW2_, rctx, gX, gW1, gW2, rws)
        for _ in range(W):
            sparse_step()
    if args.quick:
        ms = timed(sparse_step, K)
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": replicas.aggregate_tflops(flop_step, K, ms), "unit": UNIT,
                              "n_gpus": world, "steps": K, "ms_per_step": ms / K,
                              "config": {"workload": args.workload}, "quick": True}))
        return

    # ---- the timed region: exactly K sparse steps; the library records an event between its kernels
    sampler = ClockSampler(local) if rank == 0 else None
    with binding.StageTrace(13 * K) as tr:
        ms = timed(sparse_step, K)
    clocks = sampler.stop() if sampler else None
    value = replicas.aggregate_tflops(flop_step, K, ms)
    d = tr.durations_ms()
    per = {}
    for s in range(K):
        for n, v in zip(TRACE_NAMES, d[13 * s: 13 * s + 12]):
            if n:
                per.setdefault(n, []).append(v)
    path = _step_path(V, M) if not (args.flags & (binding.SF_FFN_UNFUSED_ACT | binding.SF_FFN_FUSED_ACT)) else \
        ("fused" if args.flags & binding.SF_FFN_FUSED_ACT else "two_kernel")
    not_launched = {"fused": {"vnm_sparsify", "transpose_W2", "pack_dy1"}, "two_kernel": {"transpose_W2", "pack_dy1"},
                    "plain24": {"transpose_W2", "pack_dy1"}, "venom": set()}[path]   # empty trace intervals
    kern_ms = {n: float(np.mean(v)) for n, v in per.items() if n not in not_launched}
    kern_sum = float(sum(kern_ms.values()))

    def rested_warmup(fn):
        """Every arm starts like the first one: after an idle gap (the part drops back to its idle power state)
        and W warm-up steps, so that no arm inherits the heat of the arm before it."""
        barrier()
        time.sleep(args.rest_seconds)
        for _ in range(W):
            fn()

    rested_warmup(dense_step)
    ms_dense = timed(dense_step, K)
    if binding.sf_check_status(ws) != binding.SF_OK:
        raise SystemExit("device status: a bounded wait expired")

    # ---- the routed step (Section 3.1's neuron-level experts, E = M / 4): same layer, same metric
    routed, routed_step = None, None
    E = M // 4
    if E >= 1 and F % E == 0 and (F // E) % 256 == 0 and E <= 16:
        rdesc = binding.make_router_desc(T, D, F, E, prune_mode=args.prune_mode)
        rc, rw = binding.sf_routed_ffn_workspace_size(rdesc)
        rctx = torch.zeros((rc,), dtype=torch.uint8, device="cuda")
        rws = torch.zeros((rw,), dtype=torch.uint8, device="cuda")
        means = torch.from_numpy(synth.normal_bf16((E, D), 0.0, 1.0, cfg["seed"], 9).view(np.int16)).cuda().view(torch.bfloat16)

        def routed_step():
            binding.sf_routed_ffn_fwd(rdesc, dX_, dW1_, dW2_, means, Y, rctx, rws)
            binding.sf_routed_ffn_bwd(rdesc, ddY, dX_, dW1_, dW2_, rctx, gX, gW1, gW2, rws)

        rested_warmup(routed_step)
        with binding.StageTrace(13 * K) as rtr:
            ms_r = timed(routed_step, K)
        if binding.sf_check_status(rws) != binding.SF_OK:
            raise SystemExit("device status: a bounded wait expired in the routed step")
        rd = rtr.durations_ms()
        rnames = ["prune24_W1", "route", "group_tables_gather_X", "gemm_y1", "gemm_y3", None,
                  "prune24_W2", "gather_dY", "gemm_dy1", "gemm_dX", "gemm_dW2", "gemm_dW1"]
        rper = {}
        for st in range(K):
            for n, v in zip(rnames, rd[13 * st: 13 * st + 12]):
                if n:
                    rper.setdefault(n, []).append(v)
        seg = binding.sf_routed_ctx_view(rdesc, rctx, binding.SF_RCTX_SEGMENTS).cpu().numpy()
        routed = {"experts": E, "ms_per_step": ms_r / K, "value": replicas.aggregate_tflops(flop_step, K, ms_r),
                  "speedup_vs_dense_step": ms_dense / ms_r, "kernel_ms": {n: float(np.mean(v)) for n, v in rper.items()},
                  "tokens_per_expert": seg[E + 1:].tolist(), "rows_with_padding": int(seg[E]), "gpu_launches": 15 * K,
                  "routing": "synthetic expert means ~ N(0,1): near-uniform top-1 routing",
                  "note": "Algorithm 1 line 6 as the paper words it (MoEToVenom): every product touches one expert's "
                          "F/E features per token; reported beside the magnitude-selection step, not instead of it"}

    # ---- sustained: alternate K-step blocks of the arms until each has run for the target time
    sustained = None
    if args.sustain_seconds > 0:
        target_ms = args.sustain_seconds * 1e3
        arms = [("sparse", sparse_step), ("dense", dense_step)] + ([("routed", routed_step)] if routed else [])
        blocks = {n: [] for n, _ in arms}
        sampler2 = ClockSampler(local) if rank == 0 else None
        while any(sum(b) < target_ms for b in blocks.values()):
            for n, fn in arms:
                blocks[n].append(timed(fn, K))
            if len(blocks["sparse"]) > 2000:
                break
        clocks2 = sampler2.stop() if sampler2 else None
        med = {n: float(np.median(b)) / K for n, b in blocks.items()}
        ms_s, ms_d = med["sparse"], med["dense"]
        sustained = {"ms_per_step": ms_s, "value": flop_step * world / (ms_s / 1e3) / 1e12, "dense_step_ms": ms_d,
                     "speedup_vs_dense_step": ms_d / ms_s, "blocks_per_arm": len(blocks["sparse"]), "steps_per_block": K,
                     "seconds_per_arm": sum(blocks["sparse"]) / 1e3, "clocks": clocks2}
        if routed:
            sustained["routed_ms_per_step"] = med["routed"]
            sustained["routed_speedup_vs_dense_step"] = ms_d / med["routed"]

    # ---- roofline fractions on ALGORITHMIC work, against the measured peaks
    peaks = _peaks()
    unit = 2.0 * T * D * F                   # flop of one dense product
    # Tensor work in units of one dense product: the 2:4 products do 2*T*D*F dense-equivalent flop at the 2:4 peak
    # (2 x dense), the V:N:M products (4/M) of that whichever kernel runs them, the weight-gradient products
    # 2*T*D*F at the dense peak. The step loop runs for a long time at the power cap, so the peak is the SUSTAINED
    # measured bf16 GEMM figure (the burst figure is printed beside it).
    P = peaks["bf16_tflops_sustained"]
    prod = {"gemm_y1": (1.0, 2.0), "gemm_dy1": (1.0, 2.0), "gemm_y3": (4.0 / M, 2.0), "gemm_dX": (4.0 / M, 2.0),
            "gemm_dW2": (1.0, 1.0), "gemm_dW1": (1.0, 1.0)}
    products = {}
    for n, (alg, ratio) in prod.items():
        t = kern_ms[n] / 1e3
        products[n] = {"ms": kern_ms[n], "algorithmic_dense_equiv_tflops": alg * unit / t / 1e12,
                       "peak_tflops": P * ratio, "frac": alg * unit / t / 1e12 / (P * ratio),
                       "frac_of_burst_peak": alg * unit / t / 1e12 / (peaks["bf16_tflops"] * ratio)}
    if path == "fused":
        products["gemm_y1"]["includes"] = "SquaredReLU + V:N:M selection in the epilogue"
    groups = {"2:4 tensor kernels (y1, dy1, y3, dX)": (["gemm_y1", "gemm_dy1", "gemm_y3", "gemm_dX"], 2.0),
              "dense tensor kernel (dW2, dW1)": (["gemm_dW2", "gemm_dW1"], 1.0)}
    gstat = {}
    for g, (ks, ratio) in groups.items():
        t = sum(kern_ms[k] for k in ks) / 1e3
        alg = sum(prod[k][0] for k in ks) * unit
        gstat[g] = {"ms": t * 1e3, "launches_per_step": len(ks), "achieved": alg / t / 1e12, "peak": P * ratio,
                    "frac": alg / t / 1e12 / (P * ratio), "share_of_step": t * 1e3 / kern_sum}
    dom = max(gstat, key=lambda g: gstat[g]["ms"])
    traffic = _traffic()
    roofline = {"bound": "tensor", "kernel": dom, "achieved": gstat[dom]["achieved"], "peak": gstat[dom]["peak"],
                "unit": "TFLOP/s", "frac": gstat[dom]["frac"],
                "traffic": traffic.get("kernels", {}).get(dom), "traffic_captured_on": traffic.get("captured_on"),
                "peak_source": peaks["source"] + " sustained bf16 GEMM x 2 (nominal 2:4 ratio)" if "2:4" in dom
                else peaks["source"] + " sustained bf16 GEMM",
                "work": "algorithmic dense-equivalent flop: 2TDF per 2:4 product, (4/M) 2TDF per V:N:M product",
                "avg_launch_ms": gstat[dom]["ms"] / gstat[dom]["launches_per_step"],
                "launches_per_step": gstat[dom]["launches_per_step"], "share_of_step": gstat[dom]["share_of_step"],
                "other_groups": {g: v for g, v in gstat.items() if g != dom}}
    floor_units = 0.5 + 0.5 + 2 * (4.0 / M) * 0.5 + 2.0
    floor_ms = floor_units * unit / (P * 1e12) * 1e3
    step_floor = {"dense_product_units": floor_units, "floor_ms": floor_ms, "frac": floor_ms / (ms / K),
                  "frac_sustained": floor_ms / sustained["ms_per_step"] if sustained else None,
                  "speedup_ceiling_vs_dense": 6.0 / floor_units}

    # ---- bandwidth kernels on algorithmic bytes (3.125 B/element; 2 + 4/M + 0.5/M (+ 4/M ReLU values) + colidx)
    hbm = peaks["hbm_gbs"]
    bw = {}
    for n in ("prune24_W1", "prune24_W2"):
        gbs = 3.125 * F * D / (kern_ms[n] / 1e3) / 1e9
        bw[n] = {"ms": kern_ms[n], "algorithmic_bytes": 3.125 * F * D, "gbs": gbs, "frac_of_hbm": gbs / hbm,
                 "traffic_over_algorithmic": (traffic.get("kernels", {}).get(n) or 0) / (3.125 * F * D) or None}
    vnm_alg = T * F * (2 + 4.0 / M + 0.5 / M + 4.0 / M) + (T // V) * (F // M) * 4
    if "vnm_sparsify" in kern_ms:
        gbs = vnm_alg / (kern_ms["vnm_sparsify"] / 1e3) / 1e9
        bw["vnm_sparsify"] = {"ms": kern_ms["vnm_sparsify"], "algorithmic_bytes": vnm_alg, "gbs": gbs,
                              "frac_of_hbm": gbs / hbm,
                              "traffic_over_algorithmic": (traffic.get("kernels", {}).get("vnm_sparsify") or 0) / vnm_alg or None}
    else:
        bw["vnm_sparsify"] = {"fused_into": "gemm_y1", "algorithmic_bytes": vnm_alg - 2.0 * T * F,
                              "note": "no separate kernel: y1 never leaves the chip"}
    launches_per_step = len(kern_ms)

    # ---- end to end through the host-buffer entry point (H2D of inputs and D2H of results timed)
    staging = torch.empty((binding.sf_ffn_host_staging_size(desc),), dtype=torch.uint8, device="cuda")
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
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "T": T, "D": D, "F": F, "V": V, "N": 2, "M": M,
                   "prune_mode": args.prune_mode, "flags": args.flags, "path": path,
                   "parallelism": f"replicas x{world}",
                   "arms": f"each arm (sparse, dense, routed) is timed after an idle gap of {args.rest_seconds} s and {W} warm-up steps",
                   "l2": _l2_note((2 * T * D + 2 * F * D) * 2, T * F * 2)},
        "dense_step_ms": ms_dense / K, "speedup_vs_dense_step": ms_dense / ms,
        "dense_step_tflops": replicas.aggregate_tflops(flop_step, K, ms_dense),
        "sustained": sustained, "routed_step": routed,
        "kernel_ms": kern_ms, "kernel_ms_sum": kern_sum, "kernel_ms_sum_over_step": kern_sum / (ms / K),
        "products": products, "step_floor": step_floor, "bandwidth_kernels": bw,
        "roofline": roofline, "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": UNIT, "ms_per_step": ms_e2e / K, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": launches_per_step * K,
    }
    if abs(kern_sum / (ms / K) - 1.0) > 0.05:
        out["kernel_ms_note"] = "per-kernel times do not add up to the step time within 5 %: breakdown rejected"

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


# ---- stand-alone sweeps (BASELINE configs 2 and 3, and the paper's product micro-benchmarks) ------------

def _time_cuda(fn, iters=20, warm=3, flush=None):
    """Mean device time of fn. flush: a buffer larger than the L2 that is overwritten before every timed call
    (outside the timed interval), for inputs that would otherwise stay resident in the L2."""
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in ev:
        flush.zero_()
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in ev) / iters


def run_sweep(args):
    """One JSON line: `results` holds one entry per swept shape; value = the worst fraction of the
    measured HBM bandwidth (bandwidth sweeps) or the 2:4 speed-up at the paper's shape (gemm_micro)."""
    import torch
    from paper_2602_06183_b200 import binding, build, synth
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    build.build()
    peaks = _peaks()
    hbm = peaks["hbm_gbs"]
    dev = lambda b: torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).cuda().view(torch.bfloat16)
    iters = max(args.steps, 5)
    results = []
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    roofline = None
    if args.workload == "c2_prune":
        flush = torch.empty((256 << 20,), dtype=torch.uint8, device="cuda")      # twice the L2
        for i, (rows, cols) in enumerate(synth.PRUNE_SWEEP_SHAPES):
            w = dev(synth.prune_sweep_matrix(rows, cols, seed=1000 + i))
            for group_dim in (1, 0):
                for mode in (0, 1):
                    outb = binding.sf_prune24_compress(w, group_dim, mode)
                    ms = _time_cuda(lambda: binding.sf_prune24_compress(w, group_dim, mode, out=outb), iters, args.warmup,
                                    flush=flush)
                    gbs = 3.125 * rows * cols / (ms / 1e3) / 1e9
                    results.append({"rows": rows, "cols": cols, "group_dim": group_dim, "prune_mode": mode,
                                    "us": ms * 1e3, "gbs": gbs, "frac_of_hbm": gbs / hbm})
        metric, unit, value = "prune24_compress_min_frac_of_measured_hbm", "fraction", min(r["frac_of_hbm"] for r in results)
        big = [r for r in results if r["rows"] * r["cols"] == max(x["rows"] * x["cols"] for x in results) and r["prune_mode"] == 0]
        roofline = {"bound": "hbm", "kernel": "prune24_rows_kernel / prune24_cols_kernel at the largest shape, hard pruning",
                    "achieved": min(r["gbs"] for r in big), "peak": hbm, "unit": "GB/s",
                    "frac": min(r["frac_of_hbm"] for r in big), "traffic": None,
                    "peak_source": f"{peaks['source']} copy bandwidth", "work": "3.125 algorithmic bytes per element"}
        note = ("3.125 algorithmic bytes per element; three of the four inputs would fit the 126 MB L2, so a 256 MB buffer "
                "is overwritten before every timed launch (each launch timed by its own event pair, input cold)")
    elif args.workload == "c3_act":
        Tn = Fn = 16384
        p = dev(synth.act_sweep_matrix(Tn, Fn, seed=2000))
        for V in (64, 128):
            for M in (8, 16):
                outb = binding.sf_vnm_sparsify_act(p, V, M)
                ms = _time_cuda(lambda: binding.sf_vnm_sparsify_act(p, V, M, out=outb), iters, args.warmup)
                nbytes = Tn * Fn * (2 + 4.0 / M + 0.5 / M + 4.0 / M) + (Tn // V) * (Fn // M) * 4
                gbs = nbytes / (ms / 1e3) / 1e9
                results.append({"T": Tn, "F": Fn, "V": V, "M": M, "us": ms * 1e3, "algorithmic_bytes_per_element": nbytes / (Tn * Fn),
                                "gbs": gbs, "frac_of_hbm": gbs / hbm})
        metric, unit, value = "vnm_sparsify_min_frac_of_measured_hbm", "fraction", min(r["frac_of_hbm"] for r in results)
        roofline = {"bound": "hbm", "kernel": "vnm_stream_kernel", "achieved": min(r["gbs"] for r in results), "peak": hbm,
                    "unit": "GB/s", "frac": value, "traffic": None, "peak_source": f"{peaks['source']} copy bandwidth",
                    "work": "2 + 4/M + 0.5/M + 4/M algorithmic bytes per element + colidx"}
        note = "2 + 4/M + 0.5/M + 4/M (ReLU values) bytes per element + colidx; 537 MB input, larger than the L2"
    else:
        shapes = [(4096, 16384, 4096)] if args.workload == "fp8_micro" else [(4096, 16384, 4096), (16384, 8192, 4096), (8192, 4096, 16384)]
        for (m, n, k) in shapes:
            A = torch.randn((m, k), device="cuda").to(torch.bfloat16)
            B = torch.randn((n, k), device="cuda").to(torch.bfloat16)
            Cm = torch.empty((m, n), dtype=torch.bfloat16, device="cuda")
            wsb = torch.zeros((binding.sf_gemm_workspace_size(m, k),), dtype=torch.uint8, device="cuda")
            ms_d = _time_cuda(lambda: binding.sf_gemm_dense(A, True, B, True, C_out=Cm, workspace=wsb), iters, args.warmup)
            vals, meta, _ = binding.sf_prune24_compress(A, 1, 0)
            ms_p = _time_cuda(lambda: binding.sf_prune24_compress(A, 1, 0, out=(vals, meta, None)), iters, args.warmup)
            ms_s = _time_cuda(lambda: binding.sf_gemm_sparse24_rm(vals, meta, B, True, C_out=Cm, workspace=wsb), iters, args.warmup)
            fl = 2.0 * m * n * k
            results.append({"product": "2:4 vs dense", "shape_mnk": [m, n, k], "dense_ms": ms_d, "dense_tflops": fl / ms_d / 1e9,
                            "sparse24_ms": ms_s, "sparse24_dense_equiv_tflops": fl / ms_s / 1e9, "prune_ms": ms_p,
                            "speedup_gemm_only": ms_d / ms_s, "speedup_with_prune": ms_d / (ms_s + ms_p)})
            # the same product on E4M3 operands (Section 3.2.2, last paragraph): quantisation rides on the pruning pass
            sa, sb = 64.0, 64.0
            Aq, Bq = binding.sf_fp8_quantize(A, sa), binding.sf_fp8_quantize(B, sb)
            ws8 = torch.zeros((binding.sf_gemm_fp8_workspace_size(m, k),), dtype=torch.uint8, device="cuda")
            ms_q = _time_cuda(lambda: binding.sf_fp8_quantize(B, sb, out=Bq), iters, args.warmup)
            ms_d8 = _time_cuda(lambda: binding.sf_gemm_fp8_dense(Aq, Bq, 1.0 / (sa * sb), C_out=Cm, workspace=ws8), iters, args.warmup)
            o8 = binding.sf_prune24_compress_fp8(A, 0, sa)
            ms_p8 = _time_cuda(lambda: binding.sf_prune24_compress_fp8(A, 0, sa, out=o8), iters, args.warmup)
            ms_s8 = _time_cuda(lambda: binding.sf_gemm_fp8_sparse24(o8[0], o8[1], Bq, 1.0 / (sa * sb), C_out=Cm, workspace=ws8),
                               iters, args.warmup)
            results.append({"product": "fp8 (E4M3) 2:4 vs dense", "shape_mnk": [m, n, k], "dense_fp8_ms": ms_d8,
                            "dense_fp8_tflops": fl / ms_d8 / 1e9, "sparse24_fp8_ms": ms_s8,
                            "sparse24_fp8_dense_equiv_tflops": fl / ms_s8 / 1e9, "prune_quantise_ms": ms_p8,
                            "prune_quantise_gbs": 2.625 * m * k / ms_p8 / 1e6, "quantise_B_ms": ms_q,
                            "quantise_B_gbs": 3.0 * n * k / ms_q / 1e6,
                            "speedup_gemm_only": ms_d8 / ms_s8, "speedup_with_prune": ms_d8 / (ms_s8 + ms_p8),
                            "speedup_vs_bf16_dense": ms_d / ms_s8})
            del A, B, Cm, vals, meta, Aq, Bq, o8
        if args.workload == "gemm_micro":
            Tn, Fn, Nn = 8192, 16384, 4096
            A = torch.randn((Tn, Fn), device="cuda").to(torch.bfloat16)
            Bd = torch.randn((Nn, Fn), device="cuda").to(torch.bfloat16)
            Cd = torch.empty((Tn, Nn), dtype=torch.bfloat16, device="cuda")
            wsd = torch.zeros((binding.sf_gemm_workspace_size(Tn, Fn),), dtype=torch.uint8, device="cuda")
            ms_dense = _time_cuda(lambda: binding.sf_gemm_dense(A, True, Bd, True, C_out=Cd, workspace=wsd), iters, args.warmup)
            del A, Bd, Cd
            for M in (8, 16, 32, 64):
                P = dev(synth.normal_bf16((Tn, Fn), 0.0, 1.0, seed=7))
                vals, meta, colidx, _, _ = binding.sf_vnm_sparsify_act(P, 128, M)
                Bt = torch.randn((Fn, Nn), device="cuda").to(torch.bfloat16)
                Cm = torch.empty((Tn, Nn), dtype=torch.bfloat16, device="cuda")
                wsb = torch.zeros((binding.sf_gemm_workspace_size(Tn, Fn),), dtype=torch.uint8, device="cuda")
                ms_v = _time_cuda(lambda: binding.sf_gemm_venom(vals, meta, colidx, Bt, 128, M, C_out=Cm, workspace=wsb), iters, args.warmup)
                results.append({"product": "Venom vs dense", "T": Tn, "F": Fn, "N": Nn, "V": 128, "M": M,
                                "sparsity_pct": 100.0 * (1 - 2.0 / M), "ms": ms_v, "dense_ms": ms_dense,
                                "speedup_vs_dense": ms_dense / ms_v})
        metric, unit, value = "sparse24_gemm_speedup_vs_dense_at_4096x16384x4096", "ratio", results[0]["speedup_gemm_only"]
        note = "Section 5.2.3's micro-benchmark shape first; Venom products at Table 5's sparsities"
    line = {"metric": metric, "value": value, "unit": unit, "n_gpus": 1, "steps": iters, "warmup": args.warmup,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "note": note, "hbm_peak_gbs": hbm, "peak_source": peaks["source"]},
            "results": results, "gpu_launches": iters * len(results), "clocks": sampler.stop()}
    if roofline:
        line["roofline"] = roofline
    print(json.dumps(line))


def _spawn_replicas(args):
    """`--gpus N` outside torchrun: start the N ranks (one per GPU of this node) and relay their output."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4_d4096")
    ap.add_argument("--prune-mode", type=int, default=0)
    ap.add_argument("--flags", type=int, default=0, help="sf_ffn_flags of the step (0 = the library's defaults)")
    ap.add_argument("--sustain-seconds", type=float, default=1.0,
                    help="time per arm of the alternating sparse/dense blocks (0 = skip)")
    ap.add_argument("--rest-seconds", type=float, default=0.5,
                    help="idle gap before the warm-up of the dense and the routed arm (the sparse arm starts from idle too)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true",
                    help="sparse step only (no dense step, trace, e2e, CPU baseline): for profiler captures")
    ap.add_argument("--quick-arm", default="sparse", choices=["sparse", "routed"],
                    help="with --quick: the magnitude-selection step or the routed step")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        raise SystemExit(_spawn_replicas(args))
    from paper_2602_06183_b200 import synth
    if args.workload in SWEEP_WORKLOADS:
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "the reference arm times the FFN step workloads only"}))
            return
        run_sweep(args)
        return
    cfg = synth.FFN_CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
