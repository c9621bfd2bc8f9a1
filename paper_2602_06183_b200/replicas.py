"""Replica bookkeeping for multi-GPU runs.

The step has no exchange between GPUs (V-blocks of tokens are independent; only a data-parallel
all-reduce of dW would communicate, and that is not part of this build), so N GPUs run N
independent replicas of the layer. What the ranks share is timing: a barrier on both sides of the
timed region, the maximum of the per-rank times, and the aggregate throughput.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    if world() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """The slowest rank's time: what a lock-step job would see."""
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tflops(flop_per_replica_step: float, steps: int, ms_max: float) -> float:
    """Whole-job dense-equivalent TFLOP/s: every replica did `steps` steps in `ms_max`."""
    return world() * flop_per_replica_step * steps / (ms_max / 1e3) / 1e12
