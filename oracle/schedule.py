"""Sparse/dense step schedule and the paper's speed-up arithmetic (TEST INFRASTRUCTURE ONLY).

Section 5.3.2: training runs sparse steps first and dense steps afterwards to recover accuracy,
and V:N:M sparsification only starts after a dense warm-up (1000 steps in the paper). Section 3.1
relates a per-step FFN speed-up to an end-to-end one through the FFN's share of the training
FLOPs; Section 5.1 works one example (a 2.2x faster sparse iteration on half of the iterations
gives 1.37x end to end).

Readings where the paper is silent: the warm-up steps are plain dense steps and count towards
the total; the sparse phase follows the warm-up immediately; the time of a phase is its step
count times a constant per-step time; the end-to-end effect of an FFN-only speed-up is
Amdahl's law on the FLOP share (the paper says the share "reflects the portion of the
end-to-end time spent in the FFN").
"""
from __future__ import annotations

DENSE, SPARSE = 0, 1


def step_kind(step: int, warmup_steps: int, sparse_steps: int, total_steps: int) -> int:
    """Kind of step `step` (0-based): dense warm-up, then `sparse_steps` sparse steps, then dense."""
    if not (0 <= step < total_steps) or warmup_steps < 0 or sparse_steps < 0 \
            or warmup_steps + sparse_steps > total_steps:
        raise ValueError("step outside the schedule")
    return SPARSE if warmup_steps <= step < warmup_steps + sparse_steps else DENSE


def schedule_speedup(sparse_steps: int, total_steps: int, sparse_step_speedup: float) -> float:
    """Time of `total_steps` dense steps over the time of the mixed schedule (Section 5.1)."""
    dense_steps = total_steps - sparse_steps
    return total_steps / (sparse_steps / sparse_step_speedup + dense_steps)


def ffn_flop_fraction(D: int, F: int, n_q_heads: int, n_kv_heads: int, head_dim: int) -> float:
    """FFN share of the training FLOPs, Section 3.1: 18 D F / (6 (3 D F + 2 D (N + K) H))."""
    return 18.0 * D * F / (6.0 * (3.0 * D * F + 2.0 * D * (n_q_heads + n_kv_heads) * head_dim))


def end_to_end_speedup(ffn_fraction: float, ffn_speedup: float) -> float:
    """Whole-model speed-up when only the FFN share gets `ffn_speedup` times faster."""
    return 1.0 / ((1.0 - ffn_fraction) + ffn_fraction / ffn_speedup)
