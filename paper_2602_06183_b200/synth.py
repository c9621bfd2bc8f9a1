"""Seeded synthetic inputs for the sparsified-FFN hot path.

This module only draws random tensors and converts them to bf16 bit patterns. It holds none of
the method's arithmetic (no pruning, no activation, no products), so both the CPU oracle's tests
and the CUDA path's tests/bench can take their inputs from here without sharing any logic.

All tensors are returned as ``numpy.uint16`` arrays holding bf16 bit patterns (row-major).
The generator is numpy's counter-based Philox stream keyed by ``(seed, stream)``, so a tensor is
reproducible independently of the order in which other tensors are drawn.

Shapes, distributions and structure follow the paper's workloads:
  * FFN shapes from the model table (Table 1: d_model 2048/4096, d_ffn 8192/16384) and the
    micro-benchmark shape of Section 5.2.3,
  * N(0, sigma) weights, N(0, 1) tokens and output gradients,
  * pre-activations shifted so that about 90 % of them are negative (Section 2.1 / 2.3 state that
    more than 90 % of post-activation values are zero),
  * an injector of exact magnitude ties for exercising the tie rule of the 2:4 selection.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "f32_to_bf16_bits", "bf16_bits_to_f32", "normal_bf16", "inject_ties",
    "ffn_inputs", "prune_sweep_matrix", "act_sweep_matrix",
    "FFN_CONFIGS", "PRUNE_SWEEP_SHAPES",
]

# (T, D, F, V, N, M, sigma_w) per named FFN configuration.
FFN_CONFIGS = {
    "c1_small": dict(T=1024, D=256, F=1024, V=64, N=2, M=8, sigma_w=0.02, seed=0),
    # the d_model = 4096 layer; the configuration says "V:2:8" and leaves V free: V = 64 is the block height of
    # the paper's Table 5, and three such blocks fill one token tile of the fused y1 epilogue
    "c4_d4096": dict(T=8192, D=4096, F=16384, V=64, N=2, M=8, sigma_w=0.02, seed=4),
    # the same layer with 128-token blocks (SquaredReLU + V:N:M then run as a second kernel by default)
    "c4_d4096_v128": dict(T=8192, D=4096, F=16384, V=128, N=2, M=8, sigma_w=0.02, seed=4),
    # one eighth of c4's tokens with the full-size layer: weights (134 MB each) still exceed the
    # L2, device footprint ~1.5 GB; used for profiler captures that must stay small
    "c4_slice": dict(T=1024, D=4096, F=16384, V=64, N=2, M=8, sigma_w=0.02, seed=4),
    "c4_slice_v128": dict(T=1024, D=4096, F=16384, V=128, N=2, M=8, sigma_w=0.02, seed=4),
    # the same slice with groups of 16 (87.5 % sparse activations): exercises the condensed Venom products
    "c4_slice_m16": dict(T=1024, D=4096, F=16384, V=128, N=2, M=16, sigma_w=0.02, seed=4),
    # c4 with groups of 16 (Table 5's 87.5 % row): the full-size case of the condensed Venom products
    "c4_d4096_m16": dict(T=8192, D=4096, F=16384, V=128, N=2, M=16, sigma_w=0.02, seed=4),
    "c5_d8192": dict(T=16384, D=8192, F=28672, V=64, N=2, M=8, sigma_w=0.015, seed=5),
    "c5_d8192_v128": dict(T=16384, D=8192, F=28672, V=128, N=2, M=8, sigma_w=0.015, seed=5),
}

PRUNE_SWEEP_SHAPES = [(4096, 4096), (14336, 4096), (4096, 16384), (28672, 8192)]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = (b + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(u: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 (exact)."""
    return (np.ascontiguousarray(u, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & 0xFFFFFFFFFFFFFFFF, int(stream)]))


def normal_bf16(shape, mean: float, std: float, seed: int, stream: int = 0) -> np.ndarray:
    """bf16 bit patterns of N(mean, std) samples (drawn in float32, rounded RNE)."""
    g = _rng(seed, stream)
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    if mean != 0.0:
        x += np.float32(mean)
    return f32_to_bf16_bits(x)


def inject_ties(w_bits: np.ndarray, frac: float, seed: int, stream: int = 99, axis: int = 1) -> np.ndarray:
    """Copy one element's magnitude onto another position in a fraction of the groups of four.

    Groups run along ``axis`` (1: four consecutive columns, 0: four consecutive rows). In each
    chosen group a random ordered pair (src, dst), src != dst, is drawn and dst receives
    |src| with a fresh random sign, so ties straddle every rank boundary of the selection.
    """
    w = np.array(w_bits, dtype=np.uint16, copy=True)
    view = w if axis == 1 else w.T
    rows, cols = view.shape
    assert cols % 4 == 0
    g = _rng(seed, stream)
    ngroups = rows * (cols // 4)
    chosen = np.flatnonzero(g.random(ngroups) < frac)
    src = g.integers(0, 4, size=chosen.size)
    dst = (src + g.integers(1, 4, size=chosen.size)) % 4
    sign = (g.integers(0, 2, size=chosen.size).astype(np.uint16) << np.uint16(15))
    r = chosen // (cols // 4)
    c0 = (chosen % (cols // 4)) * 4
    mag = view[r, c0 + src] & np.uint16(0x7FFF)
    view[r, c0 + dst] = mag | sign
    return w


def ffn_inputs(T: int, D: int, F: int, sigma_w: float, seed: int, act_shift: float = 0.0):
    """X [T,D] ~ N(0,1), W1 [F,D], W2 [D,F] ~ N(0,sigma_w), dY [T,D] ~ N(0,1), all bf16 bits.

    ``act_shift`` != 0 adds a constant to X's first column and to W1's first column scaled so
    that the pre-activations X.W1^T are shifted by about ``act_shift`` standard deviations,
    which reproduces the ~90 % post-ReLU sparsity the paper reports for trained models.
    """
    X = normal_bf16((T, D), 0.0, 1.0, seed, 1)
    W1 = normal_bf16((F, D), 0.0, sigma_w, seed, 2)
    W2 = normal_bf16((D, F), 0.0, sigma_w, seed, 3)
    dY = normal_bf16((T, D), 0.0, 1.0, seed, 4)
    if act_shift != 0.0:
        # y1 = X.W1^T has std sigma_w*sqrt(D); put a bias term through one feature column.
        Xf = bf16_bits_to_f32(X)
        Wf = bf16_bits_to_f32(W1)
        Xf[:, 0] = 1.0
        Wf[:, 0] = act_shift * sigma_w * np.sqrt(D)
        X = f32_to_bf16_bits(Xf)
        W1 = f32_to_bf16_bits(Wf)
    return X, W1, W2, dY


def prune_sweep_matrix(rows: int, cols: int, seed: int, tie_frac: float = 0.05, axis: int = 1) -> np.ndarray:
    """Weight matrix ~ N(0, 0.02) with exact-tie groups in ``tie_frac`` of the groups."""
    w = normal_bf16((rows, cols), 0.0, 0.02, seed, 0)
    return inject_ties(w, tie_frac, seed, axis=axis)


def act_sweep_matrix(T: int, F: int, seed: int) -> np.ndarray:
    """Pre-activations ~ N(-1.3, 1): P(x > 0) = 9.7 %, i.e. about 90 % zeros after ReLU."""
    return normal_bf16((T, F), -1.3, 1.0, seed, 0)
