"""CPU oracle for the sparsified Transformer-FFN training step (TEST INFRASTRUCTURE ONLY).

A plain, slow, numpy implementation of what the hot path computes, written from the paper:
2:4 magnitude pruning with optional soft-thresholding (Section 2.2), the V:N:M activation
format (Section 2.3), SquaredReLU (Eq. 2) and the masked FFN forward/backward products
(Eqs. 1-8 with the operand colouring of Algorithms 1 and 2), and the sparse/dense step
schedule with the paper's speed-up arithmetic (Sections 3.1, 5.1, 5.3.2; `oracle.schedule`), and
the neuron-level router that produces the V:N:M pattern from experts (Section 3.1, Algorithm 3;
`oracle.router`), and E4M3 operands whose quantisation rides on the pruning pass (Section 3.2.2, last
paragraph; `oracle.fp8`: format, scaling and order of operations are this oracle's readings, stated there).

Nothing in here is shared with, imported by, or derived from the CUDA path. Only the tests,
the smoke check and the benchmark's CPU-baseline leg may import this package; the product
never routes through it.

Pins: every function is pinned by the CPU tests (brute force, closed forms, structural
invariants, finite differences). One reading is "parity unpinned" by the paper itself: the
criterion that picks the four kept columns of a V x M block (Section 2.3 only says four columns
are retained); the oracle uses the ordered fp32 column sum of magnitudes, pinned internally by
brute force on exactly-summable data. The router's clustering details (start, balanced assignment
order) are this oracle's own choices too: any balanced partition is a valid router, so the step
functions take the routing and the feature order as inputs.
"""
from .bf16 import bf16_to_f32, f32_to_bf16
from .prune24 import prune24, decompress24, Prune24Result
from .vnm import vnm_sparsify, decompress_vnm, VnmResult
from .ffn import (sparse_ffn_fwd, sparse_ffn_bwd, dense_ffn_fwd, dense_ffn_bwd,
                  SparseFwd, SparseBwd, DenseFwd, DenseBwd, matmul_f64)

__all__ = [
    "bf16_to_f32", "f32_to_bf16",
    "prune24", "decompress24", "Prune24Result",
    "vnm_sparsify", "decompress_vnm", "VnmResult",
    "sparse_ffn_fwd", "sparse_ffn_bwd", "dense_ffn_fwd", "dense_ffn_bwd",
    "SparseFwd", "SparseBwd", "DenseFwd", "DenseBwd", "matmul_f64",
]
