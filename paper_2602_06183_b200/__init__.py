"""B200-native sparsified Transformer-FFN training step (2:4 weights, V:N:M activations).

The compute path lives in ``csrc/`` (CUDA for sm_100a behind a C ABI, ``libsparseffn.so``);
``binding`` marshals arguments to it with ctypes, ``synth`` draws the seeded synthetic inputs.
Importing the package does not load the shared library; ``binding`` does, and fails loudly if
it is missing.
"""

__all__ = ["binding", "synth", "build"]
