"""B200-native Trigger-Aware Quantization (TAQ) cross-attention.

The compute path lives in ``csrc/`` (CUDA for sm_100a behind a C ABI, built into ``libtaq.so``);
``binding`` marshals torch tensors into that ABI and ``synth`` draws the seeded benchmark inputs.
Importing the package loads nothing; ``binding.lib()`` loads the shared library on first use and
raises if it is missing (there is no CPU fallback).
"""
__all__ = ["binding", "synth", "build"]
