"""Seeded synthetic inputs for the PASK hot path: counter RNG, activations, tag streams, tables.

Serves both the CPU oracle's tests and the CUDA path's tests and benchmark. It generates inputs
only; nothing of the method itself is computed here.
"""
from . import configs, policy, rng, tags, tensors  # noqa: F401
