"""Counter-based integer random numbers shared by every seeded input generator.

The generators are pure functions of (seed, stream key, element index), so any slice of any
tensor can be regenerated anywhere (host or device, whole or sampled) and comes out identical.
Everything here is integer arithmetic on 64-bit words; the same torch code runs on CPU and on a
CUDA device and produces the same bits, because int64 multiplication wraps the same way on both.

This module holds input generation only: none of the method's arithmetic (table lookup,
quantisation, paging, attention) lives here.
"""
from __future__ import annotations

import numpy as np
import torch

MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB

BASE_SEED = 260828276


def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit constant as the signed value torch.int64 can hold."""
    x &= MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def splitmix64_int(x: int) -> int:
    """One splitmix64 output for a Python int (scalar keys)."""
    z = (x + _GOLDEN) & MASK64
    z = ((z ^ (z >> 30)) * _M1) & MASK64
    z = ((z ^ (z >> 27)) * _M2) & MASK64
    return z ^ (z >> 31)


def make_key(seed: int, *parts: int) -> int:
    """Fold a seed and a tuple of small integers (tensor id, layer, sequence, ...) into one key."""
    k = splitmix64_int(seed & MASK64)
    for p in parts:
        k = splitmix64_int((k ^ ((p & MASK64) * _GOLDEN)) & MASK64)
    return k


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right of int64 words (torch's >> is arithmetic)."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def splitmix64_torch(x: torch.Tensor) -> torch.Tensor:
    """Vectorised splitmix64 on int64 tensors holding the unsigned words' bit patterns."""
    z = x + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def hash_words(key: int, index: torch.Tensor) -> torch.Tensor:
    """64-bit hash of (key, index) for an int64 index tensor."""
    return splitmix64_torch(index + _s64(key))


def splitmix64_np(x: np.ndarray) -> np.ndarray:
    """numpy twin (uint64) used by the small host-side generators (tag streams, tables)."""
    with np.errstate(over="ignore"):
        z = x.astype(np.uint64) + np.uint64(_GOLDEN)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_M1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_M2)
        return z ^ (z >> np.uint64(31))


class CounterRng:
    """Tiny sequential view on the counter generator for host-side structure generators.

    Draw i of stream `key` is splitmix64(key + i); helpers turn draws into bounded integers
    and unit-interval floats. Deterministic and independent of numpy's / Python's own RNGs.
    """

    def __init__(self, seed: int, *parts: int):
        self.key = make_key(seed, *parts)
        self.i = 0

    def u64(self) -> int:
        v = splitmix64_int((self.key + self.i) & MASK64)
        self.i += 1
        return v

    def below(self, n: int) -> int:
        """Uniform integer in [0, n) (n << 2^64, so the modulo bias is immaterial)."""
        return self.u64() % n

    def randint(self, lo: int, hi: int) -> int:
        """Uniform integer in [lo, hi] inclusive."""
        return lo + self.below(hi - lo + 1)

    def unit(self) -> float:
        return (self.u64() >> 11) * (1.0 / (1 << 53))

    def choice(self, seq):
        return seq[self.below(len(seq))]

    def weighted(self, weights) -> int:
        tot = float(sum(weights))
        x = self.unit() * tot
        acc = 0.0
        for i, w in enumerate(weights):
            acc += w
            if x < acc:
                return i
        return len(weights) - 1
