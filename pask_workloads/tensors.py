"""Seeded synthetic Q / K / V activations (stand-ins for Qwen3 post-RoPE projections).

Values are approximately N(0,1): the sum of twelve 16-bit uniforms taken from three hash words
(Irwin-Hall, variance exactly 1), centred and scaled by 2^-16, which is exact in fp32, then
rounded to bf16 (round to nearest even). Element (tensor, layer, seq, token, head, dim) depends
only on the seed and those coordinates, so the CPU oracle can regenerate any sampled
(layer, sequence) slice of a workload that was generated on the device.
"""
from __future__ import annotations

import torch

from .rng import hash_words, make_key, _lsr

TENSOR_Q, TENSOR_K, TENSOR_V = 0, 1, 2
HEAD_DIM = 128


def normal_bf16(seed: int, tensor: int, layer: int, seq: int, token_start: int, n_tokens: int,
                n_heads: int, device="cpu", head_dim: int = HEAD_DIM) -> torch.Tensor:
    """bf16 tensor [n_tokens, n_heads, head_dim] for tokens token_start .. token_start+n_tokens-1."""
    key = make_key(seed, tensor, layer, seq)
    row = n_heads * head_dim
    n = n_tokens * row
    if n == 0:
        return torch.empty((0, n_heads, head_dim), dtype=torch.bfloat16, device=device)
    idx = torch.arange(token_start * row, token_start * row + n, dtype=torch.int64, device=device)
    total = torch.zeros(n, dtype=torch.int64, device=device)
    for w in range(3):
        h = hash_words(key, idx * 4 + w)
        total += (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + (_lsr(h, 48) & 0xFFFF)
    x = (total - 393210).to(torch.float32) * (1.0 / 65536.0)
    return x.to(torch.bfloat16).view(n_tokens, n_heads, head_dim)


def ragged_normal_bf16(seed: int, tensor: int, layer: int, seq_ids, token_starts, token_counts,
                       n_heads: int, device="cpu") -> torch.Tensor:
    """Concatenation over sequences of normal_bf16 slices: [sum(token_counts), n_heads, 128]."""
    parts = [normal_bf16(seed, tensor, layer, int(s), int(t0), int(n), n_heads, device)
             for s, t0, n in zip(seq_ids, token_starts, token_counts)]
    if not parts:
        return torch.empty((0, n_heads, HEAD_DIM), dtype=torch.bfloat16, device=device)
    return torch.cat(parts, dim=0)


def bf16_bits(x: torch.Tensor) -> torch.Tensor:
    """View a bf16 tensor as its raw 16-bit patterns (int16 storage, same shape)."""
    assert x.dtype == torch.bfloat16
    return x.view(torch.int16)
