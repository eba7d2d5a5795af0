"""The benchmark configurations as seeded synthetic workloads.

Each configuration fixes shapes (query / KV heads, layers, layer groups), the batch, the prompt
and generated lengths, how tags are produced (grammar mode or run-structured mix mode), and the
table (random, or greedy to a target normalised KV cost). A built `Workload` holds only small
host-side data (tag streams, the policy, lengths); activations are regenerated on demand from
the counter generator, on whatever device the caller asks for.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np
import torch

from . import tags as T
from .policy import (Policy, greedy_policy, random_policy, all_high_policy, write_blob, expected_cost,
                     with_dynamic_budget)
from .rng import BASE_SEED, CounterRng
from .tensors import TENSOR_K, TENSOR_Q, TENSOR_V, normal_bf16


@dataclass(frozen=True)
class Config:
    name: str
    index: int                       # position in the configuration list (seed offset)
    n_layers: int
    n_groups: int
    n_q: int
    n_kv: int
    batch: int
    prompt_len: int                  # used when len_lo == len_hi == 0
    gen_len: int
    len_lo: int = 0                  # total length drawn uniformly in [len_lo, len_hi], half prompt
    len_hi: int = 0
    budget: float = 0.33
    mode: str = "grammar"            # "grammar" | "mix"
    lut: str = "greedy"              # "greedy" | "random" | "all_high"
    bias: str = "balanced"           # greedy table flavour: "balanced" | "low" | "high"
    low_bits: int = 4                # width of the RETAIN-LOW codes: 2, 4 or 8
    protected_prompt: bool = False   # prompt tokens carry TAG_PROTECTED (tiny)
    extra_gen: int = 64              # generated tokens beyond gen_len kept ready for decode steps


TINY = Config("tiny", 0, n_layers=1, n_groups=1, n_q=8, n_kv=2, batch=1, prompt_len=512, gen_len=256,
              budget=1.0, lut="random", protected_prompt=True)
QWEN3_4B_1LAYER = Config("qwen3-4b-1layer-per-group-b8-2k+2k", 1, n_layers=4, n_groups=4, n_q=32, n_kv=8, batch=8,
                         prompt_len=2048, gen_len=2048)
QWEN3_4B_STEP = Config("qwen3-4b-36layer-b64-u2k-8k", 2, n_layers=36, n_groups=4, n_q=32, n_kv=8, batch=64,
                       prompt_len=0, gen_len=0, len_lo=2048, len_hi=8192)
QWEN3_8B_LONG = Config("qwen3-8b-36layer-b128-16k-mix", 3, n_layers=36, n_groups=4, n_q=32, n_kv=8,
                       batch=128, prompt_len=8192, gen_len=8192, mode="mix")
QWEN3_4B_SWEEP = Config("qwen3-4b-36layer-b64-8k-sweep", 4, n_layers=36, n_groups=4, n_q=32, n_kv=8,
                        batch=64, prompt_len=4096, gen_len=4096)
SWEEP_BUDGETS = (0.2, 0.33, 0.5, 0.75, 1.0)
# The shapes of the paper's latency table (Table 3): concurrency 8, 8K or 32K input tokens and
# 256 / 1024 / 2048 generated ones (here: the state after 1024 generated tokens).  Small batch, long
# context: few bytes per launch at 8K, deep splits at 32K.
TABLE3_8K = Config("qwen3-4b-36layer-c8-8k-in-1k-out", 5, n_layers=36, n_groups=4, n_q=32, n_kv=8, batch=8,
                   prompt_len=8192, gen_len=1024)
TABLE3_32K = Config("qwen3-4b-36layer-c8-32k-in-1k-out", 6, n_layers=36, n_groups=4, n_q=32, n_kv=8, batch=8,
                    prompt_len=32768, gen_len=1024)

# The one-layer configuration is run once per layer-group column: four layers, one per group.
CONFIGS = [TINY, QWEN3_4B_1LAYER, QWEN3_4B_STEP, QWEN3_8B_LONG, QWEN3_4B_SWEEP, TABLE3_8K, TABLE3_32K]


def scaled(cfg: Config, **kw) -> Config:
    """A reduced copy of a configuration (fewer layers / sequences / tokens) for parity cases."""
    return replace(cfg, **kw)


@dataclass
class Workload:
    cfg: Config
    seed: int
    prompt_tags: List[np.ndarray]
    gen_tags: List[np.ndarray]        # gen_len + extra_gen tags per sequence
    policy: Policy
    tag_counts: np.ndarray = field(default=None)

    @property
    def blob(self) -> bytes:
        return write_blob(self.policy)

    def prompt_len(self, b: int) -> int:
        return int(self.prompt_tags[b].shape[0])

    def gen_len(self, b: int) -> int:
        return int(self.gen_tags[b].shape[0]) - self.cfg.extra_gen

    def total_len(self, b: int) -> int:
        return self.prompt_len(b) + self.gen_len(b)

    def tags(self, b: int, t0: int, n: int) -> np.ndarray:
        """Tags of tokens t0 .. t0+n-1 of sequence b (prompt first, then generated)."""
        full = np.concatenate([self.prompt_tags[b], self.gen_tags[b]])
        return full[t0:t0 + n]

    def states(self, b: int, t0: int, n: int) -> np.ndarray:
        """Synthetic parser-state ids of the same tokens."""
        cache = self.__dict__.setdefault("_states", {})
        if b not in cache:
            cache[b] = T.parser_states(np.concatenate([self.prompt_tags[b], self.gen_tags[b]]))
        return cache[b][t0:t0 + n]

    def dynamic_blob(self, reserve_tokens: int = 32, budget: Optional[float] = None) -> bytes:
        """The table with critical-state flags, reserves and floors attached (version-2 blob)."""
        full = self.cfg.n_layers * 2 * self.cfg.n_kv * 128 * 2
        pol = with_dynamic_budget(self.policy, self.seed, full, reserve_tokens)
        if budget is not None:
            pol = replace(pol, budget_target=budget)
        return write_blob(pol)

    def kv(self, layer: int, b: int, t0: int, n: int, device="cpu"):
        k = normal_bf16(self.seed, TENSOR_K, layer, b, t0, n, self.cfg.n_kv, device)
        v = normal_bf16(self.seed, TENSOR_V, layer, b, t0, n, self.cfg.n_kv, device)
        return k, v

    def q(self, layer: int, b: int, t: int, device="cpu") -> torch.Tensor:
        """Query of sequence b at decode position t: [n_q, 128] bf16."""
        return normal_bf16(self.seed, TENSOR_Q, layer, b, t, 1, self.cfg.n_q, device)[0]

    def expected_cost(self) -> float:
        return expected_cost(self.policy, self.tag_counts)


def build(cfg: Config, seed: Optional[int] = None, repeat: int = 0) -> Workload:
    """Tag streams, lengths and table of a configuration; seed = base + configuration index."""
    seed = (BASE_SEED + cfg.index + repeat) if seed is None else seed
    rng = CounterRng(seed, 707)
    prompt_tags, gen_tags = [], []
    for b in range(cfg.batch):
        if cfg.len_hi:
            total = rng.randint(cfg.len_lo, cfg.len_hi)
            n_prompt = total // 2
            n_gen = total - n_prompt
        else:
            n_prompt, n_gen = cfg.prompt_len, cfg.gen_len
        if cfg.protected_prompt:
            pt = np.full(n_prompt, T.TAG_PROTECTED, dtype=np.uint8)
        elif cfg.mode == "mix":
            pt = T.mix_prompt_tags(seed, b, n_prompt)
        else:
            pt = T.grammar_prompt_tags(seed, b, n_prompt)
        n_g = n_gen + cfg.extra_gen
        gt = T.mix_decode_tags(seed, b, n_g) if cfg.mode == "mix" else T.grammar_decode_tags(seed, b, n_g)
        prompt_tags.append(pt)
        gen_tags.append(gt)
    n_tags = T.N_DECODE_TAGS if cfg.protected_prompt else T.N_ALL_TAGS
    counts = np.zeros(n_tags, dtype=np.int64)
    for pt, gt in zip(prompt_tags, gen_tags):
        for arr in (pt, gt[:len(gt) - cfg.extra_gen]):
            known = arr[arr < n_tags]
            counts += np.bincount(known, minlength=n_tags)
    if cfg.lut == "random":
        pol = random_policy(seed, n_tags, cfg.n_groups, cfg.n_layers)
    elif cfg.lut == "all_high":
        pol = all_high_policy(n_tags, cfg.n_groups, cfg.n_layers)
    else:
        pol = greedy_policy(seed, counts, cfg.n_groups, cfg.n_layers, cfg.budget, cfg.bias, cfg.low_bits)
    return Workload(cfg, seed, prompt_tags, gen_tags, pol, counts)
