"""Seeded synthetic persistence tables and the policy-blob writer.

A policy blob is the frozen output of offline calibration that the online path loads: for each
bucket (tag, layer group) the selected action, the protection floor and two adjacent-upgrade
scores, the layer -> group map, and a reserve per parser state. Calibration itself needs data
that does not exist here, so the tables are synthetic: random for the tiny case, and otherwise a
greedy adjacent-upgrade path (the shape the paper's allocation has) that stops at a target
normalised KV cost computed from the tag frequencies of the very streams it will be used on.

Little-endian layout written by `write_blob`:
    0  char[4] "PASK"      4  u32 version (1)      8  u32 n_tags       12 u32 n_groups
    16 u32 n_layers       20 u32 n_states         24 u32 budget_target_q16
    28 u32 recent_window  32 u32 low_bits (4)     36 u32 group_size (32)
    40 u8  layer_group[n_layers], zero padded to a multiple of 4 bytes
    then n_tags*n_groups entries, tag-major: u8 a0, u8 a_floor, u16 0, f32 rho_RL, f32 rho_LH
    then u32 gamma[n_states]
Version 2 (written when the policy carries critical-state flags) appends
    u32 gamma_shift (0..16: the reserve of state s is gamma[s] << gamma_shift bytes)
    u8  crit[n_states] (0 or 1), zero padded to a multiple of 4 bytes
Actions: 0 = release (drop), 1 = retain-low, 2 = retain-high.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass, field

import numpy as np

from .rng import CounterRng
from . import tags as T

R, L, H = 0, 1, 2
COST_L_OVER_H = 1152.0 / 4096.0      # int4 codes + fp16 scale per 32 values, against bf16


def cost_l_over_h(low_bits: int) -> float:
    """m(L) / m(H): codes of low_bits each plus one fp16 scale per 32 values, against bf16."""
    return (128 * low_bits / 8 + 8) / 256.0


@dataclass
class Policy:
    n_tags: int
    n_groups: int
    layer_group: np.ndarray            # u8 [n_layers]
    a0: np.ndarray                     # u8 [n_tags, n_groups]
    a_floor: np.ndarray                # u8 [n_tags, n_groups]
    rho_rl: np.ndarray                 # f32 [n_tags, n_groups]
    rho_lh: np.ndarray                 # f32 [n_tags, n_groups]
    gamma: np.ndarray = field(default_factory=lambda: np.zeros(1, dtype=np.uint32))
    budget_target: float = 1.0
    recent_window: int = 0
    low_bits: int = 4
    group_size: int = 32
    crit: np.ndarray | None = None     # u8 [n_states] critical-state flags (None: version-1 blob)
    gamma_shift: int = 0

    @property
    def n_layers(self) -> int:
        return int(self.layer_group.shape[0])


def write_blob(p: Policy) -> bytes:
    q16 = int(round(p.budget_target * 65536.0))
    out = bytearray()
    out += b"PASK"
    version = 1 if p.crit is None else 2
    out += struct.pack("<9I", version, p.n_tags, p.n_groups, p.n_layers, int(p.gamma.shape[0]), q16,
                       p.recent_window, p.low_bits, p.group_size)
    lg = bytes(np.asarray(p.layer_group, dtype=np.uint8).tolist())
    out += lg + b"\0" * ((-len(lg)) % 4)
    for z in range(p.n_tags):
        for c in range(p.n_groups):
            out += struct.pack("<BBHff", int(p.a0[z, c]), int(p.a_floor[z, c]), 0,
                               float(p.rho_rl[z, c]), float(p.rho_lh[z, c]))
    out += np.asarray(p.gamma, dtype="<u4").tobytes()
    if version == 2:
        assert p.crit.shape[0] == p.gamma.shape[0]
        out += struct.pack("<I", p.gamma_shift)
        cr = bytes(np.asarray(p.crit, dtype=np.uint8).tolist())
        out += cr + b"\0" * ((-len(cr)) % 4)
    return bytes(out)


def equal_layer_groups(n_layers: int, n_groups: int) -> np.ndarray:
    """Contiguous, equally sized layer ranges (36 layers, 4 groups -> 9 layers each)."""
    return np.asarray([min(n_groups - 1, (l * n_groups) // n_layers) for l in range(n_layers)],
                      dtype=np.uint8)


def random_policy(seed: int, n_tags: int, n_groups: int, n_layers: int) -> Policy:
    """Uniformly random selected actions and floors (the tiny case)."""
    rng = CounterRng(seed, 505)
    a0 = np.zeros((n_tags, n_groups), np.uint8)
    fl = np.zeros((n_tags, n_groups), np.uint8)
    rl = np.zeros((n_tags, n_groups), np.float32)
    lh = np.zeros((n_tags, n_groups), np.float32)
    for z in range(n_tags):
        for c in range(n_groups):
            a0[z, c] = rng.below(3)
            fl[z, c] = rng.below(3) if rng.unit() < 0.3 else 0
            rl[z, c] = rng.unit()
            lh[z, c] = rng.unit() * 0.5
    gamma = np.asarray([rng.below(1 << 20) for _ in range(8)], dtype=np.uint32)
    return Policy(n_tags, n_groups, equal_layer_groups(n_layers, n_groups), a0, fl, rl, lh, gamma,
                  budget_target=1.0)


_PRIOR = {
    T.REQUIRED_KEY: 1.00, T.ENUM_VALUE: 0.90, T.ARGUMENT_VALUE: 0.80, T.BOUNDARY: 0.50,
    T.FREE_TEXT: 0.35, T.SCAFFOLD: 0.20,
    T.P_PROTECTED: 1.00, T.P_FUNCTION_NAME: 0.90, T.P_PARAMETER_KEY: 0.75, T.P_CONSTRAINT: 0.60,
    T.P_SCHEMA_SCAFFOLD: 0.15,
}


def greedy_policy(seed: int, tag_counts: np.ndarray, n_groups: int, n_layers: int, budget: float,
                  bias: str = "balanced", low_bits: int = 4) -> Policy:
    """Greedy adjacent-upgrade table that reaches (without exceeding) a target normalised cost.

    tag_counts[z] is how many tokens of the workload carry tag z (all sequences, prompt and
    generated). Every bucket starts released; upgrade R->L of bucket (z, c) has score
    prior(z) + 0.1 c + noise and its L->H follow-up the same score minus `lh_penalty`; upgrades
    are applied in descending score while the expected cost stays within the budget, and a last
    pass adds whatever still fits. `bias` moves the L->H penalty to obtain LOW-heavy or
    HIGH-heavy tables at the same cost ("low": almost everything retained at low precision,
    "high": few tokens kept, almost all at high precision).
    """
    n_tags = int(tag_counts.shape[0])
    rng = CounterRng(seed, 606)
    lg = equal_layer_groups(n_layers, n_groups)
    w = np.bincount(lg, minlength=n_groups).astype(np.float64) / n_layers
    f = tag_counts.astype(np.float64) / max(1.0, float(tag_counts.sum()))
    a = np.zeros((n_tags, n_groups), np.uint8)
    rl = np.zeros((n_tags, n_groups), np.float32)
    lh = np.zeros((n_tags, n_groups), np.float32)
    lh_penalty = {"balanced": 0.5, "low": 5.0, "high": -5.0}[bias]
    cost_l = cost_l_over_h(low_bits)
    ups = []
    for z in range(n_tags):
        for c in range(n_groups):
            s = _PRIOR.get(z, 0.5) + 0.1 * c + (rng.unit() - 0.5) * 0.1
            rl[z, c] = s
            lh[z, c] = s - 0.5
            ups.append((s, z, c, L))
            ups.append((s - lh_penalty, z, c, H))
    if budget >= 1.0:
        a[:, :] = H
    else:
        cost = 0.0
        ups.sort(key=lambda u: (-u[0], u[1], u[2], u[3]))
        pending = list(ups)
        for _ in range(2):                                   # greedy pass, then the fill pass
            rest = []
            for s, z, c, tgt in pending:
                if a[z, c] >= tgt:
                    continue
                # an H upgrade may arrive before its L (bias="high"): take both steps at once
                step = (cost_l if a[z, c] == R else 0.0) if tgt == L else \
                       (1.0 - (cost_l if a[z, c] == L else 0.0))
                dc = f[z] * w[c] * step
                if cost + dc <= budget + 1e-12:
                    a[z, c] = tgt
                    cost += dc
                else:
                    rest.append((s, z, c, tgt))
            pending = rest
    fl = np.zeros((n_tags, n_groups), np.uint8)
    gamma = np.asarray([rng.below(1 << 20) for _ in range(16)], dtype=np.uint32)
    return Policy(n_tags, n_groups, lg, a, fl, rl, lh, gamma, budget_target=budget, low_bits=low_bits)


def all_high_policy(n_tags: int, n_groups: int, n_layers: int) -> Policy:
    """The full high-precision reference: every bucket retained at high precision."""
    z = np.zeros((n_tags, n_groups), np.float32)
    a = np.full((n_tags, n_groups), H, np.uint8)
    return Policy(n_tags, n_groups, equal_layer_groups(n_layers, n_groups), a,
                  np.zeros_like(a), z, z.copy(), np.zeros(1, np.uint32), budget_target=1.0)


def expected_cost(p: Policy, tag_counts: np.ndarray) -> float:
    """Normalised KV cost the table yields on streams with these tag counts (protected tokens,
    which are not in tag_counts, are not included)."""
    eff = np.maximum(p.a0, p.a_floor).astype(np.int64)
    w = np.bincount(p.layer_group, minlength=p.n_groups).astype(np.float64) / p.n_layers
    per = np.where(eff == H, 1.0, np.where(eff == L, cost_l_over_h(p.low_bits), 0.0))
    f = tag_counts.astype(np.float64) / max(1.0, float(tag_counts.sum()))
    return float((f[:, None] * w[None, :] * per).sum())


def with_dynamic_budget(p: Policy, seed: int, token_full_bytes: int, reserve_tokens: int = 32,
                        gamma_shift: int = 8) -> Policy:
    """A copy of `p` that carries what the budget-dependent adjustment reads: critical-state flags
    for the synthetic parser states and a reserve per state of up to `reserve_tokens` tokens' full
    cost (Eq. 9's quantile needs calibration traces; here it is a seeded random amount), plus
    floors on the required-key and enum-value rows so that protection and budget can conflict."""
    from dataclasses import replace
    rng = CounterRng(seed, 808)
    gamma = np.asarray([(rng.below(reserve_tokens + 1) * token_full_bytes) >> gamma_shift
                        for _ in range(T.N_STATES)], dtype=np.uint32)
    fl = p.a_floor.copy()
    for z in (T.REQUIRED_KEY, T.ENUM_VALUE):
        if z < p.n_tags:
            fl[z, :] = np.maximum(fl[z, :], L)
    return replace(p, a_floor=fl, gamma=gamma, gamma_shift=gamma_shift, crit=T.critical_states())
