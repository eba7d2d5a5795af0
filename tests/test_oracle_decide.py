"""Pins for the oracle's dynamic budget adjustment (Algorithm 2 steps 3-6 and 8; CPU only).

Hand-worked cases from tests/golden/decide_cases.txt, the special cases that reduce to the
frozen table or to the floors, and invariants on random tables checked by recounting.
"""
import os

import numpy as np
import pytest

from pask_workloads import policy as WP
from pask_workloads.rng import CounterRng
from pask_workloads.tensors import bf16_bits, normal_bf16

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "decide_cases.txt")
LETTER = {"R": 0, "L": 1, "H": 2}
M = {2: (0, 288, 1024), 8: (0, 1152, 4096)}       # bytes per token per layer for R, L, H


def _cases():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            fld = [x.strip() for x in line.split("|")]
            assert len(fld) == 11, line
            out.append(pytest.param(fld, id=fld[0]))
    return out


def _letters(s):
    return [LETTER[ch] for ch in s]


@pytest.mark.parametrize("fld", _cases())
def test_hand_worked_cases(oracle, fld):
    _, q16, gamma, crit, a0, fl, rl, lh, tags, want, counts = fld
    pol = WP.Policy(1, 3, np.asarray([0, 1, 2], np.uint8), np.asarray([_letters(a0)], np.uint8),
                    np.asarray([_letters(fl)], np.uint8), np.asarray([[float(x) for x in rl.split()]], np.float32),
                    np.asarray([[float(x) for x in lh.split()]], np.float32),
                    gamma=np.asarray([int(gamma)], np.uint32), budget_target=int(q16) / 65536.0,
                    crit=np.asarray([int(crit)], np.uint8))
    c = oracle.Cache(oracle.Policy(WP.write_blob(pol)), 8, 2, 1, 16, 16)
    tg = np.asarray([0xFF if t == "P" else int(t) for t in tags.split()], np.uint8)
    rc, act = c.decide([0], [0, len(tg)], tg, states=np.zeros(len(tg), np.uint16), n_groups=3)
    assert rc == 0
    assert act.tolist() == [_letters(w) for w in want.split()]
    b = c.budget(0)
    assert [b.n_demoted, b.n_promoted, b.n_floor_conflicts] == [int(x) for x in counts.split()]
    assert b.decided_full_bytes == 3072 * len(tg)
    assert b.decided_retained_bytes == sum(M[2][a] for row in act.tolist() for a in row)


def _random_policy(seed, n_tags, n_groups, n_layers, target, n_states=8, crit_p=0.5, gamma_max=1 << 14):
    rng = CounterRng(seed, 909)
    p = WP.random_policy(seed, n_tags, n_groups, n_layers)
    p.budget_target = target
    p.gamma = np.asarray([rng.below(gamma_max) for _ in range(n_states)], np.uint32)
    p.crit = np.asarray([1 if rng.unit() < crit_p else 0 for _ in range(n_states)], np.uint8)
    return p


def _stream(seed, n, n_tags, n_states):
    rng = CounterRng(seed, 910)
    tags = np.asarray([rng.below(n_tags) for _ in range(n)], np.uint8)
    states = np.asarray([rng.below(n_states + 2) for _ in range(n)], np.uint16)   # two ids past the table
    return tags, states


def _cost(act_row, layers_in_group, n_kv):
    return sum(int(layers_in_group[g]) * M[n_kv][int(a)] for g, a in enumerate(act_row))


def test_full_target_without_critical_states_is_the_frozen_table(oracle):
    # target 1, no reserve: every token's own full cost is added to R before it is charged, so
    # nothing is ever over budget; with no critical state the result is a = max(a0, floor)
    p = _random_policy(3, 6, 4, 8, 1.0, crit_p=0.0, gamma_max=1)
    c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, 2, 1, 16, 16)
    tags, states = _stream(3, 300, 6, 8)
    rc, act = c.decide([0], [0, 300], tags, states=states, n_groups=4)
    assert rc == 0
    assert np.array_equal(act, np.maximum(p.a0, p.a_floor)[tags])
    b = c.budget(0)
    assert b.n_demoted == b.n_promoted == b.n_floor_conflicts == 0


def test_zero_target_is_the_floors(oracle):
    p = _random_policy(4, 6, 4, 8, 0.0)
    c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, 2, 1, 16, 16)
    tags, states = _stream(4, 300, 6, 8)
    rc, act = c.decide([0], [0, 300], tags, states=states, n_groups=4)
    assert rc == 0
    assert np.array_equal(act, p.a_floor[tags])


def test_critical_state_with_room_promotes_to_high(oracle):
    # target 1, no reserve, every state critical: each token may spend its own full cost
    p = _random_policy(5, 6, 4, 8, 1.0, crit_p=1.1, gamma_max=1)
    c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, 2, 1, 16, 16)
    tags = _stream(5, 100, 6, 8)[0]
    rc, act = c.decide([0], [0, 100], tags, states=np.zeros(100, np.uint16), n_groups=4)
    assert rc == 0 and np.all(act == 2)


def test_no_states_means_no_reserve_and_nothing_critical(oracle):
    p = _random_policy(6, 6, 4, 8, 0.4, crit_p=1.1)
    blob = WP.write_blob(p)
    tags, _ = _stream(6, 200, 6, 8)
    c1 = oracle.Cache(oracle.Policy(blob), 8, 2, 1, 16, 16)
    rc, a1 = c1.decide([0], [0, 200], tags, states=None, n_groups=4)
    assert rc == 0
    # the same as states that all lie outside the table
    c2 = oracle.Cache(oracle.Policy(blob), 8, 2, 1, 16, 16)
    rc, a2 = c2.decide([0], [0, 200], tags, states=np.full(200, 999, np.uint16), n_groups=4)
    assert rc == 0 and np.array_equal(a1, a2)
    assert np.all(a1 <= np.maximum(p.a0, p.a_floor)[tags])       # nothing was promoted


@pytest.mark.parametrize("target", [0.1, 0.33, 0.6])
def test_invariants_by_recount(oracle, target):
    """Replays R from the returned actions alone and checks, token by token: floors are never
    crossed; a token is demoted only if the table's cost exceeded B, and then either fits or sits
    on its floors, and undoing any one demotion step would overshoot or be out of order;
    promotions occur only in critical states, fit in B, and leave no further step that fits."""
    n_tags, G, n_layers, n_kv, n_states, n = 7, 4, 10, 2, 8, 400
    p = _random_policy(11, n_tags, G, n_layers, target, n_states=n_states)
    lig = np.bincount(p.layer_group, minlength=G)
    c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, n_kv, 1, 16, 16)
    tags, states = _stream(12, n, n_tags, n_states)
    tags[::37] = 0xFF                                             # protected
    tags[5::41] = 200                                             # unknown
    rc, act = c.decide([0], [0, n], tags, states=states, n_groups=G)
    assert rc == 0
    q16 = int(round(target * 65536.0))
    full = retained = 0
    F = sum(int(lig[g]) * M[n_kv][2] for g in range(G))
    saw = {"demote": 0, "promote": 0, "conflict": 0}
    for t in range(n):
        z, s = int(tags[t]), int(states[t])
        table = z < n_tags
        fl = p.a_floor[z] if table else np.full(G, 2)
        eff = np.maximum(p.a0[z], fl) if table else np.full(G, 2)
        gam = int(p.gamma[s]) if s < n_states else 0
        crit = bool(p.crit[s]) if s < n_states else False
        full += F
        B = max(0, ((q16 * full) >> 16) - retained - gam)
        a = act[t].astype(int)
        cost = _cost(a, lig, n_kv)
        assert np.all(a >= fl)
        down = [g for g in range(G) if a[g] < eff[g]]
        up = [g for g in range(G) if a[g] > eff[g]]
        assert not (down and up) or crit
        if down:
            saw["demote"] += 1
            assert _cost(eff, lig, n_kv) > B
        if up:
            saw["promote"] += 1
            assert crit and cost <= B
        if not crit:
            assert not up
            if cost > B:                                          # still over: only floors may be left
                assert all(a[g] == fl[g] or lig[g] == 0 for g in range(G))
                saw["conflict"] += 1
            elif down:
                # the loop stops as soon as the cost fits: before its last step (the last step of
                # one of the lowered groups) the cost was still over B
                back = [int(lig[g]) * (M[n_kv][a[g] + 1] - M[n_kv][a[g]]) for g in down]
                assert cost + max(back) > B
            if down:
                # order: a group that was never lowered but could have been had its step on offer
                # the whole time, so every step taken scored no higher (equal only from an earlier group)
                rho = lambda g, lvl: float(p.rho_lh[z, g] if lvl == 2 else p.rho_rl[z, g])
                for g in range(G):
                    if g in down or a[g] <= fl[g] or lig[g] == 0:
                        continue
                    for h in down:
                        for lvl in range(a[h] + 1, eff[h] + 1):
                            assert rho(h, lvl) < rho(g, a[g]) or (rho(h, lvl) == rho(g, a[g]) and h < g)
        else:
            for g in range(G):                                    # nothing that fits was left on the table
                if a[g] < 2 and lig[g] > 0 and cost <= B:
                    assert cost + int(lig[g]) * (M[n_kv][a[g] + 1] - M[n_kv][a[g]]) > B
        retained += cost
    b = c.budget(0)
    assert b.decided_full_bytes == full and b.decided_retained_bytes == retained
    if target < 0.5:
        assert saw["demote"] > 0
    if target > 0.3:
        assert saw["promote"] > 0


def test_larger_reserve_never_retains_more(oracle):
    n_tags, G = 6, 4
    tags, _ = _stream(21, 300, n_tags, 1)
    got = []
    for gam in (0, 4096, 1 << 16, 1 << 30):
        p = _random_policy(21, n_tags, G, 8, 0.5, n_states=1, crit_p=0.0)
        p.gamma = np.asarray([gam], np.uint32)
        c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, 2, 1, 16, 16)
        rc, act = c.decide([0], [0, 300], tags, states=np.zeros(300, np.uint16), n_groups=G)
        assert rc == 0
        got.append((act, c.budget(0).decided_retained_bytes))
    # first token: a larger reserve leaves a smaller B, and Demote is monotone in B
    for (a, _), (b, _) in zip(got, got[1:]):
        assert np.all(b[0] <= a[0])
    assert np.array_equal(got[-1][0], _random_policy(21, n_tags, G, 8, 0.5, n_states=1).a_floor[tags])


def test_gamma_shift_scales_the_reserve(oracle):
    tags, _ = _stream(22, 200, 6, 1)
    res = []
    for gam, sh in ((3 << 10, 0), (3, 10)):
        p = _random_policy(22, 6, 4, 8, 0.5, n_states=1, crit_p=0.0)
        p.gamma = np.asarray([gam], np.uint32)
        p.gamma_shift = sh
        c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, 2, 1, 16, 16)
        res.append(c.decide([0], [0, 200], tags, states=np.zeros(200, np.uint16), n_groups=4)[1])
    assert np.array_equal(res[0], res[1])


def test_decide_then_append_realises_the_decided_cost(oracle):
    # step 7 after steps 1-6: appending every layer with the decided actions makes the realised
    # counters equal Algorithm 2's own running budget, and the streams hold what was decided
    n_tags, G, n_layers, n_kv, n = 6, 3, 5, 2, 150
    p = _random_policy(31, n_tags, G, n_layers, 0.35, n_states=4)
    c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, n_kv, 2, 256, 256)
    tags, states = _stream(31, n, n_tags, 4)
    cu = [0, 60, n]
    rc, act = c.decide([1, 0], cu, tags, states=states, n_groups=G)
    assert rc == 0
    for layer in range(n_layers):
        k = bf16_bits(normal_bf16(31, 1, layer, 0, 0, n, n_kv)).numpy()
        v = bf16_bits(normal_bf16(31, 2, layer, 0, 0, n, n_kv)).numpy()
        rc, used = c.append(layer, [1, 0], cu, k, v, tags, decided=act)
        assert rc == 0
        g = int(p.layer_group[layer])
        assert np.array_equal(used, act[:, g])
        for i, seq in enumerate([1, 0]):
            a = act[cu[i]:cu[i + 1], g]
            assert c.stream_len(layer, seq) == (int((a == 2).sum()), int((a == 1).sum()))
    for seq in (0, 1):
        b = c.budget(seq)
        assert b.retained_bytes == b.decided_retained_bytes
        assert b.full_bytes == b.decided_full_bytes


def test_decide_refuses_bad_calls_and_changes_nothing(oracle):
    p = _random_policy(41, 6, 4, 8, 0.5)
    c = oracle.Cache(oracle.Policy(WP.write_blob(p)), 8, 2, 2, 16, 16)
    tags, states = _stream(41, 10, 6, 8)
    assert c.decide([0, 0], [0, 5, 10], tags, states=states, n_groups=4)[0] == oracle.ERR_SEQ
    assert c.decide([0, 2], [0, 5, 10], tags, states=states, n_groups=4)[0] == oracle.ERR_SEQ
    for seq in (0, 1):
        assert c.budget(seq).decided_full_bytes == 0
    # append refuses an action outside R, L, H
    k = bf16_bits(normal_bf16(41, 1, 0, 0, 0, 10, 2)).numpy()
    bad = np.zeros((10, 4), np.uint8)
    bad[3, 0] = 3
    assert c.append(0, [0], [0, 10], k, k, tags, decided=bad)[0] == oracle.ERR_ARG
    assert c.stream_len(0, 0) == (0, 0)


def test_policy_blob_versions(oracle):
    p = _random_policy(51, 4, 2, 4, 0.5)
    blob2 = WP.write_blob(p)
    oracle.Policy(blob2)
    p.crit = None
    blob1 = WP.write_blob(p)
    oracle.Policy(blob1)
    assert len(blob2) == len(blob1) + 4 + 8
    with pytest.raises(ValueError):
        oracle.Policy(blob2[:-4])
    bad = bytearray(blob2)
    bad[-8] = 2                                                   # a critical flag that is not 0 or 1
    with pytest.raises(ValueError):
        oracle.Policy(bytes(bad))
    p2 = _random_policy(51, 4, 2, 4, 0.5)
    p2.gamma_shift = 17
    with pytest.raises(ValueError):
        oracle.Policy(WP.write_blob(p2))
    p3 = _random_policy(51, 4, 2, 4, 0.5)
    p3.rho_lh[1, 1] = np.nan
    with pytest.raises(ValueError):
        oracle.Policy(WP.write_blob(p3))
