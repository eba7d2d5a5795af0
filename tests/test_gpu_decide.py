"""GPU parity of the budget-dependent adjustment (pask_decide, Algorithm 2 steps 3-6 and 8) and of
persisting decided actions (pask_append_kv_decided), through the C ABI against the CPU oracle.
Decisions, counters, page ids and stored bytes must be identical; attention over the resulting
cache within the usual tolerance."""
import os

import numpy as np
import pytest
import torch

from pask_workloads import configs as WC
from pask_workloads import policy as WP

from parity import Pair

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "decide_cases.txt")
LETTER = {"R": 0, "L": 1, "H": 2}


@pytest.fixture(scope="module")
def pask():
    import paper_2608_28276_b200 as P      # fails loudly if libpask.so is missing
    assert torch.cuda.is_available()
    return P


def _cases():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                fld = [x.strip() for x in line.split("|")]
                out.append(pytest.param(fld, id=fld[0]))
    return out


@pytest.mark.parametrize("fld", _cases())
def test_hand_worked_cases_on_the_gpu(pask, fld):
    _, q16, gamma, crit, a0, fl, rl, lh, tags, want, counts = fld
    L = lambda s: [LETTER[ch] for ch in s]
    pol = WP.Policy(1, 3, np.asarray([0, 1, 2], np.uint8), np.asarray([L(a0)], np.uint8), np.asarray([L(fl)], np.uint8),
                    np.asarray([[float(x) for x in rl.split()]], np.float32),
                    np.asarray([[float(x) for x in lh.split()]], np.float32),
                    gamma=np.asarray([int(gamma)], np.uint32), budget_target=int(q16) / 65536.0,
                    crit=np.asarray([int(crit)], np.uint8))
    c = pask.Cache(WP.write_blob(pol), 3, 8, 2, 1, 64, 64, 16, 16)
    tg = np.asarray([0xFF if t == "P" else int(t) for t in tags.split()], np.uint8)
    d = "cuda"
    act = torch.full((len(tg), 3), 0xEE, dtype=torch.uint8, device=d)
    pask.pask_decide(c.handle, torch.tensor([0], dtype=torch.int32, device=d),
                     torch.tensor([0, len(tg)], dtype=torch.int32, device=d), torch.from_numpy(tg).to(d),
                     torch.zeros(len(tg), dtype=torch.int16, device=d), act)
    assert act.cpu().tolist() == [L(w) for w in want.split()]
    b = pask.pask_budget_state(c.handle, 0)
    assert [b.n_demoted, b.n_promoted, b.n_floor_conflicts] == [int(x) for x in counts.split()]
    assert b.decided_full_bytes == 3072 * len(tg) and b.device_status == 0
    c.close()


def _pair(pask, oracle, budget, batch=3, prompt=200, gen=120, reserve_tokens=8, **kw):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=batch, prompt_len=prompt, gen_len=gen, extra_gen=48)
    w = WC.build(cfg)
    return Pair(pask, oracle, w, blob=w.dynamic_blob(reserve_tokens=reserve_tokens, budget=budget), **kw), w


@pytest.mark.parametrize("budget", [0.15, 0.33, 0.7])
def test_prefill_then_decode_with_decided_actions(pask, oracle, budget):
    p, w = _pair(pask, oracle, budget)
    cfg = w.cfg
    seqs = [2, 0, 1]
    counts = [w.total_len(s) - 7 * i for i, s in enumerate(seqs)]      # ragged, several 32-token rounds
    starts = [0, 0, 0]
    tags, states = p.gather(seqs, counts, starts)
    _, act_o, act_g = p.decide(seqs, counts, tags, states)
    b = p.orc.budget(0)
    assert b.n_demoted > 0 and (budget < 0.5 or b.n_promoted > 0)       # the case exercises both loops
    for layer in range(cfg.n_layers):
        _, _, k, v = p.gather(seqs, counts, starts, layer)
        p.append_decided(layer, seqs, counts, k, v, tags, act_o, act_g)  # the general (plan + write) path
    p.compare_state()
    for s in range(3):
        g = pask.pask_budget_state(p.gpu.handle, s)
        assert g.retained_bytes == g.decided_retained_bytes and g.full_bytes == g.decided_full_bytes
    for layer in range(cfg.n_layers):
        p.check_attention(layer, [0, 1, 2], pos=counts[1])
    # decode: one token per sequence and step; decisions now depend on the budget left by the prefill
    pos = dict(zip(seqs, counts))
    for step in range(40):
        order = seqs if step % 2 == 0 else seqs[::-1]
        cnt, st = [1, 1, 1], [pos[s] for s in order]
        tags, states = p.gather(order, cnt, st)
        _, act_o, act_g = p.decide(order, cnt, tags, states)
        for layer in range(cfg.n_layers):
            _, _, k, v = p.gather(order, cnt, st, layer)
            p.append_decided(layer, order, cnt, k, v, tags, act_o, act_g)  # the one-launch decode path
        for s in order:
            pos[s] += 1
    p.compare_state()
    for layer in range(cfg.n_layers):
        p.check_attention(layer, [1, 2, 0], pos=pos[0])


def test_decide_without_states_and_with_unknown_ones(pask, oracle):
    p, w = _pair(pask, oracle, 0.3, batch=2, prompt=90, gen=40)
    tags, states = p.gather([0, 1], [100, 130], [0, 0])
    tags = tags.copy()
    tags[::13] = 0xFF
    tags[5::17] = 77                                                    # unknown tag: high, floor high
    p.decide([0, 1], [100, 130], tags, None)
    st = states.copy()
    st[::3] = 60000                                                     # ids past the reserve table
    p.decide([1, 0], [100, 130], tags, st)
    for s in (0, 1):
        p.compare_budget(s)


def test_decide_many_sequences_one_token_each(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=300, prompt_len=8, gen_len=8, extra_gen=8)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w, blob=w.dynamic_blob(reserve_tokens=2, budget=0.3))
    seqs = list(range(299, -1, -1))
    for t in range(12):
        tags, states = p.gather(seqs, [1] * 300, [t] * 300)
        p.decide(seqs, [1] * 300, tags, states)
    for s in (0, 17, 299):
        p.compare_budget(s)
    # empty sequences inside a ragged call
    counts = [0 if s % 3 == 0 else 2 for s in seqs]
    tags, states = p.gather(seqs, counts, [12] * 300)
    p.decide(seqs, counts, tags, states)
    for s in (0, 1, 298):
        p.compare_budget(s)


def test_refused_calls_change_nothing(pask, oracle):
    p, w = _pair(pask, oracle, 0.3, batch=2, prompt=40, gen=40)
    P, h = pask, p.gpu.handle
    tags, states = p.gather([0, 1], [5, 5], [0, 0])
    p.decide([0, 1], [5, 5], tags, states)
    before = [(P.pask_budget_state(h, s).decided_full_bytes, P.pask_budget_state(h, s).decided_retained_bytes) for s in (0, 1)]
    d = "cuda"
    act = torch.zeros((10, w.cfg.n_groups), dtype=torch.uint8, device=d)
    tg, st = torch.from_numpy(tags).to(d), torch.from_numpy(states.astype(np.int16)).to(d)

    def call(ids, cu):
        P.pask_decide(h, torch.tensor(ids, dtype=torch.int32, device=d), torch.tensor(cu, dtype=torch.int32, device=d), tg, st, act)
        return P.pask_budget_state(h, 0).device_status

    assert call([0, 0], [0, 5, 10]) & P.DEV_BAD_SEQ                     # a sequence named twice
    rc, _, _ = p.decide([0, 0], [5, 5], tags, states, expect_ok=False)
    assert rc == oracle.ERR_SEQ
    assert call([0, 5], [0, 5, 10]) & P.DEV_BAD_SEQ                     # id out of range
    assert call([0, 1], [0, 7, 5]) & P.DEV_BAD_RAGGED                   # descending offsets
    assert call([0, 1], [0, 5, 9]) & P.DEV_BAD_RAGGED                   # does not end at total_tokens
    after = [(P.pask_budget_state(h, s).decided_full_bytes, P.pask_budget_state(h, s).decided_retained_bytes) for s in (0, 1)]
    assert before == after
    # an action outside R, L, H refuses the append: one-launch path and general path
    for n in (6, 200):
        cfgn = WC.scaled(WC.QWEN3_4B_1LAYER, batch=1, prompt_len=n, gen_len=8, extra_gen=8)
        wn = WC.build(cfgn)
        q = Pair(pask, oracle, wn, blob=wn.dynamic_blob(budget=0.3))
        tags, states, k, v = q.gather([0], [n], [0], 0)
        _, act_o, act_g = q.decide([0], [n], tags, states)
        bad_o, bad_g = act_o.copy(), act_g.clone()
        bad_o[n // 2, 0] = 3
        bad_g[n // 2, 0] = 3
        rc = q.append_decided(0, [0], [n], k, v, tags, bad_o, bad_g, expect_ok=False)
        assert rc == oracle.ERR_ARG
        assert P.pask_debug_stream_len(q.gpu.handle, 0, 0) == (0, 0)
        assert P.pask_budget_state(q.gpu.handle, 0).device_status == P.DEV_BAD_ACTION
        assert P.pask_debug_pool_state(q.gpu.handle) == q.orc.pool_state()


def test_sequence_reset_clears_the_running_budget(pask, oracle):
    p, w = _pair(pask, oracle, 0.3, batch=2, prompt=40, gen=40)
    tags, states = p.gather([0, 1], [30, 30], [0, 0])
    p.decide([0, 1], [30, 30], tags, states)
    pask.pask_seq_reset(p.gpu.handle, 1)
    p.orc.seq_reset(1)
    p.compare_budget(1)
    assert pask.pask_budget_state(p.gpu.handle, 1).decided_full_bytes == 0
    tags, states = p.gather([1], [30], [0])
    p.decide([1], [30], tags, states)                                   # starts again from an empty budget
    p.compare_budget(1)
    p.compare_budget(0)


def test_protected_and_unknown_tags_in_critical_states_with_eight_groups(pask, oracle):
    # tag bytes outside the table (0xFF = protected, 200 and 254 = unknown) have no row of upgrade scores: they stay
    # at H in all eight groups whatever the budget says, are counted as floor conflicts when over budget, and the
    # scored tokens around them are adjusted exactly as the oracle adjusts them
    G, n_tags = 8, 6
    rng = np.random.default_rng(5)
    pol = WP.Policy(n_tags, G, np.arange(G, dtype=np.uint8), rng.integers(0, 3, (n_tags, G)).astype(np.uint8),
                    np.zeros((n_tags, G), np.uint8), rng.random((n_tags, G)).astype(np.float32),
                    rng.random((n_tags, G)).astype(np.float32), gamma=np.asarray([0, 4096, 0, 1 << 14], np.uint32),
                    budget_target=0.25, crit=np.asarray([1, 1, 0, 1], np.uint8))
    blob = WP.write_blob(pol)
    c = pask.Cache(blob, G, 8, 2, 1, 256, 256, 16, 16)
    orc = oracle.Cache(oracle.Policy(blob), 8, 2, 1, 16, 16)
    n = 200
    tags = rng.integers(0, n_tags, n).astype(np.uint8)
    tags[rng.random(n) < 0.3] = 0xFF
    tags[rng.random(n) < 0.1] = 200
    tags[7] = 254
    states = rng.integers(0, 4, n).astype(np.uint16)
    rc, act_o = orc.decide([0], [0, n], tags, states=states, n_groups=G)
    assert rc == 0
    d = "cuda"
    act = torch.full((n, G), 0xEE, dtype=torch.uint8, device=d)
    pask.pask_decide(c.handle, torch.tensor([0], dtype=torch.int32, device=d), torch.tensor([0, n], dtype=torch.int32, device=d),
                     torch.from_numpy(tags).to(d), torch.from_numpy(states.astype(np.int16)).to(d), act)
    got = act.cpu().numpy()
    assert np.array_equal(got, act_o)
    assert np.all(got[tags >= n_tags] == 2)
    g, o = pask.pask_budget_state(c.handle, 0), orc.budget(0)
    for f in ("decided_full_bytes", "decided_retained_bytes", "n_demoted", "n_promoted", "n_floor_conflicts"):
        assert getattr(g, f) == getattr(o, f), f
    assert g.n_floor_conflicts > 0 and g.n_demoted > 0 and g.device_status == 0
    c.close()
