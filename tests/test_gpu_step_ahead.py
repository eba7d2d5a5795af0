"""Planned-ahead decode steps (pask_plan_ahead + pask_decode_step_ahead) against the oracle and against
pask_append_attend.

The streaming kernel of such a step works from a plan of the cache before the step's append, the
append runs beside it and the merge attends the new token from the call's inputs.  The cache state
it leaves (pages, codes, scales, page ids, counters) must be bit-identical to the oracle's and to
what pask_append_attend leaves; out / lse must agree with the fp64 oracle within the usual bound."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from pask_workloads import configs as WC
from pask_workloads import policy as WP
from pask_workloads.tensors import bf16_bits

from parity import Pair, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pask():
    import paper_2608_28276_b200 as P
    assert torch.cuda.is_available()
    return P


def _pair(pask, oracle, batch, prompt, gen, low_bits=4, dynamic=False, **kw):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=batch, prompt_len=prompt, gen_len=gen, extra_gen=80, low_bits=low_bits)
    w = WC.build(cfg)
    blob = w.dynamic_blob(reserve_tokens=4, budget=0.3) if dynamic else w.blob
    return Pair(pask, oracle, w, blob=blob, **kw), w


def _ahead_step(p, area, layer, seqs, pos, acts=None):
    """One planned-ahead call on the GPU, append + attention on the oracle; compares actions and outputs."""
    d = "cuda"
    n = len(seqs)
    ones = [1] * n
    tags, states, k, v = p.gather(seqs, ones, pos, layer)
    act_o, act_g = acts if acts else (None, None)
    rc, used_o = p.orc.append(layer, seqs, list(range(n + 1)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags, decided=act_o)
    assert rc == 0
    q = torch.stack([p.w.q(layer, int(s), int(t) + 1) for s, t in zip(seqs, pos)])
    out = torch.full((n, p.cfg.n_q, 128), float("nan"), dtype=torch.float32, device=d)
    lse = torch.full((n, p.cfg.n_q), float("nan"), dtype=torch.float32, device=d)
    used_g = torch.full((n,), 0xEE, dtype=torch.uint8, device=d)
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    p.pask.pask_decode_step_ahead(p.gpu.handle, layer, ids, k.to(d), v.to(d), torch.from_numpy(tags).to(d), q.to(d), out, lse,
                                  p.gpu.workspace(n), area, actions=act_g, actions_out=used_g)
    torch.cuda.synchronize()
    assert np.array_equal(used_g.cpu().numpy(), used_o)
    oo, ol = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
    assert_close(out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), oo, ol, where=(layer, seqs))
    return out, lse, (ids, k.to(d), v.to(d), torch.from_numpy(tags).to(d), q.to(d))


@pytest.mark.parametrize("batch,low_bits,dynamic", [(5, 4, False), (64, 4, False), (7, 4, True), (3, 8, False), (3, 2, False),
                                                    (255, 4, False)])
def test_steps_ahead_against_the_oracle(pask, oracle, batch, low_bits, dynamic):
    prompt, gen = (40, 24) if batch > 8 else (150, 70)
    p, w = _pair(pask, oracle, batch, prompt, gen, low_bits=low_bits, dynamic=dynamic)
    seqs = list(range(batch))[::-1]
    lens = [w.total_len(s) - (3 * s) % 17 for s in seqs]
    if dynamic:
        tags, states = p.gather(seqs, lens, [0] * batch)
        _, act_o, act_g = p.decide(seqs, lens, tags, states)
        for layer in range(w.cfg.n_layers):
            _, _, k, v = p.gather(seqs, lens, [0] * batch, layer)
            p.append_decided(layer, seqs, lens, k, v, tags, act_o, act_g)
    else:
        for layer in range(w.cfg.n_layers):
            p.append(layer, seqs, lens, [0] * batch)
    area = torch.empty(pask.pask_plan_area_bytes(p.gpu.handle, batch), dtype=torch.uint8, device="cuda")
    ids = torch.tensor(seqs, dtype=torch.int32, device="cuda")
    for layer in range(w.cfg.n_layers):
        pask.pask_plan_ahead(p.gpu.handle, layer, ids, area)
    pos = list(lens)
    for step in range(36):                  # long enough for pages of both streams to fill up and new ones to be taken
        acts = None
        if dynamic:
            tags, states = p.gather(seqs, [1] * batch, pos)
            _, act_o, act_g = p.decide(seqs, [1] * batch, tags, states)
            acts = (act_o, act_g)
        for layer in range(w.cfg.n_layers):
            _ahead_step(p, area, layer, seqs, pos, acts)
        pos = [x + 1 for x in pos]
    p.compare_state()
    assert pask.pask_budget_state(p.gpu.handle, 0).device_status == 0


def test_same_state_and_close_outputs_as_the_fused_call(pask, oracle):
    p, w = _pair(pask, oracle, 4, 100, 60)
    p2, _ = _pair(pask, oracle, 4, 100, 60)
    seqs = [3, 1, 0, 2]
    lens = [150, 97, 160, 33]
    for layer in range(w.cfg.n_layers):
        p.append(layer, seqs, lens, [0] * 4)
        p2.append(layer, seqs, lens, [0] * 4)
    area = torch.empty(pask.pask_plan_area_bytes(p.gpu.handle, 4), dtype=torch.uint8, device="cuda")
    cu = torch.arange(5, dtype=torch.int32, device="cuda")
    for layer in range(w.cfg.n_layers):
        pask.pask_plan_ahead(p.gpu.handle, layer, torch.tensor(seqs, dtype=torch.int32, device="cuda"), area)
    pos = list(lens)
    for step in range(20):
        for layer in range(w.cfg.n_layers):
            out, lse, (ids, k, v, tags, q) = _ahead_step(p, area, layer, seqs, pos)
            out2, lse2 = torch.empty_like(out), torch.empty_like(lse)
            pask.pask_append_attend(p2.gpu.handle, layer, ids, cu, k, v, tags, q, out2, lse2, p2.gpu.workspace(4))
            torch.cuda.synchronize()
            assert float((out - out2).abs().max()) < 1e-3 and float((lse - lse2).abs().max()) < 1e-3     # (a new RETAIN-LOW token: exact here, P * scale in fp16 there)
        pos = [x + 1 for x in pos]
    # the two caches hold the same bytes
    for s in seqs:
        for layer in range(w.cfg.n_layers):
            a, b = pask.pask_debug_dump_high(p.gpu.handle, layer, s, 8), pask.pask_debug_dump_high(p2.gpu.handle, layer, s, 8)
            assert all(np.array_equal(x, y) for x, y in zip(a, b))
            a, b = pask.pask_debug_dump_low(p.gpu.handle, layer, s, 8), pask.pask_debug_dump_low(p2.gpu.handle, layer, s, 8)
            assert all(np.array_equal(x, y) for x, y in zip(a, b))
    p.compare_state()


def test_stale_plans_are_refused_or_flagged(pask, oracle):
    p, w = _pair(pask, oracle, 3, 60, 40)
    seqs = [0, 1, 2]
    for layer in range(w.cfg.n_layers):
        p.append(layer, seqs, [100] * 3, [0] * 3)
    P, h, d = pask, p.gpu.handle, "cuda"
    area = torch.empty(P.pask_plan_area_bytes(h, 3), dtype=torch.uint8, device=d)
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    tags, states, k, v = p.gather(seqs, [1] * 3, [100] * 3, 0)
    q = torch.stack([w.q(0, s, 101) for s in seqs]).to(d)
    out = torch.zeros((3, 32, 128), dtype=torch.float32, device=d)
    lse = torch.zeros((3, 32), dtype=torch.float32, device=d)
    args = (k.to(d), v.to(d), torch.from_numpy(tags).to(d), q, out, lse, p.gpu.workspace(3), area)

    def refused(layer=0, ids_=ids, a=args):
        with pytest.raises(P.PaskError) as e:
            P.pask_decode_step_ahead(h, layer, ids_, *a)
        return e.value.status

    assert refused() == P.ERR_STALE_PLAN                                  # no plan yet
    P.pask_plan_ahead(h, 0, ids, area)
    assert refused(layer=1) == P.ERR_STALE_PLAN                           # another layer
    assert refused(ids_=ids[:2].contiguous(), a=(k[:2].to(d), v[:2].to(d), torch.from_numpy(tags[:2]).to(d), q[:2].contiguous(),
                                                 out[:2], lse[:2], p.gpu.workspace(3), area)) == P.ERR_STALE_PLAN   # another batch size
    other = torch.empty_like(area)
    assert refused(a=args[:-1] + (other,)) == P.ERR_STALE_PLAN            # another plan area
    small = torch.empty(area.numel() - 256, dtype=torch.uint8, device=d)
    assert refused(a=args[:-1] + (small,)) == P.ERR_WORKSPACE
    # an append through another call forgets the plan
    p.append(0, seqs, [1] * 3, [100] * 3)
    assert refused() == P.ERR_STALE_PLAN
    # a different list of the same length is only seen on the device
    P.pask_plan_ahead(h, 0, ids, area)
    swapped = torch.tensor([1, 0, 2], dtype=torch.int32, device=d)
    P.pask_decode_step_ahead(h, 0, swapped, *args)
    torch.cuda.synchronize()
    assert P.pask_budget_state(h, 0).device_status & P.DEV_STALE_PLAN
    # a protected recent window is not served by this path
    pw = Pair(pask, oracle, w, blob=WP.write_blob(replace(w.policy, recent_window=16)))
    with pytest.raises(P.PaskError) as e:
        P.pask_plan_ahead(pw.gpu.handle, 0, ids, area)
    assert e.value.status == P.ERR_UNSUPPORTED_SHAPE


def test_refused_append_inside_a_step_ahead(pask, oracle):
    # the pools hold one page more than the history needs: within a few steps a call wants a page that is not there.
    # Nothing is written by that call, the sticky bit says why, and both sides still hold the same state.
    seqs, n0 = [0, 1], 64
    probe, w = _pair(pask, oracle, 2, 40, 20)
    for layer in range(w.cfg.n_layers):
        probe.append(layer, seqs, [n0] * 2, [0] * 2)
    used_h, _, used_l, _ = probe.orc.pool_state()
    p, w = _pair(pask, oracle, 2, 40, 20, pool_high_pages=used_h + 1, pool_low_pages=used_l + 1)
    P, h, d = pask, p.gpu.handle, "cuda"
    for layer in range(w.cfg.n_layers):
        p.append(layer, seqs, [n0] * 2, [0] * 2)
    area = torch.empty(P.pask_plan_area_bytes(h, 2), dtype=torch.uint8, device=d)
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    for layer in range(w.cfg.n_layers):
        P.pask_plan_ahead(h, layer, ids, area)
    pos, failed = n0, False
    for step in range(40):
        for layer in range(w.cfg.n_layers):
            tags, states, k, v = p.gather(seqs, [1] * 2, [pos] * 2, layer)
            rc, _ = p.orc.append(layer, seqs, [0, 1, 2], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
            q = torch.stack([w.q(layer, s, pos + 1) for s in seqs]).to(d)
            out = torch.zeros((2, 32, 128), dtype=torch.float32, device=d)
            lse = torch.zeros((2, 32), dtype=torch.float32, device=d)
            P.pask_decode_step_ahead(h, layer, ids, k.to(d), v.to(d), torch.from_numpy(tags).to(d), q, out, lse, p.gpu.workspace(2), area)
            torch.cuda.synchronize()
            st = P.pask_budget_state(h, 0).device_status
            if rc != 0:
                assert st & P.DEV_POOL_EXHAUSTED
                failed = True
                break
            assert st == 0
        if failed:
            break
        pos += 1
    assert failed
    p.compare_state(expect_status=P.DEV_POOL_EXHAUSTED)       # the refused call changed nothing on either side


def test_pipelined_host_steps_ahead(pask, oracle):
    # layer after layer from pinned host blocks, each layer's step issued as a planned-ahead one
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=5, n_layers=3, n_groups=3, prompt_len=150, gen_len=60, extra_gen=32)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [3, 0, 4, 1, 2]
    for layer in range(3):
        p.append(layer, seqs, [210] * 5, [0] * 5)
    P, h = pask, p.gpu.handle
    off, n_in = P.pask_step_packed_layout(h, 5)
    staging = torch.empty(2 * P.pask_step_staging_bytes(h, 5), dtype=torch.uint8, device="cuda")
    area = torch.empty(P.pask_plan_area_bytes(h, 5), dtype=torch.uint8, device="cuda")
    ids = torch.tensor(seqs, dtype=torch.int32, device="cuda")
    for layer in range(3):
        P.pask_plan_ahead(h, layer, ids, area)
    calls = []
    for step in range(20):
        for layer in range(3):
            k = torch.stack([w.kv(layer, b, 210 + step, 1)[0][0] for b in seqs])
            v = torch.stack([w.kv(layer, b, 210 + step, 1)[1][0] for b in seqs])
            tags = torch.from_numpy(np.array([w.tags(b, 210 + step, 1)[0] for b in seqs], np.uint8))
            q = torch.stack([w.q(layer, b, 211 + step) for b in seqs])
            block = torch.zeros(n_in, dtype=torch.uint8).pin_memory()
            for o, t in zip(off, [torch.tensor(seqs, dtype=torch.int32), torch.arange(6, dtype=torch.int32), k, v, tags, q]):
                raw = t.contiguous().view(torch.uint8).reshape(-1)
                block[o:o + raw.numel()] = raw
            out = torch.full((5, 32, 128), float("nan"), dtype=torch.float32).pin_memory()
            P.pask_decode_step_pipelined_ahead(h, layer, 5, block, out, staging, p.gpu.workspace(5), area)
            rc, _ = p.orc.append(layer, seqs, list(range(6)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags.numpy())
            assert rc == 0
            oo, ol = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
            calls.append((block, out, oo, ol))
    P.pask_decode_step_drain(h)
    torch.cuda.synchronize()
    for block, out, oo, ol in calls:
        assert_close(out.numpy().astype(np.float64), ol.copy(), oo, ol)
    p.compare_state()


def test_one_layer_called_back_to_back(pask, oracle):
    # a single layer stepped again and again: the plan a call reads was written by the call right before it, so the
    # streaming kernel may not read it ahead of its dependency wait (the handle keeps track); results stay the oracle's
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=6, n_layers=1, n_groups=1, prompt_len=90, gen_len=40, extra_gen=80)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [5, 4, 3, 2, 1, 0]
    lens = [w.total_len(s) for s in seqs]
    p.append(0, seqs, lens, [0] * 6)
    area = torch.empty(pask.pask_plan_area_bytes(p.gpu.handle, 6), dtype=torch.uint8, device="cuda")
    pask.pask_plan_ahead(p.gpu.handle, 0, torch.tensor(seqs, dtype=torch.int32, device="cuda"), area)
    d, n, pos, held = "cuda", 6, list(lens), []
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    for step in range(50):                 # no synchronisation between the calls: the kernels of consecutive steps do overlap
        tags, states, k, v = p.gather(seqs, [1] * n, pos, 0)
        rc, _ = p.orc.append(0, seqs, list(range(n + 1)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
        assert rc == 0
        q = torch.stack([w.q(0, s, t + 1) for s, t in zip(seqs, pos)])
        out = torch.full((n, cfg.n_q, 128), float("nan"), dtype=torch.float32, device=d)
        lse = torch.full((n, cfg.n_q), float("nan"), dtype=torch.float32, device=d)
        dev = (k.to(d), v.to(d), torch.from_numpy(tags).to(d), q.to(d))
        pask.pask_decode_step_ahead(p.gpu.handle, 0, ids, *dev, out, lse, p.gpu.workspace(n), area)
        held.append((dev, out, lse, p.orc.attention_batch(0, seqs, bf16_bits(q).numpy())))
        pos = [x + 1 for x in pos]
    torch.cuda.synchronize()
    for dev, out, lse, (oo, ol) in held:
        assert_close(out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), oo, ol)
    p.compare_state()


def test_two_steps_ahead_replayed_as_a_cuda_graph(pask, oracle):
    # Planned-ahead calls only enqueue work, so a stream capture can record them.  Which of a layer's two plan blocks a
    # call reads is fixed when it is recorded, so a graph that is replayed over and over must hold an even number of
    # steps: here two steps of every layer, replayed four times on new inputs.
    p, w = _pair(pask, oracle, 6, 120, 60)
    seqs = [2, 5, 0, 3, 1, 4]
    lens = [w.total_len(s) - 5 * i for i, s in enumerate(seqs)]
    L, d = w.cfg.n_layers, "cuda"
    for layer in range(L):
        p.append(layer, seqs, lens, [0] * 6)
    h = p.gpu.handle
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    area = torch.empty(pask.pask_plan_area_bytes(h, 6), dtype=torch.uint8, device=d)
    ws = p.gpu.workspace(6)
    mk = lambda shape, dt: [[torch.zeros(shape, dtype=dt, device=d) for _ in range(L)] for _ in range(2)]
    ks, vs = mk((6, w.cfg.n_kv, 128), torch.bfloat16), mk((6, w.cfg.n_kv, 128), torch.bfloat16)
    qs, outs = mk((6, w.cfg.n_q, 128), torch.bfloat16), mk((6, w.cfg.n_q, 128), torch.float32)
    lses, tgs = mk((6, w.cfg.n_q), torch.float32), mk((6,), torch.uint8)
    # first use of every kernel outside the capture, on a throw-away cache
    warm, _ = _pair(pask, oracle, 6, 120, 60)
    warm_area = torch.empty_like(area)
    pask.pask_plan_ahead(warm.gpu.handle, 0, ids, warm_area)
    pask.pask_decode_step_ahead(warm.gpu.handle, 0, ids, ks[0][0], vs[0][0], tgs[0][0], qs[0][0], outs[0][0], lses[0][0],
                                warm.gpu.workspace(6), warm_area)
    for layer in range(L):
        pask.pask_plan_ahead(h, layer, ids, area)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for half in range(2):
                for layer in range(L):
                    pask.pask_decode_step_ahead(h, layer, ids, ks[half][layer], vs[half][layer], tgs[half][layer], qs[half][layer],
                                                outs[half][layer], lses[half][layer], ws, area)
    torch.cuda.current_stream().wait_stream(side)
    pos = list(lens)
    for rep in range(4):
        want = [[None] * L for _ in range(2)]
        for half in range(2):
            for layer in range(L):
                tags, _, k, v = p.gather(seqs, [1] * 6, pos, layer)
                q = torch.stack([w.q(layer, s, t + 1) for s, t in zip(seqs, pos)])
                ks[half][layer].copy_(k); vs[half][layer].copy_(v); qs[half][layer].copy_(q)
                tgs[half][layer].copy_(torch.from_numpy(tags))
                rc, _ = p.orc.append(layer, seqs, list(range(7)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
                assert rc == 0
                want[half][layer] = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
            pos = [x + 1 for x in pos]
        graph.replay()
        torch.cuda.synchronize()
        for half in range(2):
            for layer in range(L):
                oo, ol = want[half][layer]
                assert_close(outs[half][layer].cpu().numpy().astype(np.float64), lses[half][layer].cpu().numpy().astype(np.float64),
                             oo, ol, where=(rep, half, layer))
    p.compare_state()
    assert pask.pask_budget_state(h, 0).device_status == 0


@pytest.mark.parametrize("seed,n_kv,low_bits", [(1, 8, 4), (2, 2, 4), (3, 1, 4), (4, 4, 8), (5, 8, 2), (6, 2, 4)])
def test_random_sequences_of_planned_ahead_steps(pask, oracle, seed, n_kv, low_bits):
    # Seeded differential fuzz: batches that change (and are then planned again), arbitrary per-token actions, bulk
    # appends and sequence resets in between (each makes the handle forget its plans), several layers in any order --
    # outputs of every planned-ahead call and the state after every call against the oracle.
    from pask_workloads.rng import CounterRng
    from pask_workloads.tensors import normal_bf16
    rng = CounterRng(seed, 777)
    n_layers, G, B = 3, 2, 5
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, n_kv=n_kv, n_q=4 * n_kv, n_layers=n_layers, n_groups=G, batch=B, prompt_len=8, gen_len=8,
                    extra_gen=8, low_bits=low_bits)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w, pool_high_pages=600, pool_low_pages=600, max_tokens_per_seq=2048, max_append_tokens=1024)
    P, h, d = pask, p.gpu.handle, "cuda"
    serial, planned = 0, None                    # planned: (tuple of sequences, set of layers that hold a plan)
    area = torch.empty(P.pask_plan_area_bytes(h, B), dtype=torch.uint8, device=d)

    def data(total):
        nonlocal serial
        serial += 1
        k = normal_bf16(seed, 1, serial, 0, 0, total, n_kv)
        v = normal_bf16(seed, 2, serial, 0, 0, total, n_kv)
        tags = np.asarray([rng.below(14) if rng.unit() < 0.9 else 0xFF for _ in range(total)], np.uint8)
        acts = np.asarray([[rng.weighted([3, 3, 3]) for _ in range(G)] for _ in range(total)], np.uint8).reshape(total, G)
        return k, v, tags, acts

    for call in range(60):
        u = rng.unit()
        if u < 0.08:                                                    # forget a sequence
            s = rng.below(B)
            P.pask_seq_reset(h, s)
            p.orc.seq_reset(s)
            planned = None
        elif u < 0.25:                                                  # a ragged append through the ordinary call
            n_seqs = 1 + rng.below(B)
            seqs = [int(x) for x in np.random.default_rng(seed * 1000 + call).permutation(B)[:n_seqs]]
            counts = [[1, rng.below(40), rng.below(300)][rng.below(3)] for _ in seqs]
            total = int(sum(counts))
            if total == 0:
                continue
            cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
            k, v, tags, acts = data(total)
            layer = rng.below(n_layers)
            rc, _ = p.orc.append(layer, seqs, cu, bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags, decided=acts)
            assert rc == 0
            P.pask_append_kv_decided(h, layer, torch.tensor(seqs, dtype=torch.int32, device=d), torch.from_numpy(cu).to(d),
                                     k.to(d), v.to(d), torch.from_numpy(tags).to(d), torch.from_numpy(acts).to(d), total_tokens=total)
            if planned:
                planned[1].discard(layer)
        else:                                                           # a planned-ahead step of one layer
            if planned is None or rng.unit() < 0.1:                     # a new batch (or the first one)
                n_seqs = 1 + rng.below(B)
                seqs = tuple(int(x) for x in np.random.default_rng(seed * 2000 + call).permutation(B)[:n_seqs])
                planned = (seqs, set())
            seqs = list(planned[0])
            n = len(seqs)
            ids = torch.tensor(seqs, dtype=torch.int32, device=d)
            layer = rng.below(n_layers)
            if layer not in planned[1]:
                P.pask_plan_ahead(h, layer, ids, area)
                planned[1].add(layer)
            k, v, tags, acts = data(n)
            q = normal_bf16(seed, 0, serial, 0, 0, n, 4 * n_kv)
            rc, used_o = p.orc.append(layer, seqs, list(range(n + 1)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags, decided=acts)
            assert rc == 0
            out = torch.full((n, 4 * n_kv, 128), float("nan"), dtype=torch.float32, device=d)
            lse = torch.full((n, 4 * n_kv), float("nan"), dtype=torch.float32, device=d)
            used_g = torch.full((n,), 0xEE, dtype=torch.uint8, device=d)
            P.pask_decode_step_ahead(h, layer, ids, k.to(d), v.to(d), torch.from_numpy(tags).to(d), q.to(d), out, lse, p.gpu.workspace(n),
                                     area, actions=torch.from_numpy(acts).to(d), actions_out=used_g)
            torch.cuda.synchronize()
            assert np.array_equal(used_g.cpu().numpy(), used_o)
            oo, ol = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
            assert_close(out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), oo, ol, where=(call, layer, seqs))
        torch.cuda.synchronize()
        assert P.pask_budget_state(h, 0).device_status == 0
        for s in range(B):
            for l in range(n_layers):
                assert P.pask_debug_stream_len(h, l, s) == p.orc.stream_len(l, s)
        assert P.pask_debug_pool_state(h) == p.orc.pool_state()
    p.compare_state()


@pytest.mark.parametrize("batch", [2, 12, 18, 19, 30, 37, 50])
def test_unequal_small_batches_through_both_attention_paths(pask, oracle, batch):
    # How the partials of a row are merged and how the cost line is cut depend on the batch: up to 18 sequences
    # every non-empty one gets whole CTAs of the streaming kernel; below 43 a row's partials are shared by 2, 4 or
    # 8 warps.  One long sequence, short ones of every page-boundary case and one that holds nothing, through
    # pask_decode_attention and through planned-ahead steps.
    p, w = _pair(pask, oracle, batch, 1500, 100)
    seqs = list(range(batch))
    lens = [w.total_len(0)] + [(7 * s * s + 1) % 97 for s in range(1, batch)]
    lens[-1] = 0                                     # named in every call, holds nothing until the first step
    some = [s for s in seqs if lens[s] > 0]
    for layer in range(w.cfg.n_layers):
        p.append(layer, some, [lens[s] for s in some], [0] * len(some))
        p.check_attention(layer, seqs, pos=1600)
        p.check_attention(layer, seqs[::-1][: max(1, batch // 2)], pos=1601)      # another batch size, another cut
    area = torch.empty(pask.pask_plan_area_bytes(p.gpu.handle, batch), dtype=torch.uint8, device="cuda")
    ids = torch.tensor(seqs, dtype=torch.int32, device="cuda")
    for layer in range(w.cfg.n_layers):
        pask.pask_plan_ahead(p.gpu.handle, layer, ids, area)
    pos = list(lens)
    for step in range(20):
        for layer in range(w.cfg.n_layers):
            _ahead_step(p, area, layer, seqs, pos)
        pos = [x + 1 for x in pos]
    p.compare_state()
    assert pask.pask_budget_state(p.gpu.handle, 0).device_status == 0
