"""pask_append_attend (append + attention of one layer in one call; for small batches the append's
launch also writes the attention plan) against the oracle and against the two separate calls."""
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
    import paper_2608_28276_b200 as P      # fails loudly if libpask.so is missing
    assert torch.cuda.is_available()
    return P


def _step(p, layer, seqs, counts, starts, acts=None):
    """One fused call on the GPU side, the two steps on the oracle side; returns both outputs.
    acts: (oracle actions, gpu actions) from Pair.decide for these tokens, or None (table actions)."""
    d = "cuda"
    tags, states, k, v = p.gather(seqs, counts, starts, layer)
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    act_o, act_g = acts if acts else (None, None)
    rc, used_o = p.orc.append(layer, seqs, cu, bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags, decided=act_o)
    assert rc == 0
    q = torch.stack([p.w.q(layer, int(s), int(t0 + n)) for s, n, t0 in zip(seqs, counts, starts)])
    n = len(seqs)
    out = torch.full((n, p.cfg.n_q, 128), float("nan"), dtype=torch.float32, device=d)
    lse = torch.full((n, p.cfg.n_q), float("nan"), dtype=torch.float32, device=d)
    used_g = torch.full((max(1, len(tags)),), 0xEE, dtype=torch.uint8, device=d)
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    p.pask.pask_append_attend(p.gpu.handle, layer, ids, torch.from_numpy(cu).to(d), k.to(d), v.to(d),
                              torch.from_numpy(tags).to(d), q.to(d), out, lse, p.gpu.workspace(n), actions=act_g,
                              actions_out=used_g, total_tokens=len(tags))
    torch.cuda.synchronize()
    assert np.array_equal(used_g.cpu().numpy()[:len(tags)], used_o)
    oo, ol = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
    go, gl = out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    assert_close(go, gl, oo, ol, where=(layer, seqs))
    return out, lse, (ids, torch.from_numpy(cu).to(d), k.to(d), v.to(d), torch.from_numpy(tags).to(d), q.to(d), act_g)


def _pair(pask, oracle, batch, prompt, gen, window=0, dynamic=False, **kw):
    from dataclasses import replace
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=batch, prompt_len=prompt, gen_len=gen, extra_gen=64)
    w = WC.build(cfg)
    blob = w.dynamic_blob(reserve_tokens=4, budget=0.3) if dynamic else WP.write_blob(replace(w.policy, recent_window=window))
    if dynamic and window:
        blob = blob[:28] + int(window).to_bytes(4, "little") + blob[32:]
    return Pair(pask, oracle, w, blob=blob, **kw), w


@pytest.mark.parametrize("batch,window,dynamic", [(5, 0, False), (64, 0, False), (7, 0, True), (5, 32, False), (130, 0, False), (255, 0, False), (256, 0, False),
                                                  (64, 64, False), (5, 256, False), (7, 16, True), (200, 48, False)])
def test_decode_steps(pask, oracle, batch, window, dynamic):
    prompt, gen = (40, 24) if batch > 8 else (150, 70)
    p, w = _pair(pask, oracle, batch, prompt, gen, window=window, dynamic=dynamic)
    seqs = list(range(batch))
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
    pos = list(lens)
    ones = [1] * batch
    for step in range(20):                                              # pages fill up and new ones are allocated on the way
        order = seqs if step % 2 == 0 else seqs[::-1]
        starts = [pos[s] for s in order]
        acts = None
        if dynamic:                                                     # Algorithm 2 steps 1-6 once per token, then every layer
            tags, states = p.gather(order, ones, starts)
            _, act_o, act_g = p.decide(order, ones, tags, states)
            acts = (act_o, act_g)
        for layer in range(w.cfg.n_layers):
            _step(p, layer, order, ones, starts, acts)
        pos = [x + 1 for x in pos]
    p.compare_state()


@pytest.mark.parametrize("window", [0, 16, 48, 256])
def test_ragged_small_batches_and_identity_with_separate_calls(pask, oracle, window):
    # with a recent window the one launch also counts the window's members: a ring that is not yet full,
    # bursts longer than the window, and sequences that get nothing in a call
    p, w = _pair(pask, oracle, 4, 100, 60, window=window)
    q2, _ = _pair(pask, oracle, 4, 100, 60, window=window)              # second cache: the two separate calls
    seqs = [3, 1, 0, 2]
    pos = {s: 0 for s in seqs}
    for counts in ([1, 1, 1, 1], [16, 3, 0, 31], [40, 40, 40, 8], [1, 0, 0, 2], [33, 17, 16, 15]):
        starts = [pos[s] for s in seqs]
        for layer in range(w.cfg.n_layers):
            out, lse, (ids, cu, k, v, tags, q, _) = _step(p, layer, seqs, counts, starts)
            pask.pask_append_kv(q2.gpu.handle, layer, ids, cu, k, v, tags, total_tokens=int(cu[-1]))
            out2, lse2 = torch.empty_like(out), torch.empty_like(lse)
            pask.pask_decode_attention(q2.gpu.handle, layer, ids, q, out2, lse2, q2.gpu.workspace(4))
            torch.cuda.synchronize()
            assert torch.equal(out, out2) and torch.equal(lse, lse2)    # same plan, same kernels: same bits
        pos = {s: pos[s] + n for s, n in zip(seqs, counts)}
    p.compare_state()


def test_refused_append_inside_the_fused_call(pask, oracle):
    p, w = _pair(pask, oracle, 2, 40, 20, pool_high_pages=1, pool_low_pages=1)
    d = "cuda"
    ids = torch.tensor([0, 1], dtype=torch.int32, device=d)
    n = 100                                                             # needs more pages than either pool has
    tags, states, k, v = p.gather([0, 1], [n, 20], [0, 0], 0)
    cu = torch.tensor([0, n, n + 20], dtype=torch.int32, device=d)
    q = torch.stack([w.q(0, s, 0) for s in (0, 1)]).to(d)
    out = torch.zeros((2, w.cfg.n_q, 128), device=d)
    lse = torch.zeros((2, w.cfg.n_q), device=d)
    pask.pask_append_attend(p.gpu.handle, 0, ids, cu, k.to(d), v.to(d), torch.from_numpy(tags).to(d), q, out, lse,
                            p.gpu.workspace(2), total_tokens=n + 20)
    torch.cuda.synchronize()
    st = pask.pask_budget_state(p.gpu.handle, 0)
    assert st.device_status & pask.DEV_POOL_EXHAUSTED and st.full_bytes == 0
    assert pask.pask_debug_stream_len(p.gpu.handle, 0, 0) == (0, 0)
    assert pask.pask_debug_pool_state(p.gpu.handle) == (0, 0, 0, 0)


def test_a_step_replayed_as_a_cuda_graph(pask, oracle):
    # the calls of a step only enqueue work, so a stream capture can record them; replaying the
    # graph must leave the same state and outputs as issuing the calls
    from pask_workloads.tensors import bf16_bits
    p, w = _pair(pask, oracle, 6, 120, 60, dynamic=True)
    seqs = list(range(6))
    lens = [w.total_len(s) for s in seqs]
    tags, states = p.gather(seqs, lens, [0] * 6)
    _, act_o, act_g = p.decide(seqs, lens, tags, states)
    for layer in range(w.cfg.n_layers):
        _, _, k, v = p.gather(seqs, lens, [0] * 6, layer)
        p.append_decided(layer, seqs, lens, k, v, tags, act_o, act_g)
    d = "cuda"
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    cu = torch.arange(7, dtype=torch.int32, device=d)
    G, L = w.cfg.n_groups, w.cfg.n_layers
    # static buffers the graph reads from and writes to
    tg = torch.zeros(6, dtype=torch.uint8, device=d)
    st = torch.zeros(6, dtype=torch.int16, device=d)
    act = torch.zeros((6, G), dtype=torch.uint8, device=d)
    ks = [torch.zeros((6, w.cfg.n_kv, 128), dtype=torch.bfloat16, device=d) for _ in range(L)]
    vs = [torch.zeros_like(ks[0]) for _ in range(L)]
    qs = [torch.zeros((6, w.cfg.n_q, 128), dtype=torch.bfloat16, device=d) for _ in range(L)]
    outs = [torch.zeros((6, w.cfg.n_q, 128), dtype=torch.float32, device=d) for _ in range(L)]
    lse = torch.zeros((6, w.cfg.n_q), dtype=torch.float32, device=d)
    ws = p.gpu.workspace(6)
    # warm the kernels up outside the capture on a throw-away cache (captures must not see first-use set-up)
    warm, _ = _pair(pask, oracle, 6, 120, 60, dynamic=True)
    pask.pask_decide(warm.gpu.handle, ids, cu, tg, st, act)
    pask.pask_append_attend(warm.gpu.handle, 0, ids, cu, ks[0], vs[0], tg, qs[0], outs[0], lse, warm.gpu.workspace(6), actions=act)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            pask.pask_decide(p.gpu.handle, ids, cu, tg, st, act)
            for layer in range(L):
                pask.pask_append_attend(p.gpu.handle, layer, ids, cu, ks[layer], vs[layer], tg, qs[layer], outs[layer], lse, ws,
                                        actions=act)
    torch.cuda.current_stream().wait_stream(side)
    pos = list(lens)
    for step in range(5):                                               # the same graph, new inputs each time
        tags, states = p.gather(seqs, [1] * 6, pos)
        tg.copy_(torch.from_numpy(tags)); st.copy_(torch.from_numpy(states.astype(np.int16)))
        rc, a_o = p.orc.decide(seqs, list(range(7)), tags, states=states, n_groups=G)
        assert rc == 0
        want = []
        for layer in range(L):
            _, _, k, v = p.gather(seqs, [1] * 6, pos, layer)
            q = torch.stack([w.q(layer, s, pos[s] + 1) for s in seqs])
            ks[layer].copy_(k); vs[layer].copy_(v); qs[layer].copy_(q)
            rc, _ = p.orc.append(layer, seqs, list(range(7)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags, decided=a_o)
            assert rc == 0
            want.append(p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy()))
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(act.cpu().numpy(), a_o)
        for layer in range(L):
            go = outs[layer].cpu().numpy().astype(np.float64)
            assert_close(go, want[layer][1].copy(), want[layer][0], want[layer][1], where=(step, layer))
        pos = [x + 1 for x in pos]
    p.compare_state()


def test_bulk_append_replayed_as_a_cuda_graph(pask, oracle):
    # the two-kernel bulk path recorded once and replayed on new data: the duplicate check and the
    # page numbering must behave as if the call had been issued each time
    from pask_workloads.tensors import bf16_bits
    p, w = _pair(pask, oracle, 3, 700, 100)
    d = "cuda"
    seqs = [2, 0, 1]
    counts = [200, 170, 150]
    total = sum(counts)
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(counts)]), dtype=torch.int32, device=d)
    k = torch.zeros((total, w.cfg.n_kv, 128), dtype=torch.bfloat16, device=d)
    v = torch.zeros_like(k)
    tg = torch.zeros(total, dtype=torch.uint8, device=d)
    used = torch.zeros(total, dtype=torch.uint8, device=d)
    warm, _ = _pair(pask, oracle, 3, 700, 100)
    pask.pask_append_kv(warm.gpu.handle, 0, ids, cu, k, v, tg, actions_out=used, total_tokens=total)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            pask.pask_append_kv(p.gpu.handle, 0, ids, cu, k, v, tg, actions_out=used, total_tokens=total)
    torch.cuda.current_stream().wait_stream(side)
    start = {s: 0 for s in seqs}
    for rep in range(3):
        tags, _, kk, vv = p.gather(seqs, counts, [start[s] for s in seqs], 0)
        k.copy_(kk); v.copy_(vv); tg.copy_(torch.from_numpy(tags))
        rc, act_o = p.orc.append(0, seqs, cu.cpu().numpy(), bf16_bits(kk).numpy(), bf16_bits(vv).numpy(), tags)
        assert rc == 0
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(used.cpu().numpy(), act_o)
        start = {s: start[s] + n for s, n in zip(seqs, counts)}
        p.compare_state(layers=[0])
    p.check_attention(0, [0, 1, 2], pos=600)


def test_fused_step_with_nothing_retained(pask, oracle):
    # every token released: the plan is empty, outputs are zero and lse is -inf, through the one-call form too
    a = np.zeros((11, 4), np.uint8)
    z = np.zeros((11, 4), np.float32)
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, prompt_len=40, gen_len=20, extra_gen=16)
    w = WC.build(cfg)
    pol = WP.Policy(11, 4, WP.equal_layer_groups(4, 4), a, a.copy(), z, z.copy(), np.zeros(1, np.uint32), budget_target=0.0)
    p = Pair(pask, oracle, w, blob=WP.write_blob(pol))
    for step in range(3):
        for layer in range(4):
            out, lse, _ = _step(p, layer, [2, 0, 1], [1, 1, 1], [step] * 3)
            assert torch.all(out == 0) and torch.all(torch.isinf(lse) & (lse < 0))
    assert pask.pask_debug_pool_state(p.gpu.handle) == (0, 0, 0, 0)
    p.compare_state()
