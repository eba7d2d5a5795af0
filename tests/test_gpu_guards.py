"""Memory-safety and determinism checks on the GPU: caller-owned buffers are wrapped in canary
regions that must survive every kernel, the same calls on two caches must leave byte-identical
pools, page tables and outputs, and a stream may be filled exactly to its bound."""
import numpy as np
import pytest
import torch

from pask_workloads import configs as WC

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes of canary before and after each buffer
PATTERN = 0xA5


def _guarded(nbytes, device):
    """A zero-filled buffer of nbytes (256-byte aligned) inside a larger allocation painted with a canary."""
    total = GUARD + nbytes + GUARD
    raw = torch.full((total + 256,), PATTERN, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % 256
    whole = raw[off:off + total]
    whole[GUARD:GUARD + nbytes] = 0
    return raw, whole, whole[GUARD:GUARD + nbytes]


def _canaries_intact(whole, nbytes):
    return bool((whole[:GUARD] == PATTERN).all()) and bool((whole[GUARD + nbytes:] == PATTERN).all())


def _run(P, w, device):
    """Bulk append + three decode steps + attention on caller-created, canary-guarded buffers."""
    cfg = w.cfg
    lens = [w.total_len(b) for b in range(cfg.batch)]
    pages = cfg.n_layers * (sum(lens) // 16 + 4 * cfg.batch)
    desc = P.CacheDesc(cfg.n_layers, cfg.n_q, cfg.n_kv, 128, 16, cfg.batch, max(lens) + 16, sum(lens), pages, pages)
    sizes = P.pask_cache_sizes(desc)
    bufs = [_guarded(n, device) for n in (sizes.pool_high_bytes, sizes.pool_low_bytes, sizes.meta_bytes)]
    policy = P.pask_load_policy(w.blob)
    h = P.pask_cache_create(desc, policy, bufs[0][2], bufs[1][2], bufs[2][2])
    ws_raw, ws_whole, ws = _guarded(P.pask_workspace_bytes(h, cfg.batch), device)
    ids = torch.arange(cfg.batch, dtype=torch.int32, device=device)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=device)
    tags = torch.from_numpy(np.concatenate([w.tags(b, 0, lens[b]) for b in range(cfg.batch)])).to(device)
    outs = []
    for layer in range(cfg.n_layers):
        k = torch.cat([w.kv(layer, b, 0, lens[b])[0] for b in range(cfg.batch)]).to(device)
        v = torch.cat([w.kv(layer, b, 0, lens[b])[1] for b in range(cfg.batch)]).to(device)
        P.pask_append_kv(h, layer, ids, cu, k, v, tags)
    cu1 = torch.arange(cfg.batch + 1, dtype=torch.int32, device=device)
    for step in range(3):
        for layer in range(cfg.n_layers):
            k = torch.stack([w.kv(layer, b, lens[b] + step, 1)[0][0] for b in range(cfg.batch)]).to(device)
            v = torch.stack([w.kv(layer, b, lens[b] + step, 1)[1][0] for b in range(cfg.batch)]).to(device)
            t = torch.from_numpy(np.array([w.tags(b, lens[b] + step, 1)[0] for b in range(cfg.batch)], np.uint8)).to(device)
            q = torch.stack([w.q(layer, b, lens[b] + step + 1) for b in range(cfg.batch)]).to(device)
            out = torch.empty((cfg.batch, cfg.n_q, 128), dtype=torch.float32, device=device)
            lse = torch.empty((cfg.batch, cfg.n_q), dtype=torch.float32, device=device)
            P.pask_append_kv(h, layer, ids, cu1, k, v, t)
            P.pask_decode_attention(h, layer, ids, q, out, lse, ws)
            outs.append(out)
    torch.cuda.synchronize()
    assert P.pask_budget_state(h, 0).device_status == 0
    sizes_list = (sizes.pool_high_bytes, sizes.pool_low_bytes, sizes.meta_bytes)
    for (raw, whole, inner), n in zip(bufs, sizes_list):
        assert _canaries_intact(whole, n)
    assert _canaries_intact(ws_whole, ws.numel())
    # snapshot: pools, and the meta without the status/ticket control words' volatile parts
    snap = [bufs[0][2].clone(), bufs[1][2].clone(), bufs[2][2].clone(), torch.stack(outs).clone()]
    P.pask_cache_destroy(h)
    P.pask_free_policy(policy)
    return snap


def test_canaries_survive_and_runs_are_deterministic():
    import paper_2608_28276_b200 as P
    dev = torch.device("cuda", 0)
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=5, n_layers=2, n_groups=2, prompt_len=450, gen_len=390)
    w = WC.build(cfg)
    a = _run(P, w, dev)
    b = _run(P, w, dev)
    for x, y in zip(a, b):
        assert torch.equal(x, y)          # pools, meta (tables, counters, budgets) and outputs: byte for byte


def test_stream_filled_exactly_to_its_bound():
    import paper_2608_28276_b200 as P
    d = "cuda"
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=1, n_layers=1, n_groups=1, lut="all_high")
    w = WC.build(cfg)
    cache = P.Cache(w.blob, 1, cfg.n_q, cfg.n_kv, 1, 64, 64, 4, 4)      # streams of at most 64 tokens = 4 pages
    ids = torch.zeros(1, dtype=torch.int32, device=d)
    k, v = w.kv(0, 0, 0, 64)
    tags = torch.zeros(64, dtype=torch.uint8, device=d)
    P.pask_append_kv(cache.handle, 0, ids, torch.tensor([0, 63], dtype=torch.int32, device=d), k[:63].to(d), v[:63].to(d), tags[:63].contiguous())
    P.pask_append_kv(cache.handle, 0, ids, torch.tensor([0, 1], dtype=torch.int32, device=d), k[63:].to(d), v[63:].to(d), tags[:1].contiguous())
    assert P.pask_debug_stream_len(cache.handle, 0, 0) == (64, 0)
    assert P.pask_budget_state(cache.handle, 0).device_status == 0
    assert P.pask_debug_pool_state(cache.handle) == (4, 0, 0, 0)
    # full attention over exactly four full pages equals the library routine
    q = w.q(0, 0, 64)
    out = torch.empty((1, cfg.n_q, 128), dtype=torch.float32, device=d)
    P.pask_decode_attention(cache.handle, 0, ids, q.unsqueeze(0).to(d), out, None, cache.workspace(1))
    kk = k.double().repeat_interleave(4, dim=1).permute(1, 0, 2)
    vv = v.double().repeat_interleave(4, dim=1).permute(1, 0, 2)
    sc = torch.einsum("hd,hnd->hn", q.double(), kk) / 128 ** 0.5
    ref = torch.einsum("hn,hnd->hd", torch.softmax(sc, -1), vv)
    assert float((out[0].cpu().double() - ref).abs().max()) < 2e-3
    # one more token does not fit: refused, flagged, nothing changes
    P.pask_append_kv(cache.handle, 0, ids, torch.tensor([0, 1], dtype=torch.int32, device=d), k[:1].to(d), v[:1].to(d), tags[:1].contiguous())
    assert P.pask_budget_state(cache.handle, 0).device_status == P.DEV_SEQ_OVERFLOW
    assert P.pask_debug_stream_len(cache.handle, 0, 0) == (64, 0)
    cache.close()


def test_everything_on_a_side_stream_and_after_a_cache_reset(oracle):
    import paper_2608_28276_b200 as pask
    # every call on a non-default stream (nothing may lean on the legacy default stream), with busy
    # work queued in front so that a missing dependency would show; then the cache is reset, used
    # again with decided actions and a window, and still agrees with a fresh oracle
    from dataclasses import replace
    from pask_workloads import policy as WP
    from parity import Pair
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=2, n_groups=2, prompt_len=200, gen_len=100, extra_gen=32)
    w = WC.build(cfg)
    blob = WP.write_blob(replace(w.policy, recent_window=16))
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        p = Pair(pask, oracle, w, blob=blob)
        busy = torch.randn((4096, 4096), device="cuda")
        for rnd in range(2):
            for _ in range(6):
                busy = busy @ busy * 1e-4                               # keeps the stream occupied ahead of the library's work
            seqs = [1, 2, 0]
            for layer in range(2):
                p.append(layer, seqs, [250, 260, 270], [0, 0, 0])
            for step in range(3):
                for layer in range(2):
                    p.append(layer, seqs, [1, 1, 1], [250 + step, 260 + step, 270 + step])
            p.compare_state()
            for layer in range(2):
                p.check_attention(layer, [0, 1, 2], pos=273)
            if rnd == 0:                                                # wipe both sides and go again
                pask.pask_cache_reset(p.gpu.handle)
                p.orc = oracle.Cache(oracle.Policy(blob), cfg.n_q, cfg.n_kv, p.max_seqs, p.hp, p.lp)
                assert pask.pask_debug_pool_state(p.gpu.handle) == (0, 0, 0, 0)
                assert pask.pask_budget_state(p.gpu.handle, 1).full_bytes == 0
    torch.cuda.synchronize()


def test_page_ids_beyond_the_pools_are_refused_not_dereferenced(oracle):
    # The streaming kernel checks every page id of its plan against what the pools hold.  A plan whose page-order
    # list somebody has overwritten with ids far beyond the pools must not make the kernel read there: it reads
    # page 0 instead and sets PASK_DEV_INTERNAL (the results of that call are void).
    import paper_2608_28276_b200 as pask
    from parity import Pair
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=1, n_groups=1, prompt_len=200, gen_len=100, extra_gen=16)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [0, 1, 2]
    p.append(0, seqs, [300] * 3, [0] * 3)
    h, d = p.gpu.handle, "cuda"
    ids = torch.tensor(seqs, dtype=torch.int32, device=d)
    area = torch.zeros(pask.pask_plan_area_bytes(h, 3), dtype=torch.uint8, device=d)
    pask.pask_plan_ahead(h, 0, ids, area)
    torch.cuda.synchronize()
    off, nbytes = pask.pask_debug_plan_order_span(h, 3, 0, 0)
    order = area[off:off + nbytes].view(torch.int32)
    pages = sum((x + 15) // 16 for s in seqs for x in pask.pask_debug_stream_len(h, 0, s))
    assert int((order != 0).sum()) >= pages - 1                       # this is where the plan's page list lies
    order[:pages] |= 0x07FFFFFF                                          # every id becomes the largest one an entry can hold
    k, v = w.kv(0, 0, 300, 1)
    kk = torch.cat([w.kv(0, s, 300, 1)[0] for s in seqs]).to(d)
    vv = torch.cat([w.kv(0, s, 300, 1)[1] for s in seqs]).to(d)
    tags = torch.from_numpy(np.array([w.tags(s, 300, 1)[0] for s in seqs], np.uint8)).to(d)
    q = torch.stack([w.q(0, s, 301) for s in seqs]).to(d)
    out = torch.zeros((3, cfg.n_q, 128), dtype=torch.float32, device=d)
    lse = torch.zeros((3, cfg.n_q), dtype=torch.float32, device=d)
    pask.pask_decode_step_ahead(h, 0, ids, kk, vv, tags, q, out, lse, p.gpu.workspace(3), area)
    torch.cuda.synchronize()                                             # the call returns, nothing faulted
    assert pask.pask_budget_state(h, 0).device_status & pask.DEV_INTERNAL
    # the append of that call went through as usual (it does not depend on the plan it was given)
    assert pask.pask_debug_stream_len(h, 0, 0)[0] + pask.pask_debug_stream_len(h, 0, 0)[1] >= 1
