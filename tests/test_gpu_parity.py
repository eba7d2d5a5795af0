"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs. Integer / byte / index results must be identical; attention within
max-abs 2e-3 and relative L2 1e-3 of the fp64 oracle."""
import numpy as np
import pytest
import torch

from pask_workloads import configs as WC
from pask_workloads import policy as WP
from pask_workloads.tensors import normal_bf16

from parity import Pair, assert_close, error_stats

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pask():
    import paper_2608_28276_b200 as P      # fails loudly if libpask.so is missing
    assert torch.cuda.is_available()
    return P


def _explicit_policy(actions, n_layers=1, floors=None, budget=0.5):
    a = np.asarray(actions, np.uint8)
    fl = np.zeros_like(a) if floors is None else np.asarray(floors, np.uint8)
    z = np.zeros(a.shape, np.float32)
    lg = np.asarray([l % a.shape[1] for l in range(n_layers)], np.uint8)
    return WP.Policy(a.shape[0], a.shape[1], lg, a, fl, z, z.copy(), np.zeros(2, np.uint32), budget_target=budget)


def _workload(cfg, actions=None, n_layers=None, **kw):
    w = WC.build(cfg)
    if actions is not None:
        w.policy = _explicit_policy(actions, n_layers or cfg.n_layers, **kw)
    return w


def test_tiny_bulk_append_then_decode_step(pask, oracle):
    w = WC.build(WC.TINY)
    p = Pair(pask, oracle, w)
    n = w.total_len(0)
    _, act = p.append(0, [0], [n], [0])
    assert set(np.unique(act).tolist()) == {0, 1, 2}
    p.compare_state()
    p.check_attention(0, [0])
    # one decode step: the new token is appended, then attended (if retained)
    p.append(0, [0], [1], [n])
    p.compare_state()
    p.check_attention(0, [0], pos=n + 1)


def test_tiny_token_by_token_replay_gives_identical_pages(pask, oracle):
    w = WC.build(WC.TINY)
    bulk, step = Pair(pask, oracle, w), Pair(pask, oracle, w)
    n = w.total_len(0)
    bulk.append(0, [0], [n], [0])
    for t0 in range(0, n, 1):
        step.append(0, [0], [1], [t0])
    step.compare_state()
    P = pask
    for fn in (P.pask_debug_dump_high, P.pask_debug_dump_low):
        for x, y in zip(fn(bulk.gpu.handle, 0, 0, 2), fn(step.gpu.handle, 0, 0, 2)):
            assert np.array_equal(x, y)
    a = bulk.check_attention(0, [0])[0]
    b = step.check_attention(0, [0])[0]
    assert np.array_equal(a, b)            # same pages, same schedule: bit-identical outputs


def test_qwen3_one_layer_per_group_full_config(pask, oracle):
    w = WC.build(WC.QWEN3_4B_1LAYER)
    cfg = w.cfg
    p = Pair(pask, oracle, w)
    seqs = list(range(cfg.batch))
    lens = [w.total_len(b) for b in seqs]
    for layer in range(cfg.n_layers):
        # prompt as one ragged bulk call, generated tokens in uneven chunks (ragged tails)
        p.append(layer, seqs, [w.prompt_len(b) for b in seqs], [0] * cfg.batch)
        done = [w.prompt_len(b) for b in seqs]
        chunk = 0
        while any(d < l for d, l in zip(done, lens)):
            cnt = [min(l - d, 700 + 37 * chunk + 11 * b) for b, (d, l) in enumerate(zip(done, lens))]
            p.append(layer, seqs, cnt, done)
            done = [d + c for d, c in zip(done, cnt)]
            chunk += 1
    p.compare_state()
    worst = (0.0, 0.0)
    for layer in range(cfg.n_layers):
        go, oo = p.check_attention(layer, seqs)
        e = error_stats(go, oo)
        worst = (max(worst[0], e[0]), max(worst[1], e[1]))
    print("config-2 attention error: max-abs %.3e rel-L2 %.3e" % worst)
    # realised normalised KV cost is the configured budget (Eq. 1 from the budget states)
    ret = sum(pask.pask_budget_state(p.gpu.handle, b).retained_bytes for b in seqs)
    full = sum(pask.pask_budget_state(p.gpu.handle, b).full_bytes for b in seqs)
    assert abs(ret / full - cfg.budget) < 0.01
    # a decode step on top: one token per sequence, then attention
    for layer in range(cfg.n_layers):
        p.append(layer, seqs, [1] * cfg.batch, lens)
        p.check_attention(layer, seqs, pos=lens[0] + 1)
    p.compare_state(layers=[0, 3], seqs=[0, cfg.batch - 1])


def test_batch_subsets_orders_and_empty_sequences(pask, oracle):
    # sequences: 0 all dropped, 1 empty (never appended), 2 HIGH only with a ragged tail,
    # 3 LOW only with a ragged tail, 4 mixed, 5 one token
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=6, n_layers=1, n_groups=1)
    w = _workload(cfg, actions=[[0], [1], [2]])
    p = Pair(pask, oracle, w, pool_high_pages=64, pool_low_pages=64, max_tokens_per_seq=512, max_append_tokens=2048)
    rng = np.random.default_rng(2)
    plan = {0: np.zeros(40, np.uint8), 2: np.full(131, 2, np.uint8), 3: np.full(77, 1, np.uint8),
            4: rng.integers(0, 3, 300).astype(np.uint8), 5: np.array([1], np.uint8)}
    seqs = sorted(plan)
    ks = [normal_bf16(5, 1, 0, s, 0, len(plan[s]), 8) for s in seqs]
    vs = [normal_bf16(5, 2, 0, s, 0, len(plan[s]), 8) for s in seqs]
    p.append(0, seqs, [len(plan[s]) for s in seqs], None, k=torch.cat(ks), v=torch.cat(vs),
             tags=np.concatenate([plan[s] for s in seqs]))
    p.compare_state()
    q = normal_bf16(5, 0, 0, 0, 0, 6, 32)
    base = p.attention(0, [0, 1, 2, 3, 4, 5], q=q)
    assert_close(*base)
    assert np.all(base[0][0] == 0) and np.all(np.isneginf(base[1][0]))       # everything dropped
    assert np.all(base[0][1] == 0) and np.all(np.isneginf(base[1][1]))       # never appended
    # a permuted subset gives the same rows
    order = [4, 1, 5, 2]
    sub = p.attention(0, order, q=q[order])
    assert_close(*sub)
    for i, s in enumerate(order):
        assert np.abs(sub[0][i] - base[0][s]).max() < 1e-5
    # single-sequence calls
    for s in (2, 3, 5):
        assert_close(*p.attention(0, [s], q=q[[s]]))


def test_split_count_does_not_change_the_result(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=1, n_groups=1, prompt_len=600, gen_len=500)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [0, 1, 2]
    p.append(0, seqs, [w.total_len(b) for b in seqs], [0, 0, 0])
    ref = None
    for n_ctas in (1, 2, 3, 17, 148, 296, 1000):
        pask.pask_debug_set_attention_ctas(p.gpu.handle, n_ctas)
        go, gl, oo, ol = p.attention(0, seqs)
        assert_close(go, gl, oo, ol, where=n_ctas)
        ref = go if ref is None else ref
        # the split changes the running maxima and with them the fp16 rounding of P * scale
        assert np.abs(go - ref).max() < 3e-4


def test_all_high_policy_and_full_kv_kernel(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=2, n_layers=2, n_groups=2, prompt_len=300, gen_len=211, lut="all_high")
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    for layer in range(2):
        p.append(layer, [0, 1], [511, 511], [0, 0])
    p.compare_state()
    for b in (0, 1):
        st = pask.pask_budget_state(p.gpu.handle, b)
        assert st.retained_bytes == st.full_bytes == 2 * 511 * 4096 and st.remaining_bytes == 0
    for layer in range(2):
        a = p.attention(0 + layer, [0, 1])
        f = p.attention(0 + layer, [1, 0], full=True)
        assert_close(*a)
        assert_close(*f)
        # the reference policy equals plain full attention on the raw inputs (library routine)
        for i, b in enumerate((0, 1)):
            k, v = w.kv(layer, b, 0, 511)
            qq = w.q(layer, b, 511).double()
            kk = k.double().repeat_interleave(4, dim=1).permute(1, 0, 2)
            vv = v.double().repeat_interleave(4, dim=1).permute(1, 0, 2)
            sc = torch.einsum("hd,hnd->hn", qq, kk) / 128 ** 0.5
            ref = torch.einsum("hn,hnd->hd", torch.softmax(sc, -1), vv).numpy()
            assert np.abs(a[0][i] - ref).max() < 2e-3
            assert np.abs(f[0][1 - i] - ref).max() < 2e-3


def test_low_only_and_extreme_magnitudes(pask, oracle):
    # all tokens at low precision, with K/V scaled far away from unit variance
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=2, n_layers=1, n_groups=1)
    w = _workload(cfg, actions=[[1]])
    p = Pair(pask, oracle, w, pool_high_pages=8, pool_low_pages=128, max_tokens_per_seq=1024, max_append_tokens=4096)
    n = 517
    for scale_k, scale_v, seq in ((1.0, 1e-3, 0), (0.05, 300.0, 1)):
        k = (normal_bf16(9, 1, 0, seq, 0, n, 8).float() * scale_k).to(torch.bfloat16)
        v = (normal_bf16(9, 2, 0, seq, 0, n, 8).float() * scale_v).to(torch.bfloat16)
        k[5] = 0                                      # an all-zero token: scale 0, codes 8
        p.append(0, [seq], [n], None, k=k, v=v, tags=np.zeros(n, np.uint8))
    p.compare_state()
    q = normal_bf16(9, 0, 0, 0, 0, 2, 32)
    go, gl, oo, ol = p.attention(0, [0, 1], q=q)
    # tolerances are absolute for unit-scale outputs: compare after normalising each row's scale
    for i, sv in enumerate((1e-3, 300.0)):
        assert_close(go[i:i + 1] / sv, gl[i:i + 1], oo[i:i + 1] / sv, ol[i:i + 1], where=("scaled", i))


def test_subnormal_and_saturated_scales_through_both_append_paths(pask, oracle):
    # groups whose fp16 scale is subnormal (coarsely rounded: the clamp of the codes bites) or saturates at 65504,
    # next to ordinary ones, through the bulk path (full pages) and the one-launch path; stored bytes bit for bit
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=2, n_layers=1, n_groups=1)
    w = _workload(cfg, actions=[[1]])
    p = Pair(pask, oracle, w, pool_high_pages=8, pool_low_pages=128, max_tokens_per_seq=1024, max_append_tokens=4096)
    n = 200
    for seq, scales in ((0, (3e-6, 1e-7, 1.0)), (1, (4e5, 3e6, 1.0))):
        k = normal_bf16(19, 1, 0, seq, 0, n, 8).float()
        v = normal_bf16(19, 2, 0, seq, 0, n, 8).float()
        for i, sc in enumerate(scales):                # every third token at each magnitude, heads alternate too
            k[i::3] *= sc
            v[i::3, ::2] *= sc
        k, v = k.to(torch.bfloat16), v.to(torch.bfloat16)
        tags = np.zeros(n, np.uint8)
        p.append(0, [seq], [n - 7], None, k=k[:n - 7], v=v[:n - 7], tags=tags[:n - 7])
        for t in range(n - 7, n):
            p.append(0, [seq], [1], None, k=k[t:t + 1], v=v[t:t + 1], tags=tags[t:t + 1])
    p.compare_state()
    kc, ks, _, _, _ = pask.pask_debug_dump_low(p.gpu.handle, 0, 0, 8)
    sub = (ks > 0) & (ks < 0x0400)
    assert sub.any() and (ks == 0).any()                # subnormal scales and scales that underflowed to zero
    _, ks1, _, _, _ = pask.pask_debug_dump_low(p.gpu.handle, 0, 1, 8)
    assert (ks1 == 0x7BFF).any()                        # saturated scales


def test_device_side_refusals_leave_the_cache_untouched(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=1, n_groups=1)
    w = _workload(cfg, actions=[[1], [2]])
    p = Pair(pask, oracle, w, pool_high_pages=3, pool_low_pages=2, max_tokens_per_seq=64, max_append_tokens=256)
    P, h, d = pask, p.gpu.handle, "cuda"
    k, v = normal_bf16(3, 1, 0, 0, 0, 64, 8), normal_bf16(3, 2, 0, 0, 0, 64, 8)
    p.append(0, [0], [40], None, k=k[:40], v=v[:40], tags=np.ones(40, np.uint8))       # 3 HIGH pages: pool empty
    p.compare_state()
    # needs one more HIGH page than the pool has: refused as a whole, LOW part included
    rc, _ = p.append(0, [1], [20], None, expect_ok=False, k=k[:20], v=v[:20],
                     tags=np.array([0] * 10 + [1] * 10, np.uint8))
    assert rc == oracle.ERR_POOL
    p.compare_budget(1, expect_status=P.DEV_POOL_EXHAUSTED)
    assert P.pask_debug_stream_len(h, 0, 1) == (0, 0)
    assert P.pask_debug_pool_state(h) == p.orc.pool_state()
    # repeated sequence id, id out of range, bad ragged offsets: refused, flagged, nothing changes
    ids = torch.tensor([1, 1], dtype=torch.int32, device=d)
    cu = torch.tensor([0, 1, 2], dtype=torch.int32, device=d)
    tg = torch.zeros(2, dtype=torch.uint8, device=d)
    P.pask_append_kv(h, 0, ids, cu, k[:2].to(d), v[:2].to(d), tg)
    assert P.pask_budget_state(h, 1).device_status & P.DEV_BAD_SEQ
    P.pask_cache_reset(h)
    p.orc.seq_reset(0)
    ids = torch.tensor([7], dtype=torch.int32, device=d)
    P.pask_append_kv(h, 0, ids, cu[:2].contiguous(), k[:1].to(d), v[:1].to(d), tg[:1].contiguous())
    assert P.pask_budget_state(h, 0).device_status == P.DEV_BAD_SEQ
    P.pask_cache_reset(h)
    ids = torch.tensor([0, 1], dtype=torch.int32, device=d)
    bad_cu = torch.tensor([0, 2, 1], dtype=torch.int32, device=d)
    P.pask_append_kv(h, 0, ids, bad_cu, k[:2].to(d), v[:2].to(d), tg)
    assert P.pask_budget_state(h, 0).device_status & P.DEV_BAD_RAGGED
    assert P.pask_debug_stream_len(h, 0, 0) == (0, 0) and P.pask_debug_pool_state(h) == (0, 0, 0, 0)
    P.pask_cache_reset(h)
    # a stream that would outgrow max_tokens_per_seq (64 tokens = 4 pages) is refused
    tags65 = torch.zeros(65, dtype=torch.uint8, device=d)
    kk = normal_bf16(3, 1, 0, 1, 0, 65, 8).to(d)
    P.pask_append_kv(h, 0, torch.tensor([2], dtype=torch.int32, device=d),
                     torch.tensor([0, 65], dtype=torch.int32, device=d), kk, kk, tags65)
    assert P.pask_budget_state(h, 2).device_status == P.DEV_SEQ_OVERFLOW
    assert P.pask_debug_stream_len(h, 0, 2) == (0, 0)
    # host-visible argument errors return at once
    with pytest.raises(P.PaskError) as e:
        P.pask_append_kv(h, 5, ids, cu, k[:2].to(d), v[:2].to(d), tg)
    assert e.value.status == P.ERR_INVALID_ARG
    with pytest.raises(P.PaskError) as e:
        P.pask_append_kv(h, 0, ids, cu, k[:2].to(d), v[:2].to(d), tg, total_tokens=10 ** 6)
    assert e.value.status == P.ERR_INVALID_ARG
    small = torch.empty(256, dtype=torch.uint8, device=d)
    out = torch.empty((2, 32, 128), dtype=torch.float32, device=d)
    with pytest.raises(P.PaskError) as e:
        P.pask_decode_attention(h, 0, ids, torch.zeros((2, 32, 128), dtype=torch.bfloat16, device=d), out, None, small)
    assert e.value.status == P.ERR_WORKSPACE


def test_unknown_and_protected_tags_and_floors(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=1, n_layers=2, n_groups=2)
    w = _workload(cfg, actions=[[0, 1], [1, 0], [2, 2]], floors=[[0, 2], [0, 0], [0, 0]])
    p = Pair(pask, oracle, w, pool_high_pages=16, pool_low_pages=16, max_tokens_per_seq=256, max_append_tokens=256)
    tags = np.array([0, 1, 2, 0xFF, 3, 200, 0, 1] * 9, np.uint8)
    k, v = normal_bf16(4, 1, 0, 0, 0, len(tags), 8), normal_bf16(4, 2, 0, 0, 0, len(tags), 8)
    _, a0 = p.append(0, [0], [len(tags)], None, k=k, v=v, tags=tags)
    _, a1 = p.append(1, [0], [len(tags)], None, k=k, v=v, tags=tags)
    assert a0[:8].tolist() == [0, 1, 2, 2, 2, 2, 0, 1] and a1[:8].tolist() == [2, 0, 2, 2, 2, 2, 2, 0]
    p.compare_state()
    assert pask.pask_budget_state(p.gpu.handle, 0).bad_tags == 2 * 2 * 9
    p.check_attention(0, [0], pos=0)
    p.check_attention(1, [0], pos=0)


def test_sequence_reset_returns_pages_lifo(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=2, n_groups=2, prompt_len=100, gen_len=60)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w, pool_high_pages=40, pool_low_pages=40)
    for layer in range(2):
        p.append(layer, [0, 1, 2], [160, 160, 160], [0, 0, 0])
    p.compare_state()
    pask.pask_seq_reset(p.gpu.handle, 1)
    p.orc.seq_reset(1)
    p.compare_state()
    # sequence 1 starts over and reuses the returned pages in reverse order
    for layer in range(2):
        p.append(layer, [1], [90], [0])
    p.compare_state()
    p.check_attention(0, [0, 1, 2], pos=500)
    p.check_attention(1, [2, 1], pos=500)


def test_decode_step_from_host_buffers(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=4, n_layers=1, n_groups=1, prompt_len=200, gen_len=100)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [0, 1, 2, 3]
    p.append(0, seqs, [300] * 4, [0] * 4)
    P, h = pask, p.gpu.handle
    k = torch.stack([w.kv(0, b, 300, 1)[0][0] for b in seqs]).pin_memory()
    v = torch.stack([w.kv(0, b, 300, 1)[1][0] for b in seqs]).pin_memory()
    tags = torch.from_numpy(np.array([w.tags(b, 300, 1)[0] for b in seqs], np.uint8)).pin_memory()
    q = torch.stack([w.q(0, b, 301) for b in seqs]).pin_memory()
    ids = torch.tensor(seqs, dtype=torch.int32).pin_memory()
    out = torch.empty((4, 32, 128), dtype=torch.float32).pin_memory()
    staging = torch.empty(P.pask_step_staging_bytes(h, 4), dtype=torch.uint8, device="cuda")
    P.pask_decode_step_host(h, 0, ids, k, v, tags, q, out, staging, p.gpu.workspace(4))
    torch.cuda.synchronize()
    from pask_workloads.tensors import bf16_bits
    rc, _ = p.orc.append(0, seqs, [0, 1, 2, 3, 4], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags.numpy())
    assert rc == 0
    oo, ol = p.orc.attention_batch(0, seqs, bf16_bits(q).numpy())
    go = out.numpy().astype(np.float64)
    assert_close(go, ol.copy(), oo, ol)
    p.compare_state()


def test_decode_step_from_one_packed_host_block(pask, oracle):
    # the same step with all inputs in one pinned block (one host-to-device copy)
    from pask_workloads.tensors import bf16_bits
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=4, n_layers=1, n_groups=1, prompt_len=200, gen_len=100)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [2, 0, 3, 1]
    p.append(0, seqs, [300] * 4, [0] * 4)
    P, h = pask, p.gpu.handle
    k = torch.stack([w.kv(0, b, 300, 1)[0][0] for b in seqs])
    v = torch.stack([w.kv(0, b, 300, 1)[1][0] for b in seqs])
    tags = torch.from_numpy(np.array([w.tags(b, 300, 1)[0] for b in seqs], np.uint8))
    q = torch.stack([w.q(0, b, 301) for b in seqs])
    off, n_in = P.pask_step_packed_layout(h, 4)
    block = torch.zeros(n_in, dtype=torch.uint8).pin_memory()
    parts = [torch.tensor(seqs, dtype=torch.int32), torch.arange(5, dtype=torch.int32), k, v, tags, q]
    for o, t in zip(off, parts):
        raw = t.contiguous().view(torch.uint8).reshape(-1)
        block[o:o + raw.numel()] = raw
    out = torch.empty((4, 32, 128), dtype=torch.float32).pin_memory()
    staging = torch.empty(P.pask_step_staging_bytes(h, 4), dtype=torch.uint8, device="cuda")
    P.pask_decode_step_packed(h, 0, 4, block, out, staging, p.gpu.workspace(4))
    torch.cuda.synchronize()
    rc, _ = p.orc.append(0, seqs, [0, 1, 2, 3, 4], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags.numpy())
    assert rc == 0
    oo, ol = p.orc.attention_batch(0, seqs, bf16_bits(q).numpy())
    assert_close(out.numpy().astype(np.float64), ol.copy(), oo, ol)
    p.compare_state()


def test_pipelined_host_steps(pask, oracle):
    # layer after layer from host blocks with the copies on the cache's own streams: every output is
    # that of the oracle, whatever overlapped with whatever
    from pask_workloads.tensors import bf16_bits
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=5, n_layers=3, n_groups=3, prompt_len=150, gen_len=60, extra_gen=32)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [3, 0, 4, 1, 2]
    for layer in range(3):
        p.append(layer, seqs, [210] * 5, [0] * 5)
    P, h = pask, p.gpu.handle
    off, n_in = P.pask_step_packed_layout(h, 5)
    staging = torch.empty(2 * P.pask_step_staging_bytes(h, 5), dtype=torch.uint8, device="cuda")
    calls = []
    for step in range(6):
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
            P.pask_decode_step_pipelined(h, layer, 5, block, out, staging, p.gpu.workspace(5))
            rc, _ = p.orc.append(layer, seqs, list(range(6)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags.numpy())
            assert rc == 0
            oo, ol = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
            calls.append((block, out, oo, ol))
    P.pask_decode_step_drain(h)
    torch.cuda.synchronize()
    for block, out, oo, ol in calls:
        assert_close(out.numpy().astype(np.float64), ol.copy(), oo, ol)
    p.compare_state()


def test_pipelined_host_steps_with_a_batch_that_changes_from_call_to_call(pask, oracle):
    # consecutive pipelined calls with different n_seqs: the two staging slots are the buffer's fixed halves, so a
    # call's slot never reaches into the slot the call before is still reading; outputs are the oracle's throughout
    from pask_workloads.tensors import bf16_bits
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=6, n_layers=2, n_groups=2, prompt_len=120, gen_len=60, extra_gen=64)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    everyone = [3, 0, 4, 1, 2, 5]
    for layer in range(2):
        p.append(layer, everyone, [180] * 6, [0] * 6)
    P, h = pask, p.gpu.handle
    staging = torch.empty(2 * P.pask_step_staging_bytes(h, 6), dtype=torch.uint8, device="cuda")
    pos = {s: 180 for s in everyone}
    calls = []
    for step, seqs in enumerate(([3, 0, 4, 1, 2, 5], [5], [0, 1, 2, 3], [4, 2], [1, 5, 0, 3, 2, 4], [2], [0, 5, 1])):
        n = len(seqs)
        off, n_in = P.pask_step_packed_layout(h, n)
        for layer in range(2):
            k = torch.stack([w.kv(layer, b, pos[b], 1)[0][0] for b in seqs])
            v = torch.stack([w.kv(layer, b, pos[b], 1)[1][0] for b in seqs])
            tags = torch.from_numpy(np.array([w.tags(b, pos[b], 1)[0] for b in seqs], np.uint8))
            q = torch.stack([w.q(layer, b, pos[b] + 1) for b in seqs])
            block = torch.zeros(n_in, dtype=torch.uint8).pin_memory()
            for o, t in zip(off, [torch.tensor(seqs, dtype=torch.int32), torch.arange(n + 1, dtype=torch.int32), k, v, tags, q]):
                raw = t.contiguous().view(torch.uint8).reshape(-1)
                block[o:o + raw.numel()] = raw
            out = torch.full((n, 32, 128), float("nan"), dtype=torch.float32).pin_memory()
            P.pask_decode_step_pipelined(h, layer, n, block, out, staging, p.gpu.workspace(n))
            rc, _ = p.orc.append(layer, seqs, list(range(n + 1)), bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags.numpy())
            assert rc == 0
            oo, ol = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
            calls.append((block, out, oo, ol))
        for b in seqs:
            pos[b] += 1
    P.pask_decode_step_drain(h)
    torch.cuda.synchronize()
    for block, out, oo, ol in calls:
        assert_close(out.numpy().astype(np.float64), ol.copy(), oo, ol)
    p.compare_state()
    # halves too small for the batch are refused
    small = torch.empty(2 * P.pask_step_staging_bytes(h, 6) - 512, dtype=torch.uint8, device="cuda")
    with pytest.raises(P.PaskError) as e:
        P.pask_decode_step_pipelined(h, 0, 6, calls[0][0], calls[0][1], small, p.gpu.workspace(6))
    assert e.value.status == P.ERR_WORKSPACE


def test_the_streaming_kernel_times_itself_on_request(pask, oracle):
    # pask_cache_set_timing_span: the next streaming kernel leaves its earliest start and latest end (GPU global timer);
    # one launch only, results unaffected
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=1, n_groups=1, prompt_len=300, gen_len=100)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [0, 1, 2]
    p.append(0, seqs, [400] * 3, [0] * 3)
    span = torch.tensor([-1, 0], dtype=torch.int64, device="cuda")
    pask.pask_cache_set_timing_span(p.gpu.handle, span)
    p.check_attention(0, seqs)
    a, b = span.tolist()
    assert 0 < a < b and b - a < 10_000_000            # a few microseconds, in nanoseconds
    p.check_attention(0, seqs)                          # the request was for one launch
    assert span.tolist() == [a, b]
