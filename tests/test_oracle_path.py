"""Pins for the oracle's append / paging / budget / attention path (CPU only).

Attention is pinned to a library routine (torch CPU fp64 softmax and matmul) on inputs prepared
independently of the oracle's own attention code, to closed forms, and to brute force on tiny
inputs; paging and budget to recounts and closed forms.
"""
import numpy as np
import pytest
import torch

from pask_workloads import configs as WC
from pask_workloads import policy as WP
from pask_workloads import tags as WT
from pask_workloads.tensors import bf16_bits, normal_bf16

H_BYTES = {2: 1024, 8: 4096}
L_BYTES = {2: 288, 8: 1152}


def _policy(actions, n_layers=1, floors=None):
    """Policy with explicit per-(tag, group) actions; layer l belongs to group l % n_groups."""
    a = np.asarray(actions, np.uint8)
    n_tags, n_groups = a.shape
    fl = np.zeros_like(a) if floors is None else np.asarray(floors, np.uint8)
    z = np.zeros(a.shape, np.float32)
    lg = np.asarray([l % n_groups for l in range(n_layers)], np.uint8)
    return WP.Policy(n_tags, n_groups, lg, a, fl, z, z.copy(), np.zeros(2, np.uint32), budget_target=0.5)


def _rand_kv(seed, n, n_kv):
    k = normal_bf16(seed, 1, 0, 0, 0, n, n_kv)
    v = normal_bf16(seed, 2, 0, 0, 0, n, n_kv)
    return k, v


def _ref_attention(q, k, v):
    """Library routine: fp64 softmax(q k^T / sqrt(d)) v with GQA head repeat.
    q [n_q,128], k/v [n,n_kv,128] (any float dtype) -> out [n_q,128], lse [n_q]."""
    q, k, v = q.double(), k.double(), v.double()
    g = q.shape[0] // k.shape[1]
    kk = k.repeat_interleave(g, dim=1).permute(1, 0, 2)          # [n_q, n, 128]
    vv = v.repeat_interleave(g, dim=1).permute(1, 0, 2)
    s = torch.einsum("hd,hnd->hn", q, kk) / (128.0 ** 0.5)
    return torch.einsum("hn,hnd->hd", torch.softmax(s, dim=-1), vv), torch.logsumexp(s, dim=-1)


def _dequant(codes, scale_bits):
    """(code - 8) * scale with the fp16 scale decoded by numpy: [n,n_kv,128] float64."""
    s = scale_bits.view(np.float16).astype(np.float64)           # [n,n_kv,4]
    return (codes.astype(np.float64) - 8.0) * np.repeat(s, 32, axis=-1)


def _mk(oracle, pol, n_q=8, n_kv=2, max_seqs=2, hp=256, lp=256):
    p = oracle.Policy(WP.write_blob(pol))
    return oracle.Cache(p, n_q, n_kv, max_seqs, hp, lp)


def _append(cache, layer, seq, k, v, tags):
    rc, act = cache.append(layer, [seq], [0, len(tags)], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
    assert rc == 0
    return act


def test_all_high_equals_full_attention(oracle):
    # the reference policy keeps everything at high precision: plain full attention, cost exactly 1
    n = 333
    c = _mk(oracle, _policy([[2], [2], [2]]))
    k, v = _rand_kv(1, n, 2)
    tags = (np.arange(n) % 3).astype(np.uint8)
    act = _append(c, 0, 0, k, v, tags)
    assert np.all(act == 2)
    q = normal_bf16(1, 0, 0, 0, n, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    ro, rl = _ref_attention(q, k, v)
    assert np.abs(out - ro.numpy()).max() < 1e-12
    assert np.abs(lse - rl.numpy()).max() < 1e-12
    b = c.budget(0)
    assert b.retained_bytes == b.full_bytes == n * H_BYTES[2]


def test_dropped_tokens_contribute_exactly_nothing(oracle):
    # release removes a token from future attention: same result as deleting it from the inputs
    n = 257
    c = _mk(oracle, _policy([[0], [2]]))
    k, v = _rand_kv(2, n, 2)
    rng = np.random.default_rng(0)
    tags = rng.integers(0, 2, n).astype(np.uint8)
    act = _append(c, 0, 0, k, v, tags)
    assert np.array_equal(act, tags * 2)
    keep = torch.from_numpy(tags == 1)
    q = normal_bf16(2, 0, 0, 0, n, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    ro, rl = _ref_attention(q, k[keep], v[keep])
    assert np.abs(out - ro.numpy()).max() < 1e-12
    assert np.abs(lse - rl.numpy()).max() < 1e-12
    # poisoning the dropped tokens' values changes nothing
    k2, v2 = k.clone(), v.clone()
    k2[~keep] = 1e4
    v2[~keep] = -1e4
    c2 = _mk(oracle, _policy([[0], [2]]))
    _append(c2, 0, 0, k2, v2, tags)
    out2, _ = c2.attention(0, 0, bf16_bits(q).numpy())
    assert np.array_equal(out, out2)


def test_mixed_streams_equal_library_attention_on_dequantised_inputs(oracle):
    n = 300
    c = _mk(oracle, _policy([[0], [1], [2]]))
    k, v = _rand_kv(3, n, 2)
    rng = np.random.default_rng(1)
    tags = rng.integers(0, 3, n).astype(np.uint8)
    _append(c, 0, 0, k, v, tags)
    hk, hv, _ = c.dump_high(0, 0)
    kc, ks, vc, vs, _ = c.dump_low(0, 0)
    # HIGH stream holds the original bits of the H tokens, in arrival order
    assert np.array_equal(hk, bf16_bits(k).numpy().view(np.uint16)[tags == 2])
    assert np.array_equal(hv, bf16_bits(v).numpy().view(np.uint16)[tags == 2])
    k_all = torch.cat([k[torch.from_numpy(tags == 2)].double(), torch.from_numpy(_dequant(kc, ks))])
    v_all = torch.cat([v[torch.from_numpy(tags == 2)].double(), torch.from_numpy(_dequant(vc, vs))])
    q = normal_bf16(3, 0, 0, 0, n, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    ro, rl = _ref_attention(q, k_all, v_all)
    assert np.abs(out - ro.numpy()).max() < 1e-12
    assert np.abs(lse - rl.numpy()).max() < 1e-12
    # and the LOW codes are what the group quantiser gives for those tokens
    kb = bf16_bits(k).numpy().view(np.uint16)[tags == 1]
    for t in (0, kb.shape[0] - 1):
        for h in range(2):
            for g in range(4):
                sb, codes = oracle.quantize_group(kb[t, h, 32 * g:32 * g + 32])
                assert sb == ks[t, h, g] and np.array_equal(codes, kc[t, h, 32 * g:32 * g + 32])


def test_softmax_core_closed_forms(oracle):
    # one retained token: the output is that token's value, exactly; lse is its score
    c = _mk(oracle, _policy([[2]]))
    k, v = _rand_kv(4, 1, 2)
    _append(c, 0, 0, k, v, np.zeros(1, np.uint8))
    q = normal_bf16(4, 0, 0, 0, 0, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    for h in range(8):
        assert np.array_equal(out[h], v[0, h // 4].double().numpy())
        s = float((q[h].double() * k[0, h // 4].double()).sum()) / 128 ** 0.5
        assert abs(lse[h] - s) < 1e-12
    # identical keys: uniform weights, output is the mean of the values
    n = 7
    c = _mk(oracle, _policy([[2]]))
    k = k.expand(n, 2, 128).contiguous()
    v = normal_bf16(5, 2, 0, 0, 0, n, 2)
    _append(c, 0, 0, k, v, np.zeros(n, np.uint8))
    out, lse2 = c.attention(0, 0, bf16_bits(q).numpy())
    for h in range(8):
        assert np.abs(out[h] - v[:, h // 4].double().mean(0).numpy()).max() < 1e-14
        assert abs(lse2[h] - (lse[h] + np.log(n))) < 1e-12
    # two tokens: weights are the logistic function of the score difference
    c = _mk(oracle, _policy([[2]]))
    k, v = _rand_kv(6, 2, 2)
    _append(c, 0, 0, k, v, np.zeros(2, np.uint8))
    out, _ = c.attention(0, 0, bf16_bits(q).numpy())
    for h in range(8):
        kk, vv = k[:, h // 4].double(), v[:, h // 4].double()
        d = float((q[h].double() * (kk[0] - kk[1])).sum()) / 128 ** 0.5
        w0 = 1.0 / (1.0 + np.exp(-d))
        assert np.abs(out[h] - (w0 * vv[0] + (1 - w0) * vv[1]).numpy()).max() < 1e-13


def test_empty_retained_set(oracle):
    c = _mk(oracle, _policy([[0]]))
    k, v = _rand_kv(7, 5, 2)
    _append(c, 0, 0, k, v, np.zeros(5, np.uint8))
    q = normal_bf16(7, 0, 0, 0, 0, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    assert np.all(out == 0) and np.all(np.isneginf(lse))
    b = c.budget(0)
    assert b.retained_bytes == 0 and b.full_bytes == 5 * 1024 and b.n_drop[0] == 5


def test_split_combine_identity(oracle):
    # any partition of the retained set, merged with the log-sum-exp rule, gives the same result
    n = 200
    k, v = _rand_kv(8, n, 2)
    q = normal_bf16(8, 0, 0, 0, n, 1, 8)[0]
    c = _mk(oracle, _policy([[2]]))
    _append(c, 0, 0, k, v, np.zeros(n, np.uint8))
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    for cuts in ([0, 1, 200], [0, 37, 101, 200], [0, 16, 32, 48, 199, 200]):
        parts = []
        for a, b in zip(cuts[:-1], cuts[1:]):
            cc = _mk(oracle, _policy([[2]]))
            _append(cc, 0, 0, k[a:b], v[a:b], np.zeros(b - a, np.uint8))
            parts.append(cc.attention(0, 0, bf16_bits(q).numpy()))
        m = np.max([p[1] for p in parts], axis=0)
        w = np.stack([np.exp(p[1] - m) for p in parts])                 # [parts, n_q]
        merged = sum(wi[:, None] * p[0] for wi, p in zip(w, parts)) / w.sum(0)[:, None]
        assert np.abs(merged - out).max() < 1e-12
        assert np.abs(m + np.log(w.sum(0)) - lse).max() < 1e-12


def test_unknown_and_protected_tags(oracle):
    c = _mk(oracle, _policy([[0], [1]]))
    k, v = _rand_kv(9, 4, 2)
    act = _append(c, 0, 0, k, v, np.array([0, 1, 0xFF, 7], np.uint8))
    assert act.tolist() == [0, 1, 2, 2]
    b = c.budget(0)
    assert b.bad_tags == 1 and b.n_high[0] == 2 and b.n_low[0] == 1 and b.n_drop[0] == 1


def test_floor_takes_priority(oracle):
    c = _mk(oracle, _policy([[0], [1], [2]], floors=[[2], [0], [1]]))
    k, v = _rand_kv(10, 3, 2)
    act = _append(c, 0, 0, k, v, np.array([0, 1, 2], np.uint8))
    assert act.tolist() == [2, 1, 2]


def test_layer_groups_diverge(oracle):
    # the same tag may be low precision in an early group and high precision in a late one
    pol = _policy([[1, 2], [0, 1]], n_layers=4)
    c = _mk(oracle, pol)
    k, v = _rand_kv(11, 6, 2)
    tags = np.array([0, 1, 0, 1, 1, 0], np.uint8)
    for layer in range(4):
        act = _append(c, layer, 0, k, v, tags)
        want = np.where(tags == 0, 1, 0) if layer % 2 == 0 else np.where(tags == 0, 2, 1)
        assert np.array_equal(act, want)
    assert c.stream_len(0, 0) == (0, 3) and c.stream_len(1, 0) == (3, 3)
    b = c.budget(0)
    assert b.n_seen[0] == 12 and b.n_seen[1] == 12
    assert b.n_low[0] == 6 and b.n_drop[0] == 6 and b.n_high[1] == 6 and b.n_low[1] == 6


def test_budget_recount_and_closed_form(oracle):
    w = WC.build(WC.TINY)
    cfg = w.cfg
    c = _mk(oracle, w.policy, cfg.n_q, cfg.n_kv, 1, 64, 64)
    n = w.total_len(0)
    k, v = w.kv(0, 0, 0, n)
    tags = w.tags(0, 0, n)
    act = _append(c, 0, 0, k, v, tags)
    b = c.budget(0)
    nh, nl = c.stream_len(0, 0)
    assert (nh, nl) == (int((act == 2).sum()), int((act == 1).sum()))
    assert b.retained_bytes == nh * 1024 + nl * 288                   # recount from the streams
    assert b.full_bytes == n * 1024
    assert b.n_seen[0] == n and b.n_drop[0] == n - nh - nl
    assert b.pages_high == (nh + 15) // 16 and b.pages_low == (nl + 15) // 16
    q16 = int(round(w.policy.budget_target * 65536))
    assert b.remaining_bytes == (q16 * b.full_bytes >> 16) - b.retained_bytes
    c_kv = b.retained_bytes / b.full_bytes                            # Eq. 1 from the counts
    assert abs(c_kv - (nh * 1.0 + nl * 0.28125) / n) < 1e-15


def test_paging_invariants_and_bulk_equals_stepwise(oracle):
    pol = _policy([[0], [1], [2]])
    n = 150
    rng = np.random.default_rng(5)
    tags = [rng.integers(0, 3, n).astype(np.uint8) for _ in range(2)]
    kv = [(normal_bf16(12, 1, 0, s, 0, n, 2), normal_bf16(12, 2, 0, s, 0, n, 2)) for s in range(2)]
    bulk = _mk(oracle, pol)
    k = torch.cat([kv[0][0], kv[1][0]])
    v = torch.cat([kv[0][1], kv[1][1]])
    rc, act = bulk.append(0, [0, 1], [0, n, 2 * n], bf16_bits(k).numpy(), bf16_bits(v).numpy(),
                          np.concatenate(tags))
    assert rc == 0
    # sequence-major page order: sequence 0 owns the first ids of each pool
    for s in range(2):
        hk, hv, ph = bulk.dump_high(0, s)
        kc, ks, vc, vs, pl = bulk.dump_low(0, s)
        nh, nl = bulk.stream_len(0, s)
        assert len(ph) == (nh + 15) // 16 and len(pl) == (nl + 15) // 16
        assert np.array_equal(hk, bf16_bits(kv[s][0]).numpy().view(np.uint16)[tags[s] == 2])
    p0h = bulk.dump_high(0, 0)[2]
    p1h = bulk.dump_high(0, 1)[2]
    assert np.array_equal(np.concatenate([p0h, p1h]), np.arange(len(p0h) + len(p1h)))
    p0l, p1l = bulk.dump_low(0, 0)[4], bulk.dump_low(0, 1)[4]
    assert np.array_equal(np.concatenate([p0l, p1l]), np.arange(len(p0l) + len(p1l)))
    # token-by-token replay (both sequences per call, one token each): same streams, codes, scales
    step = _mk(oracle, pol)
    for t in range(n):
        kk = torch.stack([kv[0][0][t], kv[1][0][t]])
        vv = torch.stack([kv[0][1][t], kv[1][1][t]])
        rc, a = step.append(0, [0, 1], [0, 1, 2], bf16_bits(kk).numpy(), bf16_bits(vv).numpy(),
                            np.array([tags[0][t], tags[1][t]], np.uint8))
        assert rc == 0 and a[0] == act[t] and a[1] == act[n + t]
    for s in range(2):
        for x, y in zip(bulk.dump_high(0, s)[:2], step.dump_high(0, s)[:2]):
            assert np.array_equal(x, y)
        for x, y in zip(bulk.dump_low(0, s)[:4], step.dump_low(0, s)[:4]):
            assert np.array_equal(x, y)
        # page ids differ between the two schedules (interleaved arrival) but stay unique per pool
    ids = np.concatenate([step.dump_high(0, 0)[2], step.dump_high(0, 1)[2]])
    assert len(set(ids.tolist())) == len(ids)
    assert step.budget(0).retained_bytes == bulk.budget(0).retained_bytes


def test_pool_exhaustion_is_atomic_and_pages_are_reused_lifo(oracle):
    pol = _policy([[1], [2]])
    c = _mk(oracle, pol, hp=3, lp=2)
    k, v = _rand_kv(13, 40, 2)
    _append(c, 0, 0, k[:40], v[:40], np.ones(40, np.uint8))              # 3 HIGH pages: pool now empty
    before = (c.stream_len(0, 0), c.budget(0).retained_bytes, c.pool_state())
    rc, _ = c.append(0, [1], [0, 20], bf16_bits(k[:20]).numpy(), bf16_bits(v[:20]).numpy(),
                     np.array([0] * 10 + [1] * 10, np.uint8))             # needs 1 LOW + 1 HIGH page
    assert rc == oracle.ERR_POOL
    assert (c.stream_len(0, 0), c.budget(0).retained_bytes, c.pool_state()) == before
    assert c.stream_len(0, 1) == (0, 0) and c.budget(1).full_bytes == 0
    # a call that fits still works, including filling the partial page without a new one
    rc, _ = c.append(0, [0], [0, 8], bf16_bits(k[:8]).numpy(), bf16_bits(v[:8]).numpy(), np.ones(8, np.uint8))
    assert rc == 0 and c.stream_len(0, 0) == (48, 0)
    # reset returns pages; the next allocations pop them in reverse push order
    assert c.dump_high(0, 0)[2].tolist() == [0, 1, 2]
    c.seq_reset(0)
    assert c.pool_state() == (3, 3, 0, 0)
    _append(c, 0, 1, k[:33], v[:33], np.ones(33, np.uint8))
    assert c.dump_high(0, 1)[2].tolist() == [2, 1, 0]
    assert c.budget(0).full_bytes == 0


def test_bad_blobs_are_rejected(oracle):
    good = WP.write_blob(_policy([[0], [1]]))
    oracle.Policy(good)
    for bad in (good[:-1], good + b"\0", b"XASK" + good[4:], good[:4] + b"\2\0\0\0" + good[8:], b""):
        with pytest.raises(ValueError):
            oracle.Policy(bad)
    broken = bytearray(good)
    broken[40 + 4] = 3                                                    # action out of range
    with pytest.raises(ValueError):
        oracle.Policy(bytes(broken))


def test_generators_are_reproducible_and_slice_consistent():
    a = normal_bf16(99, 1, 3, 5, 0, 64, 8)
    b = normal_bf16(99, 1, 3, 5, 16, 8, 8)
    assert torch.equal(a[16:24], b)
    assert not torch.equal(normal_bf16(99, 2, 3, 5, 0, 8, 8), a[:8])
    x = normal_bf16(1, 1, 0, 0, 0, 4096, 8).float()
    assert abs(float(x.mean())) < 0.01 and abs(float(x.std()) - 1.0) < 0.01
    w1, w2 = WC.build(WC.TINY), WC.build(WC.TINY)
    assert np.array_equal(w1.gen_tags[0], w2.gen_tags[0]) and w1.blob == w2.blob
    assert set(np.unique(w1.gen_tags[0]).tolist()) <= set(range(WT.N_DECODE_TAGS))


def test_eight_bit_low_stream_against_library_attention(oracle):
    # policy low_bits = 8: the LOW stream holds int8 codes (offset 128) and is attended as (code - 128) * scale
    from dataclasses import replace
    n = 200
    pol = replace(_policy([[1], [2], [0], [1]]), low_bits=8)
    c = _mk(oracle, pol)
    k, v = _rand_kv(8, n, 2)
    tags = (np.arange(n) % 4).astype(np.uint8)
    act = _append(c, 0, 0, k, v, tags)
    kc, ks, vc, vs, _ = c.dump_low(0, 0)
    assert kc.min() >= 1 and kc.max() > 200                       # the codes use the 8-bit range
    hk, hv, _ = c.dump_high(0, 0)
    s = lambda b: b.view(np.float16).astype(np.float64)
    dq = lambda codes, sc: (codes.astype(np.float64) - 128.0) * np.repeat(s(sc), 32, axis=-1)
    from_bits = lambda b: torch.from_numpy(b.astype(np.int32) << 16).view(torch.float32).double()
    K = torch.cat([from_bits(hk), torch.from_numpy(dq(kc, ks))])
    V = torch.cat([from_bits(hv), torch.from_numpy(dq(vc, vs))])
    q = normal_bf16(8, 0, 0, 0, n, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    ro, rl = _ref_attention(q, K, V)
    assert np.abs(out - ro.numpy()).max() < 1e-12 and np.abs(lse - rl.numpy()).max() < 1e-12
    # the int8 copy of a token is close to the token itself: relative error of a row below 1 %
    kl = k[act == 1].double().numpy()
    assert np.abs(dq(kc, ks) - kl).max() <= 0.5 * s(ks).max() * 1.01
    b = c.budget(0)
    n_l, n_h = int((act == 1).sum()), int((act == 2).sum())
    assert b.retained_bytes == n_h * H_BYTES[2] + n_l * 2 * 2 * (128 + 8)   # codes at one byte each + scales


def test_two_bit_low_stream_against_library_attention(oracle):
    # policy low_bits = 2: the LOW stream holds the codes 1, 2, 3 and is attended as (code - 2) * scale
    from dataclasses import replace
    n = 200
    pol = replace(_policy([[1], [2], [0], [1]]), low_bits=2)
    c = _mk(oracle, pol)
    k, v = _rand_kv(9, n, 2)
    tags = (np.arange(n) % 4).astype(np.uint8)
    act = _append(c, 0, 0, k, v, tags)
    kc, ks, vc, vs, _ = c.dump_low(0, 0)
    assert set(np.unique(kc).tolist()) == {1, 2, 3} and set(np.unique(vc).tolist()) == {1, 2, 3}
    hk, hv, _ = c.dump_high(0, 0)
    s = lambda b: b.view(np.float16).astype(np.float64)
    dq = lambda codes, sc: (codes.astype(np.float64) - 2.0) * np.repeat(s(sc), 32, axis=-1)
    from_bits = lambda b: torch.from_numpy(b.astype(np.int32) << 16).view(torch.float32).double()
    K = torch.cat([from_bits(hk), torch.from_numpy(dq(kc, ks))])
    V = torch.cat([from_bits(hv), torch.from_numpy(dq(vc, vs))])
    q = normal_bf16(8, 0, 0, 0, n, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    ro, rl = _ref_attention(q, K, V)
    assert np.abs(out - ro.numpy()).max() < 1e-12 and np.abs(lse - rl.numpy()).max() < 1e-12
    # every value is within half a step of its level, the step being the group's amax
    kl = k[act == 1].double().numpy()
    assert np.abs(dq(kc, ks) - kl).max() <= 0.5 * s(ks).max() * 1.01
    b = c.budget(0)
    n_l, n_h = int((act == 1).sum()), int((act == 2).sum())
    assert b.retained_bytes == n_h * H_BYTES[2] + n_l * 2 * 2 * (32 + 8)     # four codes per byte + scales
