"""Pins for the oracle's protected recent window (Section 3.1: release and the low-precision format
apply to a KV state only after it has left the window).  CPU only.

The window is pinned to a library routine (torch fp64 softmax attention) on inputs the test
assembles itself: raw bf16 rows for the window, and for older tokens the rows of the dumped
streams, cut by a recount of the returned actions."""
import numpy as np
import pytest
import torch

from pask_workloads import policy as WP
from pask_workloads.rng import CounterRng
from pask_workloads.tensors import bf16_bits, normal_bf16


def _policy(seed, n_tags, window, n_layers=1, n_groups=1):
    p = WP.random_policy(seed, n_tags, n_groups, n_layers)
    p.recent_window = window
    return p


def _ref_attention(q, k, v):
    q, k, v = q.double(), k.double(), v.double()
    g = q.shape[0] // k.shape[1]
    kk = k.repeat_interleave(g, dim=1).permute(1, 0, 2)
    vv = v.repeat_interleave(g, dim=1).permute(1, 0, 2)
    s = torch.einsum("hd,hnd->hn", q, kk) / (128.0 ** 0.5)
    return torch.einsum("hn,hnd->hd", torch.softmax(s, dim=-1), vv), torch.logsumexp(s, dim=-1)


def _from_bits(b):
    return torch.from_numpy(b.astype(np.int32) << 16).view(torch.float32)


def _dequant(codes, scale_bits):
    s = scale_bits.view(np.float16).astype(np.float64)
    return (codes.astype(np.float64) - 8.0) * np.repeat(s, 32, axis=-1)


def _inputs(seed, n, n_tags, n_kv=2):
    rng = CounterRng(seed, 111)
    tags = np.asarray([rng.below(n_tags) for _ in range(n)], np.uint8)
    return normal_bf16(seed, 1, 0, 0, 0, n, n_kv), normal_bf16(seed, 2, 0, 0, 0, n, n_kv), tags


def _cache(oracle, pol, n_kv=2, pages=256):
    return oracle.Cache(oracle.Policy(WP.write_blob(pol)), 4 * n_kv, n_kv, 1, pages, pages)


def _expected(c, k, v, act, window, q):
    """softmax attention over: dumped streams minus their last window members, plus raw window rows."""
    n = len(act)
    nw = min(n, window)
    wa = act[n - nw:]
    hk, hv, _ = c.dump_high(0, 0)
    kc, ks, vc, vs, _ = c.dump_low(0, 0)
    nh, nl = hk.shape[0] - int((wa == 2).sum()), kc.shape[0] - int((wa == 1).sum())
    K = torch.cat([_from_bits(hk[:nh]).double(), torch.from_numpy(_dequant(kc[:nl], ks[:nl])), k[n - nw:].double()])
    V = torch.cat([_from_bits(hv[:nh]).double(), torch.from_numpy(_dequant(vc[:nl], vs[:nl])), v[n - nw:].double()])
    return _ref_attention(q, K, V)


@pytest.mark.parametrize("window,n", [(16, 5), (16, 16), (16, 17), (32, 100), (64, 333), (256, 300)])
def test_window_against_library_attention(oracle, window, n):
    pol = _policy(7, 6, window)
    c = _cache(oracle, pol)
    k, v, tags = _inputs(window * 1000 + n, n, 6)
    rc, act = c.append(0, [0], [0, n], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
    assert rc == 0 and set(np.unique(act).tolist()) <= {0, 1, 2}
    q = normal_bf16(9, 0, 0, 0, n, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    ro, rl = _expected(c, k, v, act, window, q)
    assert np.abs(out - ro.numpy()).max() < 1e-12
    assert np.abs(lse - rl.numpy()).max() < 1e-12


def test_window_covering_everything_is_full_attention(oracle):
    # while no token has left the window, actions do not matter: plain attention on the raw inputs
    pol = _policy(8, 6, 128)
    c = _cache(oracle, pol)
    k, v, tags = _inputs(81, 128, 6)
    rc, act = c.append(0, [0], [0, 128], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
    assert rc == 0 and (act == 0).any() and (act == 1).any()
    q = normal_bf16(10, 0, 0, 0, 0, 1, 8)[0]
    out, lse = c.attention(0, 0, bf16_bits(q).numpy())
    ro, rl = _ref_attention(q, k, v)
    assert np.abs(out - ro.numpy()).max() < 1e-12 and np.abs(lse - rl.numpy()).max() < 1e-12


def test_released_token_is_attended_until_it_leaves_the_window(oracle):
    # one tag, always released, window 16: the newest 16 tokens are all there is to attend
    a = np.zeros((1, 1), np.uint8)
    z = np.zeros((1, 1), np.float32)
    pol = WP.Policy(1, 1, np.zeros(1, np.uint8), a, a.copy(), z, z.copy(), np.zeros(1, np.uint32), recent_window=16)
    c = _cache(oracle, pol)
    k, v, _ = _inputs(82, 40, 1)
    tags = np.zeros(40, np.uint8)
    q = normal_bf16(11, 0, 0, 0, 0, 1, 8)[0]
    for t in range(40):
        rc, act = c.append(0, [0], [0, 1], bf16_bits(k[t:t + 1]).numpy(), bf16_bits(v[t:t + 1]).numpy(), tags[t:t + 1])
        assert rc == 0 and act[0] == 0
        out, lse = c.attention(0, 0, bf16_bits(q).numpy())
        lo = max(0, t + 1 - 16)
        ro, rl = _ref_attention(q, k[lo:t + 1], v[lo:t + 1])
        assert np.abs(out - ro.numpy()).max() < 1e-12
    assert c.stream_len(0, 0) == (0, 0) and c.budget(0).retained_bytes == 0


def test_token_by_token_equals_bulk_and_budget_ignores_the_window(oracle):
    n, window = 150, 32
    k, v, tags = _inputs(83, n, 6)
    q = normal_bf16(12, 0, 0, 0, 0, 1, 8)[0]
    bulk, step, plain = (_cache(oracle, _policy(9, 6, w)) for w in (window, window, 0))
    bulk.append(0, [0], [0, n], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
    plain.append(0, [0], [0, n], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
    for t0 in range(0, n, 7):
        t1 = min(n, t0 + 7)
        step.append(0, [0], [0, t1 - t0], bf16_bits(k[t0:t1]).numpy(), bf16_bits(v[t0:t1]).numpy(), tags[t0:t1])
    ob, lb = bulk.attention(0, 0, bf16_bits(q).numpy())
    os_, ls = step.attention(0, 0, bf16_bits(q).numpy())
    assert np.array_equal(ob, os_) and np.array_equal(lb, ls)
    # the streams and the accounting are those of the window-less cache: the window only changes what is attended
    for a, b in zip(bulk.dump_high(0, 0) + bulk.dump_low(0, 0), plain.dump_high(0, 0) + plain.dump_low(0, 0)):
        assert np.array_equal(a, b)
    assert bulk.budget(0).retained_bytes == plain.budget(0).retained_bytes
    op, _ = plain.attention(0, 0, bf16_bits(q).numpy())
    assert np.abs(op - ob).max() > 1e-6                                   # and it does change that


def test_window_sizes_accepted(oracle):
    for w, ok in ((0, True), (16, True), (256, True), (8, False), (24, False), (272, False)):
        blob = WP.write_blob(_policy(10, 4, w))
        if ok:
            oracle.Policy(blob)
        else:
            with pytest.raises(ValueError):
                oracle.Policy(blob)
