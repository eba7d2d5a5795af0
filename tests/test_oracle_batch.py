"""Pins for the oracle's batched attention entry (`orc_attention_batch`), the one every GPU attention
comparison goes through.  CPU only.

The batch entry is a loop over (row of the call, query head) that looks the sequence up through
`seq_ids`; what can go wrong in it is indexing: the row -> sequence map, the row stride of q / out /
lse, the layer, and the sharing of the loop among host threads.  It is pinned, row by row, to the
single-sequence entry and to a library routine (torch fp64 softmax attention) on inputs this test
assembles itself from the raw tensors and the dumped streams, for sequences of different lengths
and mixes (one never appended, one with every token released, one all high, one all low), with the
ids permuted, repeated, and a strict subset of the cache's sequences, on two layers of different
groups, with and without a protected recent window, on one host thread and on many."""
import numpy as np
import pytest
import torch

from pask_workloads import policy as WP
from pask_workloads.rng import CounterRng
from pask_workloads.tensors import bf16_bits, normal_bf16

N_KV, N_Q, N_SEQ = 2, 8, 7
R_TAG, L_TAG, H_TAG = 0, 1, 2            # the table below maps these tags to one action in every group


def _policy(window):
    # tags 0..2 fixed to R / L / H in both groups; tags 3..5 differ between the groups
    a0 = np.asarray([[0, 0], [1, 1], [2, 2], [0, 2], [1, 0], [2, 1]], np.uint8)
    z = np.zeros(a0.shape, np.float32)
    p = WP.Policy(6, 2, np.asarray([0, 1], np.uint8), a0, np.zeros_like(a0), z, z.copy(), np.zeros(2, np.uint32),
                  budget_target=0.5)
    p.recent_window = window
    return p


def _ref_attention(q, k, v):
    """Library routine: fp64 softmax(q k^T / sqrt(d)) v with GQA head repeat."""
    q, k, v = q.double(), k.double(), v.double()
    if k.shape[0] == 0:
        return torch.zeros(q.shape[0], 128, dtype=torch.float64), torch.full((q.shape[0],), -np.inf, dtype=torch.float64)
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


def _tags(seq, n):
    """Sequence 0: never appended.  1: every token released.  2: all high.  3: all low.  Others: a seeded mix."""
    if seq == 1:
        return np.full(n, R_TAG, np.uint8)
    if seq == 2:
        return np.full(n, H_TAG, np.uint8)
    if seq == 3:
        return np.full(n, L_TAG, np.uint8)
    rng = CounterRng(77, seq)
    return np.asarray([rng.below(6) for _ in range(n)], np.uint8)


LENGTHS = [0, 40, 33, 50, 129, 17, 301]


def _build(oracle, window):
    c = oracle.Cache(oracle.Policy(WP.write_blob(_policy(window))), N_Q, N_KV, N_SEQ, 512, 512)
    raw = {}
    for layer in (0, 1):
        for seq, n in enumerate(LENGTHS):
            if n == 0:
                continue
            k = normal_bf16(5, 1, layer, seq, 0, n, N_KV)
            v = normal_bf16(5, 2, layer, seq, 0, n, N_KV)
            rc, act = c.append(layer, [seq], [0, n], bf16_bits(k).numpy(), bf16_bits(v).numpy(), _tags(seq, n))
            assert rc == 0
            raw[(layer, seq)] = (k, v, act)
    return c, raw


def _expected(c, raw, layer, seq, window, q):
    """Library attention over what the sequence retains: the dumped streams without their last window
    members, plus the window's raw bf16 rows."""
    if (layer, seq) not in raw:
        return _ref_attention(q, torch.zeros(0, N_KV, 128), torch.zeros(0, N_KV, 128))
    k, v, act = raw[(layer, seq)]
    n = len(act)
    nw = min(n, window)
    wa = act[n - nw:]
    hk, hv, _ = c.dump_high(layer, seq)
    kc, ks, vc, vs, _ = c.dump_low(layer, seq)
    nh, nl = hk.shape[0] - int((wa == 2).sum()), kc.shape[0] - int((wa == 1).sum())
    K = torch.cat([_from_bits(hk[:nh]).double(), torch.from_numpy(_dequant(kc[:nl], ks[:nl])), k[n - nw:].double()])
    V = torch.cat([_from_bits(hv[:nh]).double(), torch.from_numpy(_dequant(vc[:nl], vs[:nl])), v[n - nw:].double()])
    return _ref_attention(q, K, V)


@pytest.mark.parametrize("window", [0, 32])
@pytest.mark.parametrize("threads", [1, 0])          # 0: as many as the host offers
def test_batch_rows_against_single_entry_and_library_attention(oracle, window, threads):
    c, raw = _build(oracle, window)
    before = oracle.max_threads()
    oracle.set_threads(threads if threads else max(4, before))
    try:
        orders = [
            [6, 0, 3, 1, 5, 2, 4],        # every sequence, permuted
            [4, 1, 6],                    # a strict subset, not in order
            [5, 5, 2],                    # a sequence named twice: two independent rows
            [3],
        ]
        for layer in (0, 1):
            for call, ids in enumerate(orders):
                # every row gets its own query, so a row read or written at the wrong stride cannot go unnoticed
                q = normal_bf16(900 + call, 0, layer, 0, 0, len(ids), N_Q)
                out, lse = c.attention_batch(layer, ids, bf16_bits(q).numpy())
                assert out.shape == (len(ids), N_Q, 128) and lse.shape == (len(ids), N_Q)
                for row, seq in enumerate(ids):
                    so, sl = c.attention(layer, seq, bf16_bits(q[row]).numpy())
                    assert np.array_equal(out[row], so) and np.array_equal(lse[row], sl)
                    ro, rl = _expected(c, raw, layer, seq, window, q[row])
                    assert np.abs(out[row] - ro.numpy()).max() < 1e-12
                    if LENGTHS[seq] == 0 or (seq == 1 and window == 0):
                        assert np.all(out[row] == 0.0) and np.all(np.isneginf(lse[row]))     # nothing retained
                    else:
                        assert np.abs(lse[row] - rl.numpy()).max() < 1e-12
    finally:
        oracle.set_threads(before)


def test_batch_rows_differ_where_they_should(oracle):
    # the fixture would be blind to a row -> sequence mix-up if the sequences were alike: they are not
    c, _ = _build(oracle, 0)
    q = normal_bf16(901, 0, 0, 0, 0, 1, N_Q)
    qb = bf16_bits(q.repeat(N_SEQ, 1, 1)).numpy()
    out, _ = c.attention_batch(0, list(range(N_SEQ)), qb)
    for a in range(2, N_SEQ):
        for b in range(a + 1, N_SEQ):
            assert np.abs(out[a] - out[b]).max() > 1e-3
    # and the two layers of one sequence differ too (different K/V, different group column of the table)
    out1, _ = c.attention_batch(1, list(range(N_SEQ)), qb)
    assert np.abs(out[4] - out1[4]).max() > 1e-3


def test_batch_refuses_bad_ids_and_layers(oracle):
    c, _ = _build(oracle, 0)
    import ctypes as C
    q = np.zeros((1, N_Q, 128), np.uint16)
    out, lse = np.zeros((1, N_Q, 128)), np.zeros((1, N_Q))
    L = oracle.lib()
    for ids, layer, rc in (([N_SEQ], 0, oracle.ERR_SEQ), ([-1], 0, oracle.ERR_SEQ), ([0], 2, oracle.ERR_ARG), ([0], -1, oracle.ERR_ARG)):
        a = np.asarray(ids, np.int32)
        got = L.orc_attention_batch(c.h, layer, 1, a.ctypes.data_as(C.c_void_p), q.ctypes.data_as(C.c_void_p),
                                    out.ctypes.data_as(C.c_void_p), lse.ctypes.data_as(C.c_void_p))
        assert got == rc
