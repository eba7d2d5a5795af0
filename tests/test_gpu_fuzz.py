"""Seeded differential fuzz of the cache machinery: arbitrary per-token actions (fed through
pask_append_kv_decided), ragged call sizes that hit the one-launch path and the bulk path, sequence
resets in between, small pools that sometimes refuse a call -- state compared with the oracle
after every call, attention at the end."""
import numpy as np
import pytest
import torch

from pask_workloads import configs as WC
from pask_workloads import policy as WP
from pask_workloads.rng import CounterRng
from pask_workloads.tensors import bf16_bits, normal_bf16

from parity import Pair

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pask():
    import paper_2608_28276_b200 as P      # fails loudly if libpask.so is missing
    assert torch.cuda.is_available()
    return P


@pytest.mark.parametrize("seed,n_kv,window,low_bits", [(1, 2, 0, 4), (2, 8, 0, 4), (3, 4, 16, 4), (4, 1, 48, 4), (5, 8, 0, 4),
                                                       (6, 2, 0, 4), (7, 8, 0, 8), (8, 2, 32, 8), (9, 1, 0, 8), (10, 8, 0, 2),
                                                       (11, 2, 16, 2), (12, 4, 0, 2)])
def test_random_call_sequences(pask, oracle, seed, n_kv, window, low_bits):
    from dataclasses import replace
    rng = CounterRng(seed, 4242)
    n_layers, G, B = 2, 2, 4
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, n_kv=n_kv, n_q=4 * n_kv, n_layers=n_layers, n_groups=G, batch=B, prompt_len=8,
                    gen_len=8, extra_gen=8)
    w = WC.build(cfg)
    tight = seed % 2 == 0                                               # every other case runs out of pages now and then
    pages = 16 if tight else 400
    p = Pair(pask, oracle, w, blob=WP.write_blob(replace(w.policy, recent_window=window, low_bits=low_bits)), pool_high_pages=pages,
             pool_low_pages=pages, max_tokens_per_seq=4096, max_append_tokens=2048)
    d = "cuda"
    serial = 0
    refused = 0
    for call in range(16):
        if rng.unit() < 0.15:                                           # forget a sequence, its pages go back on the stacks
            s = rng.below(B)
            pask.pask_seq_reset(p.gpu.handle, s)
            p.orc.seq_reset(s)
        n_seqs = 1 + rng.below(B)
        seqs = list(np.random.default_rng(seed * 100 + call).permutation(B)[:n_seqs])
        kind = rng.below(3)
        counts = [[1, 1 + rng.below(3), rng.below(40), rng.below(400)][rng.below(2) + kind] for _ in seqs]
        total = int(sum(counts))
        cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        serial += 1
        k = normal_bf16(seed, 1, serial, 0, 0, total, n_kv)
        v = normal_bf16(seed, 2, serial, 0, 0, total, n_kv)
        tags = np.asarray([rng.below(14) if rng.unit() < 0.9 else 0xFF for _ in range(total)], np.uint8)
        acts = np.asarray([[rng.weighted([3, 3, 3]) for _ in range(G)] for _ in range(total)], np.uint8).reshape(total, G)
        layer = rng.below(n_layers)
        rc, used_o = p.orc.append(layer, seqs, cu, bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags, decided=acts)
        used_g = torch.full((max(1, total),), 0xEE, dtype=torch.uint8, device=d)
        if total:
            pask.pask_append_kv_decided(p.gpu.handle, layer, torch.tensor(seqs, dtype=torch.int32, device=d),
                                        torch.from_numpy(cu).to(d), k.to(d), v.to(d), torch.from_numpy(tags).to(d),
                                        torch.from_numpy(acts).to(d), actions_out=used_g, total_tokens=total)
        torch.cuda.synchronize()
        st = pask.pask_budget_state(p.gpu.handle, 0).device_status
        if rc == 0:
            assert np.array_equal(used_g.cpu().numpy()[:total], used_o)
        else:
            assert rc == oracle.ERR_POOL and st & pask.DEV_POOL_EXHAUSTED
            refused += 1
        assert (st & ~pask.DEV_POOL_EXHAUSTED) == 0
        for s in range(B):                                              # lengths, page ids and pool state after every call
            for l in range(n_layers):
                assert pask.pask_debug_stream_len(p.gpu.handle, l, s) == p.orc.stream_len(l, s)
        assert pask.pask_debug_pool_state(p.gpu.handle) == p.orc.pool_state()
    # full state (stored bytes, page ids, budgets; the sticky exhaustion bit aside) and attention at the end
    for s in range(B):
        for l in range(n_layers):
            for a, b in zip(pask.pask_debug_dump_high(p.gpu.handle, l, s, n_kv), p.orc.dump_high(l, s)):
                assert np.array_equal(a, b)
            for a, b in zip(pask.pask_debug_dump_low(p.gpu.handle, l, s, n_kv), p.orc.dump_low(l, s)):
                assert np.array_equal(a, b)
        p.compare_budget(s, expect_status=pask.DEV_POOL_EXHAUSTED if refused else 0)
    q = normal_bf16(seed, 0, 0, 0, 0, B, 4 * n_kv)
    for l in range(n_layers):
        p.check_attention(l, list(range(B)), q=q)
