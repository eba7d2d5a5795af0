"""Every supported head shape (1, 2, 4 or 8 KV heads, 4 query heads each) through the bulk append,
the one-launch decode append, the fused step, the recent window and attention, against the oracle."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from pask_workloads import configs as WC
from pask_workloads import policy as WP

from parity import Pair

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pask():
    import paper_2608_28276_b200 as P      # fails loudly if libpask.so is missing
    assert torch.cuda.is_available()
    return P


@pytest.mark.parametrize("n_kv", [1, 2, 4, 8])
@pytest.mark.parametrize("window", [0, 32])
def test_shape(pask, oracle, n_kv, window):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, n_kv=n_kv, n_q=4 * n_kv, n_layers=2, n_groups=2, batch=3, prompt_len=190,
                    gen_len=130, extra_gen=64)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w, blob=WP.write_blob(replace(w.policy, recent_window=window)))
    seqs = [2, 0, 1]
    counts = [w.total_len(s) - 5 * i for i, s in enumerate(seqs)]
    for layer in range(2):
        p.append(layer, seqs, counts, [0, 0, 0])                        # bulk path: whole pages and partly filled ones
    p.compare_state()
    for layer in range(2):
        p.check_attention(layer, [0, 1, 2], pos=counts[0])
    pos = dict(zip(seqs, counts))
    for n in (1, 1, 3, 1, 20, 1):                                       # one-launch path, pages filling up
        for layer in range(2):
            p.append(layer, seqs, [n] * 3, [pos[s] for s in seqs])
        pos = {s: pos[s] + n for s in pos}
    p.compare_state()
    for layer in range(2):
        p.check_attention(layer, [1, 2, 0], pos=pos[0])
    # a second bulk call continues partly filled pages
    for layer in range(2):
        p.append(layer, seqs, [14, 14, 14], [pos[s] for s in seqs], expect_ok=True)
    p.compare_state()
    p.check_attention(1, [0, 1, 2], pos=pos[0] + 14)


def test_largest_call_1024_sequences(pask, oracle):
    # PASK_MAX_SEQS_PER_CALL sequences in one append and one attention call, some of them empty
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, n_kv=2, n_q=8, n_layers=1, n_groups=1, batch=1024, prompt_len=20, gen_len=20,
                    extra_gen=8)
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = list(range(1023, -1, -1))
    counts = [0 if s % 97 == 0 else 17 + s % 23 for s in seqs]
    p.append(0, seqs, counts, [0] * 1024)
    for step in range(3):
        p.append(0, seqs, [1] * 1024, [c + step for c in counts])
    p.compare_state(seqs=[0, 1, 96, 97, 500, 1023])
    assert pask.pask_debug_pool_state(p.gpu.handle) == p.orc.pool_state()
    p.check_attention(0, list(range(1024)), pos=40)
    p.check_attention(0, seqs[:300], pos=40)


def test_one_stream_of_more_than_65536_pages(pask, oracle):
    # past 2^16 pages per sequence the work partition switches to 64-bit arithmetic: one sequence of
    # 1.2 M retained tokens (one KV head, one layer), appended in bulk, then one decode step
    n = 1_200_000
    a = np.asarray([[2], [1], [2], [1]], np.uint8)                      # every tag retained, half high half low
    z = np.zeros(a.shape, np.float32)
    pol = WP.Policy(4, 1, np.zeros(1, np.uint8), a, np.zeros_like(a), z, z.copy(), np.zeros(1, np.uint32), budget_target=1.0)
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, n_kv=1, n_q=4, n_layers=1, n_groups=1, batch=1, prompt_len=16, gen_len=16)
    w = WC.build(cfg)
    pages = n // 16 + 8
    P_ = pask
    gpu = P_.Cache(WP.write_blob(pol), 1, 4, 1, 1, n + 64, n + 64, pages, pages)
    orc = oracle.Cache(oracle.Policy(WP.write_blob(pol)), 4, 1, 1, pages, pages)
    from pask_workloads.tensors import bf16_bits, normal_bf16
    d = "cuda"
    k = normal_bf16(7, 1, 0, 0, 0, n, 1, d)
    v = normal_bf16(7, 2, 0, 0, 0, n, 1, d)
    tags = ((torch.arange(n, device=d) * 2654435761) >> 7).remainder(4).to(torch.uint8)
    ids = torch.zeros(1, dtype=torch.int32, device=d)
    cu = torch.tensor([0, n], dtype=torch.int32, device=d)
    P_.pask_append_kv(gpu.handle, 0, ids, cu, k, v, tags)
    rc, _ = orc.append(0, [0], [0, n], bf16_bits(k.cpu()).numpy(), bf16_bits(v.cpu()).numpy(), tags.cpu().numpy())
    assert rc == 0
    nh, nl = P_.pask_debug_stream_len(gpu.handle, 0, 0)
    assert (nh, nl) == orc.stream_len(0, 0) and (nh + 15) // 16 + (nl + 15) // 16 > 65536
    hi_g, lo_g = P_.pask_debug_page_ids(gpu.handle, 0, 0)
    _, _, hi_o = orc.dump_high(0, 0)
    assert np.array_equal(hi_g, hi_o)
    q = normal_bf16(7, 0, 0, 0, 0, 1, 4)
    out = torch.empty((1, 4, 128), dtype=torch.float32, device=d)
    lse = torch.empty((1, 4), dtype=torch.float32, device=d)
    P_.pask_decode_attention(gpu.handle, 0, ids, q.to(d), out, lse, gpu.workspace(1))
    torch.cuda.synchronize()
    oo, ol = orc.attention_batch(0, [0], bf16_bits(q).numpy())
    from parity import assert_close
    assert_close(out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), oo, ol, where="1.2M tokens")
    assert P_.pask_budget_state(gpu.handle, 0).device_status == 0
    gpu.close()
