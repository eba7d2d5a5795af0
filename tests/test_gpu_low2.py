"""GPU parity for the 2-bit variant of RETAIN-LOW (policy low_bits = 2: the levels -s, 0, +s): stored
codes and scales, page ids, budgets bit for bit; attention within the usual tolerance."""
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


def _pair(pask, oracle, n_kv=8, window=0, bias="balanced", batch=3, prompt=260, gen=180, n_layers=2, **kw):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, n_kv=n_kv, n_q=4 * n_kv, n_layers=n_layers, n_groups=2, batch=batch,
                    prompt_len=prompt, gen_len=gen, extra_gen=64, bias=bias)
    w = WC.build(cfg)
    blob = WP.write_blob(replace(w.policy, low_bits=2, recent_window=window))
    return Pair(pask, oracle, w, blob=blob, **kw), w


@pytest.mark.parametrize("n_kv,window,bias", [(8, 0, "balanced"), (2, 0, "low"), (1, 0, "low"), (4, 32, "balanced"), (8, 0, "low")])
def test_bulk_then_decode(pask, oracle, n_kv, window, bias):
    p, w = _pair(pask, oracle, n_kv=n_kv, window=window, bias=bias)
    sizes = pask.pask_cache_sizes(p.gpu.desc)
    assert sizes.low_page_bytes == n_kv * 1280
    seqs = [1, 0, 2]
    counts = [w.total_len(s) - 9 * i for i, s in enumerate(seqs)]
    for layer in range(2):
        p.append(layer, seqs, counts, [0, 0, 0])                        # bulk path: full pages through the shared-memory image
    p.compare_state()
    b = pask.pask_budget_state(p.gpu.handle, 0)
    assert b.retained_bytes == sum(b.n_high) * 2 * n_kv * 256 + sum(b.n_low) * 2 * n_kv * 40
    for layer in range(2):
        p.check_attention(layer, [0, 1, 2], pos=counts[0])
    pos = dict(zip(seqs, counts))
    for n in (1, 1, 1, 2, 19, 1, 1):                                    # one-launch path, pages filling up
        for layer in range(2):
            p.append(layer, seqs, [n] * 3, [pos[s] for s in seqs])
        pos = {s: pos[s] + n for s in pos}
        p.check_attention(n % 2, [2, 1, 0], pos=pos[0])
    p.compare_state()


def test_fused_step_and_decide_with_two_bit_costs(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, n_layers=4, n_groups=4, batch=3, prompt_len=200, gen_len=100, extra_gen=48)
    w = WC.build(cfg)
    from pask_workloads.policy import with_dynamic_budget
    full = cfg.n_layers * 2 * cfg.n_kv * 256
    pol = replace(with_dynamic_budget(w.policy, w.seed, full, 6), low_bits=2, budget_target=0.3)
    p = Pair(pask, oracle, w, blob=WP.write_blob(pol))
    seqs = [0, 2, 1]
    counts = [w.total_len(s) for s in seqs]
    tags, states = p.gather(seqs, counts, [0, 0, 0])
    _, act_o, act_g = p.decide(seqs, counts, tags, states)               # Demote / Promote count 2-bit bytes for L
    for layer in range(cfg.n_layers):
        _, _, k, v = p.gather(seqs, counts, [0, 0, 0], layer)
        p.append_decided(layer, seqs, counts, k, v, tags, act_o, act_g)
    p.compare_state()
    for s in range(3):
        g = pask.pask_budget_state(p.gpu.handle, s)
        assert g.retained_bytes == g.decided_retained_bytes
    # decode steps through the one-call form
    d = "cuda"
    from pask_workloads.tensors import bf16_bits
    from parity import assert_close
    pos = dict(zip(seqs, counts))
    for step in range(6):
        for layer in range(cfg.n_layers):
            tags, states, k, v = p.gather(seqs, [1, 1, 1], [pos[s] for s in seqs], layer)
            rc, _ = p.orc.append(layer, seqs, [0, 1, 2, 3], bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
            assert rc == 0
            q = torch.stack([w.q(layer, s, pos[s] + 1) for s in seqs])
            out = torch.empty((3, cfg.n_q, 128), dtype=torch.float32, device=d)
            lse = torch.empty((3, cfg.n_q), dtype=torch.float32, device=d)
            pask.pask_append_attend(p.gpu.handle, layer, torch.tensor(seqs, dtype=torch.int32, device=d),
                                    torch.arange(4, dtype=torch.int32, device=d), k.to(d), v.to(d),
                                    torch.from_numpy(tags).to(d), q.to(d), out, lse, p.gpu.workspace(3))
            torch.cuda.synchronize()
            oo, ol = p.orc.attention_batch(layer, seqs, bf16_bits(q).numpy())
            assert_close(out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), oo, ol, where=(step, layer))
        pos = {s: pos[s] + 1 for s in pos}
    p.compare_state()


def test_policy_and_cache_must_agree_on_the_width(pask):
    w = WC.build(WC.scaled(WC.QWEN3_4B_1LAYER, batch=1, prompt_len=16, gen_len=16))
    blob2 = WP.write_blob(replace(w.policy, low_bits=2))
    with pytest.raises(pask.PaskError) as e:
        pask.Cache(blob2, 4, 32, 8, 1, 64, 64, 16, 16, low_bits=4)
    assert e.value.status == pask.ERR_INVALID_ARG
    with pytest.raises(pask.PaskError) as e:
        pask.Cache(w.blob, 4, 32, 8, 1, 64, 64, 16, 16, low_bits=2)
    assert e.value.status == pask.ERR_INVALID_ARG
