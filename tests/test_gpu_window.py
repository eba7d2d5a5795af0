"""GPU parity with a protected recent window W > 0: the last W tokens are attended at full
precision whatever their action; streams, page ids and budget states stay those of W = 0."""
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


def _pair(pask, oracle, window, batch=3, prompt=150, gen=90, budget=0.33, **kw):
    from dataclasses import replace
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=batch, prompt_len=prompt, gen_len=gen, extra_gen=48, budget=budget)
    w = WC.build(cfg)
    blob = WP.write_blob(replace(w.policy, recent_window=window))
    return Pair(pask, oracle, w, blob=blob, **kw), w


@pytest.mark.parametrize("window", [16, 64, 256])
def test_prefill_then_decode(pask, oracle, window):
    p, w = _pair(pask, oracle, window)
    cfg = w.cfg
    seqs = [1, 2, 0]
    counts = [w.total_len(s) - 11 * i for i, s in enumerate(seqs)]
    for layer in range(cfg.n_layers):
        p.append(layer, seqs, counts, [0, 0, 0])                        # the bulk path fills the ring with the last W
    p.compare_state()
    for layer in range(cfg.n_layers):
        p.check_attention(layer, [0, 1, 2], pos=counts[0])
    pos = dict(zip(seqs, counts))
    for step in range(window + 5 if window < 64 else 24):               # the ring wraps around
        for layer in range(cfg.n_layers):
            p.append(layer, seqs, [1, 1, 1], [pos[s] for s in seqs])    # the one-launch decode path
        for s in seqs:
            pos[s] += 1
        if step % 5 == 0:
            p.check_attention(step % cfg.n_layers, [2, 0, 1], pos=pos[0])
    p.compare_state()
    for layer in range(cfg.n_layers):
        p.check_attention(layer, [0, 1, 2], pos=pos[0])


def test_window_not_yet_full_and_short_calls(pask, oracle):
    # fewer tokens than W, a few at a time through the one-launch path: partly filled ring pages
    p, w = _pair(pask, oracle, 64, batch=2, prompt=40, gen=20)
    pos = {0: 0, 1: 0}
    for n in (1, 3, 16, 5, 17, 9):
        for layer in range(w.cfg.n_layers):
            p.append(layer, [0, 1], [n, n], [pos[0], pos[1]])
        pos = {s: pos[s] + n for s in pos}
        for layer in range(w.cfg.n_layers):
            p.check_attention(layer, [1, 0], pos=pos[0])
    p.compare_state()


def test_everything_released_leaves_only_the_window(pask, oracle):
    a = np.zeros((11, 4), np.uint8)
    z = np.zeros((11, 4), np.float32)
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=2, prompt_len=100, gen_len=60, extra_gen=16)
    w = WC.build(cfg)
    pol = WP.Policy(11, 4, WP.equal_layer_groups(4, 4), a, a.copy(), z, z.copy(), np.zeros(1, np.uint32),
                    budget_target=0.0, recent_window=32)
    p = Pair(pask, oracle, w, blob=WP.write_blob(pol))
    for layer in range(4):
        p.append(layer, [0, 1], [160, 150], [0, 0])
        assert pask.pask_debug_stream_len(p.gpu.handle, layer, 0) == (0, 0)
        go, _ = p.check_attention(layer, [0, 1], pos=160)
        assert np.abs(go).max() > 0                                     # 32 window tokens are attended
    p.compare_state()


def test_full_kv_kernel_and_sequence_reset_with_a_window(pask, oracle):
    from dataclasses import replace
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=2, prompt_len=70, gen_len=30, extra_gen=16, lut="all_high")
    w = WC.build(cfg)
    p = Pair(pask, oracle, w, blob=WP.write_blob(replace(w.policy, recent_window=48)))
    for layer in range(cfg.n_layers):
        p.append(layer, [0, 1], [100, 100], [0, 0])
    p.check_attention(0, [0, 1], pos=100, full=True)                    # all-high: window members sit in both places
    pask.pask_seq_reset(p.gpu.handle, 1)
    p.orc.seq_reset(1)
    for layer in range(cfg.n_layers):
        p.append(layer, [1], [5], [0])                                  # starts again with an empty window
    p.check_attention(1, [1, 0], pos=5)
    p.compare_state()


def test_window_must_match_between_policy_and_cache(pask):
    from dataclasses import replace
    w = WC.build(WC.scaled(WC.QWEN3_4B_1LAYER, batch=1, prompt_len=16, gen_len=16))
    blob = WP.write_blob(replace(w.policy, recent_window=32))
    with pytest.raises(pask.PaskError) as e:
        pask.Cache(blob, 4, 32, 8, 1, 64, 64, 16, 16, recent_window=16)
    assert e.value.status == pask.ERR_INVALID_ARG
    sizes0 = pask.pask_cache_sizes(pask.CacheDesc(4, 32, 8, 128, 16, 2, 64, 64, 16, 16, 0))
    sizes32 = pask.pask_cache_sizes(pask.CacheDesc(4, 32, 8, 128, 16, 2, 64, 64, 16, 16, 32))
    assert sizes32.pool_high_bytes - sizes0.pool_high_bytes == 2 * 4 * 2 * sizes0.high_page_bytes
