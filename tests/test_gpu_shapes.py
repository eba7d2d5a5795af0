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
