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
