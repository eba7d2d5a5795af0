"""GPU parity of pask_distortion (Eq. 4's inner term) and its use on the kernel pair: the outputs of
the full high-precision kernel against the outputs under a policy."""
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


@pytest.mark.parametrize("rows,n_q", [(1, 8), (37, 32), (300, 4)])
def test_matches_oracle(pask, oracle, rows, n_q):
    g = torch.Generator().manual_seed(rows)
    a = torch.randn((rows, n_q, 128), generator=g)
    b = a + 0.05 * torch.randn((rows, n_q, 128), generator=g)
    per = torch.full((rows,), float("nan"), device="cuda")
    acc = torch.full((1,), 2.5, dtype=torch.float64, device="cuda")      # the sum is added to what is there
    pask.pask_distortion(a.cuda(), b.cuda(), per, acc)
    want, total = oracle.distortion(a.numpy(), b.numpy())
    got = per.cpu().numpy().astype(np.float64)
    assert np.abs(got - want).max() <= 1e-5 * want.max()                  # fp32 sums of 128 squares
    assert abs(acc.item() - 2.5 - total) <= 1e-5 * total
    pask.pask_distortion(a.cuda(), a.cuda(), per, None)
    assert torch.all(per == 0)


def test_distortion_of_a_policy_against_the_full_cache(pask, oracle):
    # the same history in an all-high cache and under the budget-0.33 table: D > 0 for the policy,
    # exactly 0 for the all-high cache against itself, and the GPU figure agrees with the oracle's
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, prompt_len=300, gen_len=200, extra_gen=16)
    w = WC.build(cfg)
    full_blob = WP.write_blob(WP.all_high_policy(w.policy.n_tags, cfg.n_groups, cfg.n_layers))
    pol, full = Pair(pask, oracle, w), Pair(pask, oracle, w, blob=full_blob)
    lens = [w.total_len(b) for b in range(3)]
    acc = torch.zeros(1, dtype=torch.float64, device="cuda")
    total_o = 0.0
    for layer in range(cfg.n_layers):
        for p in (pol, full):
            p.append(layer, [0, 1, 2], lens, [0, 0, 0])
        go_p, _, oo_p, _ = pol.attention(layer, [0, 1, 2])
        go_f, _, oo_f, _ = full.attention(layer, [0, 1, 2], full=True)
        a, b = torch.from_numpy(go_f).float().cuda(), torch.from_numpy(go_p).float().cuda()
        per = torch.empty(3, device="cuda")
        pask.pask_distortion(a, b, per, acc)
        want, tot = oracle.distortion(oo_f.astype(np.float32), oo_p.astype(np.float32))
        total_o += tot
        assert np.all(want > 0)
        # both sides carry the attention tolerance (2e-3 per element) into the difference
        assert np.abs(per.cpu().numpy() - want).max() <= 0.05 * want.max() + 1e-4
    assert acc.item() > 0 and abs(acc.item() - total_o) <= 0.05 * total_o + 1e-3
