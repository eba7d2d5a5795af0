"""The decode-attention kernel's bounded wait, made to run out in the safe form.

The kernel's only device-side waits are for its own bulk copies into shared memory.  Nothing is
made to go wrong on the GPU here: `pask_debug_set_wait` shortens the limit and lets every warp
announce, for its first copy, a few bytes more than the copy brings.  The copy lands as always; the
barrier cannot complete; the wait gives up after the limit.  The call must return, the sticky
status must carry PASK_DEV_TIMEOUT, the outputs must be finite (the merge skips the abandoned
partials), and after a reset the same cache must give the oracle's results again."""
import numpy as np
import pytest
import torch

from pask_workloads import configs as WC

from parity import Pair

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def pask():
    import paper_2608_28276_b200 as P
    assert torch.cuda.is_available()
    return P


@pytest.mark.parametrize("full", [False, True])
def test_a_wait_that_runs_out_reports_and_leaves_the_cache_usable(pask, oracle, full):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=1, n_groups=1, prompt_len=300, gen_len=200,
                    **({"lut": "all_high", "budget": 1.0} if full else {}))
    w = WC.build(cfg)
    p = Pair(pask, oracle, w)
    seqs = [0, 1, 2]
    lens = [w.total_len(s) for s in seqs]
    P, h = pask, p.gpu.handle

    def fill():
        p.append(0, seqs, lens, [0, 0, 0])

    fill()
    p.check_attention(0, seqs, full=full)                       # the normal path first

    P.pask_debug_set_wait(h, 100_000, 16)                       # ~50 us limit, 16 bytes announced that never come
    d = "cuda"
    q = torch.stack([w.q(0, s, lens[s]) for s in seqs]).to(d)
    out = torch.full((3, cfg.n_q, 128), float("nan"), dtype=torch.float32, device=d)
    lse = torch.full((3, cfg.n_q), float("nan"), dtype=torch.float32, device=d)
    fn = P.pask_decode_attention_full if full else P.pask_decode_attention
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    fn(h, 0, torch.tensor(seqs, dtype=torch.int32, device=d), q, out, lse, p.gpu.workspace(3))
    t1.record()
    torch.cuda.synchronize()                                    # the call returns
    assert t0.elapsed_time(t1) < 1000.0                         # and well within a second
    st = P.pask_budget_state(h, 0)
    assert st.device_status & P.DEV_TIMEOUT
    assert bool(torch.isfinite(out).all())                      # abandoned partials are skipped, not merged
    assert bool((out == 0).all()) and bool(torch.isinf(lse).all())   # every warp gave up before its first page

    # back to normal: reset clears the sticky bit, the same cache serves the oracle's results again
    P.pask_debug_set_wait(h)
    P.pask_cache_reset(h)
    p.orc = oracle.Cache(oracle.Policy(w.blob), cfg.n_q, cfg.n_kv, p.max_seqs, p.hp, p.lp)
    torch.cuda.synchronize()
    assert P.pask_budget_state(h, 0).device_status == 0
    fill()
    p.check_attention(0, seqs, full=full)
    p.compare_state()


def test_wait_setter_refuses_nonsense(pask, oracle):
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=1, n_layers=1, n_groups=1, prompt_len=32, gen_len=16)
    p = Pair(pask, oracle, WC.build(cfg))
    for limit, surplus in ((0, 0), (100_000, 8), (100_000, 1 << 20)):
        with pytest.raises(pask.PaskError) as e:
            pask.pask_debug_set_wait(p.gpu.handle, limit, surplus)
        assert e.value.status == pask.ERR_INVALID_ARG
