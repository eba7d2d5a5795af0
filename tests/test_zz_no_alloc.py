"""pask_decode_attention_static: decode attention for callers that cannot allocate a workspace.

An engine that has already given all free device memory to its own block pool, or code running
where a device allocation is not allowed, cannot hand the library a scratch buffer. This entry
point uses a fixed scratch array built into the library instead. The test calls it through the
C ABI twice in a row and compares both results with the CPU oracle's attention over the same
history (the parity bound of every other attention test) and, as a second check, with
pask_decode_attention on the same cache.
(The file name makes pytest collect it after every other test.)"""
import numpy as np
import pytest
import torch

from pask_workloads import configs as WC

from pask_workloads.tensors import bf16_bits

from parity import ATOL_MAX, RTOL_L2, assert_close

pytestmark = pytest.mark.gpu


def test_static_workspace_matches_oracle_and_caller_workspace_twice_in_a_row(oracle):
    import paper_2608_28276_b200 as P
    assert torch.cuda.is_available()
    d = "cuda"
    cfg = WC.scaled(WC.QWEN3_4B_1LAYER, batch=3, n_layers=1, n_groups=1, prompt_len=700, gen_len=333)
    w = WC.build(cfg)
    lens = [w.total_len(b) for b in range(cfg.batch)]
    pages = sum(lens) // 16 + 16
    cache = P.Cache(w.blob, 1, cfg.n_q, cfg.n_kv, cfg.batch, max(lens) + 16, sum(lens), pages, pages)
    ids = torch.arange(cfg.batch, dtype=torch.int32, device=d)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device=d)
    k = torch.cat([w.kv(0, b, 0, lens[b])[0] for b in range(cfg.batch)]).to(d)
    v = torch.cat([w.kv(0, b, 0, lens[b])[1] for b in range(cfg.batch)]).to(d)
    tags = torch.from_numpy(np.concatenate([w.tags(b, 0, lens[b]) for b in range(cfg.batch)])).to(d)
    P.pask_append_kv(cache.handle, 0, ids, cu, k, v, tags)
    assert P.pask_budget_state(cache.handle, 0).device_status == 0
    orc = oracle.Cache(oracle.Policy(w.blob), cfg.n_q, cfg.n_kv, cfg.batch, pages, pages)
    rc, _ = orc.append(0, list(range(cfg.batch)), cu.cpu().numpy(), bf16_bits(k.cpu()).numpy(), bf16_bits(v.cpu()).numpy(),
                       tags.cpu().numpy())
    assert rc == 0

    def run(fn, q, *extra):
        out = torch.full((cfg.batch, cfg.n_q, 128), float("nan"), dtype=torch.float32, device=d)
        lse = torch.full((cfg.batch, cfg.n_q), float("nan"), dtype=torch.float32, device=d)
        fn(cache.handle, 0, ids, q, out, lse, *extra)
        torch.cuda.synchronize()
        return out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)

    assert P.pask_workspace_bytes(cache.handle, cfg.batch) <= P.STATIC_WORKSPACE_BYTES
    for call in range(2):                                   # two calls in a row, different queries
        q = torch.stack([w.q(0, b, lens[b] + call) for b in range(cfg.batch)]).to(d)
        ref_out, ref_lse = run(P.pask_decode_attention, q, cache.workspace(cfg.batch))
        got_out, got_lse = run(P.pask_decode_attention_static, q)
        orc_out, orc_lse = orc.attention_batch(0, list(range(cfg.batch)), bf16_bits(q.cpu()).numpy())
        assert_close(got_out, got_lse, orc_out, orc_lse, where=("static scratch vs oracle, call", call))
        for b in range(cfg.batch):
            assert np.abs(got_out[b] - ref_out[b]).max() <= ATOL_MAX
            assert np.linalg.norm(got_out[b] - ref_out[b]) <= RTOL_L2 * np.linalg.norm(ref_out[b])
        assert np.abs(got_lse - ref_lse).max() <= 1e-3

    # a batch whose partials do not fit the built-in scratch is refused, nothing is launched
    P.pask_debug_set_attention_ctas(cache.handle, 4096)
    assert P.pask_workspace_bytes(cache.handle, cfg.batch) > P.STATIC_WORKSPACE_BYTES
    out = torch.zeros((cfg.batch, cfg.n_q, 128), dtype=torch.float32, device=d)
    with pytest.raises(P.PaskError) as e:
        P.pask_decode_attention_static(cache.handle, 0, ids, q, out, None)
    assert e.value.status == P.ERR_WORKSPACE
    cache.close()
