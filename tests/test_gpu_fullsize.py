"""Parity at the benchmark's full size, in the launch configuration bench.py times: the Qwen3-4B
decode step (36 layers, 4 layer groups, batch 64, lengths U[2K, 8K], KV budget 0.33) is built
exactly as the benchmark builds it, one decode step is run, and sampled (layer, sequence) pairs
are compared with the oracle, which regenerates those slices from the same seeded generators.
What the oracle cannot recompute at this size is checked through properties that hold at any
size (page ids unique, counts consistent)."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from pask_workloads import configs as WC
from pask_workloads.tensors import TENSOR_K, TENSOR_V, bf16_bits, normal_bf16

from parity import assert_close

pytestmark = pytest.mark.gpu

LAYERS = (0, 9, 18, 35)


# the headline configuration in both of its call forms, and the longest sequences any configuration has (the
# concurrency-8, 32K-input shape of the paper's latency table: 33 792 tokens, 2112-entry page tables, deep splits)
@pytest.mark.parametrize("mode,base,SEQS", [("ahead", WC.QWEN3_4B_STEP, (0, 17, 42, 63)), ("fused", WC.QWEN3_4B_STEP, (0, 17, 42, 63)),
                                            ("ahead", WC.TABLE3_32K, (0, 3, 7))])
def test_full_size_decode_step_sampled_against_oracle(oracle, mode, base, SEQS):
    import bench
    import paper_2608_28276_b200 as P
    dev = torch.device("cuda", 0)
    cfg = WC.scaled(base, extra_gen=16)
    w = WC.build(cfg)
    job = bench.Job(P, w, dev, 6)
    job.fill()
    # "ahead": the call bench.py times by default -- planned-ahead steps; three of them, so that the last one streams from
    # a plan written by the step before and sets its pipeline up ahead of its dependency wait.  "fused": one
    # pask_append_attend per layer (the append launch carries the plan), bench.py --no-ahead.
    n_steps = 3 if mode == "ahead" else 1
    job.prepare_steps(n_steps)
    if mode == "ahead":
        job.plan_ahead()
    outs = {}
    h = job.cache.handle
    for step in range(n_steps):
        for layer, (k, v, q, tags) in enumerate(job.steps[step]):      # whole decode steps, keeping the last one's sampled outputs
            if mode == "ahead":
                P.pask_decode_step_ahead(h, layer, job.ids, k, v, tags, q, job.out, job.lse, job.ws, job.area)
            else:
                P.pask_append_attend(h, layer, job.ids, job.cu1, k, v, tags, q, job.out, job.lse, job.ws)
            if layer in LAYERS and step == n_steps - 1:
                outs[layer] = (job.out.cpu().numpy().astype(np.float64), job.lse.cpu().numpy().astype(np.float64))
    torch.cuda.synchronize()
    assert P.pask_budget_state(h, 0).device_status == 0

    # ---- the oracle on the sampled sequences: every layer for the counters, real K/V on sampled layers
    lens = [w.total_len(b) for b in SEQS]
    pages = cfg.n_layers * (sum(lens) // 16 + 8 * len(SEQS))
    orc = oracle.Cache(oracle.Policy(w.blob), cfg.n_q, cfg.n_kv, len(SEQS), pages, pages)
    ids = list(range(len(SEQS)))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    tags_hist = np.concatenate([w.tags(b, 0, n) for b, n in zip(SEQS, lens)])
    zeros = np.zeros((int(cu[-1]), cfg.n_kv, 128), np.uint16)
    zeros1 = np.zeros((len(SEQS), cfg.n_kv, 128), np.uint16)
    one = np.arange(len(SEQS) + 1, dtype=np.int32)
    for layer in range(cfg.n_layers):
        if layer in LAYERS:
            k = torch.cat([normal_bf16(w.seed, TENSOR_K, layer, b, 0, n, cfg.n_kv, dev) for b, n in zip(SEQS, lens)]).cpu()
            v = torch.cat([normal_bf16(w.seed, TENSOR_V, layer, b, 0, n, cfg.n_kv, dev) for b, n in zip(SEQS, lens)]).cpu()
            rc, _ = orc.append(layer, ids, cu, bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags_hist)
        else:
            rc, _ = orc.append(layer, ids, cu, zeros, zeros, tags_hist)
        assert rc == 0
        for step in range(n_steps):
            ks, vs, qs, st = bench.step_inputs(w, layer, step, "cpu")
            if layer in LAYERS:
                rc, _ = orc.append(layer, ids, one, bf16_bits(ks[list(SEQS)]).numpy(), bf16_bits(vs[list(SEQS)]).numpy(), st[list(SEQS)])
            else:
                rc, _ = orc.append(layer, ids, one, zeros1, zeros1, st[list(SEQS)])
            assert rc == 0

    # ---- budget states (all 36 layers of accounting), bit exact
    for i, b in enumerate(SEQS):
        g, o = P.pask_budget_state(h, b), orc.budget(i)
        for f in ("n_seen", "n_high", "n_low", "n_drop"):
            assert list(getattr(g, f)) == list(getattr(o, f)), (f, b)
        for f in ("retained_bytes", "full_bytes", "remaining_bytes", "bad_tags", "pages_high", "pages_low"):
            assert getattr(g, f) == getattr(o, f), (f, b)

    # ---- stored streams and attention on the sampled (layer, sequence) pairs
    for layer in LAYERS:
        q = bench.step_inputs(w, layer, n_steps - 1, "cpu")[2]
        oo, ol = orc.attention_batch(layer, ids, bf16_bits(q[list(SEQS)]).numpy())
        go, gl = outs[layer]
        assert_close(go[list(SEQS)], gl[list(SEQS)], oo, ol, where=("full size", layer))
        for i, b in enumerate(SEQS):
            assert P.pask_debug_stream_len(h, layer, b) == orc.stream_len(layer, i)
            for x, y in zip(P.pask_debug_dump_high(h, layer, b, cfg.n_kv)[:2], orc.dump_high(layer, i)[:2]):
                assert np.array_equal(x, y), ("high stream", layer, b)
            for x, y in zip(P.pask_debug_dump_low(h, layer, b, cfg.n_kv)[:4], orc.dump_low(layer, i)[:4]):
                assert np.array_equal(x, y), ("low stream", layer, b)

    # ---- properties that hold at any size: page ids are unique per pool and within the pools
    hi_next, hi_free, lo_next, lo_free = P.pask_debug_pool_state(h)
    assert hi_free == 0 and lo_free == 0
    seen_hi, seen_lo = [], []
    for layer in LAYERS:
        prev_first = -1
        for b in range(cfg.batch):
            ph, pl = P.pask_debug_page_ids(h, layer, b)
            nh, nl = P.pask_debug_stream_len(h, layer, b)
            assert len(ph) == (nh + 15) // 16 and len(pl) == (nl + 15) // 16
            seen_hi.append(ph); seen_lo.append(pl)
            if len(ph):                                   # the bulk fill numbered pages sequence-major
                assert ph[0] > prev_first
                prev_first = ph[0]
    for seen, nxt in ((np.concatenate(seen_hi), hi_next), (np.concatenate(seen_lo), lo_next)):
        assert len(np.unique(seen)) == len(seen) and seen.max() < nxt
    # all sequences: out finite, lse finite
    for layer in LAYERS:
        assert np.all(np.isfinite(outs[layer][0])) and np.all(np.isfinite(outs[layer][1]))
