"""Drive the CPU oracle and the CUDA library side by side on one seeded workload and compare.

Decisions, codes, scales, page ids and counters must agree bit for bit; attention outputs within
max-abs 2e-3 and relative L2 1e-3 per (sequence, layer) tensor [n_q, 128] against the fp64 oracle.
"""
from __future__ import annotations

import numpy as np
import torch

from pask_workloads.tensors import bf16_bits

ATOL_MAX = 2e-3
RTOL_L2 = 1e-3


class Pair:
    def __init__(self, pask, oracle, workload, max_seqs=None, pool_high_pages=None, pool_low_pages=None,
                 max_tokens_per_seq=None, max_append_tokens=None, blob=None):
        self.pask, self.oracle, self.w = pask, oracle, workload
        cfg = workload.cfg
        self.cfg = cfg
        self.max_seqs = max_seqs or cfg.batch
        longest = max(workload.total_len(b) for b in range(cfg.batch)) + cfg.extra_gen
        self.max_tokens = max_tokens_per_seq or longest
        total = sum(workload.total_len(b) + cfg.extra_gen for b in range(cfg.batch))
        pages = cfg.n_layers * (total // 16 + 2 * cfg.batch)
        self.hp = pool_high_pages if pool_high_pages is not None else pages
        self.lp = pool_low_pages if pool_low_pages is not None else pages
        blob = blob or workload.blob
        window = int.from_bytes(blob[28:32], "little")                  # the policy's protected recent window
        self.gpu = pask.Cache(blob, cfg.n_layers, cfg.n_q, cfg.n_kv, self.max_seqs, self.max_tokens,
                              max_append_tokens or total, self.hp, self.lp, recent_window=window,
                              low_bits=int.from_bytes(blob[32:36], "little"))
        self.orc = oracle.Cache(oracle.Policy(blob), cfg.n_q, cfg.n_kv, self.max_seqs, self.hp, self.lp)

    # ------------------------------------------------------------------ append
    def append(self, layer, seq_ids, counts, starts, expect_ok=True, k=None, v=None, tags=None):
        """Append tokens starts[i] .. starts[i]+counts[i]-1 of each sequence to both sides."""
        w = self.w
        cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        if k is None:
            ks, vs, ts = [], [], []
            for s, n, t0 in zip(seq_ids, counts, starts):
                kk, vv = w.kv(layer, int(s), int(t0), int(n))
                ks.append(kk); vs.append(vv); ts.append(w.tags(int(s), int(t0), int(n)))
            k = torch.cat(ks) if ks else torch.empty((0, self.cfg.n_kv, 128), dtype=torch.bfloat16)
            v = torch.cat(vs) if vs else torch.empty((0, self.cfg.n_kv, 128), dtype=torch.bfloat16)
            tags = np.concatenate(ts) if ts else np.zeros(0, np.uint8)
        rc, act_o = self.orc.append(layer, seq_ids, cu, bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
        d = "cuda"
        act_g = torch.full((max(1, len(tags)),), 0xEE, dtype=torch.uint8, device=d)
        self.pask.pask_append_kv(self.gpu.handle, layer, torch.tensor(seq_ids, dtype=torch.int32, device=d),
                                 torch.from_numpy(cu).to(d), k.to(d), v.to(d), torch.from_numpy(tags).to(d),
                                 actions_out=act_g, total_tokens=len(tags))
        torch.cuda.synchronize()
        if expect_ok:
            assert rc == 0
            assert np.array_equal(act_g.cpu().numpy()[:len(tags)], act_o), "actions differ"
        return rc, act_o

    # ------------------------------------------------------------------ dynamic budget adjustment
    def gather(self, seq_ids, counts, starts, layer=None):
        """tags, states (and k, v of `layer`) of tokens starts[i] .. +counts[i]-1, call order."""
        w = self.w
        ts = [w.tags(int(s), int(t0), int(n)) for s, n, t0 in zip(seq_ids, counts, starts)]
        ss = [w.states(int(s), int(t0), int(n)) for s, n, t0 in zip(seq_ids, counts, starts)]
        tags = np.concatenate(ts) if ts else np.zeros(0, np.uint8)
        states = np.concatenate(ss) if ss else np.zeros(0, np.uint16)
        if layer is None:
            return tags, states
        kv = [w.kv(layer, int(s), int(t0), int(n)) for s, n, t0 in zip(seq_ids, counts, starts)]
        return tags, states, torch.cat([a for a, _ in kv]), torch.cat([b for _, b in kv])

    def decide(self, seq_ids, counts, tags, states, expect_ok=True):
        """pask_decide on both sides; returns (oracle status, oracle actions, gpu actions tensor)."""
        d = "cuda"
        cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        G = self.cfg.n_groups
        rc, act_o = self.orc.decide(seq_ids, cu, tags, states=states, n_groups=G)
        act_g = torch.full((max(1, len(tags)), G), 0xEE, dtype=torch.uint8, device=d)
        st = None if states is None else torch.from_numpy(states.astype(np.int16)).to(d)
        self.pask.pask_decide(self.gpu.handle, torch.tensor(seq_ids, dtype=torch.int32, device=d),
                              torch.from_numpy(cu).to(d), torch.from_numpy(tags).to(d), st, act_g)
        torch.cuda.synchronize()
        if expect_ok:
            assert rc == 0
            assert np.array_equal(act_g.cpu().numpy()[:len(tags)], act_o), "decided actions differ"
        return rc, act_o, act_g

    def append_decided(self, layer, seq_ids, counts, k, v, tags, act_o, act_g, expect_ok=True):
        d = "cuda"
        cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
        rc, used_o = self.orc.append(layer, seq_ids, cu, bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags, decided=act_o)
        used_g = torch.full((max(1, len(tags)),), 0xEE, dtype=torch.uint8, device=d)
        self.pask.pask_append_kv_decided(self.gpu.handle, layer, torch.tensor(seq_ids, dtype=torch.int32, device=d),
                                         torch.from_numpy(cu).to(d), k.to(d), v.to(d), torch.from_numpy(tags).to(d),
                                         act_g, actions_out=used_g, total_tokens=len(tags))
        torch.cuda.synchronize()
        if expect_ok:
            assert rc == 0
            assert np.array_equal(used_g.cpu().numpy()[:len(tags)], used_o), "persisted actions differ"
        return rc

    # ------------------------------------------------------------------ state
    def compare_state(self, layers=None, seqs=None, expect_status=0):
        P, h = self.pask, self.gpu.handle
        layers = range(self.cfg.n_layers) if layers is None else layers
        seqs = range(self.max_seqs) if seqs is None else seqs
        for s in seqs:
            for l in layers:
                assert P.pask_debug_stream_len(h, l, s) == self.orc.stream_len(l, s), (l, s)
                gk, gv, gp = P.pask_debug_dump_high(h, l, s, self.cfg.n_kv)
                ok, ov, op = self.orc.dump_high(l, s)
                assert np.array_equal(gp, op), ("high page ids", l, s, gp[:8], op[:8])
                assert np.array_equal(gk, ok), ("high K", l, s)
                assert np.array_equal(gv, ov), ("high V", l, s)
                gkc, gks, gvc, gvs, gpl = P.pask_debug_dump_low(h, l, s, self.cfg.n_kv)
                okc, oks, ovc, ovs, opl = self.orc.dump_low(l, s)
                assert np.array_equal(gpl, opl), ("low page ids", l, s)
                assert np.array_equal(gks, oks), ("low K scales", l, s)
                assert np.array_equal(gvs, ovs), ("low V scales", l, s)
                assert np.array_equal(gkc, okc), ("low K codes", l, s)
                assert np.array_equal(gvc, ovc), ("low V codes", l, s)
            self.compare_budget(s, expect_status=expect_status)
        assert P.pask_debug_pool_state(h) == self.orc.pool_state()

    def compare_budget(self, s, expect_status=0):
        g, o = self.pask.pask_budget_state(self.gpu.handle, s), self.orc.budget(s)
        for f in ("n_seen", "n_high", "n_low", "n_drop"):
            assert list(getattr(g, f)) == list(getattr(o, f)), (f, s)
        for f in ("retained_bytes", "full_bytes", "remaining_bytes", "bad_tags", "pages_high", "pages_low",
                  "decided_full_bytes", "decided_retained_bytes", "n_demoted", "n_promoted", "n_floor_conflicts"):
            assert getattr(g, f) == getattr(o, f), (f, s, getattr(g, f), getattr(o, f))
        assert g.device_status == expect_status, g.device_status
        return g

    # ------------------------------------------------------------------ attention
    def attention(self, layer, seq_ids, pos=None, full=False, q=None):
        """Decode attention for the given sequences on both sides; returns (gpu out, gpu lse,
        oracle out, oracle lse)."""
        w, d = self.w, "cuda"
        if q is None:
            q = torch.stack([w.q(layer, int(s), w.total_len(int(s)) if pos is None else pos) for s in seq_ids])
        n = len(seq_ids)
        out = torch.full((n, self.cfg.n_q, 128), float("nan"), dtype=torch.float32, device=d)
        lse = torch.full((n, self.cfg.n_q), float("nan"), dtype=torch.float32, device=d)
        fn = self.pask.pask_decode_attention_full if full else self.pask.pask_decode_attention
        fn(self.gpu.handle, layer, torch.tensor(seq_ids, dtype=torch.int32, device=d), q.to(d), out, lse,
           self.gpu.workspace(n))
        torch.cuda.synchronize()
        oo, ol = self.orc.attention_batch(layer, seq_ids, bf16_bits(q).numpy())
        return out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), oo, ol

    def check_attention(self, layer, seq_ids, **kw):
        go, gl, oo, ol = self.attention(layer, seq_ids, **kw)
        assert_close(go, gl, oo, ol, where=(layer, list(seq_ids)))
        return go, oo


def assert_close(go, gl, oo, ol, where=""):
    assert np.all(np.isfinite(go)), ("non-finite output", where)
    for i in range(go.shape[0]):
        err = np.abs(go[i] - oo[i]).max()
        den = np.linalg.norm(oo[i])
        rel = np.linalg.norm(go[i] - oo[i]) / den if den > 0 else np.linalg.norm(go[i])
        assert err <= ATOL_MAX, ("max-abs", err, where, i)
        assert rel <= RTOL_L2, ("rel-L2", rel, where, i)
        fin = np.isfinite(ol[i])
        assert np.array_equal(np.isfinite(gl[i]), fin), ("lse finiteness", where, i)
        if fin.any():
            assert np.abs(gl[i][fin] - ol[i][fin]).max() <= 1e-3, ("lse", where, i)


def error_stats(go, oo):
    rel = [np.linalg.norm(go[i] - oo[i]) / max(np.linalg.norm(oo[i]), 1e-300) for i in range(go.shape[0])]
    return float(np.abs(go - oo).max()), float(max(rel))
