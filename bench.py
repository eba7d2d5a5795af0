#!/usr/bin/env python
"""Benchmark of the PASK online hot path on B200.

A step is one decode step of the whole path for one batch: for every layer, pask_append_kv of
the new token of each sequence (table lookup, drop / int4 / bf16 persist, paging, budget state)
followed by pask_decode_attention over the mixed-precision cache. The default workload is the
Qwen3-4B full decode step (36 layers, 4 layer groups, batch 64, sequence lengths uniform in
[2K, 8K], KV budget 0.33); metric = decode tokens/s (batch / step time).

    python bench.py --gpus 1 --steps 20 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N   (weak scaling: every
        rank runs its own batch, no collective on the data path)
    python bench.py --impl reference      times the CPU oracle on a bounded sample instead

Prints one JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from pask_workloads import configs as WC                      # noqa: E402
from pask_workloads.tensors import TENSOR_K, TENSOR_Q, TENSOR_V, normal_bf16, bf16_bits  # noqa: E402

METRIC = "mixed-KV decode-attn tokens/s at KV budget 0.33"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) over algorithmic bytes of the streaming kernel, from the ncu capture
# summarised in profiles/decode_attn_kernel__qwen3-4b-step-first-4-layers.md (mean of three launches
# of a 4-layer cut of this workload; traffic grows in proportion to the pages streamed)
NCU_TRAFFIC_RATIO = 1.009
NCU_TRAFFIC_PROFILE = "profiles/decode_attn_kernel__qwen3-4b-step-first-4-layers.md"
STEP_STREAM = 1_000_000          # decode-step inputs of step i come from generator stream (layer, STEP_STREAM + i)

CONFIGS = {c.name: c for c in WC.CONFIGS}
DEFAULT_CONFIG = WC.QWEN3_4B_STEP.name


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ------------------------------------------------------------------------------------------------
# workload bookkeeping (host side, inputs only)

def stream_counts(w):
    """Tokens each (sequence, layer group) keeps at high / low precision, from tags and table."""
    pol = w.policy
    eff = np.maximum(pol.a0, pol.a_floor)
    B, G = w.cfg.batch, pol.n_groups
    nh = np.zeros((B, G), np.int64)
    nl = np.zeros((B, G), np.int64)
    for b in range(B):
        tags = w.tags(b, 0, w.total_len(b))
        prot = tags == 0xFF
        known = tags[~prot]
        cnt = np.bincount(known[known < pol.n_tags], minlength=pol.n_tags)
        unknown = int((known >= pol.n_tags).sum()) + int(prot.sum())
        for g in range(G):
            nh[b, g] = int(cnt[eff[:, g] == 2].sum()) + unknown
            nl[b, g] = int(cnt[eff[:, g] == 1].sum())
    return nh, nl


def step_inputs(w, layer, step, device):
    """K, V, Q and tags of decode step `step` at `layer` for the whole batch (row b = sequence b)."""
    cfg = w.cfg
    k = normal_bf16(w.seed, TENSOR_K, layer, STEP_STREAM + step, 0, cfg.batch, cfg.n_kv, device)
    v = normal_bf16(w.seed, TENSOR_V, layer, STEP_STREAM + step, 0, cfg.batch, cfg.n_kv, device)
    q = normal_bf16(w.seed, TENSOR_Q, layer, STEP_STREAM + step, 0, cfg.batch, cfg.n_q, device)
    tags = np.array([w.gen_tags[b][w.gen_len(b) + step] for b in range(cfg.batch)], np.uint8)
    return k, v, q, tags


def max_over_ranks(x: float, device) -> float:
    """MAX of a per-rank scalar over the job (identity on one rank). Works on NCCL and gloo groups."""
    if torch.distributed.is_available() and torch.distributed.is_initialized() and torch.distributed.get_world_size() > 1:
        t = torch.tensor([x], dtype=torch.float64, device=device)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        return float(t.item())
    return float(x)


def whole_job_tokens_per_s(world: int, batch_per_rank: int, steps: int, max_ms: float) -> float:
    """Every rank decodes its own batch (weak scaling): units all ranks processed / slowest rank's time."""
    return world * batch_per_rank * steps / (max_ms * 1e-3)


def rank_workload(cfg, rank: int):
    """Rank r runs its own sequences: the same configuration, seed offset by the rank."""
    return WC.build(cfg, repeat=rank)


def kernel_events(n_layers, n_steps, stride):
    """CUDA-event pairs for timing the streaming kernel live inside the timed region. Recording an
    event between two kernels gives up the launch overlap of that pair, so only every `stride`-th
    launch is timed, rotating over the layers from step to step (every layer is covered)."""
    evs = []
    for s in range(n_steps):
        row = {l: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for l in range(n_layers) if (l + s) % stride == 0}
        for a, b in row.values():
            a.record(); b.record()          # creates the CUDA handles before they are handed to the library
        evs.append(row)
    return evs


def kernel_spans(n_layers, n_steps, stride, device):
    """Device words for the in-kernel timing of launches that carry NO events (so that they overlap their launch
    with their neighbours as in the un-timed step): per step {layer: int64[2] preset to (all ones, 0)}."""
    out = []
    for s in range(n_steps):
        out.append({l: torch.tensor([-1, 0], dtype=torch.int64, device=device)
                    for l in range(n_layers) if (l + s) % stride == stride // 2 and stride > 1})
    return out


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 20 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [r.split(", ") for r in open(self.path).read().strip().splitlines() if r.strip()]
            os.unlink(self.path)
            sm = [float(r[0]) for r in rows]
            out["sm_mhz"] = statistics.median(sm) if sm else None
            out["sm_max_mhz"] = float(rows[0][1]) if rows else None
            out["power_w_max"] = max(float(r[2]) for r in rows) if rows else None
            out["samples"] = len(rows)
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            for i, nme in enumerate(names):
                if any(r[4 + i].strip().lower().startswith("active") for r in rows):
                    out["reasons"].append(nme)
        except Exception:
            pass
        return out


# ------------------------------------------------------------------------------------------------
# the CUDA arm

class Job:
    """One rank's cache, filled with the workload's history, ready to run decode steps."""

    def __init__(self, P, w, device, total_steps, policy_blob=None, label="pask", dynamic=False):
        self.P, self.w, self.device, self.label = P, w, device, label
        self.dynamic = dynamic
        cfg = w.cfg
        self.cfg = cfg
        self.B = cfg.batch
        blob = policy_blob or w.blob
        nh, nl = stream_counts(w)
        if policy_blob is not None:                      # the all-high comparison cache
            tot = np.array([w.total_len(b) for b in range(self.B)], np.int64)
            nh = np.repeat(tot[:, None], w.policy.n_groups, axis=1)
            nl = np.zeros_like(nh)
        if dynamic:
            # actions depend on the running budget: size both pools for the worst case (the
            # realised counts are read back from the budget states after the fill)
            blob = w.dynamic_blob()
            tot = np.array([w.total_len(b) for b in range(self.B)], np.int64)
            nh = np.repeat(tot[:, None], w.policy.n_groups, axis=1)
            nl = nh.copy()
        self.nh, self.nl = nh, nl
        lg = w.policy.layer_group.astype(np.int64)
        extra = total_steps + 1
        pages_h = int(sum(((nh[:, lg[l]] + extra + 15) // 16).sum() for l in range(cfg.n_layers))) + 64
        pages_l = int(sum(((nl[:, lg[l]] + extra + 15) // 16).sum() for l in range(cfg.n_layers))) + 64
        self.lens = [w.total_len(b) for b in range(self.B)]
        self.total_tokens = int(sum(self.lens))
        self.window = int.from_bytes(blob[28:32], "little")
        self.low_bits = int.from_bytes(blob[32:36], "little")
        self.cache = P.Cache(blob, cfg.n_layers, cfg.n_q, cfg.n_kv, self.B, max(self.lens) + extra + 16,
                             self.total_tokens, pages_h, pages_l, device=device, recent_window=self.window,
                             low_bits=self.low_bits)
        self.ids = torch.arange(self.B, dtype=torch.int32, device=device)
        self.cu1 = torch.arange(self.B + 1, dtype=torch.int32, device=device)
        self.ws = self.cache.workspace(self.B)
        self.out = torch.empty((self.B, cfg.n_q, 128), dtype=torch.float32, device=device)
        self.lse = torch.empty((self.B, cfg.n_q), dtype=torch.float32, device=device)
        self.attn = P.pask_decode_attention_full if policy_blob is not None else P.pask_decode_attention
        self.fused = False
        self.ahead = False          # planned-ahead steps (pask_decode_step_ahead): set by plan_ahead()
        self.area = None

    def plan_ahead(self):
        """Plan every layer's next decode step from the cache as it stands; run_step then uses pask_decode_step_ahead."""
        self.area = torch.empty(self.P.pask_plan_area_bytes(self.cache.handle, self.B), dtype=torch.uint8, device=self.device)
        for layer in range(self.cfg.n_layers):
            self.P.pask_plan_ahead(self.cache.handle, layer, self.ids, self.area)
        self.ahead = True

    def fill(self):
        """Append the whole history, one ragged bulk call per layer (generated on the device)."""
        w, cfg, d = self.w, self.cfg, self.device
        cu = torch.tensor(np.concatenate([[0], np.cumsum(self.lens)]), dtype=torch.int32, device=d)
        tags = torch.from_numpy(np.concatenate([w.tags(b, 0, self.lens[b]) for b in range(self.B)])).to(d)
        decided = None
        if self.dynamic:
            states = torch.from_numpy(np.concatenate([w.states(b, 0, self.lens[b]) for b in range(self.B)]).astype(np.int16)).to(d)
            decided = torch.empty((self.total_tokens, cfg.n_groups), dtype=torch.uint8, device=d)
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            self.P.pask_decide(self.cache.handle, self.ids, cu, tags, states, decided)
            b_.record()
            torch.cuda.synchronize()
            self.prefill_decide_ms = a.elapsed_time(b_)
        evs = []
        for layer in range(cfg.n_layers):
            k = torch.cat([normal_bf16(w.seed, TENSOR_K, layer, b, 0, self.lens[b], cfg.n_kv, d) for b in range(self.B)])
            v = torch.cat([normal_bf16(w.seed, TENSOR_V, layer, b, 0, self.lens[b], cfg.n_kv, d) for b in range(self.B)])
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if decided is None:
                self.P.pask_append_kv(self.cache.handle, layer, self.ids, cu, k, v, tags)
            else:
                self.P.pask_append_kv_decided(self.cache.handle, layer, self.ids, cu, k, v, tags, decided)
            b_.record()
            evs.append((a, b_))
            del k, v
        torch.cuda.synchronize()
        # bulk (prefill-style) append: one ragged call per layer over the whole history; layer 0 is the warm-up
        self.fill_ms = [a.elapsed_time(b_) for a, b_ in evs]
        st = self.P.pask_budget_state(self.cache.handle, 0)
        if st.device_status:
            raise RuntimeError(f"device status {st.device_status:#x} after fill")
        if self.dynamic:       # what was actually kept, per (sequence, group), in tokens per layer
            lig = np.bincount(w.policy.layer_group, minlength=cfg.n_groups)
            for b in range(self.B):
                st = self.P.pask_budget_state(self.cache.handle, b)
                for g in range(cfg.n_groups):
                    self.nh[b, g] = st.n_high[g] // max(1, lig[g])
                    self.nl[b, g] = st.n_low[g] // max(1, lig[g])

    def prepare_steps(self, n_steps):
        w, cfg, d = self.w, self.cfg, self.device
        self.steps = []
        for s in range(n_steps):
            per_layer = []
            for layer in range(cfg.n_layers):
                k, v, q, tags = step_inputs(w, layer, s, d)
                per_layer.append((k, v, q, torch.from_numpy(tags).to(d)))
            self.steps.append(per_layer)
        if self.dynamic:
            self.step_states = [torch.from_numpy(np.array([w.states(b, w.total_len(b) + s, 1)[0] for b in range(self.B)],
                                                          np.int16)).to(d) for s in range(n_steps)]
            self.decided = torch.empty((self.B, cfg.n_groups), dtype=torch.uint8, device=d)

    def capture_steps(self, first, n_steps):
        """One CUDA graph per step (its inputs are fixed buffers): the step's launches are then
        issued by a single graph launch."""
        self.graphs = {}
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for s in range(first, first + n_steps):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    self.run_step(s)
                self.graphs[s] = g
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()

    def run_step(self, s, events=None, spans=None):
        """events: {layer: (start, stop)} for the launches of this step whose streaming kernel is timed;
        spans: {layer: int64[2]} for those that time themselves from inside (pask_cache_set_timing_span)."""
        P, h = self.P, self.cache.handle
        if self.dynamic:       # Algorithm 2 steps 1-6 once per token, then step 7 layer by layer
            P.pask_decide(h, self.ids, self.cu1, self.steps[s][0][3], self.step_states[s], self.decided)
        for layer, (k, v, q, tags) in enumerate(self.steps[s]):
            if events is not None and layer in events:
                P.pask_cache_set_timing_events(h, *events[layer])
            if spans is not None and layer in spans:
                P.pask_cache_set_timing_span(h, spans[layer])
            if self.ahead:     # streaming from the plan made a step ahead, the append beside it
                P.pask_decode_step_ahead(h, layer, self.ids, k, v, tags, q, self.out, self.lse, self.ws, self.area,
                                         actions=self.decided if self.dynamic else None)
                continue
            if self.fused:     # the library's one-call form of append + attention for a layer
                P.pask_append_attend(h, layer, self.ids, self.cu1, k, v, tags, q, self.out, self.lse, self.ws,
                                     actions=self.decided if self.dynamic else None)
                continue
            if self.dynamic:
                P.pask_append_kv_decided(h, layer, self.ids, self.cu1, k, v, tags, self.decided)
            else:
                P.pask_append_kv(h, layer, self.ids, self.cu1, k, v, tags)
            self.attn(h, layer, self.ids, q, self.out, self.lse, self.ws)

    def algorithmic_bytes_per_layer(self, steps_done=0):
        """Bytes one launch of the streaming kernel must move, averaged over layers: K/V payload of the
        retained tokens (codes + scales, or bf16), the queries, the page-order list, and the split
        partials it writes. Dropped tokens and page slack are not counted."""
        cfg = self.cfg
        lg = self.w.policy.layer_group.astype(np.int64)
        n_ctas = 2 * torch.cuda.get_device_properties(self.device).multi_processor_count
        tot = 0.0
        win_h = win_l = np.zeros((self.B, self.w.policy.n_groups), np.int64)
        if self.window:     # window members are read from the bf16 ring instead of from their streams
            eff = np.maximum(self.w.policy.a0, self.w.policy.a_floor)
            win_h, win_l = win_h.copy(), win_l.copy()
            for b in range(self.B):
                tags = self.w.tags(b, self.lens[b] + steps_done - self.window, self.window)
                acts = np.where(tags[:, None] < self.w.policy.n_tags, eff[np.minimum(tags, self.w.policy.n_tags - 1)], 2)
                win_h[b], win_l[b] = (acts == 2).sum(0), (acts == 1).sum(0)
        for l in range(cfg.n_layers):
            nh, nl = self.nh[:, lg[l]] + steps_done - win_h[:, lg[l]] + self.window, self.nl[:, lg[l]] - win_l[:, lg[l]]
            tot += float((nh * cfg.n_kv * 512).sum() + (nl * cfg.n_kv * {8: 272, 4: 144, 2: 80}[self.low_bits]).sum())
            tot += float((((nh + 15) // 16) + ((nl + 15) // 16)).sum() * 4)
        per_layer = tot / cfg.n_layers
        per_layer += self.B * cfg.n_q * 128 * 2
        per_layer += (n_ctas + self.B) * cfg.n_q * 130 * 4
        return per_layer


class Runner:
    """Times decode steps of one Job: blocks of exactly K steps bracketed by a barrier and a device
    synchronisation on both sides, CUDA events on the launching stream, MAX over ranks."""

    def __init__(self, args, world, device):
        self.args, self.world, self.device = args, world, device

    def barrier(self):
        if self.world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    def block(self, job, first_step, n_steps, with_events=True, graph=False):
        """One timed block; returns (ms of the block, [ms of each timed streaming-kernel launch])."""
        evs = kernel_events(job.cfg.n_layers, n_steps, self.args.event_stride) if (with_events and not graph) else None
        sps = kernel_spans(job.cfg.n_layers, n_steps, self.args.event_stride, self.device) if evs else None
        self.barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for i in range(n_steps):
            if graph:
                job.graphs[first_step + i].replay()
            else:
                job.run_step(first_step + i, evs[i] if evs else None, sps[i] if sps else None)
        t1.record()
        self.barrier()
        ms = max_over_ranks(t0.elapsed_time(t1), self.device)
        kern = [a.elapsed_time(b) for row in (evs or []) for a, b in row.values()]
        # in-kernel spans (ns of the GPU's global timer) of launches that carried no events
        self.last_spans_ms = [float(v[1] - v[0]) * 1e-6 for row in (sps or []) for v in (t.tolist() for t in row.values())
                              if v[1] > 0 and v[0] > 0]
        return ms, kern


def kernel_figures(job, kern_ms, steps_done, peak):
    """Roofline figures of the streaming kernel from its live launch times."""
    alg = job.algorithmic_bytes_per_layer(steps_done)
    if not kern_ms:
        return {"algorithmic_bytes_per_launch": alg, "avg_launch_ms": None, "achieved": None, "frac": None}
    k_ms = sum(kern_ms) / len(kern_ms)
    achieved = alg / (k_ms * 1e-3) / 1e9
    return {"algorithmic_bytes_per_launch": alg, "avg_launch_ms": k_ms, "launches_timed": len(kern_ms),
            "achieved": achieved, "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}


def check_status(P, job, where):
    st = P.pask_budget_state(job.cache.handle, 0)
    if st.device_status:
        raise RuntimeError(f"device status {st.device_status:#x} {where}")


def quick_point(P, runner, cfg, device, steps, peak, repeat=0, policy_blob=None, label="pask", clocks_index=None):
    """One further measurement point: build the workload, fill the cache, 3 warm-up steps, one timed block.
    Returns a small dict (tokens/s, ms/step, streaming-kernel GB/s and fraction of the peak, clocks)."""
    warm = 3
    cfg = WC.scaled(cfg, extra_gen=max(cfg.extra_gen, warm + steps + 8))
    t_setup = time.time()
    w = WC.build(cfg, repeat=repeat)
    if policy_blob == "all_high":                 # the dense comparison cache: every token kept at bf16
        from pask_workloads.policy import all_high_policy, write_blob
        policy_blob = write_blob(all_high_policy(w.policy.n_tags, cfg.n_groups, cfg.n_layers))
    job = Job(P, w, device, warm + steps + 4, policy_blob=policy_blob, label=label)
    job.fused = policy_blob is None
    job.fill()
    job.prepare_steps(warm + steps)
    if job.fused and job.B <= 255 and runner.args.ahead:
        job.plan_ahead()
    t_setup = time.time() - t_setup
    for i in range(warm):
        job.run_step(i)
    sampler = ClockSampler(clocks_index if clocks_index is not None else (device.index or 0))
    sampler.start()
    ms, kern = runner.block(job, warm, steps)
    clocks = sampler.stop()
    check_status(P, job, f"after {cfg.name}")
    ret = sum(P.pask_budget_state(job.cache.handle, b).retained_bytes for b in range(job.B))
    full = sum(P.pask_budget_state(job.cache.handle, b).full_bytes for b in range(job.B))
    fig = kernel_figures(job, kern, warm + steps // 2, peak)
    spans = runner.last_spans_ms
    out = {"workload": cfg.name, "kernel": label, "batch": job.B, "layers": cfg.n_layers, "kv_budget_target": cfg.budget,
           "kv_budget_realised": ret / full, "table": f"{cfg.lut}/{cfg.bias}", "steps": steps, "warmup": warm,
           "tokens_per_s": job.B * steps / (ms * 1e-3), "ms_per_step": ms / steps,
           "kernel_GBs": fig["achieved"], "frac": fig["frac"], "frac_of_nominal_8TBs": fig.get("frac_of_nominal_8TBs"),
           "avg_launch_ms": fig["avg_launch_ms"], "algorithmic_bytes_per_launch": fig["algorithmic_bytes_per_launch"],
           "clocks": clocks, "setup_s": round(t_setup, 1)}
    if spans:      # the kernel timed from inside on launches without events (see roofline.in_kernel of the headline)
        sp = sum(spans) / len(spans)
        out["in_kernel_span_ms"] = sp
        out["in_kernel_frac"] = fig["algorithmic_bytes_per_launch"] / (sp * 1e-3) / 1e9 / peak
    if len(job.fill_ms) > 1:
        out["bulk_append_ms_per_layer_call"] = sum(job.fill_ms[1:]) / (len(job.fill_ms) - 1)
        out["tokens_in_cache"] = job.total_tokens
    job.cache.close()
    del job
    torch.cuda.empty_cache()
    return out


def other_configs(P, runner, device, peak, args):
    """The configurations of the metric's list besides the headline one, each measured in this run:
    the budget sweep at the batch-64 8K shape against the full-KV kernel, the batch-128 16K case, the
    concurrency-8 shapes of the paper's latency table, the LOW-heavy and HIGH-heavy tables at the
    headline shape, and the one-layer batch-8 shape with its layer rotated over replicas."""
    out, steps = [], max(4, min(args.steps, 10))

    def add(fn, what):
        try:
            out.append(fn())
        except Exception as e:                      # e.g. out of memory on a smaller part: say so, keep going
            out.append({"workload": what, "unavailable": str(e)[:200]})
            torch.cuda.empty_cache()

    for b in WC.SWEEP_BUDGETS:
        cfg = WC.scaled(WC.QWEN3_4B_SWEEP, budget=b, lut="all_high" if b >= 1.0 else "greedy")
        add(lambda: quick_point(P, runner, cfg, device, steps, peak), f"{cfg.name} @ {b}")

    def full_kv_sweep():
        r = quick_point(P, runner, WC.QWEN3_4B_SWEEP, device, steps, peak, policy_blob="all_high", label="full-kv bf16 kernel")
        r["kv_budget_target"] = 1.0
        return r
    add(full_kv_sweep, "full-KV at the sweep shape")
    add(lambda: dict(quick_point(P, runner, WC.QWEN3_8B_LONG, device, max(3, steps // 2), peak),
                     note="the dense comparison cache of this shape (309 GB) does not fit one GPU: PASK only"),
        WC.QWEN3_8B_LONG.name)
    for cfg in (WC.TABLE3_8K, WC.TABLE3_32K):
        add(lambda: quick_point(P, runner, cfg, device, steps, peak), cfg.name)
    for bias in ("low", "high"):
        cfg = WC.scaled(WC.QWEN3_4B_STEP, bias=bias, name=f"{WC.QWEN3_4B_STEP.name}[{bias.upper()}-heavy table]")
        add(lambda: quick_point(P, runner, cfg, device, steps, peak), cfg.name)

    def one_layer_rotated():
        # 16 layers = 4 replicas of each layer-group column, every one with its own pages: a step walks
        # 16 distinct ~45 MB working sets (together far beyond L2), so no launch finds its pages in L2
        reps = 4
        base = WC.QWEN3_4B_1LAYER
        cfg = WC.scaled(base, n_layers=base.n_groups * reps, name=f"{base.name}[x{reps} replicas per column]")
        r = quick_point(P, runner, cfg, device, 2 * steps, peak)
        r["layer_tokens_per_s"] = r["tokens_per_s"] * cfg.n_layers
        r["tokens_per_s_at_36_layers"] = r["layer_tokens_per_s"] / 36.0
        r["note"] = ("one-layer shape: tokens_per_s counts a pass over all 16 replica layers as one step; "
                     "layer_tokens_per_s = batch x layer launches / s; L2: rotated over 16 distinct layer caches")
        return r
    add(one_layer_rotated, "one-layer shape, rotated")
    return out


def run_cuda(args, rank, world):
    import paper_2608_28276_b200 as P
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(device)
    cfg = CONFIGS[args.config]
    if args.budget is not None or args.bias != "balanced":
        cfg = WC.scaled(cfg, budget=args.budget if args.budget is not None else cfg.budget, bias=args.bias,
                        lut="all_high" if (args.budget or 0) >= 1.0 else cfg.lut)
    if args.low_bits != 4:
        cfg = WC.scaled(cfg, low_bits=args.low_bits, name=f"{cfg.name}[{args.low_bits}-bit low]")
    if args.layers:
        cfg = WC.scaled(cfg, n_layers=args.layers, name=f"{cfg.name}[first {args.layers} layers]")
    repeats = max(1, args.repeats)
    total_steps = args.warmup + repeats * args.steps
    e2e_steps = min(args.steps, 10)
    e2e_warm = 2                       # untimed end-to-end steps (the first call creates the library's copy streams)
    cfg = WC.scaled(cfg, extra_gen=max(cfg.extra_gen, 2 * total_steps + e2e_steps + e2e_warm + 8))
    w = rank_workload(cfg, rank)
    if args.window:
        from dataclasses import replace as _replace
        w.policy = _replace(w.policy, recent_window=args.window)
    runner = Runner(args, world, device)
    peak, peak_kind = measured_peaks()
    t_setup = time.time()
    job = Job(P, w, device, 2 * total_steps + e2e_steps + e2e_warm + 4, dynamic=args.dynamic)
    job.fused = not args.unfused
    job.fill()
    job.prepare_steps(total_steps)
    use_ahead = args.ahead and job.fused and job.B <= 255 and not args.window
    if use_ahead:
        job.plan_ahead()
    # launches per layer: planned-ahead step = streaming kernel + the kernel that ends the step (append and merge);
    # pask_append_attend = append (+ plan), streaming kernel, combine; the two separate calls = four
    per_layer_launches = 2 if use_ahead else 3 if (job.fused and job.B <= 255) else 4
    t_setup = time.time() - t_setup
    ret = sum(P.pask_budget_state(job.cache.handle, b).retained_bytes for b in range(job.B))
    full = sum(P.pask_budget_state(job.cache.handle, b).full_bytes for b in range(job.B))

    for i in range(args.warmup):
        job.run_step(i)
    if args.graph:
        job.capture_steps(args.warmup, repeats * args.steps)
    sampler = ClockSampler(device.index or 0)
    if rank == 0:
        sampler.start()
    # the timed region, `repeats` times over: each block is exactly --steps steps between two barriers
    blocks, kern_ms, kern_by_block, span_ms = [], [], [], []
    for r in range(repeats):
        ms, kern = runner.block(job, args.warmup + r * args.steps, args.steps, graph=args.graph)
        blocks.append(ms)
        kern_ms += kern
        span_ms += runner.last_spans_ms
        kern_by_block.append(sum(kern) / len(kern) if kern else None)
    clocks = sampler.stop() if rank == 0 else {}
    check_status(P, job, "after the timed region")
    per_block = [whole_job_tokens_per_s(world, job.B, args.steps, ms) for ms in blocks]
    ms = statistics.median(blocks)
    value = whole_job_tokens_per_s(world, job.B, args.steps, ms)

    # ---- end to end: the same step through the host-buffer entry point, copies inside the region
    e2e = None
    if (rank == 0 or world > 1) and not args.dynamic:   # the host-buffer entry point applies the frozen table
        e2e = end_to_end(P, runner, job, w, cfg, total_steps, e2e_warm, e2e_steps, world, device)

    if rank != 0:
        return
    fig = kernel_figures(job, kern_ms, args.warmup + repeats * args.steps // 2, peak)
    alg = fig["algorithmic_bytes_per_launch"]
    covered = job.low_bits == 4 and not args.window and cfg.name == DEFAULT_CONFIG and args.bias == "balanced"
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": f"bf16/int{job.low_bits} storage, bf16 / fp16 tensor-core operands with fp32 accumulation", "data": "synthetic",
        "config": {"workload": cfg.name, "batch_per_gpu": job.B, "layers": cfg.n_layers, "layer_groups": cfg.n_groups,
                   "kv_budget_target": cfg.budget, "kv_budget_realised": ret / full, "table": f"greedy/{cfg.bias}",
                   "recent_window": args.window,
                   "step_call": "pask_decode_step_ahead (plan made a step ahead, append beside the streaming kernel)" if use_ahead
                                else "pask_append_attend" if job.fused else "pask_append_kv + pask_decode_attention",
                   "tokens_in_cache_per_gpu": job.total_tokens, "page_tokens": 16,
                   "l2": "inputs larger than L2: each layer streams its own ~%.0f MB of pages" % (alg / 1e6),
                   "setup_s": round(t_setup, 1)},
        "repeats": {"n": repeats, "statistic": "value = median over the timed blocks, each exactly `steps` steps",
                    "tokens_per_s": per_block, "min": min(per_block), "max": max(per_block),
                    "ms_per_block": blocks, "kernel_avg_launch_ms_per_block": kern_by_block},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": (per_layer_launches * cfg.n_layers + (1 if args.dynamic else 0)) * args.steps,
        "roofline": {"bound": "hbm", "kernel": f"decode_attn_kernel<{job.low_bits}>", "achieved": fig["achieved"], "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": fig["frac"],
                     "frac_of_nominal_8TBs": fig.get("frac_of_nominal_8TBs"), "algorithmic_bytes_per_launch": alg,
                     "avg_launch_ms": fig["avg_launch_ms"], "launches_timed": fig.get("launches_timed"),
                     "traffic": alg * NCU_TRAFFIC_RATIO if covered else None,
                     "traffic_source": (f"estimated: {NCU_TRAFFIC_RATIO} x algorithmic bytes, the ratio of ncu "
                                        "dram__bytes_read+write to algorithmic bytes in the capture summarised in "
                                        f"{NCU_TRAFFIC_PROFILE} (a 4-layer cut of this workload)") if covered else
                                       "no ncu capture covers this configuration"},
    }
    if span_ms and line["roofline"]:
        sp = sum(span_ms) / len(span_ms)
        line["roofline"]["in_kernel"] = {
            "avg_span_ms": sp, "launches": len(span_ms), "achieved": alg / (sp * 1e-3) / 1e9, "frac": alg / (sp * 1e-3) / 1e9 / peak,
            "what": "the same kernel timed from inside (pask_cache_set_timing_span: first CTA released -> last CTA done, GPU "
                    "global timer) on launches of the timed region that carry no events and so keep their launch overlap; "
                    "the event figure above adds the launch and completion latency around a kernel that stands alone"}
    if fig["avg_launch_ms"]:
        k_ms = fig["avg_launch_ms"]
        in_ms = sum(span_ms) / len(span_ms) if span_ms else None
        # Share of the step spent in the streaming kernel.  From the in-kernel spans when there are any: an event-timed
        # launch stands alone (nothing overlaps its launch and completion latency, ~9 us here), so n_layers x its
        # duration can exceed the un-timed step, in which every launch overlaps its neighbours.
        line["attention_share_of_step"] = (in_ms or k_ms) * cfg.n_layers * args.steps / ms
        line["attention_share_of_step_by_events"] = k_ms * cfg.n_layers * args.steps / ms
        line["attention_share_note"] = ("share = n_layers x streaming-kernel time / step time; the first uses the kernel's own span "
                                        "(launches that keep their overlap), the second the duration between a pair of events, "
                                        "which includes launch and completion latency that the un-timed step hides and can "
                                        "therefore exceed 1")
        line["attention_only_tokens_per_s"] = world * job.B / ((in_ms or k_ms) * 1e-3 * cfg.n_layers)
    if args.graph:
        line["config"]["launch"] = "one CUDA graph per step"
        line["roofline"] = None
    if len(job.fill_ms) > 1:
        f_ms = sum(job.fill_ms[1:]) / (len(job.fill_ms) - 1)
        lg = w.policy.layer_group.astype(np.int64)
        kept = sum(float((job.nh[:, lg[l]] + job.nl[:, lg[l]]).sum()) for l in range(cfg.n_layers)) / cfg.n_layers
        in_b = kept * 2 * cfg.n_kv * 256 + job.total_tokens * 5        # K, V rows of retained tokens (bf16), tag + list word
        out_b = ret / cfg.n_layers                                     # payload written, per layer
        line["bulk_append"] = {"tokens_per_call": job.total_tokens, "ms_per_layer_call": f_ms,
                               "token_layers_per_s": job.total_tokens / (f_ms * 1e-3),
                               "achieved_gbs": (in_b + out_b) / (f_ms * 1e-3) / 1e9,
                               "frac_of_peak": (in_b + out_b) / (f_ms * 1e-3) / 1e9 / peak,
                               "algorithmic_bytes_per_call": in_b + out_b,
                               "retained_tokens_per_layer": kept,
                               "note": "one ragged pask_append_kv call per layer over the whole history (plan + write "
                                       "kernels); rows of dropped tokens are never read"}
    if args.dynamic:
        sts = [P.pask_budget_state(job.cache.handle, b) for b in range(job.B)]
        line["dynamic_budget"] = {"prefill_decide_ms": job.prefill_decide_ms, "prefill_tokens": job.total_tokens,
                                  "demoted": sum(s.n_demoted for s in sts), "promoted": sum(s.n_promoted for s in sts),
                                  "floor_conflicts": sum(s.n_floor_conflicts for s in sts)}
        line["config"]["table"] += " + budget-dependent adjustment (pask_decide)"
    job.cache.close()
    del job
    torch.cuda.empty_cache()
    if world == 1:
        if args.seeds > 1:       # the same configuration from the next seeds: spread over inputs, not over time
            pts = [quick_point(P, runner, cfg, device, args.steps, peak, repeat=r) for r in range(1, args.seeds)]
            vals = [value] + [p["tokens_per_s"] for p in pts]
            fr = [fig["frac"]] + [p["frac"] for p in pts]
            line["seeds"] = {"n": args.seeds, "tokens_per_s": vals, "kernel_frac": fr, "median": statistics.median(vals),
                             "min": min(vals), "max": max(vals),
                             "note": "seed + 0 is the headline run (its median block); + 1, + 2: one timed block each"}
        if args.full_kv:
            r = quick_point(P, runner, cfg, device, args.steps, peak, policy_blob="all_high", label="full-kv bf16 kernel")
            line["full_kv"] = {"value": r["tokens_per_s"], "unit": UNIT, "ms_per_step": r["ms_per_step"],
                               "achieved_GBs": r["kernel_GBs"], "frac": r["frac"],
                               "algorithmic_bytes_per_launch": r["algorithmic_bytes_per_launch"],
                               "avg_launch_ms": r["avg_launch_ms"]}
        if args.other_configs:
            line["other_configs"] = other_configs(P, runner, device, peak, args)
        if args.cpu_seconds > 0:          # the oracle beside it: rank 0 at N = 1 only
            line["cpu_baseline"] = cpu_baseline(w, budget_s=args.cpu_seconds, n_seqs=args.ref_seqs)
    print(json.dumps(line))


def end_to_end(P, runner, job, w, cfg, first_step, e2e_warm, e2e_steps, world, device):
    """The same steps through pask_decode_step_pipelined: inputs start in pinned host memory and the
    attention output ends there, every layer, inside the timed region."""
    staging = torch.empty(2 * P.pask_step_staging_bytes(job.cache.handle, job.B), dtype=torch.uint8, device=device)
    off, in_bytes = P.pask_step_packed_layout(job.cache.handle, job.B)
    host = []
    for s in range(e2e_warm + e2e_steps):   # a layer's inputs sit in one pinned block, as an engine would stage them
        rows = []
        for layer in range(cfg.n_layers):
            k, v, q, tags = step_inputs(w, layer, first_step + s, "cpu")
            block = torch.zeros(in_bytes, dtype=torch.uint8).pin_memory()
            parts = [torch.arange(job.B, dtype=torch.int32), torch.arange(job.B + 1, dtype=torch.int32), k, v,
                     torch.from_numpy(tags), q]
            for o, t in zip(off, parts):
                raw = t.contiguous().view(torch.uint8).reshape(-1)
                block[o:o + raw.numel()] = raw
            rows.append(block)
        host.append(rows)
    out_h = torch.empty((job.B, cfg.n_q, 128), dtype=torch.float32).pin_memory()
    if job.ahead:        # the timed steps before have left every layer's plan for this batch in job.area
        def call(layer, block):
            P.pask_decode_step_pipelined_ahead(job.cache.handle, layer, job.B, block, out_h, staging, job.ws, job.area)
    else:
        def call(layer, block):
            P.pask_decode_step_pipelined(job.cache.handle, layer, job.B, block, out_h, staging, job.ws)
    for rows in host[:e2e_warm]:
        for layer, block in enumerate(rows):
            call(layer, block)
    P.pask_decode_step_drain(job.cache.handle)
    runner.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for rows in host[e2e_warm:]:
        for layer, block in enumerate(rows):
            call(layer, block)
    P.pask_decode_step_drain(job.cache.handle)      # the host holds every output before the clock stops
    t1.record()
    runner.barrier()
    e_ms = max_over_ranks(t0.elapsed_time(t1), device)
    h2d = cfg.n_layers * in_bytes
    d2h = cfg.n_layers * job.B * cfg.n_q * 128 * 4
    return {"value": whole_job_tokens_per_s(world, job.B, e2e_steps, e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e_ms / e2e_steps,
            "api": ("pask_decode_step_pipelined_ahead" if job.ahead else "pask_decode_step_pipelined") + ": one pinned host block in, attention output out, per layer; the "
                   "copies run on the library's copy streams and overlap the neighbouring layers' kernels"}


# ------------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands on a bounded sample of the same workload

class OracleSample:
    """The oracle's cache holding the history of a few (layer, sequence) pairs of the workload;
    step(i) runs decode step i on them (append one token per sequence, fp64 attention) and returns
    the wall time. Building the history is not timed, as the GPU arm's fill is not either."""

    def __init__(self, w, n_seqs, layers):
        import oracle
        self.oracle, self.w, self.layers = oracle, w, list(layers)
        cfg = w.cfg
        self.B = min(cfg.batch, n_seqs)
        lens = [w.total_len(b) for b in range(self.B)]
        pages = len(self.layers) * (sum(lens) // 16 + 8 * self.B) + 64
        self.cache = oracle.Cache(oracle.Policy(w.blob), cfg.n_q, cfg.n_kv, self.B, pages, pages)
        gen = "cuda" if torch.cuda.is_available() else "cpu"   # same generator, same bits, either device
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        tags = np.concatenate([w.tags(b, 0, lens[b]) for b in range(self.B)])
        for layer in self.layers:
            k = torch.cat([normal_bf16(w.seed, TENSOR_K, layer, b, 0, lens[b], cfg.n_kv, gen) for b in range(self.B)]).cpu()
            v = torch.cat([normal_bf16(w.seed, TENSOR_V, layer, b, 0, lens[b], cfg.n_kv, gen) for b in range(self.B)]).cpu()
            rc, _ = self.cache.append(layer, list(range(self.B)), cu, bf16_bits(k).numpy(), bf16_bits(v).numpy(), tags)
            assert rc == 0
            del k, v

    def step(self, i):
        """Decode step i on the sampled layers; returns the wall seconds of each sampled layer."""
        B, ts = self.B, []
        for layer in self.layers:
            k, v, q, tags = step_inputs(self.w, layer, i, "cpu")
            kb, vb, qb = bf16_bits(k[:B]).numpy(), bf16_bits(v[:B]).numpy(), bf16_bits(q[:B]).numpy()
            t0 = time.perf_counter()
            self.cache.append(layer, list(range(B)), np.arange(B + 1, dtype=np.int32), kb, vb, tags[:B])
            self.cache.attention_batch(layer, list(range(B)), qb)
            ts.append(time.perf_counter() - t0)
        return ts

    def full_step_seconds(self, per_layer):
        """Seconds of a decode step over all layers for the sampled sequences: every sampled layer stands
        for the layers of its layer group (the groups keep different shares of the tokens)."""
        lg = self.w.policy.layer_group.astype(np.int64)
        t = 0.0
        for layer, sec in zip(self.layers, per_layer):
            t += sec * int((lg == lg[layer]).sum())
        return t

    def tokens_per_s(self, per_layer):
        return self.B / self.full_step_seconds(per_layer)

    def describe(self, n_steps, seconds):
        cfg = self.w.cfg
        return (f"layers {self.layers} (the first of each layer group) of {cfg.n_layers} x {self.B} of {cfg.batch} sequences, "
                f"{n_steps} decode steps (append + fp64 attention), {seconds:.1f} s wall on the host cores; each sampled "
                f"layer scaled by the {cfg.n_layers // cfg.n_groups} layers of its group")


def group_layers(w):
    """The first layer of every layer group that owns layers."""
    lg = w.policy.layer_group.astype(np.int64)
    return [int(np.argmax(lg == g)) for g in range(w.policy.n_groups) if (lg == g).any()]


def cpu_baseline(w, budget_s=15.0, n_seqs=64):
    smp = OracleSample(w, n_seqs, group_layers(w))
    cores = smp.oracle.max_threads()
    smp.step(0)                                    # untimed first touch
    acc, wall, n = np.zeros(len(smp.layers)), 0.0, 0
    while n < 16 and wall < budget_s:
        ts = smp.step(1 + n)
        acc += np.asarray(ts)
        wall += sum(ts)
        n += 1
    return {"value": smp.tokens_per_s(acc / n), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": smp.describe(n, wall), "measured_s_per_sampled_step": wall / n,
            "extrapolated_s_per_full_step": smp.full_step_seconds(acc / n)}


def run_reference(args, rank, world):
    if rank != 0:
        return
    cfg = CONFIGS[args.config]
    cfg = WC.scaled(cfg, extra_gen=max(cfg.extra_gen, args.warmup + args.steps + 8))
    w = WC.build(cfg)
    smp = OracleSample(w, args.ref_seqs, group_layers(w))
    if world > 1:      # the launcher pins every rank to one OpenMP thread; rank 0 runs alone and takes the host's cores
        smp.oracle.set_threads(os.cpu_count() or 1)
    for i in range(args.warmup):
        smp.step(i)
    acc = np.zeros(len(smp.layers))
    for i in range(args.steps):
        acc += np.asarray(smp.step(args.warmup + i))
    wall = float(acc.sum())
    value = smp.tokens_per_s(acc / args.steps)
    base = {"value": value, "unit": UNIT, "cores": smp.oracle.max_threads(), "kind": "oracle",
            "sample": smp.describe(args.steps, wall), "measured_s_per_sampled_step": wall / args.steps,
            "extrapolated_s_per_full_step": smp.full_step_seconds(acc / args.steps)}
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * smp.full_step_seconds(acc / args.steps) * cfg.batch / smp.B,
            "measured_ms_per_sampled_step": 1e3 * wall / args.steps,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "kv_budget_target": cfg.budget,
                       "note": "ms_per_step is extrapolated from the sampled layers to all layers; "
                               "measured_ms_per_sampled_step is the wall time actually spent per step"},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--config", default=DEFAULT_CONFIG, choices=sorted(CONFIGS))
    ap.add_argument("--budget", type=float, default=None, help="override the KV budget of the table")
    ap.add_argument("--bias", default="balanced", choices=["balanced", "low", "high"])
    ap.add_argument("--no-full-kv", dest="full_kv", action="store_false")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="0 skips the CPU-oracle leg")
    ap.add_argument("--event-stride", type=int, default=9, help="time the streaming kernel of every n-th launch")
    ap.add_argument("--low-bits", type=int, default=4, choices=[2, 4, 8], help="width of the RETAIN-LOW codes")
    ap.add_argument("--unfused", action="store_true",
                    help="issue pask_append_kv and pask_decode_attention separately instead of pask_append_attend")
    ap.add_argument("--no-ahead", dest="ahead", action="store_false",
                    help="use pask_append_attend per layer instead of the planned-ahead step (pask_decode_step_ahead)")
    ap.add_argument("--window", type=int, default=0, help="protected recent window in tokens (multiple of 16, <= 256)")
    ap.add_argument("--graph", action="store_true", help="replay each timed step as one CUDA graph (launch-bound shapes)")
    ap.add_argument("--dynamic", action="store_true",
                    help="decide every token against the running budget (pask_decide) instead of the frozen table alone")
    ap.add_argument("--layers", type=int, default=None, help="profiling aid: keep only the first N layers")
    ap.add_argument("--ref-seqs", type=int, default=64, help="sequences in the oracle's timed sample")
    ap.add_argument("--repeats", type=int, default=5, help="timed blocks of --steps steps each; value = their median")
    ap.add_argument("--seeds", type=int, default=3, help="N = 1: also run the configuration from the next seeds (1 = only the first)")
    ap.add_argument("--no-other-configs", dest="other_configs", action="store_false",
                    help="N = 1: skip the further configurations (budget sweep, batch-128 16K, latency-table shapes, ...)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl")
    try:
        run_cuda(args, rank, world)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
