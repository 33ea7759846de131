#!/usr/bin/env python
"""Benchmark of the FreeCache denoising step on B200.

One "step" is one pass of the whole hot path for one denoising step of the Dream-7B-shaped
workload: attention of the active block over [cache ; fresh rows] for all 28 layers (one
layer-batched launch: all layers' synthetic Q/K/V exist up front), confidence scoring + top-4
unmasking over vocab 152064, and the cache commit (4 staged rows, or the whole block when it
completes).  Steps cycle through the 64-step generation schedule (8 blocks x 8 steps; cache
1024 -> 1248 rows, 32 -> 4 masked positions).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config NAME]

Prints one JSON line (rank 0).  `value` is denoise steps/s with inputs resident in HBM; `e2e`
is the same with the step's inputs copied from pinned host memory and the result read back.
L2 is flushed between timed steps (the cache of this workload is smaller than L2).
With --impl reference the CPU oracle is timed on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from workloads import (get_config, make_attn_inputs, make_cache, make_kv_rows, make_logits,  # noqa: E402
                       seed_for, widen, bf16_bits)

# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch, per workload, from an ncu capture of the
# attention kernel as it stands (see profiles/).  A workload without a capture, or whose capture predates a
# change of the kernel, has no entry and the line prints null.
ATTN_DRAM_TRAFFIC_BYTES = {
    "dream7b": 68.7e6,             # 67.08 MB read + 1.6 MB written (profiles/attn_step_sm100_dream7b.md)
    "dream7b_window256": 226.5e6,   # 176.9 MB read + 49.6 MB written, the lower of two launches (profiles/attn_step_sm100_window256.md)
}

L2_BYTES = 126 << 20

METRIC = "denoise_steps_per_s"
UNIT = "steps/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed region runs (NVML reads only; falls back to
    nvidia-smi when the NVML binding is missing)."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index):
        self.index, self.sm, self.mx, self.reasons = index, [], None, set()
        self._stop = threading.Event()
        self.thread = None
        self.note = None

    def _loop(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.mx = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self._stop.is_set():
                self.sm.append(int(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                r = int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
                time.sleep(0.002)
        except Exception as e:   # noqa: BLE001
            self.note = f"nvml unavailable: {type(e).__name__}"
            self._smi_once()

    def _smi_once(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
            except Exception:   # noqa: BLE001
                return
            f = [x.strip() for x in out.strip().split(",")]
            if len(f) >= 6 and f[0].isdigit():
                self.sm.append(int(f[0])); self.mx = int(f[1])
                for n, v in zip(names, f[2:6]):
                    if v.lower().startswith("active"):
                        self.reasons.add(n)

    def start(self):
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def mark(self):
        """Samples taken from here on count as "under load" (the timed region starts)."""
        self.t_mark = len(self.sm)

    def stop(self):
        self._stop.set()
        if self.thread:
            self.thread.join(timeout=10)
        load = self.sm[getattr(self, "t_mark", 0):]
        out = {"sm_mhz": statistics.median(load) if load else None, "sm_max_mhz": self.mx,
               "samples": len(load), "samples_with_warmup": len(self.sm), "reasons": sorted(self.reasons)}
        if self.note:
            out["note"] = self.note
        return out


class Schedule:
    """The 64-step generation schedule of the top-k policy (host-side bookkeeping only)."""

    def __init__(self, cfg):
        self.cfg = cfg
        # guided policy: the number of steps a block takes depends on the data; the schedule gives it 8
        # (about 4.2 positions are accepted per step of a 32-position block) and then moves on
        self.steps_per_block = cfg.steps_per_block if cfg.policy == "topk" else 8
        self.n = cfg.n_blocks * self.steps_per_block

    def at(self, t):
        cfg = self.cfg
        t %= self.n
        block, s = divmod(t, self.steps_per_block)
        return {"block": block, "step_in_block": s, "cache_len": cfg.prompt_len + block * cfg.block_len,
                "n_masked": cfg.block_len - s * cfg.top_k, "last": s == self.steps_per_block - 1}


def attn_bytes(cfg, cache_len):
    """Algorithmic bytes of one layer-batched attention launch: K/V rows read once per KV head, Q read,
    O written (bf16)."""
    L = cache_len + cfg.block_len
    kv = 2 * 2 * cfg.batch * cfg.n_kv_heads * L * cfg.head_dim
    qo = 2 * 2 * cfg.batch * cfg.n_q_heads * cfg.block_len * cfg.head_dim
    return cfg.n_layers * (kv + qo)


def attn_flops(cfg, cache_len):
    return cfg.n_layers * 4 * cfg.batch * cfg.n_q_heads * cfg.block_len * (cache_len + cfg.block_len) * cfg.head_dim


def sets_needed(bytes_per_set):
    """Input sets to rotate over so that a set has left L2 (2.5x its size in other data) before its next use."""
    return max(1, -(-int(2.5 * L2_BYTES) // max(int(bytes_per_set), 1)))


def time_rotating(calls, min_launches=24, replays=5):
    """Average duration of one launch when the launches run back to back on one stream: `calls[i]()` enqueues
    the kernel on input set i; the sets together are larger than L2 (see sets_needed), so every launch reads
    cold data without an L2 flush in between, and consecutive launches overlap only as far as the library's
    programmatic dependent launch lets them (set-up of the next under the tail of the previous).  One CUDA
    graph holds ceil(min_launches / len(calls)) rounds over the sets; the events bracket `replays` replays.
    Returns seconds per launch."""
    rounds = -(-min_launches // len(calls))
    for c in calls:
        c()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=torch.cuda.Stream()):
        for _ in range(rounds):
            for c in calls:
                c()
    g.replay()
    torch.cuda.synchronize()
    best = None
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(replays):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        t = e0.elapsed_time(e1) * 1e-3 / (replays * rounds * len(calls))
        best = t if best is None else min(best, t)
    return best


class Workload:
    """Device-resident state of one sequence batch plus the per-step launch sequence."""

    N_POOL = 2   # distinct synthetic input sets cycled across steps

    def __init__(self, cfg, cfg_index, device):
        import paper_2505_21467_b200 as dlm
        self.dlm, self.cfg, self.dev = dlm, cfg, device
        self.ctx = dlm.dlm_create(device.index)
        s = seed_for(cfg_index)
        B, Lblk, V = cfg.batch, cfg.block_len, cfg.vocab
        self.ck, self.cv = make_cache(cfg.n_layers, B, cfg.n_kv_heads, cfg.capacity, cfg.head_dim, s, device)
        self.cache_len = torch.full((B,), cfg.prompt_len, dtype=torch.int32, device=device)
        self.cache = dlm.make_kv_cache(self.ck, self.cv, self.cache_len)
        self.pool = [make_attn_inputs(cfg.n_layers, B, cfg.n_q_heads, cfg.n_kv_heads, Lblk, cfg.head_dim, s + 1 + i,
                                      device) for i in range(self.N_POOL)]
        self.logits = [make_logits(B, Lblk, V, cfg.logit_sigma, s + 10 + i, device) for i in range(self.N_POOL)]
        self.out = torch.empty_like(self.pool[0][0])
        self.masked = torch.ones(B, Lblk, dtype=torch.uint8, device=device)
        self.tokens = torch.full((B, Lblk), -1, dtype=torch.int32, device=device)
        self.tok = torch.empty(B, Lblk, dtype=torch.int32, device=device)
        self.conf = torch.empty(B, Lblk, dtype=torch.float32, device=device)
        self.sel_idx = torch.empty(B, max(cfg.top_k, 1), dtype=torch.int32, device=device)
        self.n_sel = torch.empty(B, dtype=torch.int32, device=device)
        self.attn_ws = torch.empty(max(dlm.dlm_attn_workspace_bytes(self.ctx, self.cache, cfg.n_layers, cfg.n_q_heads,
                                                                    Lblk), 256), dtype=torch.uint8, device=device)
        self.unmask_ws = torch.empty(max(dlm.dlm_unmask_workspace_bytes(self.ctx, B, Lblk, V), 256),
                                     dtype=torch.uint8, device=device)
        self.flush = torch.empty(512 << 20, dtype=torch.uint8, device=device)   # 4x the 126 MB L2
        self.guided = cfg.policy == "guided"
        if self.guided:
            # the guider's argmax for every position: agrees with the DLM's argmax with probability p_agree
            self.q_len = torch.full((B,), Lblk, dtype=torch.int32, device=device)
            self.accept = torch.empty(B, Lblk, dtype=torch.uint8, device=device)
            self.acc_idx = torch.empty(B, Lblk, dtype=torch.int32, device=device)
            self.n_acc = torch.empty(B, dtype=torch.int32, device=device)
            self.tok_ar = []
            from workloads import make_tok_ar
            for i in range(self.N_POOL):
                self.masked.fill_(1)
                dlm.dlm_unmask_select(self.ctx, self.logits[i], B, Lblk, V, self.masked, self.tokens, 0, self.tok, self.conf,
                                      None, None, self.unmask_ws)
                self.tok_ar.append(make_tok_ar(self.tok.cpu(), cfg.p_agree, V, s + 20 + i).to(device))
        self.sched = Schedule(cfg)
        self.t = 0

    def reset_block_state(self, st):
        """Puts the device state where step `t` of the schedule expects it (not timed)."""
        self.cache_len.fill_(st["cache_len"])
        if self.guided:     # accepted positions form a prefix: a block starts fully masked
            if st["step_in_block"] == 0:
                self.masked.fill_(1)
            self.q_len.copy_(self.masked.sum(1))
            return
        self.masked.zero_()
        self.masked[:, :st["n_masked"]] = 1

    def launch_attn(self, st, q, kn, vn):
        dlm, cfg = self.dlm, self.cfg
        dlm.dlm_freecache_attn_step(self.ctx, self.cache, 0, cfg.n_layers, q, kn, vn, cfg.n_q_heads, cfg.block_len,
                                    self.q_len if self.guided else None, 0.0, st["cache_len"], self.out, None, self.attn_ws)

    def launch_rest(self, last, kn, vn, lg):
        """Unmask, then the commit: the 4 staged rows, or the whole block when it completes."""
        dlm, cfg = self.dlm, self.cfg
        if self.guided:
            # propose (argmax for every masked position), accept the prefix the guider agrees with, append the
            # accepted rows (visible at once); the window shrinks to the still-masked rows
            i = 0 if lg is self.logits[0] else 1
            dlm.dlm_unmask_select(self.ctx, lg, cfg.batch, cfg.block_len, cfg.vocab, self.masked, self.tokens, 0,
                                  self.tok, self.conf, None, None, self.unmask_ws)
            dlm.dlm_guided_accept(self.ctx, self.tok, self.tok_ar[i], cfg.batch, cfg.block_len, self.masked, self.tokens, 0,
                                  self.accept, self.acc_idx, self.n_acc)
            dlm.dlm_kv_cache_commit(self.ctx, self.cache, kn, vn, cfg.block_len, self.acc_idx, None, dlm.DLM_DST_APPEND,
                                    self.n_acc, cfg.block_len, 1, 0, cfg.n_layers)
            self.q_len.copy_(self.masked.sum(1))
            return
        dlm.dlm_unmask_select(self.ctx, lg, cfg.batch, cfg.block_len, cfg.vocab, self.masked, self.tokens, cfg.top_k,
                              self.tok, self.conf, self.sel_idx, self.n_sel, self.unmask_ws)
        if last:      # block complete: freeze all of its rows and make them visible
            dlm.dlm_kv_cache_commit(self.ctx, self.cache, kn, vn, cfg.block_len, None, None, dlm.DLM_DST_APPEND, None,
                                    cfg.block_len, 1, 0, cfg.n_layers)
        else:         # stage the rows unmasked in this step at their own slots
            dlm.dlm_kv_cache_commit(self.ctx, self.cache, kn, vn, cfg.block_len, self.sel_idx, None,
                                    dlm.DLM_DST_WINDOW, self.n_sel, cfg.top_k, 0, 0, cfg.n_layers)

    def launch_step(self, st, inputs=None, logits=None):
        """Enqueues one denoising step through the C-ABI: attention (all layers), unmask, commit."""
        q, kn, vn = inputs if inputs is not None else self.pool[self.t % self.N_POOL]
        lg = logits if logits is not None else self.logits[self.t % self.N_POOL]
        self.launch_attn(st, q, kn, vn)
        self.launch_rest(st["last"], kn, vn, lg)

    def capture(self):
        """Captures the C-ABI calls of a step into CUDA graphs (the lengths and masks they read live in device
        memory, so one capture serves every step): per input set and per form of the commit, one graph holding the
        attention call, unmask and commit, with timing events recorded inside the graph (external event nodes) before
        the attention call, after it, and after the commit.  Replaying removes the host's launch latency from the
        device-side timing; the kernels and their arguments are exactly those of the direct calls."""
        dlm = self.dlm
        st = self.sched.at(0)
        self.reset_block_state(st)
        torch.cuda.synchronize()
        # Two graphs per (input set, form of the commit): the step as it is launched, with event nodes only at
        # its two ends (self.graphs_step: whole-step time), and the same step with one more event node after the
        # attention launch (self.graphs: the attention launch's own duration; the node costs the step a kernel ->
        # event -> kernel gap and the overlap of the unmask kernel's prologue with the attention kernel's tail).
        self.graphs, self.graphs_step = [], []   # [pool index][last] -> (graph, (e0, e1, e2), kernel launches)
        side = torch.cuda.Stream()
        for i in range(self.N_POOL):
            q, kn, vn = self.pool[i]
            pair, pair_step = [], []
            for last in (False, True):
                for with_mid, dest in ((True, pair), (False, pair_step)):
                    ev = tuple(torch.cuda.Event(enable_timing=True, external=True) for _ in range(3))
                    g = torch.cuda.CUDAGraph()
                    c0 = dlm.dlm_launch_count(self.ctx)
                    with torch.cuda.graph(g, stream=side):
                        ev[0].record()
                        self.launch_attn(st, q, kn, vn)
                        if with_mid:
                            ev[1].record()
                        self.launch_rest(last, kn, vn, self.logits[i])
                        ev[2].record()
                    dest.append((g, ev, dlm.dlm_launch_count(self.ctx) - c0))
            self.graphs.append(pair)
            self.graphs_step.append(pair_step)
        torch.cuda.synchronize()

    def run_timed(self, steps, attention_events=False):
        """`steps` steps replayed from the graphs; L2 flushed before each; the CUDA events inside the graph bracket
        the whole step (and, with attention_events, the attention call) on the stream the kernels run on (the flush
        and the graph's launch latency are outside both).  Returns (total_ms, attn_ms, attn_bytes, attn_flops,
        kernel launches); attn_ms is 0 without attention_events."""
        tot = attn = 0.0
        launches = 0
        nbytes = nflops = 0
        for _ in range(steps):
            st = self.sched.at(self.t)
            if st["step_in_block"] == 0:
                self.reset_block_state(st)
            g, ev, n = (self.graphs if attention_events else self.graphs_step)[self.t % self.N_POOL][1 if st["last"] else 0]
            self.flush.zero_()                      # evict L2 between timed steps
            g.replay()
            ev[2].synchronize()
            tot += ev[0].elapsed_time(ev[2])
            if attention_events:
                attn += ev[0].elapsed_time(ev[1])
            launches += n
            nbytes += attn_bytes(self.cfg, st["cache_len"])
            nflops += attn_flops(self.cfg, st["cache_len"])
            self.t += 1
        torch.cuda.synchronize()
        return tot, attn, nbytes, nflops, launches

    def run(self, steps, e2e=False, host=None):
        """Direct (uncaptured) calls: warm-up, and the end-to-end leg with host buffers.  Returns wall ms."""
        tot = 0.0
        for _ in range(steps):
            st = self.sched.at(self.t)
            if st["step_in_block"] == 0 or not e2e:
                self.reset_block_state(st)
            if e2e:
                hq, hk, hv, hl, h_sel, h_n, h_tok = host
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                q, kn, vn = (x.to(self.dev, non_blocking=True) for x in (hq, hk, hv))
                lg = hl.to(self.dev, non_blocking=True)
                self.launch_step(st, (q, kn, vn), lg)
                h_sel.copy_(self.sel_idx, non_blocking=True)
                h_n.copy_(self.n_sel, non_blocking=True)
                h_tok.copy_(self.tokens, non_blocking=True)
                torch.cuda.synchronize()
                tot += (time.perf_counter() - t0) * 1e3
            else:
                self.launch_step(st)
            self.t += 1
        torch.cuda.synchronize()
        return tot

    # ---- single-kernel measurements reported beside the step (same inputs, L2 flushed before each launch)
    def time_call(self, fn, reps=10):
        evs = []
        for _ in range(reps):
            self.flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        ts = sorted(a.elapsed_time(b) for a, b in evs)
        return ts[len(ts) // 2] * 1e-3

    def per_layer_attention(self):
        """The attention of one step issued the way a real model would: one call per layer, here all in one graph,
        at the first step's lengths (the headline number uses the layer-batched call, which only a synthetic stack,
        whose layers' Q/K/V all exist up front, can make)."""
        dlm, cfg = self.dlm, self.cfg
        st = self.sched.at(0)
        self.reset_block_state(st)
        q, kn, vn = self.pool[0]
        ws = torch.empty(max(dlm.dlm_attn_workspace_bytes(self.ctx, self.cache, 1, cfg.n_q_heads, cfg.block_len), 256),
                         dtype=torch.uint8, device=self.dev)

        def layers():
            for l in range(cfg.n_layers):
                dlm.dlm_freecache_attn_step(self.ctx, self.cache, l, l + 1, q[l:l + 1], kn[l:l + 1], vn[l:l + 1], cfg.n_q_heads,
                                            cfg.block_len, self.q_len if self.guided else None, 0.0, st["cache_len"],
                                            self.out[l:l + 1], None, ws)
        layers()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=torch.cuda.Stream()):
            layers()
        t = self.time_call(g.replay)
        sch = dlm.dlm_selftest_attn_schedule(self.ctx, self.cache, 1, cfg.n_q_heads, cfg.block_len, st["cache_len"])
        return {"us_per_step": t * 1e6, "us_per_layer": t * 1e6 / cfg.n_layers, "calls": cfg.n_layers,
                "schedule": ("team of %d blocks per unit" % sch["team"]) if sch["team"] > 1 else
                            ("whole units" if sch["whole_units"] else "units split across blocks"),
                "grid": sch["grid"], "rows_per_unit": sch["chunk_rows"]}

    def other_kernels(self, peak_gbs):
        """HBM-bound kernels of the path, each timed alone: the unmask pass over a fully masked block and the cache
        refresh that (re)writes the whole prompt.  `us` is one launch from a captured graph after an L2 flush, with
        the graph's launch gap inside the events; `us_back_to_back` is the average over launches running back to
        back on rotating input sets larger than L2 (time_rotating), and `frac` is taken from that one."""
        dlm, cfg = self.dlm, self.cfg
        B, Lblk, V = cfg.batch, cfg.block_len, cfg.vocab
        side = torch.cuda.Stream()
        res = {}
        # unmask over all Lblk rows: k = 0 (propose only) keeps the mask full for every repetition
        self.masked.fill_(1)
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            dlm.dlm_unmask_select(self.ctx, self.logits[0], B, Lblk, V, self.masked, self.tokens, 0, self.tok, self.conf,
                                  None, None, self.unmask_ws)
        t = self.time_call(g.replay)
        nb = B * Lblk * V * 4
        n_sets = sets_needed(nb)
        pool = list(self.logits) + [make_logits(B, Lblk, V, cfg.logit_sigma, seed_for(0) + 50 + i, self.dev)
                                    for i in range(max(0, n_sets - len(self.logits)))]
        tb = time_rotating([(lambda lg=lg: dlm.dlm_unmask_select(self.ctx, lg, B, Lblk, V, self.masked, self.tokens, 0,
                                                                 self.tok, self.conf, None, None, self.unmask_ws))
                            for lg in pool[:n_sets]])
        del pool
        res["unmask_full_block"] = {"us": t * 1e6, "us_back_to_back": tb * 1e6, "input_sets": n_sets, "algorithmic_bytes": nb,
                                    "GB/s": nb / tb / 1e9, "frac": nb / tb / 1e9 / peak_gbs,
                                    "GB/s_single_launch": nb / t / 1e9}
        # prompt refresh: rows [0, prompt_len) of every layer rewritten from a source of the same shape (identity
        # placement: dst_pos NULL, rows appended from slot 0 of an empty cache view)
        shape = (cfg.n_layers, B, cfg.n_kv_heads, cfg.prompt_len, cfg.head_dim)
        nb = 2 * 2 * cfg.n_layers * B * cfg.n_kv_heads * cfg.prompt_len * cfg.head_dim * 2
        zero_len = torch.zeros(B, dtype=torch.int32, device=self.dev)
        n_sets = sets_needed(nb)
        srcs = [(make_kv_rows(shape, 5 + 2 * i, self.dev), make_kv_rows(shape, 6 + 2 * i, self.dev)) for i in range(n_sets)]
        caches = [self.cache] + [dlm.make_kv_cache(torch.empty_like(self.ck), torch.empty_like(self.cv), zero_len)
                                 for _ in range(n_sets - 1)]
        view0 = dlm.make_kv_cache(self.ck, self.cv, zero_len)      # the bench's cache seen as empty: append = refresh
        caches[0] = view0

        def refresh(i):
            dlm.dlm_kv_cache_commit(self.ctx, caches[i], srcs[i][0], srcs[i][1], cfg.prompt_len, None, None,
                                    dlm.DLM_DST_APPEND, None, cfg.prompt_len, 0, 0, cfg.n_layers)
        g2 = torch.cuda.CUDAGraph()
        refresh(0)
        torch.cuda.synchronize()
        with torch.cuda.graph(g2, stream=side):
            refresh(0)
        t = self.time_call(g2.replay)
        tb = time_rotating([(lambda i=i: refresh(i)) for i in range(n_sets)])
        res["commit_prompt_refresh"] = {"us": t * 1e6, "us_back_to_back": tb * 1e6, "input_sets": n_sets, "algorithmic_bytes": nb,
                                        "GB/s": nb / tb / 1e9, "frac": nb / tb / 1e9 / peak_gbs,
                                        "GB/s_single_launch": nb / t / 1e9}
        del srcs, caches
        return res

    def attention_back_to_back(self, peaks):
        """The layer-batched attention launch of the first step, back to back over rotating caches and inputs
        larger than L2 (time_rotating): the kernel's sustained rate without the timing events of the step graph
        around every launch."""
        dlm, cfg = self.dlm, self.cfg
        st = self.sched.at(0)
        self.reset_block_state(st)
        per_set = attn_bytes(cfg, st["cache_len"])
        n_sets = sets_needed(per_set)
        sets = [(self.cache, self.pool[0], self.out)]
        for i in range(1, n_sets):
            ck, cv = torch.empty_like(self.ck).copy_(self.ck), torch.empty_like(self.cv).copy_(self.cv)
            sets.append((dlm.make_kv_cache(ck, cv, self.cache_len), self.pool[i % self.N_POOL] if i < self.N_POOL else
                         tuple(torch.empty_like(x).copy_(x) for x in self.pool[0]), torch.empty_like(self.out)))

        def call(cache, qkv, out):
            dlm.dlm_freecache_attn_step(self.ctx, cache, 0, cfg.n_layers, qkv[0], qkv[1], qkv[2], cfg.n_q_heads, cfg.block_len,
                                        self.q_len if self.guided else None, 0.0, st["cache_len"], out, None, self.attn_ws)
        t = time_rotating([(lambda c=c, q=q, o=o: call(c, q, o)) for c, q, o in sets], min_launches=16)
        del sets
        fl = attn_flops(cfg, st["cache_len"])
        t_roof = max(per_set / (peaks["hbm_gbs"] * 1e9), fl / (peaks["bf16_tflops"] * 1e12))
        return {"us_per_launch": t * 1e6, "input_sets": n_sets, "algorithmic_bytes": per_set, "GB/s": per_set / t / 1e9,
                "TFLOP/s": fl / t / 1e12, "frac_of_roofline": t_roof / t}


def max_over_ranks(values, device, world):
    """Element-wise maximum of per-rank timings over all ranks (the job runs as slow as its slowest rank)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(world, steps, total_ms):
    """Whole-job steps/s: every rank runs `steps` steps of its own replica in `total_ms` (max over ranks)."""
    return world * steps / (total_ms * 1e-3)


def cpu_oracle_sample(cfg, cfg_index, n_layers_sample):
    """Times the CPU oracle, as it stands, on a bounded sample of one denoising step: attention for
    `n_layers_sample` of the layers at the first step's lengths, one unmask over the full block and one
    4-row commit; extrapolates to a whole step."""
    import oracle
    s = seed_for(cfg_index)
    B, Lblk = cfg.batch, cfg.block_len
    ck, cv = make_cache(1, B, cfg.n_kv_heads, cfg.capacity, cfg.head_dim, s)
    q, kn, vn = make_attn_inputs(1, B, cfg.n_q_heads, cfg.n_kv_heads, Lblk, cfg.head_dim, s + 1)
    args = (widen(ck[0]), widen(cv[0]), np.full((B,), cfg.prompt_len, np.int32), widen(q[0]), widen(kn[0]), widen(vn[0]))
    t0 = time.perf_counter()
    for _ in range(n_layers_sample):
        oracle.attn_step(*args)
    t_attn = (time.perf_counter() - t0) / n_layers_sample
    logits = make_logits(B, Lblk, cfg.vocab, cfg.logit_sigma, s + 10).numpy()
    masked, tokens = np.ones((B, Lblk), np.uint8), np.zeros((B, Lblk), np.int32)
    cks, cvs = bf16_bits(ck), bf16_bits(cv)
    knb, vnb = bf16_bits(kn), bf16_bits(vn)
    lens = np.full((B,), cfg.prompt_len, np.int32)
    if cfg.policy == "guided":
        from workloads import make_tok_ar
        t0 = time.perf_counter()
        tok, _, _, _ = oracle.unmask_select(logits, masked, tokens, 0)
        tok_ar = make_tok_ar(torch.from_numpy(tok), cfg.p_agree, cfg.vocab, s + 20).numpy()
        _, idx, n = oracle.guided_accept(tok, tok_ar, masked, tokens, 0)
        t_unmask = time.perf_counter() - t0
        t0 = time.perf_counter()
        oracle.kv_cache_commit(cks, cvs, lens, knb, vnb, idx, None, n, Lblk, True)
        t_commit = (time.perf_counter() - t0) * cfg.n_layers
        what = "one propose + guided accept"
    else:
        t0 = time.perf_counter()
        _, _, sel, n = oracle.unmask_select(logits, masked, tokens, cfg.top_k)
        t_unmask = time.perf_counter() - t0
        t0 = time.perf_counter()
        oracle.kv_cache_commit(cks, cvs, lens, knb, vnb, sel, None, n, cfg.top_k, dst_mode=1)
        t_commit = (time.perf_counter() - t0) * cfg.n_layers
        what = "one unmask"
    step_s = cfg.n_layers * t_attn + t_unmask + t_commit
    return {"value": 1.0 / step_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"attention of {n_layers_sample} of {cfg.n_layers} layers at cache_len {cfg.prompt_len} "
                      f"(x{cfg.n_layers}/{n_layers_sample}), {what} over {B}x{Lblk}x{cfg.vocab} logits, one commit of the chosen rows",
            "seconds_per_step": step_s}


WINDOW_CONFIGS = {
    # name: (base config, cached rows, active rows): the paper's own window (all remaining generation rows are
    # recomputed every step) and its initial full pass; tensor-bound shapes of the same attention kernel
    "dream7b_window256": ("dream7b", 1024, 256),
    "dream7b_prefill1280": ("dream7b", 0, 1280),
    "llada8b_window512": ("llada8b", 2048, 512),
}


def bench_window(name, args, rank, world, local_rank):
    """Attention of a large active window (Sec. 3.2.1: the window holds every row not yet frozen; the initial pass
    holds the whole sequence): one layer-batched launch per step, timed back to back over rotating input sets."""
    base, cached, q_cap = WINDOW_CONFIGS[name]
    cfg = get_config(base)
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    import paper_2505_21467_b200 as dlm
    from paper_2505_21467_b200 import build as _b
    _b.build()
    ctx = dlm.dlm_create(device.index)
    B, NL, Hq, Hkv, D = cfg.batch, cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    cap = max(cached, 128)
    kv_bytes = 2 * 2 * NL * B * Hkv * (cached + q_cap) * D
    qo_bytes = 2 * 2 * NL * B * Hq * q_cap * D
    flops = 4 * NL * B * Hq * q_cap * (cached + q_cap) * D
    n_sets = sets_needed(kv_bytes + qo_bytes)
    cache_len = torch.full((B,), cached, dtype=torch.int32, device=device)
    sets = []
    for i in range(n_sets):
        ck, cv = make_cache(NL, B, Hkv, cap, D, 900 + i, device)
        q, kn, vn = make_attn_inputs(NL, B, Hq, Hkv, q_cap, D, 950 + i, device)
        sets.append((dlm.make_kv_cache(ck, cv, cache_len), q, kn, vn, torch.empty_like(q)))
    ws = torch.empty(max(dlm.dlm_attn_workspace_bytes(ctx, sets[0][0], NL, Hq, q_cap), 256), dtype=torch.uint8, device=device)

    def call(c, q, kn, vn, out):
        dlm.dlm_freecache_attn_step(ctx, c, 0, NL, q, kn, vn, Hq, q_cap, None, 0.0, cached, out, None, ws)
    c0 = dlm.dlm_launch_count(ctx)
    sampler = ClockSampler(local_rank)
    sampler.start()
    calls = [(lambda x=x: call(*x)) for x in sets]
    for _ in range(max(args.warmup, 3)):
        calls[0]()
    torch.cuda.synchronize()
    sampler.mark()
    t = time_rotating(calls, min_launches=max(args.steps, len(calls)), replays=3)
    clocks = sampler.stop()
    launches = dlm.dlm_launch_count(ctx) - c0
    status = dlm.dlm_get_status(ctx)
    if status != 0:
        raise SystemExit(f"device status {status}: {dlm.dlm_strerror(status)}")
    peaks = measured_peaks()
    t_flops, t_bytes = flops / (peaks["bf16_tflops"] * 1e12), (kv_bytes + qo_bytes) / (peaks["hbm_gbs"] * 1e9)
    bound = "tensor" if t_flops >= t_bytes else "hbm"
    ach = flops / t / 1e12 if bound == "tensor" else (kv_bytes + qo_bytes) / t / 1e9
    peak = peaks["bf16_tflops"] if bound == "tensor" else peaks["hbm_gbs"]
    print(json.dumps({
        "metric": "attention_window_steps_per_s", "value": world / t, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{name}: {base}-shaped attention stack, batch {B} per GPU, {NL} layers, {Hq}q/{Hkv}kv heads x {D}, "
                               f"{cached} cached rows + {q_cap} active rows, attention only",
                   "l2": f"{n_sets} input sets rotated, larger than L2 together; launches back to back",
                   "launch": "CUDA graph of the C-ABI calls, events around the replays"},
        "clocks": clocks, "gpu_launches": int(launches),
        "roofline": {"kernel": "attention step (all layers, one launch)", "bound": bound, "achieved": ach, "peak": peak,
                     "unit": "TFLOP/s" if bound == "tensor" else "GB/s", "frac": ach / peak, "peak_source": peaks["source"],
                     "traffic": ATTN_DRAM_TRAFFIC_BYTES.get(name), "us_per_launch": t * 1e6, "flops_per_launch": flops,
                     "algorithmic_bytes_per_launch": kv_bytes + qo_bytes}}))


PROJ_CONFIGS = {
    # name: (base config, d_model, rows per sequence): the window's fused Q/K/V projection and its output projection,
    # one call per layer over the layers' own weights (so every call streams weights that are not in L2)
    "dream7b_proj32": ("dream7b", 3584, 32),
    "dream7b_proj256": ("dream7b", 3584, 256),
    "llada8b_proj64": ("llada8b", 4096, 64),
}


def bench_proj(name, args, rank, world, local_rank):
    """Fused Q/K/V projection (and the output projection) of the active window with random weights of the model's
    widths: a step is one pass over all layers, one call per layer."""
    base, dm, q_cap = PROJ_CONFIGS[name]
    cfg = get_config(base)
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    import paper_2505_21467_b200 as dlm
    from paper_2505_21467_b200 import build as _b
    _b.build()
    ctx = dlm.dlm_create(device.index)
    B, NL, Hq, Hkv, D = cfg.batch, cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    if B * q_cap > 256:
        B = max(1, 256 // q_cap)
    n_out = (Hq + 2 * Hkv) * D
    gen = torch.Generator(device).manual_seed(4242)
    w = (torch.randn(NL, n_out, dm, generator=gen, device=device) * dm ** -0.5).to(torch.bfloat16)
    wo = (torch.randn(NL, dm, Hq * D, generator=gen, device=device) * (Hq * D) ** -0.5).to(torch.bfloat16)
    x = make_kv_rows((B, q_cap, dm), 7, device)
    q = torch.empty(B, Hq, q_cap, D, dtype=torch.bfloat16, device=device)
    k = torch.empty(B, Hkv, q_cap, D, dtype=torch.bfloat16, device=device)
    v = torch.empty_like(k)
    y = torch.empty(B, q_cap, dm, dtype=torch.bfloat16, device=device)
    ws = torch.empty(max(dlm.dlm_window_proj_workspace_bytes(ctx, B * q_cap, n_out, dm),
                         dlm.dlm_window_proj_workspace_bytes(ctx, B * q_cap, dm, Hq * D), 256), dtype=torch.uint8, device=device)
    sampler = ClockSampler(local_rank)
    sampler.start()
    c0 = dlm.dlm_launch_count(ctx)
    qkv_calls = [(lambda l=l: dlm.dlm_window_qkv_project(ctx, x, w[l], None, B, q_cap, dm, Hq, Hkv, D, q, k, v, ws)) for l in range(NL)]
    out_calls = [(lambda l=l: dlm.dlm_window_out_project(ctx, q, wo[l], None, B, q_cap, dm, Hq, D, y, ws)) for l in range(NL)]
    for c in qkv_calls[:3] + out_calls[:3]:
        c()
    torch.cuda.synchronize()
    sampler.mark()
    t_qkv = time_rotating(qkv_calls, min_launches=NL, replays=max(3, args.steps))
    t_out = time_rotating(out_calls, min_launches=NL, replays=max(3, args.steps))
    clocks = sampler.stop()
    launches = dlm.dlm_launch_count(ctx) - c0
    status = dlm.dlm_get_status(ctx)
    if status != 0:
        raise SystemExit(f"device status {status}: {dlm.dlm_strerror(status)}")
    peaks = measured_peaks()

    def roof(t, n, kk):
        rows = B * q_cap
        nbytes, flops = 2 * (n * kk + rows * kk + rows * n), 2 * rows * n * kk
        t_b, t_f = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
        bound = "tensor" if t_f > t_b else "hbm"
        ach, peak = (flops / t / 1e12, peaks["bf16_tflops"]) if bound == "tensor" else (nbytes / t / 1e9, peaks["hbm_gbs"])
        return {"bound": bound, "achieved": ach, "peak": peak, "unit": "TFLOP/s" if bound == "tensor" else "GB/s", "frac": ach / peak,
                "peak_source": peaks["source"], "us_per_launch": t * 1e6, "algorithmic_bytes_per_launch": nbytes,
                "flops_per_launch": flops, "traffic": None}
    step_s = NL * (t_qkv + t_out)
    print(json.dumps({
        "metric": "window_projection_steps_per_s", "value": world / step_s, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{name}: fused Q/K/V projection and output projection of a {B} x {q_cap}-row window, d_model {dm}, "
                               f"{Hq}q/{Hkv}kv heads x {D}, {NL} layers with their own random weights, one call per layer",
                   "l2": "every call streams another layer's weights; the layers together are larger than L2",
                   "launch": "CUDA graph of the C-ABI calls, launches back to back, events around the replays"},
        "clocks": clocks, "gpu_launches": int(launches),
        "roofline": dict(kernel="window_proj_kernel (fused Q/K/V projection)", **roof(t_qkv, n_out, dm)),
        "other_kernels": {"out_projection": roof(t_out, dm, Hq * D)}}))


def spawn_ranks(n, argv):
    """`python bench.py --gpus N` outside a launcher: start N ranks on this node, one per GPU, the way the
    launcher would (python -m torch.distributed.run), and pass their output through."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="dream7b")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.config in WINDOW_CONFIGS or args.config in PROJ_CONFIGS:
        if args.impl == "reference" or world > 1:
            raise SystemExit("the window and projection configs run on one GPU with --impl ours")
        return (bench_window if args.config in WINDOW_CONFIGS else bench_proj)(args.config, args, rank, world, local_rank)
    cfg = get_config(args.config)
    cfg_index = ["tiny", "dream7b", "llada8b", "longctx", "guided"].index(cfg.name)
    policy = (f"{cfg.steps_per_block} steps/block, vocab {cfg.vocab}, top-{cfg.top_k}" if cfg.policy == "topk" else
              f"guided accept (p_agree {cfg.p_agree}), vocab {cfg.vocab}; every block is given a fixed 8 steps, an approximation of "
              "running each sequence until it finishes")
    config = {"workload": f"{cfg.name}: {'LLaDA-8B' if cfg.name == 'llada8b' else 'Dream-7B'}-shaped attention stack, batch {cfg.batch} per GPU, {cfg.n_layers} layers, "
                          f"{cfg.n_q_heads}q/{cfg.n_kv_heads}kv heads x {cfg.head_dim}, prompt {cfg.prompt_len} + {cfg.n_blocks} blocks of "
                          f"{cfg.block_len}, {policy}",
              "attention_launch": "layer-batched (all layers in one call; synthetic stack)",
              "l2": "flushed between timed steps (512 MB write, outside the timed events)",
              "launch": "each step replayed from one CUDA graph captured from the C-ABI calls, timing event nodes at the two ends of the graph", "parallelism": f"replicated x{world} (independent sequences)"}

    if args.impl == "reference":
        if rank != 0:
            return
        vals = []
        for _ in range(args.warmup):
            cpu_oracle_sample(cfg, cfg_index, 1)
        # each step is a bounded sample (attention of one or two layers, scaled up to all layers); one layer when
        # many steps are asked for, so that the whole run stays within a few minutes
        n_sample = 2 if args.steps <= 64 else 1
        for _ in range(args.steps):
            vals.append(cpu_oracle_sample(cfg, cfg_index, n_sample))
        sec = statistics.mean(v["seconds_per_step"] for v in vals)
        base = dict(vals[-1]); base["value"] = 1.0 / sec
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": 1.0 / sec, "unit": UNIT, "n_gpus": args.gpus,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                          "cpu_baseline": base,
                          "e2e": {"value": 1.0 / sec, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2505_21467_b200 import build as _b
    if rank == 0:
        _b.build()
    if world > 1:
        dist.barrier()
    wl = Workload(cfg, cfg_index, device)
    dlm = wl.dlm

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)   # runs through the warm-up too; the median is over the timed region
    sampler.start()
    wl.run(max(args.warmup, 3))          # direct calls: first-use set-up happens here, outside any capture
    wl.capture()
    wl.t = 0
    wl.run_timed(max(args.warmup, 3))
    wl.t = 0
    wl.run_timed(max(args.warmup, 3), attention_events=True)
    # The timed region: passes of exactly `steps` steps each, repeated until the region has lasted about a
    # second (a single pass of a 60 us step is too short for the clock sampler); the median pass is reported.
    passes = []
    barrier()
    sampler.mark()
    t_region = time.perf_counter()
    while len(passes) < 3 or (time.perf_counter() - t_region < 1.0 and len(passes) < 25):
        wl.t = 0
        passes.append(wl.run_timed(args.steps))
    barrier()
    clocks = sampler.stop()
    passes.sort(key=lambda r: r[0])
    tot_ms, _, nbytes, nflops, launches = passes[len(passes) // 2]
    # the attention launch's own duration: the same steps again, from the graphs that carry an event node after it
    apasses = []
    for _ in range(3):
        wl.t = 0
        apasses.append(wl.run_timed(args.steps, attention_events=True))
    apasses.sort(key=lambda r: r[1])
    tot_attn_ms, attn_ms = apasses[1][0], apasses[1][1]
    status = dlm.dlm_get_status(wl.ctx)
    if status != 0:
        raise SystemExit(f"device status {status}: {dlm.dlm_strerror(status)}")

    # end to end: the step's inputs come from pinned host memory, the result goes back
    pin = lambda t: t.cpu().pin_memory()  # noqa: E731
    q, kn, vn = wl.pool[0]
    host = (pin(q), pin(kn), pin(vn), pin(wl.logits[0]), pin(wl.sel_idx), pin(wl.n_sel), pin(wl.tokens))
    h2d = sum(x.numel() * x.element_size() for x in host[:4])
    d2h = sum(x.numel() * x.element_size() for x in host[4:])
    wl.t = 0
    wl.run(3, e2e=True, host=host)
    wl.t = 0
    e2e_steps = min(args.steps, 64)
    e2e_ms = wl.run(e2e_steps, e2e=True, host=host)

    tot_ms, attn_ms, e2e_ms, tot_attn_ms = max_over_ranks([tot_ms, attn_ms, e2e_ms, tot_attn_ms], device, world)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    attn_s = attn_ms * 1e-3
    # the roofline of the attention launch: the slower of its bytes at HBM speed and its FLOPs at the bf16 peak
    t_bytes, t_flops = nbytes / (peaks["hbm_gbs"] * 1e9), nflops / (peaks["bf16_tflops"] * 1e12)
    bound = "tensor" if t_flops > t_bytes else "hbm"
    ach = nflops / attn_s / 1e12 if bound == "tensor" else nbytes / attn_s / 1e9
    peak = peaks["bf16_tflops"] if bound == "tensor" else peaks["hbm_gbs"]
    line = {
        "metric": METRIC, "value": job_throughput(world, args.steps, tot_ms), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
        "timed_passes": len(passes), "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": job_throughput(world, e2e_steps, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "roofline": {"kernel": "attention step (all layers, one launch)", "bound": bound, "achieved": ach,
                     "peak": peak, "unit": "TFLOP/s" if bound == "tensor" else "GB/s", "frac": ach / peak,
                     "peak_source": peaks["source"], "traffic": ATTN_DRAM_TRAFFIC_BYTES.get(cfg.name),
                     "protocol": "events inside the step graph around the attention launch, L2 flushed before the step; a pass of "
                                 "its own over the same steps, because the event node after the launch lengthens the step",
                     "ms_per_step_with_that_event": tot_attn_ms / args.steps,
                     "attn_us_per_launch": attn_ms * 1e3 / args.steps,
                     "attn_tflops": nflops / attn_s / 1e12, "attn_GB/s": nbytes / attn_s / 1e9,
                     "frac_of_bytes_roof": t_bytes / attn_s, "frac_of_flops_roof": t_flops / attn_s,
                     "algorithmic_bytes_per_launch": nbytes / args.steps,
                     "back_to_back": wl.attention_back_to_back(peaks)},
        "other_kernels": wl.other_kernels(peaks["hbm_gbs"]),
        "attention_per_layer_calls": wl.per_layer_attention(),
        "cpu_baseline": cpu_oracle_sample(cfg, cfg_index, max(1, min(4, int(2.5e9 / max(attn_flops(cfg, cfg.prompt_len) / cfg.n_layers, 1))))),
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
