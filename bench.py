#!/usr/bin/env python
"""Benchmark of the WnW decode hot path on B200.

One "step" is one generated token: the whole hot path (text append, anchor attention with fused chunk scores,
split merge, top-k selection, residency update, recall, tidal and fixed sparse attention) for every layer of the
stack, through the C ABI.  Workload at one GPU: the 3B Voxtral-shaped stack of the configuration list (30 layers,
32 q / 8 KV heads, head_dim 128, 3000 audio + 64 text tokens, chunk 64, 20 % audio budget, batch 1), synthetic
seeded inputs.  With N GPUs every rank serves its own sequence (no data-path collective): weak scaling.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg1|cfg3]

Prints ONE JSON line on rank 0.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from workloads import ROLE_ANCHOR, ROLE_FIXED, ROLE_TIDAL, Synth, config1, config2, config3, config4
from workloads.synth import bf16_bits

METRIC = "wnw_decode_tokens_per_s_at_20pct_audio_budget"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 512 << 20
SWEEP_STEPS_OVERRIDE = 0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def make_workload(name: str, n_steps: int, seed: int):
    if name == "cfg1":
        w = config1(seed=0, n_steps=n_steps)
    elif name == "cfg2":
        w = config2(seed=0, n_steps=n_steps)
    elif name == "cfg3":
        w = config3(seed=0, n_steps=n_steps)
    elif name in ("prof", "hbm"):   # many long sequences, config-1 heads: 4 layers (profiler captures) or 12 layers (HBM-bound case)
        n_l = 4 if name == "prof" else 12
        w = config4(seed=0, budget=0.2, chunk=64, batch=16, n_steps=n_steps)
        w.n_layers = n_l; w.roles = w.roles[:n_l]; w.jump_every = 0; w.sweep_steps = 128; w.name = f"{name}_{n_l}layers_b16_7500"
    elif name.startswith("b") and "x" in name:   # b<batch>x<audio tokens>[L<layers>]: config-1 heads, 12 layers unless given
        nb, na = name[1:].split("x")
        n_l = 12
        if "L" in na:
            na, n_l = na.split("L")
        n_l = int(n_l)
        w = config4(seed=0, budget=0.2, chunk=64, batch=int(nb), n_steps=n_steps)
        w.audio_lens = [int(na)] * int(nb)
        w.n_layers = n_l; w.roles = w.roles[:n_l]; w.jump_every = 0; w.sweep_steps = 256; w.name = f"cfg1heads_{n_l}layers_{name}"
    else:
        raise SystemExit(f"unknown workload {name}")
    if SWEEP_STEPS_OVERRIDE:
        w.sweep_steps = SWEEP_STEPS_OVERRIDE   # slower or faster drift of the decode focus through the clip
        w.name += f"_sweep{SWEEP_STEPS_OVERRIDE}"
    return w


# ------------------------------------------------------------------------------------------------- multi-rank helpers
def shard_plan(world: int, batch_per_rank: int) -> dict:
    """The path shards by sequence: every rank serves its own sequences on its own GPU with no data-path collective,
    so the whole job is `world` independent replicas of the per-rank workload (weak scaling)."""
    return {"scaling": "weak", "sequences_per_rank": batch_per_rank, "total_sequences": world * batch_per_rank,
            "collective": None}


def dist_max(x: float, device, world: int) -> float:
    """Max over ranks of a device-timed duration (the only cross-rank exchange; not on the data path)."""
    if world <= 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, batch_per_rank: int, ms_per_step_max: float) -> float:
    """All ranks step together; the job emits world * batch tokens per step, paced by the slowest rank."""
    return world * batch_per_rank / (ms_per_step_max * 1e-3)


# ------------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.gpu)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [x for x in sm if x > 0.5 * max(sm)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------- job state
class Job:
    """Caches, resident inputs and launch helpers of one rank."""

    layer_dependency = 3   # WNW_LAYERS_*: how the layers of a step are issued (set from --layer-dependency)
    kv_fp8 = False         # tiered caches keep their tidal tier as e4m3 (set from --tidal-kv fp8)

    def __init__(self, w, seed, device, wnw, score_scope=0, residency=0, evict_lag=3):
        self.score_scope = score_scope
        self.residency, self.evict_lag = residency, evict_lag
        self.w, self.dev, self.wnw = w, device, wnw
        self.syn = Synth(w, seed=seed, device=str(device))
        self.B = w.batch
        self.caches = {}
        self.fp8_keys = set()
        L, n = w.n_layers, w.n_steps
        # decode inputs resident in HBM; one step is one contiguous slab [q of all layers | k_new | v_new]
        nq, nk = L * self.B * w.n_q_heads * w.head_dim, L * self.B * w.n_kv_heads * w.head_dim
        self.slab = torch.empty((n, nq + 2 * nk), dtype=torch.bfloat16, device=device)
        self.q = self.slab[:, :nq].view(n, L, self.B, w.n_q_heads, w.head_dim)
        self.kn = self.slab[:, nq:nq + nk].view(n, L, self.B, w.n_kv_heads, w.head_dim)
        self.vn = self.slab[:, nq + nk:].view(n, L, self.B, w.n_kv_heads, w.head_dim)
        for b in range(self.B):
            for l in range(L):
                d = self.syn.decode(b, l)
                self.q[:, l, b] = d["q"]; self.kn[:, l, b] = d["k_new"]; self.vn[:, l, b] = d["v_new"]
        # static buffers a captured step reads from / writes to (a producer kernel would fill them in a real decoder)
        self.sslab = torch.zeros(nq + 2 * nk, dtype=torch.bfloat16, device=device)
        self.sq = self.sslab[:nq].view(L, self.B, w.n_q_heads, w.head_dim)
        self.skn = self.sslab[nq:nq + nk].view(L, self.B, w.n_kv_heads, w.head_dim)
        self.svn = self.sslab[nq + nk:].view(L, self.B, w.n_kv_heads, w.head_dim)
        self.out = torch.zeros((L, self.B, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device=device)
        self.flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
        self.flush_buf2 = torch.zeros(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
        self.stream = torch.cuda.Stream(device=device)
        self.captured = set()

    def create(self, key, mode, recall_mode=0, layer_dependency=None, kv_fp8=None):
        """kv_fp8: the tidal tier (host mirror, slot pool) as e4m3 with a scale per chunk; default: the job's setting."""
        w, wnw = self.w, self.wnw
        kv_fp8 = Job.kv_fp8 if kv_fp8 is None else kv_fp8
        h = wnw.wnw_create(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, self.B, max(w.audio_lens), w.text_capacity,
                           w.chunk, w.budget, w.roles, topk=w.topk, device=self.dev.index or 0, mode=mode,
                           recall_mode=recall_mode, score_scope=self.score_scope, residency=self.residency,
                           evict_lag=self.evict_lag,
                           tidal_kv_format=wnw.WNW_TIDAL_KV_FP8_E4M3 if kv_fp8 and mode == wnw.WNW_MODE_TIERED else wnw.WNW_TIDAL_KV_BF16)
        if kv_fp8 and mode == wnw.WNW_MODE_TIERED:
            self.fp8_keys.add(key)
        wnw.wnw_set_layer_dependency(h, Job.layer_dependency if layer_dependency is None else layer_dependency)
        self.caches[key] = h
        return h

    def place_all(self, keys, keep_host=None, token=None):
        """Generates each (seq, layer) prefill once on the device and places it into every cache in `keys`.
        token = (retention [n_layers][n_kv_heads], segment_tokens, variant): fixed heads compressed token by token."""
        w, wnw = self.w, self.wnw
        for b in range(self.B):
            for l in range(w.n_layers):
                p = self.syn.prefill(b, l)
                for key in keys:
                    if token is not None:
                        wnw.wnw_place_prefill_tokens(self.caches[key], b, l, p["k"], p["v"], p["audio_begin"], p["audio_end"],
                                                     p["q_last"][None], token[0][l], token[1], token[2])
                    else:
                        wnw.wnw_place_prefill(self.caches[key], b, l, p["k"], p["v"], p["audio_begin"], p["audio_end"], p["q_last"])
                if keep_host is not None and keep_host(b, l):
                    keep_host.store[(b, l)] = (bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_last"]), p["audio_begin"],
                                               p["audio_end"])
                torch.cuda.synchronize(self.dev)
        for key in keys:
            wnw.wnw_sync(self.caches[key])

    def flush_l2(self):
        """Writes a buffer larger than L2, then reads another one: the write evicts every cached input, the read
        evicts the dirty lines the write left behind, so the timed step starts on a cold and clean L2 (otherwise its
        first 126 MB of reads also pay for the write-back of the flush's own lines)."""
        self.flush_buf.fill_(1)
        self.flush_sink = self.flush_buf2.view(torch.int32).sum()

    def step(self, key, t, full=False, q=None, kn=None, vn=None, out=None):
        wnw, h = self.wnw, self.caches[key]
        q = self.q[t] if q is None else q
        kn = self.kn[t] if kn is None else kn
        vn = self.vn[t] if vn is None else vn
        out = self.out if out is None else out
        fn = wnw.wnw_decode_layer_full if full else wnw.wnw_decode_layer
        wnw.wnw_step_begin(h, list(range(self.B)))
        for l in range(self.w.n_layers):
            fn(h, l, q[l], kn[l], vn[l], out[l])
        wnw.wnw_step_end(h)

    def capture(self, key, full=False):
        """Captures one step of cache `key` on the job's stream as a CUDA graph that reads the static buffers."""
        wnw, h = self.wnw, self.caches[key]
        torch.cuda.synchronize(self.dev)
        wnw.wnw_graph_begin(h, list(range(self.B)), self.stream)
        fn = wnw.wnw_decode_layer_full if full else wnw.wnw_decode_layer
        wnw.wnw_step_begin(h, list(range(self.B)))
        for l in range(self.w.n_layers):
            fn(h, l, self.sq[l], self.skn[l], self.svn[l], self.out[l], stream=self.stream)
        wnw.wnw_step_end(h, stream=self.stream)
        wnw.wnw_graph_end(h, self.stream)
        self.captured.add(key)

    def stage_inputs(self, t, src=None):
        """Puts a step's inputs where the captured step reads them (the static buffers): one copy."""
        self.sslab.copy_(self.slab[t] if src is None else src, non_blocking=True)

    def graph_step(self, key, t, src=None):
        """One replayed step from host or device inputs: the copy into the static buffers, then one graph launch."""
        self.stage_inputs(t, src)
        self.wnw.wnw_graph_launch(self.caches[key], self.stream)

    def timed_steps(self, key, t0, n, full=False, flush=True, graph=True):
        """Device time of n consecutive steps, L2 flushed (untimed) before each.  Returns per-step ms.
        graph=True replays the captured step; otherwise the layers are issued eagerly."""
        if graph and key not in self.captured:
            self.capture(key, full=full)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        with torch.cuda.stream(self.stream):
            for i in range(n):
                # a replayed step reads its inputs from the static buffers: they are resident there (in HBM: the flush
                # follows) before the timed region starts; the eager step reads them where they are
                if graph:
                    self.stage_inputs(t0 + i)
                if flush:
                    self.flush_l2()
                evs[i][0].record()
                if graph:
                    self.wnw.wnw_graph_launch(self.caches[key], self.stream)
                else:
                    self.step(key, t0 + i, full=full)
                evs[i][1].record()
        torch.cuda.synchronize(self.dev)
        return [a.elapsed_time(b) for a, b in evs]

    def timed_region(self, key, t0, n, full=False):
        """Device time of n consecutive replayed steps in ONE event bracket, nothing between them but the copy of the
        next step's inputs into the static buffers: continuous decoding, in which the recall of a step overlaps the
        next step and has to pay for what it cannot hide.  No L2 flush: for use where one step reads more than L2
        holds.  Returns ms per step."""
        if key not in self.captured:
            self.capture(key, full=full)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            self.flush_l2()
            a.record()
            for i in range(n):
                self.stage_inputs(t0 + i)
                self.wnw.wnw_graph_launch(self.caches[key], self.stream)
            b.record()
        torch.cuda.synchronize(self.dev)
        self.wnw.wnw_sync(self.caches[key])
        return a.elapsed_time(b) / n

    def kv_bytes_of_step(self, key, full=False):
        """Algorithmic K,V bytes one step reads: 4*d bytes per (KV head, visible token), summed over layers; from the
        residency tables as they stand (the tables the next step's attention will use)."""
        w, wnw, h = self.w, self.wnw, self.caches[key]
        total = 0
        per_layer = []
        half_tok = 0
        for l in range(w.n_layers):
            lb = 0
            for b in range(self.B):
                T_a, T_t, C, S = wnw.wnw_get_seq_dims(h, b)
                T_t += 1  # the appended token is visible to its own step
                clen = lambda c: min(w.chunk, T_a - c * w.chunk)
                if full:
                    tok = w.n_kv_heads * (T_t + T_a)
                else:
                    roles = w.roles[l]
                    tok = int((roles == ROLE_ANCHOR).sum()) * (T_t + T_a)
                    n_tid = int((roles == ROLE_TIDAL).sum())
                    if n_tid:
                        tab, _ = wnw.wnw_get_residency(h, b, l)
                        res = sum(clen(c) for c in tab.tolist() if c >= 0)
                        if key in self.fp8_keys:      # an e4m3 slot row is d bytes for K and d for V: half a bf16 row
                            tok += n_tid * T_t
                            half_tok += n_tid * res
                        else:
                            tok += n_tid * (T_t + res)
                    for hh in np.nonzero(roles == ROLE_FIXED)[0]:
                        tok += T_t + sum(clen(c) for c in wnw.wnw_get_fixed_set(h, b, l, int(hh)).tolist())
                lb += tok * 4 * w.head_dim + half_tok * 2 * w.head_dim
                half_tok = 0
            per_layer.append(lb)
            total += lb
        return total, per_layer

    def set_dependency(self, keys, dep):
        """Switches how the layers of a step are issued for the given caches (a captured step keeps the form it was
        captured with, so the captures are dropped)."""
        for key in keys:
            self.wnw.wnw_sync(self.caches[key])
            self.wnw.wnw_set_layer_dependency(self.caches[key], dep)
            self.captured.discard(key)

    def regen_queries(self, sweep_steps):
        """New decode queries whose focus crosses the clip in `sweep_steps` steps (k_new, v_new stay)."""
        self.w.sweep_steps = sweep_steps
        for b in range(self.B):
            for l in range(self.w.n_layers):
                self.q[:, l, b] = self.syn.decode(b, l)["q"]

    def rows_fetched_and_visible(self, key):
        """(rows the kernels fetch, rows that are visible) per step of a batch-1 cache whose non-anchor heads keep a
        token-granular base: every store keeps a chunk or segment of n tokens in ceil(n / 16) * 16 rows and the kernels
        fetch whole 16-row granules of whatever is resident, so short segments move padding."""
        w, wnw, h = self.w, self.wnw, self.caches[key]
        pad = lambda n: -(-n // 16) * 16
        T_a, T_t, C, S = wnw.wnw_get_seq_dims(h, 0)
        T_t += 1
        st = wnw.wnw_get_stats(h)
        visible = st["resident_audio_tokens"] + w.n_layers * w.n_kv_heads * T_t
        fetched = 0
        for l in range(w.n_layers):
            tab = None
            for hh in range(w.n_kv_heads):
                role = w.roles[l, hh]
                fetched += pad(T_t)
                if role == ROLE_ANCHOR:
                    fetched += C * pad(w.chunk)
                    continue
                kept = len(wnw.wnw_get_fixed_tokens(h, 0, l, hh))
                fetched += -(-kept // w.chunk) * pad(w.chunk)
                if role == ROLE_TIDAL:
                    if tab is None:
                        tab, _ = wnw.wnw_get_residency(h, 0, l)
                    fetched += int((tab >= 0).sum()) * pad(w.chunk)
        return fetched, visible

    def destroy(self):
        for h in self.caches.values():
            self.wnw.wnw_destroy(h)
        self.caches.clear()


# ------------------------------------------------------------------------------------------------- oracle timing
def time_oracle(w, store, syn_dec, n_layers_sample, n_steps, warm, seqs):
    """Times the CPU oracle, as it stands, on the first `n_layers_sample` layers of the workload for `n_steps` decode
    steps of the sequences in `seqs`; returns (seconds per sampled step, threads)."""
    from oracle.wnw_oracle import Oracle
    threads = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    Ls = n_layers_sample
    o = Oracle(Ls, w.n_q_heads, w.n_kv_heads, w.head_dim, len(seqs), max(w.audio_lens), w.text_capacity, w.chunk, w.topk,
               w.budget, w.roles[:Ls])
    for i, b in enumerate(seqs):
        for l in range(Ls):
            kb, vb, qb, ab, ae = store[(b, l)]
            o.place_prefill(i, l, kb, vb, ab, ae, qb)
    times = []
    for t in range(warm + n_steps):
        t0 = time.perf_counter()
        o.step_begin(list(range(len(seqs))))
        for l in range(Ls):
            q, kn, vn = syn_dec(t, l, seqs)
            o.decode_layer(l, q, kn, vn)
        o.step_end()
        if t >= warm:
            times.append(time.perf_counter() - t0)
    o.close()
    return sum(times) / len(times), threads


# ------------------------------------------------------------------------------------------------- main arms
def run_reference(args, rank, world):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    total = args.steps + args.warmup
    w = make_workload(args.workload, max(total, 3), 0)   # the probe below runs three steps
    syn = Synth(w, seed=0, device="cpu")
    threads = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    # bound the run: sample the first Ls layers of sequence 0 so that (K+W) steps stay within about two minutes
    probe_layers = 1
    store = {}
    for l in range(probe_layers):
        p = syn.prefill(0, l)
        store[(0, l)] = (bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_last"]), p["audio_begin"], p["audio_end"])
    dec = {}

    def syn_dec(t, l, seqs):
        if l not in dec:
            d = syn.decode(0, l)
            dec[l] = (bf16_bits(d["q"]), bf16_bits(d["k_new"]), bf16_bits(d["v_new"]))
        q, kn, vn = dec[l]
        return q[t][None], kn[t][None], vn[t][None]

    per_layer_s, _ = time_oracle(w, store, syn_dec, 1, 2, 1, [0])
    budget_s = 120.0
    Ls = int(max(1, min(w.n_layers, budget_s / max(per_layer_s * total, 1e-9))))
    for l in range(probe_layers, Ls):
        p = syn.prefill(0, l)
        store[(0, l)] = (bf16_bits(p["k"]), bf16_bits(p["v"]), bf16_bits(p["q_last"]), p["audio_begin"], p["audio_end"])
    sec, threads = time_oracle(w, store, syn_dec, Ls, args.steps, args.warmup, [0])
    ms_step = sec * (w.n_layers / Ls) * w.batch * 1e3
    value = w.batch / (ms_step * 1e-3)
    sample = (f"sequence 0, first {Ls} of {w.n_layers} layers, {args.steps} decode steps; time scaled by "
              f"{w.n_layers}/{Ls} layers and x{w.batch} sequences")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            # the oracle runs the layers of a step one after the other with the default settings of the method
            "config": method_config(w), "issue": {"launch": "host loops over layers, OpenMP over query heads"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


ISSUE_NAMES = {0: "independent", 1: "chained", 2: "serial", 3: "all_layers_together"}


def method_config(w, layer_dependency=1, score_scope=0, residency=0, kv_fp8=False):
    """The `config` of a benchmark line: the workload and the method's settings, the same keys in both arms (how an arm
    launches its steps is reported outside it)."""
    return dict(workload_config(w), layer_issue=ISSUE_NAMES[layer_dependency], score_scope="global" if score_scope else "per layer",
                residency="segment lag" if residency else "hard budget", tidal_kv="fp8_e4m3" if kv_fp8 else "bf16")


def workload_config(w):
    return {"workload": w.name, "layers": w.n_layers, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "batch": w.batch, "audio_tokens": w.audio_lens if w.batch <= 4 else
            {"min": min(w.audio_lens), "max": max(w.audio_lens), "mean": sum(w.audio_lens) / w.batch},
            "text_tokens": w.n_text, "chunk": w.chunk, "audio_budget": w.budget, "topk": w.topk,
            "l2": f"flushed between steps ({L2_FLUSH_BYTES >> 20} MiB write, then {L2_FLUSH_BYTES >> 20} MiB read, untimed)"}


def run_recall_sweep(args, wnw, dev):
    """Recall-stress grid (config-1 shapes, batch 8, 7500 audio tokens, focus jumping every 4 steps):
    budget x chunk; per point the step time with recall, with recall copies skipped, the bytes recalled per step,
    the sustained recall rate and the measured host-link bandwidth.  Steps run back to back in one timed region
    (continuous decoding; a step's inputs exceed L2 many times over), so every recalled byte is paid for inside it."""
    link_copy, link_kernel = wnw.wnw_measure_host_link(dev.index or 0, 256 << 20, 5)
    K, W = args.steps if args.steps != 200 else 48, max(args.warmup, 4)
    points = []
    for budget in (0.1, 0.2, 0.4):
        for chunk in (16, 64, 256):
            w = config4(seed=0, budget=budget, chunk=chunk, batch=8, n_steps=W + K)
            job = Job(w, seed=0, device=dev, wnw=wnw)
            job.create("wnw", wnw.WNW_MODE_TIERED)
            job.create("skip", wnw.WNW_MODE_TIERED, recall_mode=wnw.WNW_RECALL_SKIP)
            job.create("count", wnw.WNW_MODE_TIERED)
            job.place_all(["wnw", "skip", "count"])
            for t in range(W):
                job.step("wnw", t); job.step("skip", t); job.step("count", t)
            torch.cuda.synchronize(dev)
            # bytes recalled by every single step (a drained run of the same steps on a cache of its own: the selections are
            # deterministic): the jumps make the demand bursty, and a selection made at step s is used at step s+1, so the copies
            # of a step can hide behind one step of attention at most
            per_step, last = [], wnw.wnw_get_stats(job.caches["count"])["recall_bytes"]
            for t in range(W, W + K):
                job.step("count", t)
                wnw.wnw_sync(job.caches["count"])
                now = wnw.wnw_get_stats(job.caches["count"])["recall_bytes"]
                per_step.append(now - last)
                last = now
            s0 = wnw.wnw_get_stats(job.caches["wnw"])
            ms = job.timed_region("wnw", W, K)          # a step reads 1.6-3.6 GB: far more than L2 holds
            s1 = wnw.wnw_get_stats(job.caches["wnw"])
            ms_skip = job.timed_region("skip", W, K)
            rb = (s1["recall_bytes"] - s0["recall_bytes"]) / K
            T_a, _, C, S = wnw.wnw_get_seq_dims(job.caches["wnw"], 0)
            floor_ms = sum(max(ms_skip, b / (link_kernel * 1e9) * 1e3) for b in per_step) / K
            points.append({"budget": budget, "chunk": chunk, "chunks": C, "slots": S, "step_us": ms * 1e3,
                           "step_us_copies_skipped": ms_skip * 1e3, "exposed_recall_us": (ms - ms_skip) * 1e3,
                           "recall_MB_per_step": rb / 1e6, "misses_per_step": (s1["misses"] - s0["misses"]) / K,
                           "sustained_recall_GBps": rb / (ms * 1e-3) / 1e9,
                           "sustained_over_link": rb / (ms * 1e-3) / 1e9 / link_kernel,
                           "largest_step_recall_MB": max(per_step) / 1e6,
                           "floor_us": floor_ms * 1e3, "step_over_floor": ms / floor_ms,
                           "floor_note": "mean over the steps of max(step with copies skipped, that step's recalled bytes / "
                                         "link_kernel_GBps): a step's copies are needed by the next step"})
            job.destroy()
            del job
            torch.cuda.empty_cache()
    print(json.dumps({"workload": "cfg4_recall_stress_sweep", "batch": 8, "audio_tokens": 7500, "steps": K, "warmup": W,
                      "tidal_kv": "fp8_e4m3" if Job.kv_fp8 else "bf16",
                      "link_memcpy_GBps": link_copy, "link_kernel_GBps": link_kernel, "points": points}), flush=True)


def _peak_frac(nbytes, ms, peak_gbs):
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"ms_per_step": ms, "GBps": gbs, "frac": gbs / peak_gbs}


def measure_block(wnw, dev, w, peak_gbs, steps=10, warm=3, speech_rate_sweep=0):
    """One workload, three caches (WnW, WnW with recall copies skipped, own full-cache kernel), each measured in the two
    ways a step can be issued: `overlapped` (every layer's inputs resident before the step: all layers issued together
    where they fit one launch, else one overlapping launch per layer) and `chained` (a layer's kernel waits for its
    predecessor before it reads q: layers that feed one another).  Per form: the replayed step with L2 flushed before
    it, and K steps back to back in one event bracket (continuous decoding: recall has to pay for what it cannot hide)."""
    n_total = 2 * (warm + 3 * steps) + (2 * steps + warm if speech_rate_sweep else 0) + 4
    w.n_steps = n_total
    job = Job(w, seed=0, device=dev, wnw=wnw)
    job.create("wnw", wnw.WNW_MODE_TIERED)
    job.create("skip", wnw.WNW_MODE_TIERED, recall_mode=wnw.WNW_RECALL_SKIP)
    job.create("full", wnw.WNW_MODE_FULL)
    fp8 = w.head_dim == 128
    if fp8:   # the same workload with the tidal tier stored as e4m3 (half the recalled bytes, half the bytes tidal heads read)
        job.create("wnw8", wnw.WNW_MODE_TIERED, kv_fp8=True)
        job.create("skip8", wnw.WNW_MODE_TIERED, recall_mode=wnw.WNW_RECALL_SKIP, kv_fp8=True)
    job.place_all(["wnw", "skip", "full"] + (["wnw8", "skip8"] if fp8 else []))
    out = {"workload": w.name, "layers": w.n_layers, "batch": w.batch}
    t = 0
    for form, dep in (("overlapped", wnw.WNW_LAYERS_BATCHED), ("chained", wnw.WNW_LAYERS_CHAINED)):
        job.set_dependency(["wnw", "skip", "full"] + (["wnw8", "skip8"] if fp8 else []), dep)
        for tt in range(t, t + warm):
            for key, full in (("wnw", False), ("skip", False), ("full", True)) + ((("wnw8", False), ("skip8", False)) if fp8 else ()):
                job.step(key, tt, full=full)
        t += warm
        torch.cuda.synchronize(dev)
        nb, _ = job.kv_bytes_of_step("wnw")
        nbf, _ = job.kv_bytes_of_step("full", full=True)
        s0 = wnw.wnw_get_stats(job.caches["wnw"])
        ms_w = sum(job.timed_steps("wnw", t, steps)) / steps
        ms_s = sum(job.timed_steps("skip", t, steps)) / steps
        ms_f = sum(job.timed_steps("full", t, steps, full=True)) / steps
        t += steps
        if fp8:
            nb8, _ = job.kv_bytes_of_step("wnw8")
            z0 = wnw.wnw_get_stats(job.caches["wnw8"])
            ms_w8 = sum(job.timed_steps("wnw8", t - steps, steps)) / steps
            ms_s8 = sum(job.timed_steps("skip8", t - steps, steps)) / steps
        bb_w = job.timed_region("wnw", t, steps)
        bb_s = job.timed_region("skip", t, steps)
        job.timed_region("full", t, steps, full=True)
        if fp8:
            bb_w8 = job.timed_region("wnw8", t, steps)
            bb_s8 = job.timed_region("skip8", t, steps)
            z1 = wnw.wnw_get_stats(job.caches["wnw8"])
        t += steps
        s1 = wnw.wnw_get_stats(job.caches["wnw"])
        recall_b = (s1["recall_bytes"] - s0["recall_bytes"]) / (2 * steps)
        out[form] = {"wnw_copies_skipped": _peak_frac(nb, ms_s, peak_gbs), "full_cache": _peak_frac(nbf, ms_f, peak_gbs),
                     "wnw": {"ms_per_step": ms_w, "back_to_back_ms_per_step": bb_w, "back_to_back_copies_skipped_ms": bb_s,
                             "exposed_recall_us_per_step": (bb_w - bb_s) * 1e3, "recall_MB_per_step": recall_b / 1e6,
                             "tokens_per_s": w.batch / (bb_w * 1e-3)},
                     "wnw_step_over_full_step": {"flushed": ms_w / ms_f, "copies_skipped": ms_s / ms_f}}
        if fp8:
            out[form]["wnw_fp8_tidal_tier"] = {
                "copies_skipped": _peak_frac(nb8, ms_s8, peak_gbs), "ms_per_step": ms_w8, "back_to_back_ms_per_step": bb_w8,
                "back_to_back_copies_skipped_ms": bb_s8, "exposed_recall_us_per_step": (bb_w8 - bb_s8) * 1e3,
                "recall_MB_per_step": (z1["recall_bytes"] - z0["recall_bytes"]) / (2 * steps) / 1e6,
                "tokens_per_s": w.batch / (bb_w8 * 1e-3), "back_to_back_over_bf16_tier": bb_w8 / bb_w}
        out["GB_per_step"], out["full_cache_GB_per_step"] = nb / 1e9, nbf / 1e9
    if speech_rate_sweep:
        # the decode focus moving at a speech-like rate (the synthetic sweep crosses the clip 10x faster): same caches
        job.regen_queries(speech_rate_sweep)
        for tt in range(t, t + warm):
            job.step("wnw", tt); job.step("skip", tt)
        t += warm
        s0 = wnw.wnw_get_stats(job.caches["wnw"])
        bb_w = job.timed_region("wnw", t, steps)
        bb_s = job.timed_region("skip", t, steps)
        s1 = wnw.wnw_get_stats(job.caches["wnw"])
        out["speech_rate"] = {"sweep_steps": speech_rate_sweep, "form": "chained", "back_to_back_ms_per_step": bb_w,
                              "back_to_back_copies_skipped_ms": bb_s, "exposed_recall_us_per_step": (bb_w - bb_s) * 1e3,
                              "recall_MB_per_step": (s1["recall_bytes"] - s0["recall_bytes"]) / steps / 1e6}
    job.destroy()
    del job
    torch.cuda.empty_cache()
    return out


def chained_batch_sweep(wnw, dev, batches, audio_tokens, steps=8, warm=3):
    """Chained layers, config-1 shapes at growing batch: the replayed WnW step at 20 % budget against the own full-cache
    step, L2 flushed before every step: from which batch on the tiered cache is the faster one."""
    points = []
    for b in batches:
        w = make_workload(f"b{b}x{audio_tokens}L30", warm + steps + 2, 0)
        job = Job(w, seed=0, device=dev, wnw=wnw)
        job.create("wnw", wnw.WNW_MODE_TIERED, layer_dependency=wnw.WNW_LAYERS_CHAINED)
        job.create("full", wnw.WNW_MODE_FULL, layer_dependency=wnw.WNW_LAYERS_CHAINED)
        job.place_all(["wnw", "full"])
        for tt in range(warm):
            job.step("wnw", tt); job.step("full", tt, full=True)
        torch.cuda.synchronize(dev)
        ms_w = sum(job.timed_steps("wnw", warm, steps)) / steps
        ms_f = sum(job.timed_steps("full", warm, steps, full=True)) / steps
        points.append({"batch": b, "wnw_step_us": ms_w * 1e3, "full_cache_step_us": ms_f * 1e3, "wnw_over_full": ms_w / ms_f})
        job.destroy()
        del job
        torch.cuda.empty_cache()
    below = [p["batch"] for p in points if p["wnw_over_full"] < 1.0]
    return {"audio_tokens": audio_tokens, "layers": 30, "form": "chained, replayed, L2 flushed, recall on", "points": points,
            "smallest_batch_with_wnw_below_full_cache": min(below) if below else None}


def run_ours(args, rank, world, local_rank):
    import paper_2608_22704_b200 as wnw
    wnw.lib()  # fails loudly if the CUDA library is missing
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    peak_gbs, peak_kind = load_peaks()
    if args.workload == "cfg4":
        if rank == 0:
            run_recall_sweep(args, wnw, dev)
        return
    K, W = args.steps, args.warmup
    R = args.roofline_steps
    DEP = args.layer_dependency
    dep_names = {0: "one overlapping launch per layer (inputs of every layer resident before the step)",
                 1: "chained: a layer's kernel waits for its predecessor before it reads q, k_new, v_new (layers that feed one another); its K/V prefetch runs ahead",
                 2: "serial launches",
                 3: "all layers issued together (inputs of every layer resident before the step, outputs read after it)"}
    extras = not (args.quick or args.eager)
    Kx = min(K, args.alt_steps) if extras else 0        # steps of each alternative issue form
    Kb = min(K, args.back_to_back_steps) if extras else 0
    total = W + R + K + Kb + 3 * Kx + 4
    w = make_workload(args.workload, total, 0)
    if args.segment_tokens > 0:
        w.chunk = args.segment_tokens
        w.name += f"_seg{args.segment_tokens}"
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    sampler.start()          # read-only nvidia-smi queries from here to the end of the measured sections
    job = Job(w, seed=rank, device=dev, wnw=wnw, score_scope=args.score_scope, residency=args.residency, evict_lag=args.evict_lag)
    job.create("wnw", wnw.WNW_MODE_FULL if args.quick_full else wnw.WNW_MODE_TIERED, recall_mode=args.recall_mode)
    if args.quick:   # profiler mode: the WnW steps only, nothing else launched
        job.place_all(["wnw"])
        for t in range(W):
            job.step("wnw", t, full=args.quick_full)
        torch.cuda.synchronize(dev)
        wnw.wnw_set_kernel_timing(job.caches["wnw"], True)
        per_step = job.timed_steps("wnw", W, K, full=args.quick_full, flush=not args.no_flush, graph=not args.eager)
        ms, n = wnw.wnw_get_kernel_time(job.caches["wnw"])
        kv_bytes, _ = job.kv_bytes_of_step("wnw", full=args.quick_full)
        ms_step = sum(per_step) / K
        sampler.stop()
        print(json.dumps({"quick": True, "workload": w.name, "ms_per_step": ms_step, "steps": K,
                          "attn_us_per_launch": ms * 1e3 / max(n, 1), "kv_GB_per_step": kv_bytes / 1e9,
                          "kv_GBps": kv_bytes / (ms_step * 1e-3) / 1e9, "frac_of_peak": kv_bytes / (ms_step * 1e-3) / 1e9 / peak_gbs}),
              flush=True)
        job.destroy()
        return
    job.create("full", wnw.WNW_MODE_FULL)
    job.create("skip", wnw.WNW_MODE_TIERED, recall_mode=wnw.WNW_RECALL_SKIP)
    keys3 = (("wnw", False), ("full", True), ("skip", False))

    class Keep:
        store = {}

        def __call__(self, b, l):
            return rank == 0 and b == 0 and l < args.oracle_layers
    keep = Keep()
    job.place_all(["wnw", "full", "skip"], keep_host=keep)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    # ---- warm-up (all caches take the same steps so their states stay comparable)
    for t in range(W):
        for key, full in keys3:
            job.step(key, t, full=full)
    torch.cuda.synchronize(dev)

    # ---- eager launches bracketed by CUDA events inside the library (kept for reference: includes host pacing)
    wnw.wnw_set_kernel_timing(job.caches["wnw"], True)
    algo_bytes = 0
    for t in range(W, W + R):
        b_step, _ = job.kv_bytes_of_step("wnw")
        algo_bytes += b_step
        job.flush_l2(); job.step("wnw", t)
        job.step("full", t, full=True); job.step("skip", t)
    attn_ms, attn_n = wnw.wnw_get_kernel_time(job.caches["wnw"])
    wnw.wnw_set_kernel_timing(job.caches["wnw"], False)

    # ---- headline: K replayed steps in the configured issue form, device time, L2 flushed before every step
    stats0 = wnw.wnw_get_stats(job.caches["wnw"])
    barrier()
    bytes_before, _ = job.kv_bytes_of_step("wnw")
    bytes_full, _ = job.kv_bytes_of_step("full", full=True)
    launches0 = wnw.wnw_get_launch_counts(job.caches["wnw"])
    wall0 = time.perf_counter()
    per_step = job.timed_steps("wnw", W + R, K, graph=not args.eager)
    barrier()
    wall = time.perf_counter() - wall0
    stats1 = wnw.wnw_get_stats(job.caches["wnw"])
    launches1 = wnw.wnw_get_launch_counts(job.caches["wnw"])
    region_launches = [b - a for a, b in zip(launches0, launches1)]   # attention, selection, recall, step-end kernels
    bytes_after, _ = job.kv_bytes_of_step("wnw")
    attn_per_step = region_launches[0] / K
    region_bytes_per_launch = 0.5 * (bytes_before + bytes_after) / attn_per_step   # the text grows by one token per step
    ms_per_step = dist_max(sum(per_step), dev, world) / K
    value = whole_job_tokens_per_s(world, w.batch, ms_per_step)

    # ---- the same steps: own full-cache kernel in the same issue form, and WnW with recall copies skipped
    ms_full = dist_max(sum(job.timed_steps("full", W + R, K, full=True, graph=not args.eager)), dev, world) / K
    ms_skip = dist_max(sum(job.timed_steps("skip", W + R, K, graph=not args.eager)), dev, world) / K
    t_next = W + R + K
    barrier()
    # ---- continuous decoding: steps back to back in one timed region (no flush gaps in which a recall could finish for
    # free); the difference to the run with copies skipped is the recall time that overlap cannot hide
    bb = None
    if Kb > 0:
        ms_bb = dist_max(job.timed_region("wnw", t_next, Kb), dev, world)
        ms_bb_skip = dist_max(job.timed_region("skip", t_next, Kb), dev, world)
        ms_bb_full = dist_max(job.timed_region("full", t_next, Kb, full=True), dev, world)
        t_next += Kb
        bb = {"steps": Kb, "ms_per_step": ms_bb, "ms_per_step_copies_skipped": ms_bb_skip, "full_cache_ms_per_step": ms_bb_full,
              "exposed_recall_us_per_step": (ms_bb - ms_bb_skip) * 1e3, "tokens_per_s": whole_job_tokens_per_s(world, w.batch, ms_bb),
              "note": "K steps in one event bracket, no L2 flush between them (a step reads more than L2 holds only on the "
                      "larger workloads), input staging copies inside the bracket"}

    # ---- end to end: inputs start in pinned host memory, outputs end there, copies inside the timed region
    n_e2e = min(K, 64)
    hslab = job.slab[W + R:W + R + n_e2e].cpu().pin_memory()
    hout = torch.empty((n_e2e,) + tuple(job.out.shape), dtype=torch.bfloat16).pin_memory()
    job.create("e2e", wnw.WNW_MODE_TIERED)
    job.place_all(["e2e"])
    for tt in range(W + R):
        job.step("e2e", tt)
    torch.cuda.synchronize(dev)
    if not args.eager:
        job.capture("e2e")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_ms = 0.0
    with torch.cuda.stream(job.stream):
        for i in range(n_e2e):
            job.flush_l2()
            e0.record()
            if args.eager:
                job.sslab.copy_(hslab[i], non_blocking=True)
                job.step("e2e", W + R + i, q=job.sq, kn=job.skn, vn=job.svn)
            else:
                job.graph_step("e2e", W + R + i, src=hslab[i])      # host -> device copy of the step's inputs, then the step
            hout[i].copy_(job.out, non_blocking=True)               # device -> host read of the step's outputs
            e1.record()
            e1.synchronize()
            e2e_ms += e0.elapsed_time(e1)
    e2e_value = whole_job_tokens_per_s(world, w.batch, dist_max(e2e_ms, dev, world) / n_e2e)
    h2d = job.sslab.numel() * 2
    d2h = job.out.numel() * 2
    wnw.wnw_destroy(job.caches.pop("e2e"))

    # ---- the other ways to issue the layers of a step, on the same caches (the state simply continues)
    forms = {}
    if Kx > 0:
        others = [(n_, d_) for n_, d_ in (("chained", wnw.WNW_LAYERS_CHAINED), ("upper_bound_all_layers_together", wnw.WNW_LAYERS_BATCHED),
                                          ("per_layer_overlapped", wnw.WNW_LAYERS_INDEPENDENT), ("serial", wnw.WNW_LAYERS_SERIAL)) if d_ != DEP]
        for name, mode in others:
            keys = ["wnw"] if mode == wnw.WNW_LAYERS_SERIAL else ["wnw", "full"]
            job.set_dependency(keys, mode)
            nb, _ = job.kv_bytes_of_step("wnw")
            l0 = wnw.wnw_get_launch_counts(job.caches["wnw"])[0]
            ms = dist_max(sum(job.timed_steps("wnw", t_next, Kx)), dev, world) / Kx
            n_l = (wnw.wnw_get_launch_counts(job.caches["wnw"])[0] - l0) / Kx
            forms[name] = {"step_us": ms * 1e3, "tokens_per_s": whole_job_tokens_per_s(world, w.batch, ms), "attention_launches_per_step": n_l,
                           "achieved": nb / (ms * 1e-3) / 1e9, "frac": nb / (ms * 1e-3) / 1e9 / peak_gbs, "steps": Kx}
            if "full" in keys:
                ms_f = dist_max(sum(job.timed_steps("full", t_next, Kx, full=True)), dev, world) / Kx
                forms[name]["full_cache_step_us"] = ms_f * 1e3
                forms[name]["wnw_step_over_full_step"] = ms / ms_f
            t_next += Kx
        job.set_dependency(["wnw", "full"], DEP)
    clocks = sampler.stop()
    clocks["window"] = "all measured sections of this run (warm-up to the last issue form); the headline region lies inside it"

    if rank != 0:
        job.destroy()
        return

    # ---- host link
    try:
        link_copy, link_kernel = wnw.wnw_measure_host_link(dev.index or 0, 256 << 20, 5)
    except Exception:
        link_copy = link_kernel = None

    # ---- CPU baseline: the oracle on a bounded sample
    cpu = None
    if args.oracle_layers > 0:
        dec_host = {}

        def syn_dec(tt, l, seqs):
            if l not in dec_host:
                dec_host[l] = (bf16_bits(job.q[:, l, 0].cpu()), bf16_bits(job.kn[:, l, 0].cpu()), bf16_bits(job.vn[:, l, 0].cpu()))
            q, kn, vn = dec_host[l]
            return q[tt][None], kn[tt][None], vn[tt][None]
        Ls = args.oracle_layers
        sec, threads = time_oracle(w, keep.store, syn_dec, Ls, args.oracle_steps, 1, [0])
        ms_oracle = sec * (w.n_layers / Ls) * w.batch * 1e3
        cpu = {"value": w.batch / (ms_oracle * 1e-3), "unit": UNIT, "cores": threads, "kind": "oracle",
               "ms_per_step": ms_oracle,
               "sample": f"sequence 0, first {Ls} of {w.n_layers} layers, {args.oracle_steps} decode steps; time scaled by "
                         f"{w.n_layers}/{Ls} layers and x{w.batch} sequences"}
    retention = {"r_gpu": stats1["resident_audio_tokens"] / max(stats1["full_audio_tokens"], 1),
                 "r_gpu_cpu": (stats1["resident_audio_tokens"] + stats1["host_audio_tokens"]) / max(stats1["full_audio_tokens"], 1)}
    job.destroy()
    torch.cuda.empty_cache()

    # ---- the other configurations of the list, bounded: the 10-minute stack at batch 1, the ragged batch of 32, and the
    # many-long-sequences case that is HBM-bound at 12 layers; then the chained batch sweep
    blocks = {}
    if not args.no_blocks:
        blocks["hbm_bound_case"] = measure_block(wnw, dev, make_workload("hbm", 64, 0), peak_gbs, steps=10)
        blocks["cfg2"] = measure_block(wnw, dev, make_workload("cfg2", 64, 0), peak_gbs, steps=10)
        blocks["cfg3"] = measure_block(wnw, dev, make_workload("cfg3", 96, 0), peak_gbs, steps=8, speech_rate_sweep=1200)
        blocks["chained_batch_sweep"] = chained_batch_sweep(wnw, dev, (1, 2, 4, 8, 16, 32), 3000)

    # ---- the paper's own form of the method on the same model shape: segments of 2 s (25 tokens at 12.5 tokens/s, 50 at
    # 25), chunks of two segments, permanent prefill base with lag-3 release, scores summed over all anchor layers
    paper_form = None
    if not args.no_paper_form:
        n_pf, n_bb = 24, 24
        wq = make_workload(args.workload, 2 * (W + n_pf) + n_bb + 2, 0)
        wq.chunk = 50 if args.workload == "cfg2" else 25
        jq = Job(wq, seed=0, device=dev, wnw=wnw, score_scope=wnw.WNW_SCOPE_GLOBAL, residency=wnw.WNW_RESIDENCY_SEGMENT_LAG_TOKEN_BASE,
                 evict_lag=3)
        jq.create("wnw", wnw.WNW_MODE_TIERED)
        jq.create("skip", wnw.WNW_MODE_TIERED, recall_mode=wnw.WNW_RECALL_SKIP)
        # tidal bases and fixed heads: token-granular per-segment top-k with per-head retention from Eq. 1 (seeded
        # importances in [0,1], lambda = 2 x budget, so the mean retention is the budget)
        lam_q = 2.0 * wq.budget
        ret_q = wnw.wnw_retention_schedule(np.random.RandomState(0).rand(wq.n_layers * wq.n_kv_heads), lam_q)
        jq.place_all(["wnw", "skip"], token=(ret_q.reshape(wq.n_layers, wq.n_kv_heads), wq.chunk, 0))
        res_q = {}
        tq = 0
        for form, dep in (("chained", wnw.WNW_LAYERS_CHAINED), ("upper_bound_all_layers_together", wnw.WNW_LAYERS_BATCHED)):
            jq.set_dependency(["wnw", "skip"], dep)
            for tt in range(tq, tq + W):
                jq.step("wnw", tt); jq.step("skip", tt)
            tq += W
            torch.cuda.synchronize(dev)
            ms_q = sum(jq.timed_steps("wnw", tq, n_pf)) / n_pf
            jq.timed_steps("skip", tq, n_pf)
            tq += n_pf
            res_q[form] = {"step_us": ms_q * 1e3, "tokens_per_s": wq.batch / (ms_q * 1e-3)}
        fetched_q, visible_q = jq.rows_fetched_and_visible("wnw")
        st0 = wnw.wnw_get_stats(jq.caches["wnw"])
        ms_q_bb = jq.timed_region("wnw", tq, n_bb)
        ms_q_bb_skip = jq.timed_region("skip", tq, n_bb)
        st1 = wnw.wnw_get_stats(jq.caches["wnw"])
        T_a_q, _, C_q, S_q = wnw.wnw_get_seq_dims(jq.caches["wnw"], 0)
        paper_form = {"segment_tokens": wq.chunk, "segments": C_q, "slots": S_q, "base_slots": wnw.wnw_get_base_slots(jq.caches["wnw"], 0),
                      "evict_lag": 3, "score_scope": "global",
                      "prefill_compression": f"token-granular for tidal bases and fixed heads: per segment top floor(retention*n_s); retention = min(s*{lam_q:g}, 1), s ~ U[0,1] seeded",
                      **res_q,
                      "back_to_back_step_us": ms_q_bb * 1e3, "back_to_back_exposed_recall_us": (ms_q_bb - ms_q_bb_skip) * 1e3,
                      "back_to_back_form": "all layers issued together",
                      "recall_bytes_per_step": (st1["recall_bytes"] - st0["recall_bytes"]) / n_bb,
                      "fetched_rows_over_visible_rows": fetched_q / max(visible_q, 1),
                      "fetched_rows_note": "K,V rows the kernels fetch per step (25-token segments and base blocks are stored and fetched as 32 rows) over the rows that are visible",
                      "r_gpu": st1["resident_audio_tokens"] / max(st1["full_audio_tokens"], 1)}
        jq.destroy()

    attn_us = attn_ms * 1e3 / max(attn_n, 1)
    region_us_per_launch = ms_per_step * 1e3 / attn_per_step
    region_achieved = region_bytes_per_launch / (region_us_per_launch * 1e-6) / 1e9
    bytes_per_launch = algo_bytes / max(attn_n, 1)
    achieved = bytes_per_launch / (attn_us * 1e-6) / 1e9 if attn_us > 0 else 0.0
    recall_bytes_step = (stats1["recall_bytes"] - stats0["recall_bytes"]) / K
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "attn_traffic.json")
    if os.path.exists(tpath):
        try:
            traffic = json.load(open(tpath)).get(w.name + (":all_layers_together" if DEP == 3 and not args.eager else ""))
        except Exception:
            traffic = None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "step_us": ms_per_step * 1e3,
        "step_us_median": float(np.median(per_step)) * 1e3, "step_us_p95": float(np.percentile(per_step, 95)) * 1e3,   # this rank's K steps
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": method_config(w, DEP, args.score_scope, args.residency, Job.kv_fp8),
        "issue": {"launch": "eager" if args.eager else "cuda graph replay of the step", "layers": dep_names[DEP]},
        "clocks": clocks, "gpu_launches": int(sum(region_launches)),
        "launches": {"attention": region_launches[0], "selection": region_launches[1], "recall": region_launches[2],
                     "step_end": region_launches[3], "layers_per_attention_launch": w.n_layers / attn_per_step},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e},
        # achieved: algorithmic K,V bytes of one launch / the launch's share of the timed region (CUDA events around every
        # replayed step; the attention kernels are the only work on the timed stream; with chained layers one launch per
        # layer, each waiting for its predecessor, so the share of one is step time / layers).  The other issue forms are
        # reported under their names: `upper_bound_all_layers_together` needs every layer's q before the step starts (no
        # decoder whose layers feed one another can run it), `per_layer_overlapped` likewise; `serial` is plain stream order.
        "roofline": {"bound": "hbm", "kernel": "wnw_attn_multi_kernel" if DEP == 3 and not args.eager else "wnw_attn_kernel",
                     "achieved": region_achieved, "peak": peak_gbs, "unit": "GB/s",
                     "frac": region_achieved / peak_gbs, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                     "bytes_per_launch": region_bytes_per_launch, "us_per_launch": region_us_per_launch,
                     "launches": region_launches[0],
                     "duration_kind": "timed region / attention launches",
                     **forms,
                     "eager_event_bracket": {"us_per_launch": attn_us, "achieved": achieved, "frac": achieved / peak_gbs,
                                             "launches": attn_n},
                     "regime": f"{region_bytes_per_launch / 1e6:.1f} MB per launch would take "
                               f"{region_bytes_per_launch / (peak_gbs * 1e3):.2f} us at peak; the batch-1 step is bound by the "
                               f"chain of dependent phases of a layer, not by bytes (see hbm_bound_case and cfg3 for the HBM-bound regime)"},
        "cpu_baseline": cpu,
        "full_cache": {"ms_per_step": ms_full, "tokens_per_s": w.batch / (ms_full * 1e-3), "layer_issue": "as the headline",
                       "GB_per_step": bytes_full / 1e9, "GBps": bytes_full / (ms_full * 1e-3) / 1e9,
                       "frac": bytes_full / (ms_full * 1e-3) / 1e9 / peak_gbs, "wnw_step_over_full_step": ms_per_step / ms_full},
        "recall": {"bytes_per_step": recall_bytes_step, "hits": stats1["hits"] - stats0["hits"],
                   "misses": stats1["misses"] - stats0["misses"], "link_memcpy_GBps": link_copy, "link_kernel_GBps": link_kernel,
                   "ms_per_step_copies_skipped": ms_skip, "exposed_us_per_step": (ms_per_step - ms_skip) * 1e3,
                   "note": "in the flushed runs the out-of-graph recall of a step may finish during the untimed flush; "
                           "`back_to_back` has no such gaps"},
        "back_to_back": bb,
        **blocks,
        "paper_form": paper_form,
        "retention": retention,
        "wall_s_timed_region": wall,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg1",
                    help="cfg1 | cfg2 | cfg3 | cfg4 (recall sweep) | prof | hbm | b<batch>x<audio tokens> (config-1 heads, 12 layers)")
    ap.add_argument("--no-paper-form", action="store_true",
                    help="skip the extra measurement of the paper's own form (2 s segments, lag release, global scores)")
    ap.add_argument("--quick", action="store_true", help="only the WnW steps (for profiler captures); prints a short line")
    ap.add_argument("--no-flush", action="store_true", help="with --quick: do not flush L2 between steps")
    ap.add_argument("--recall-mode", type=int, default=0, help="with --quick: 0 side stream, 1 inline, 2 copies skipped")
    ap.add_argument("--quick-full", action="store_true", help="with --quick: time the full-cache comparison path instead")
    ap.add_argument("--tidal-kv", default="bf16", choices=["bf16", "fp8"],
                    help="storage of the tidal tier in every tiered cache of the run (the default line stays bf16 and reports "
                         "the e4m3 tier beside it in its workload blocks)")
    ap.add_argument("--score-scope", type=int, default=0, choices=[0, 1],
                    help="0: every layer ranks by its own (or the nearest) anchor heads; 1: Eq. 2's sum over all anchor layers")
    ap.add_argument("--residency", type=int, default=0, choices=[0, 1],
                    help="0: hard budget (fixed slot pool); 1: SEGMENT_LAG (overlapping two-segment chunks, lag release)")
    ap.add_argument("--evict-lag", type=int, default=3, help="delta of SEGMENT_LAG")
    ap.add_argument("--segment-tokens", type=int, default=0, help="override the workload's chunk_tokens (e.g. the paper's 25 / 50)")
    ap.add_argument("--eager", action="store_true", help="issue every layer eagerly instead of replaying a captured step")
    ap.add_argument("--roofline-steps", type=int, default=16)
    ap.add_argument("--layer-dependency", type=int, default=1, choices=[0, 1, 2, 3],
                    help="how the layers of a step are issued: 1 chained (default: a layer waits for its predecessor before it "
                         "reads q, what a decoder whose layers feed one another runs), 3 all layers together (needs every "
                         "layer's inputs before the step: a labelled upper bound), 0 one overlapping launch per layer, 2 serial")
    ap.add_argument("--alt-steps", type=int, default=32, help="steps timed in each of the other issue forms (0 = skip)")
    ap.add_argument("--no-blocks", action="store_true", help="skip the extra workloads (hbm_bound_case, cfg2, cfg3, chained batch sweep)")
    ap.add_argument("--back-to-back-steps", type=int, default=32,
                    help="steps timed in one region without L2 flushes (continuous decoding; exposes recall). 0 = skip")
    ap.add_argument("--oracle-layers", type=int, default=6, help="layers of sequence 0 the CPU baseline samples (0 = skip)")
    ap.add_argument("--oracle-steps", type=int, default=4)
    ap.add_argument("--sweep-steps", type=int, default=0,
                    help="decode steps for one sweep of the focus through the clip (0: the workload's own; e.g. 1200 on cfg3 is "
                         "about 4 audio tokens per generated token, a speech-like rate)")
    args = ap.parse_args()
    global SWEEP_STEPS_OVERRIDE
    SWEEP_STEPS_OVERRIDE = args.sweep_steps
    Job.layer_dependency = args.layer_dependency
    Job.kv_fp8 = args.tidal_kv == "fp8"
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    try:
        run_ours(args, rank, world, local_rank)
    finally:
        if world > 1:
            torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
