#!/usr/bin/env python
"""Benchmark of the Breadcrumbs decode hot path on B200.

Workload (the compression-ratio sweep): one layer, batch 64, 32 query /
8 KV heads, head_dim 128, bf16, prompt 512, 16384 decode steps, c in {2,4,8,16,32} with
page_size = c, plus the uncompressed run (c = 1, page 16) as a reported row.

One "step" of the JSON line = one decode step (bc_append + bc_decode_attn; when the token fills the
window, bc_decode_attn_pair instead -- the token's and the beacon's queries in one pass over the
cache -- and bc_compress; --no-pair runs the beacon's attention as a second pass) at EACH of the
five compressed ratios, i.e. 5 x 64 generated tokens.  The ratios are timed one after the other, K steps each, centred on the middle
of the 16384-step generation (cache length grows linearly with t, so the mean over a window centred
on the midpoint equals the mean over the whole run).  `value` = tokens / second over all of that.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

RATIOS = (2, 4, 8, 16, 32)
METRIC = "decode tokens/s (and KV-read HBM GB/s) over the compression-ratio sweep c in {2,4,8,16,32}"


# ------------------------------------------------------------------------------ accounting
def entries_attended(P, n, c):
    """Cache entries the n-th generated token's query reads (its own entry included)."""
    if c <= 1:
        return P + n
    return P + (n - 1) // c + (n - 1) % c + 1


def step_kinds(t_begin, K, c):
    """(regular, window-filling) decode steps among steps t_begin + 1 .. t_begin + K at ratio c."""
    fill = sum(1 for n in range(t_begin + 1, t_begin + K + 1) if c > 1 and n % c == 0)
    return K - fill, fill


def entries_beacon_query(P, t, c):
    """Stored entries the beacon query reads when the window fills at t (t % c == 0)."""
    return P + (t // c - 1) + c


# DRAM traffic of one attention launch over algorithmic KV bytes, per ratio: ncu
# dram__bytes_read.sum + dram__bytes_write.sum with warm caches (--cache-control none) on the small
# case of each ratio (--profile-case C: same bytes per launch and page size as mid-generation), for
# the library version named here; see profiles/.  Slightly below 1: part of the stream stays in L2
# from the previous step.  A different library version invalidates the figures (traffic: null).
TRAFFIC_FOR_VERSION = 231
TRAFFIC_OVER_ALGORITHMIC = {2: 0.997, 4: 0.983, 8: 0.962, 16: 0.947, 32: 0.982}


def traffic_per_launch(c, algorithmic_bytes):
    from paper_2510_13797_b200 import binding
    if binding.lib().bc_version() != TRAFFIC_FOR_VERSION or c not in TRAFFIC_OVER_ALGORITHMIC:
        return None
    return TRAFFIC_OVER_ALGORITHMIC[c] * algorithmic_bytes


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc, self.index = None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ one ratio on the GPU
def make_runner(w, device, seed_offset=0, paired=True, fused=False):
    """A DecodeDriver (one cache, batch B at ratio c, driven through the C ABI) plus the timed passes."""
    import torch
    from paper_2510_13797_b200.driver import DecodeDriver
    r = type("RatioRunner", (_Passes, DecodeDriver), {})(w, device, seed_offset, fused=fused, paired=paired)
    r.torch = torch
    return r


class _Passes:
    """Accounting and timed passes over a DecodeDriver."""

    def host_bytes_per_step(self):
        w = self.w
        qb = self.n * w.q_heads * w.head_dim * 2
        kb = self.n * w.kv_heads * w.head_dim * 2
        per_beacon = 1.0 / self.c if self.c > 1 else 0.0
        return (qb + 2 * kb) * (1 + per_beacon), qb * (1 + per_beacon)

    # -- accounting ------------------------------------------------------------------------------
    def kv_bytes(self, t_from, steps):
        """Algorithmic KV bytes read by the attention launches of steps t_from+1 .. t_from+steps:
        (regular launches, beacon-query launches)."""
        E = self.w.entry_bytes
        reg = sum(entries_attended(self.P, n, self.c) for n in range(t_from + 1, t_from + steps + 1))
        bea = sum(entries_beacon_query(self.P, n, self.c) for n in range(t_from + 1, t_from + steps + 1)
                  if self.c > 1 and n % self.c == 0)
        if getattr(self, "paired", False):
            bea = 0          # the beacon's queries ride on the token's pass over the cache: no second read
        return reg * E * self.n, bea * E * self.n

    def cache_bytes(self, t):
        E = self.w.entry_bytes
        live = self.P + (t // self.c + t % self.c if self.c > 1 else t)
        return live * E * self.n, (self.P + t) * E * self.n

    # -- timed passes ------------------------------------------------------------------------------
    def timed_graph(self, K, W, replays=3):
        """W warm-up steps, then exactly K steps timed with CUDA events as ONE replay of a CUDA graph that
        holds exactly those K steps (whatever K is: no remainder runs as plain launches).  The graph is
        captured at t_begin, replayed once untimed to warm it, the caches are put back to t_begin through
        the library's own calls, and the graph is replayed again under the event pair: that replay is the
        reported time.  `replays` - 1 further rewind-and-replay rounds only feed the spread of step times."""
        torch = self.torch
        cyc = self.c if self.c > 1 else 16
        while W > 0 or self.t % cyc:
            self.step(); W -= 1
        t_begin = self.t
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        l0 = self.cache.bc_kernel_launches()
        with torch.cuda.graph(graph, stream=s, capture_error_mode="thread_local"):
            for _ in range(K):
                self.step()
        per_graph = self.cache.bc_kernel_launches() - l0     # the capture enqueued nothing
        torch.cuda.current_stream().wait_stream(s)
        graph.replay()                                         # warm the instantiated graph
        torch.cuda.synchronize()
        self.window_step_ms, first = [], None
        for _ in range(max(1, replays)):
            self.reset_to(t_begin)                            # rewind: the same K steps again
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.nvtx.range_push("timed")
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
            torch.cuda.nvtx.range_pop()
            ms = e0.elapsed_time(e1)
            first = ms if first is None else first
            self.window_step_ms.append(ms / K)
        self.t = t_begin + K
        self.graph_steps = step_kinds(t_begin, K, self.c)
        return first, t_begin, per_graph

    def timed_kernels(self, K, W):
        """K steps with plain launches; every decode-attention kernel is bracketed by CUDA events on the
        launching stream.  Returns (sum of kernel ms, launches, algorithmic bytes, whole-region ms)."""
        torch = self.torch
        for _ in range(W):
            self.step()
        torch.cuda.synchronize()
        t_begin = self.t
        n_launch = K + (sum(1 for n in range(t_begin + 1, t_begin + K + 1) if n % self.c == 0)
                        if self.c > 1 and not self.paired else 0)
        self.cache.bc_profile_enable(n_launch)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.nvtx.range_push("kernels")
        e0.record()
        for _ in range(K):
            self.step()
        e1.record()
        torch.cuda.synchronize()
        torch.cuda.nvtx.range_pop()
        got, ms = self.cache.bc_profile_read()
        assert got == n_launch, (got, n_launch)
        reg, bea = self.kv_bytes(t_begin, K)
        return ms, got, reg + bea, e0.elapsed_time(e1)

    def timed_attn_stream(self, n_launch, W):
        """n_launch decode-attention launches back to back on the cache as it stands (nothing else in
        the timed region), one CUDA-event pair around all of them on the launching stream.  Returns
        (ms, launches, algorithmic KV bytes): the kernel's average duration without the event
        overhead that bracketing every single launch adds."""
        torch = self.torch
        live = self.P + (self.t // self.c + self.t % self.c if self.c > 1 else self.t)
        for i in range(max(W, 3)):
            self.cache.bc_decode_attn(0, self.slots, self.q[i % self.ring], self.out, self.w.sm_scale)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.nvtx.range_push("attn_stream")
        e0.record()
        for i in range(n_launch):
            self.cache.bc_decode_attn(0, self.slots, self.q[i % self.ring], self.out, self.w.sm_scale)
        e1.record()
        torch.cuda.synchronize()
        torch.cuda.nvtx.range_pop()
        return e0.elapsed_time(e1), n_launch, n_launch * live * self.w.entry_bytes * self.n

    def timed_host(self, K, W):
        torch = self.torch
        for _ in range(W):
            self.step_host()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        t0 = time.perf_counter()
        for _ in range(K):
            self.step_host()
        self.host_enqueue_ms = (time.perf_counter() - t0) * 1e3   # what the calls cost the host thread (no synchronisation inside)
        self.cache.bc_host_outputs_ready()            # the last outputs' copies, before the closing event
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)


# ------------------------------------------------------------------------------ the oracle on host cores
def oracle_sample(w, t_mid, seqs, steps, seed=0):
    """Times the CPU oracle, as it stands, on `steps` decode steps of `seqs` sequences whose caches
    are at generation step t_mid.  Returns (seconds, tokens processed, cpu seconds)."""
    import numpy as np
    import psutil
    from oracle.breadcrumbs_oracle import SeqCache
    rng = np.random.RandomState(seed)
    c, P = w.cs[0], w.prompt_lens[0]
    Hkv, Hq, D = w.kv_heads, w.q_heads, w.head_dim
    t0 = (t_mid // c) * c if c > 1 else t_mid
    caches = []
    for _ in range(seqs):
        s = SeqCache(1, c)
        s.prefill(0, rng.standard_normal((P, Hkv, D)), rng.standard_normal((P, Hkv, D)))
        nb = t0 // c if c > 1 else 0
        for m in range(nb):                     # beacons are inputs: the state at t0 is built directly
            s.cache[0].append(("beacon", m + 1, rng.standard_normal((Hkv, D)), rng.standard_normal((Hkv, D))))
        if c <= 1:
            for i in range(t0):
                s.cache[0].append(("token", i, rng.standard_normal((Hkv, D)), rng.standard_normal((Hkv, D))))
        caches.append(s)
    proc = psutil.Process()
    cpu0, t_start = proc.cpu_times(), time.perf_counter()
    for _ in range(steps):
        for s in caches:
            s.append(0, rng.standard_normal((Hkv, D)), rng.standard_normal((Hkv, D)))
            s.attend(0, rng.standard_normal((Hq, D)), w.sm_scale)
            if c > 1 and s.window_len(0) == c:
                bk, bv = rng.standard_normal((Hkv, D)), rng.standard_normal((Hkv, D))
                s.beacon_attend(0, rng.standard_normal((Hq, D)), bk, bv, w.sm_scale)
                s.compress(0, bk, bv)
    wall = time.perf_counter() - t_start
    cpu1 = proc.cpu_times()
    cpu = (cpu1.user - cpu0.user) + (cpu1.system - cpu0.system)
    return wall, seqs * steps, cpu


def _oracle_worker(job):
    name, c, t_mid, seqs, steps, seed = job
    from paper_2510_13797_b200.workloads import make_workload
    return oracle_sample(make_workload(name, c=c), t_mid, seqs, steps, seed)


def oracle_sample_all_cores(c, t_mid, seqs, steps):
    """The same oracle, one process per host core, the sequences dealt out over them (sequences are
    independent).  Returns (wall seconds, tokens, processes)."""
    import multiprocessing as mp
    procs = max(1, min(os.cpu_count() or 1, seqs))
    share = [seqs // procs + (1 if i < seqs % procs else 0) for i in range(procs)]
    jobs = [("sweep", c, t_mid, n, steps, 100 + i) for i, n in enumerate(share) if n]
    with mp.get_context("spawn").Pool(len(jobs)) as pool:
        pool.map(_oracle_worker, [(j[0], j[1], j[2], 1, 1, j[5]) for j in jobs])      # start the workers, import numpy
        t0 = time.perf_counter()
        res = pool.map(_oracle_worker, jobs)
        wall = time.perf_counter() - t0
    return wall, sum(r[1] for r in res), len(jobs)


def run_reference(args):
    """The reference arm: the CPU oracle timed on this machine's host cores, same workload and metric.
    Each step decodes a bounded sample of the batch at every ratio."""
    from paper_2510_13797_b200.workloads import make_workload
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K, W = args.steps, args.warmup
    T = make_workload("sweep", c=16).steps
    budget = 150.0 / max(K + W, 1)                   # seconds per step over the five ratios
    probe = {}
    for c in RATIOS:
        w = make_workload("sweep", c=c)
        wall, _, _ = oracle_sample(w, T // 2, 1, 1)
        probe[c] = wall
    seqs = int(max(1, min(64, budget / max(sum(probe.values()), 1e-9))))
    total_wall = total_tok = total_cpu = 0.0
    for c in RATIOS:
        w = make_workload("sweep", c=c)
        oracle_sample(w, T // 2, seqs, max(W, 0))
        wall, tok, cpu = oracle_sample(w, T // 2, seqs, K)
        total_wall += wall; total_tok += tok; total_cpu += cpu
    value = total_tok / total_wall
    cores = max(1, round(total_cpu / total_wall))
    sample = f"{seqs} of 64 sequences per ratio, {K} decode steps at the mid-generation cache state, c in {list(RATIOS)}"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": K,
        "warmup": W, "ms_per_step": 1e3 * total_wall / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "sweep: B=64, 32/8 heads, D=128, P=512, T=16384, c in {2,4,8,16,32} (CPU oracle on a sample)"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_profile_case(args):
    """A few plain decode steps at one ratio on a cache whose prompt is as long as the sweep's
    mid-generation cache (same bytes per launch, same page granularity, few launches before them)."""
    import torch
    from paper_2510_13797_b200.workloads import make_workload
    c = args.profile_case
    w = make_workload("sweep", c=c)
    mid = entries_attended(w.prompt_lens[0], w.steps // 2, c)
    w = make_workload("sweep", c=c, prompt_lens=[mid] * w.batch, gen_lens=[4 * max(c, 16) + args.steps + 64] * w.batch)
    torch.cuda.set_device(0)
    r = make_runner(w, torch.device("cuda", 0), fused=not args.no_fused)
    r.reset_to(0)
    ms, n, nbytes, region = r.timed_kernels(args.steps, max(args.warmup, 3))
    r.check_error()
    print(json.dumps({"profile_case": c, "prompt": mid, "steps": args.steps, "attn_launches": n,
                      "attn_kernel_us": 1e3 * ms / n, "attn_kernel_gbs": nbytes / (ms * 1e-3) / 1e9,
                      "kv_bytes_per_launch": nbytes / n, "plain_ms_per_step": region / args.steps}))


def run_timeline(args):
    """Where a decode-attention launch spends its time (bc_attn_timeline): per-block stamps of the last
    three attention launches of (a) back-to-back bc_decode_attn calls and (b) whole decode steps, on the
    small case of ratio C (prompt as long as the sweep's mid-generation cache).  Prints, per launch and
    stamp, the mean / min / max over the blocks in microseconds after the first block entered the
    kernel, the launch's span, and the gap to the launch before it."""
    import numpy as np
    import torch
    from paper_2510_13797_b200.workloads import make_workload
    c = args.timeline
    w = make_workload("sweep", c=c)
    mid = entries_attended(w.prompt_lens[0], w.steps // 2, c)
    w = make_workload("sweep", c=c, prompt_lens=[mid] * w.batch, gen_lens=[8 * max(c, 16) + 64] * w.batch)
    if args.timeline_shape == "depth":     # one layer of the full-depth configuration: batch 256, 12/2 heads, page = c
        d = make_workload("depth", c=c)
        mid = entries_attended(d.prompt_lens[0], d.steps // 2, c)
        w = make_workload("sweep", c=c, batch=d.batch, q_heads=d.q_heads, kv_heads=d.kv_heads, page_size=d.page_size,
                          prompt_lens=[mid] * d.batch, gen_lens=[8 * max(c, 16) + 64] * d.batch, cs=[c] * d.batch)
    torch.cuda.set_device(0)
    r = make_runner(w, torch.device("cuda", 0), fused=args.fused)
    r.reset_to(1)
    WORDS, BLOCKS, KEEP = 16, 304, 3
    bufs = [torch.zeros(BLOCKS * WORDS, dtype=torch.int64, device="cuda") for _ in range(KEEP)]
    names = ["enter", "planned", "waited", "first_tile", "last_tile", "piece_out", "ticket_known", "leave"]

    def summarise(mode):
        torch.cuda.synchronize()
        out, prev_end = [], None
        for b in bufs:
            a = b.cpu().numpy().reshape(BLOCKS, WORDS)
            live = a[:, 2] > 0                             # blocks that had tiles
            t0 = a[a[:, 0] > 0, 0].min()
            row = {"blocks": int(live.sum()), "span_us": float((a[live, 7].max() - t0) / 1e3),
                   "tiles_per_block": float((a[live, 8] >> 32).mean())}
            for k, nm in enumerate(names):
                x = (a[live, k] - t0) / 1e3
                row[nm] = [round(float(x.mean()), 2), round(float(x.min()), 2), round(float(x.max()), 2)]
            row["leave_after_last_tile"] = [round(float(v), 2) for v in
                                            ((a[live, 7] - a[live, 4]) / 1e3).mean(keepdims=True).tolist()
                                            + [((a[live, 7] - a[live, 4]) / 1e3).min(), ((a[live, 7] - a[live, 4]) / 1e3).max()]]
            tail = (a[live, 7] - a[live, 4]) / 1e3
            path = a[live, 9]
            row["leave_after_last_tile_by_ending"] = {
                name: [int(sel.sum()), round(float(tail[sel].mean()), 2) if sel.any() else None]
                for name, sel in (("whole", (path & 1) > 0), ("merged_at_once", (path & 2) > 0),
                                  ("published_only", ((path & 4) > 0) & ((path & 24) == 0)),
                                  ("published_then_merged", ((path & 4) > 0) & ((path & 16) > 0)),
                                  ("merged_first_piece_too", (path & 8) > 0))}
            if args.timeline_raw:     # per block: [tiles, first sequence, ending bits, then the eight stamps in us]
                row["blocks_raw"] = [[int(a[b, 8] >> 32), int(a[b, 8] & 0xffffffff), int(a[b, 9])] +
                                     [round(float((a[b, k] - t0) / 1e3), 2) for k in range(8)] for b in range(BLOCKS) if live[b]]
            if prev_end is not None:
                row["enter_after_previous_launch_left_us"] = round(float((t0 - prev_end) / 1e3), 2)
            prev_end = a[live, 7].max()
            out.append(row)
            b.zero_()
        return {"mode": mode, "launches": out}

    res = []
    N = max(args.steps, 8)
    for i in range(N):                                     # (a) the attention call alone, back to back
        r.cache.bc_attn_timeline(bufs[i - (N - KEEP)] if i >= N - KEEP else None, BLOCKS)
        r.cache.bc_decode_attn(0, r.slots, r.q[i % r.ring], r.out, r.w.sm_scale)
    res.append(summarise("bc_decode_attn back to back"))
    r.cache.bc_attn_timeline(None)
    while (r.t + N) % max(c, 2) != max(c, 2) // 2:          # (b) whole steps; the stamped ones are regular steps
        r.step()
    for i in range(N):
        r.cache.bc_attn_timeline(bufs[i - (N - KEEP)] if i >= N - KEEP else None, BLOCKS)
        r.step()
    res.append(summarise("decode steps" + (" (bc_decode_step)" if args.fused else " (bc_append, bc_decode_attn)")))
    r.cache.bc_attn_timeline(None)
    r.check_error()
    print(json.dumps({"timeline_case": c, "prompt": mid, "batch": w.batch, "kv_bytes_per_launch": mid * w.entry_bytes * w.batch,
                      "stamps": "mean / min / max over the blocks, us after the first block entered", "runs": res}))


# ------------------------------------------------------------------------------ the other configurations
def _percentiles(xs):
    """[p50, p99, windows] of the per-step times of the graph-replayed windows (rank 0's)."""
    if not xs:
        return None
    xs = sorted(xs)
    pick = lambda q: xs[min(len(xs) - 1, int(math.ceil(q * len(xs))) - 1)]
    return [pick(0.50), pick(0.99), len(xs)]


def _event_pair(torch):
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def report_cfg2(args):
    """The small single-layer configuration: batch 32, 12/2 heads, prompt 256, 4096 steps, c = 16.  ~13 MB of KV
    per step: L2-resident and launch-bound, so the figures are microseconds per call."""
    import torch
    from paper_2510_13797_b200.workloads import make_workload
    torch.cuda.set_device(0)
    w = make_workload("cfg2")
    r = make_runner(w, torch.device("cuda", 0), paired=not args.no_pair, fused=not args.no_fused)
    K = max(16, (min(args.steps, 1024) // 16) * 16)
    t_mid = ((w.steps - K) // 2 // 16) * 16
    r.reset_to(t_mid - 32)
    ms, t_begin, launches = r.timed_graph(K, 16)
    reg, bea = r.kv_bytes(t_begin, K)
    a_ms, a_n, a_bytes = r.timed_attn_stream(256, 8)
    # bc_append and bc_compress alone: plain launches, one event pair around each call
    app, comp = [], []
    for _ in range(4 * 16):
        j = r.t % r.ring
        e0, e1 = _event_pair(torch)
        e0.record(); r.cache.bc_append(0, r.slots, r.k[j], r.v[j]); e1.record()
        app.append((e0, e1))
        r.t += 1
        if r.t % 16 == 0:
            bsel = (r.t // 16) % 4
            e0, e1 = _event_pair(torch)
            e0.record(); r.cache.bc_compress(0, r.slots, r.bk[bsel], r.bv[bsel]); e1.record()
            comp.append((e0, e1))
    torch.cuda.synchronize()
    r.check_error()
    med = lambda prs: statistics.median(1e3 * a.elapsed_time(b_) for a, b_ in prs)
    live, unc = r.cache_bytes(t_begin + K // 2)
    print(json.dumps({
        "workload": "cfg2: 1 layer, B=32, 12/2 heads, D=128, P=256, T=4096, c=16, page 16, keys pre-scaled, sm_scale 1",
        "steps": K, "t_window": [t_begin, t_begin + K], "us_per_step_graph": 1e3 * ms / K,
        "tokens_per_s": w.batch * K / (ms * 1e-3), "kv_bytes_per_step": (reg + bea) / K,
        "kv_gbs_step": (reg + bea) / (ms * 1e-3) / 1e9,
        "us_per_bc_decode_attn": 1e3 * a_ms / a_n, "attn_kernel_gbs": a_bytes / (a_ms * 1e-3) / 1e9,
        "us_per_bc_append_bracketed": med(app), "us_per_bc_compress_bracketed": med(comp),
        "cache_bytes_mid": live, "uncompressed_bytes_mid": unc, "gpu_launches": int(launches),
        "steps_through": "bc_append + bc_decode_attn (+ bc_decode_attn_pair, bc_compress)" if args.no_fused else "bc_decode_step, bc_fill_step",
        "note": "13 MB of KV per step stays in L2: the HBM roofline does not bound this configuration"}))


def report_ragged(args):
    """The ragged configuration: batch 128, 12/2 heads, page 16; prompt U[64,1024], generation
    U[1024,32768], c from {4,8,16} per sequence.  The whole run, plain launches: sequences finish at
    their own step and free their pages on the device."""
    import numpy as np
    import torch
    from paper_2510_13797_b200 import binding as B
    from paper_2510_13797_b200.workloads import InputStream, make_workload
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = make_workload("ragged")
    Bn, ps = w.batch, w.page_size
    P, T, C = np.array(w.prompt_lens), np.array(w.gen_lens), np.array(w.cs)
    cd = lambda a, b_: -(-a // b_)
    pps = cd(P, ps) + cd(C, ps) + cd(cd(T, C), ps) + 1
    cache = B.Cache(1, w.kv_heads, w.q_heads, w.head_dim, 1, ps, max_seqs=Bn, num_pages=int(pps.sum()),
                    max_pages_per_seq=int(pps.max()), device=dev)
    stream = InputStream(w, dev)
    pk, pv = stream.prompt_kv(0)
    ring = 16
    q, k, v = stream.step_chunk(0, 0, ring)
    bq, bk, bv = stream.beacon_chunk(0, 0, 4)
    i32 = lambda xs: torch.tensor(np.asarray(xs), dtype=torch.int32, device=dev)
    cu = np.concatenate([[0], np.cumsum(P)])
    all_slots = np.arange(Bn)
    cache.bc_seq_open(i32(all_slots), i32(P), i32(C))
    cache.bc_prefill(0, i32(all_slots), i32(cu), int(cu[-1]), pk, pv)
    out, outb, out2 = cache.new_out(Bn), cache.new_out(Bn), cache.new_out(Bn)
    paired = args.pair        # off by default here: with the small, shrinking batches of this run the paired
                              # kernel's longer per-tile arithmetic costs more than the saved traffic gains (measured)
    order = np.argsort(T, kind="stable")
    T_max = int(T.max())
    PERIOD = 16                                        # the call pattern of a fixed batch repeats every 16 steps

    def make_epoch(live):
        """Device tensors of one epoch (the batch stays as it is until the next sequence finishes)."""
        idx = torch.tensor(live, dtype=torch.int64, device=dev)
        ep = {"sl": i32(live), "k": k.index_select(1, idx), "v": v.index_select(1, idx), "q": q.index_select(1, idx),
              "groups": []}
        Cl = C[live]
        for ph in range(PERIOD):                       # sequences whose window fills at steps t = ph (mod 16)
            fill = ((ph % Cl) == 0) if ph else np.ones(len(live), dtype=bool)
            pos, rest = np.nonzero(fill)[0], np.nonzero(~fill)[0]
            if len(pos):
                gi = torch.tensor(live[pos], dtype=torch.int64, device=dev)
                grp = [i32(live[pos]), bq[0].index_select(0, gi), bk[0].index_select(0, gi), bv[0].index_select(0, gi)]
                if paired:      # the step's own queries of the two groups (step t uses ring row (t - 1) % 16)
                    jq = (ph - 1) % ring
                    pi, ri = torch.tensor(pos, dtype=torch.int64, device=dev), torch.tensor(rest, dtype=torch.int64, device=dev)
                    grp += [ep["q"][jq].index_select(0, pi).contiguous(),
                            (i32(live[rest]), ep["q"][jq].index_select(0, ri).contiguous()) if len(rest) else None]
                ep["groups"].append(tuple(grp))
            else:
                ep["groups"].append(None)
        return ep

    def step(t, ep):
        """Decode step t (1-based) of the epoch's batch: append, attend, and the beacon step where due."""
        j = (t - 1) % ring
        grp = ep["groups"][t % PERIOD]
        if not args.no_fused and not (grp is not None and paired):
            # append and attention of the whole batch in one launch behind the bookkeeping kernel
            cache.bc_decode_step(0, ep["sl"], ep["q"][j], ep["k"][j], ep["v"][j], out, w.sm_scale)
            if grp is not None:
                gsl, gq, gk, gv = grp[:4]
                cache.bc_decode_attn(0, gsl, gq, outb, w.sm_scale, gk, gv)
                cache.bc_compress(0, gsl, gk, gv)
            return
        cache.bc_append(0, ep["sl"], ep["k"][j], ep["v"][j])
        if grp is not None and paired:
            # the sequences whose window this token fills: token and beacon queries in one pass; the rest: plain
            gsl, gq, gk, gv, tq, rest = grp
            cache.bc_decode_attn_pair(0, gsl, tq, out, gq, outb, w.sm_scale, gk, gv)
            if rest is not None:
                cache.bc_decode_attn(0, rest[0], rest[1], out2, w.sm_scale)
            cache.bc_compress(0, gsl, gk, gv)
            return
        cache.bc_decode_attn(0, ep["sl"], ep["q"][j], out, w.sm_scale)
        if grp is not None:
            gsl, gq, gk, gv = grp[:4]
            cache.bc_decode_attn(0, gsl, gq, outb, w.sm_scale, gk, gv)
            cache.bc_compress(0, gsl, gk, gv)

    side = torch.cuda.Stream()
    graphs = []                                         # kept alive until the run is over
    torch.cuda.synchronize()
    e0, e1 = _event_pair(torch)
    t_host = time.perf_counter()
    e0.record()
    t, live, n_launch0 = 0, all_slots, cache.bc_kernel_launches()
    done_ptr, replayed_launches = 0, 0
    while len(live):
        t_end = int(T[order[done_ptr]])
        ep = make_epoch(live)
        while t < t_end and (t % PERIOD or t_end - t < 2 * PERIOD):
            t += 1; step(t, ep)                         # up to the next period boundary, or a short rest
        if t_end - t >= 2 * PERIOD:
            g = torch.cuda.CUDAGraph()
            l0 = cache.bc_kernel_launches()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):               # captured while the GPU still works on earlier steps
                g.capture_begin()
                for i in range(1, PERIOD + 1):
                    step(t + i, ep)
                g.capture_end()
            per_graph = cache.bc_kernel_launches() - l0
            graphs.append((g, ep))
            reps = (t_end - t) // PERIOD
            for _ in range(reps):
                g.replay()
            t += reps * PERIOD
            replayed_launches += (reps - 1) * per_graph
            while t < t_end:
                t += 1; step(t, ep)
        fin = []
        while done_ptr < Bn and T[order[done_ptr]] == t:
            fin.append(order[done_ptr]); done_ptr += 1
        cache.bc_seq_close(i32(fin))
        gone = set(fin)
        live = np.array([s for s in live if s not in gone], dtype=np.int64)
    e1.record()
    torch.cuda.synchronize()
    host_s = time.perf_counter() - t_host
    ms = e0.elapsed_time(e1)
    # accounting, outside the timed region: entries read and pages in use at every step (closed forms)
    kv_entries, high_water, high_water_unc = 0, 0, 0
    for t in range(1, T_max + 1):
        alive = T >= t
        Cl, Pl = C[alive], P[alive]
        kv_entries += int((Pl + (t - 1) // Cl + (t - 1) % Cl + 1).sum())
        full = (t % Cl) == 0
        if not paired:           # the beacon's second pass over the cache
            kv_entries += int((Pl[full] + (t // Cl[full] - 1) + Cl[full]).sum())
        if t % 16 == 0 or t == T_max:
            nbp, wl2 = t // Cl, t % Cl
            high_water = max(high_water, int((cd(Pl, ps) + cd(nbp, ps) + cd(wl2, ps)).sum()))
            high_water_unc = max(high_water_unc, int(cd(Pl + t, ps).sum()))
    code, slot, call = cache.bc_poll_error()
    assert code == 0, (code, slot, call)
    free = cache.bc_get_free_list()
    assert len(free) == int(pps.sum()), "pages were lost"
    E = w.entry_bytes
    tokens = int(T.sum())
    print(json.dumps({
        "workload": "ragged: 1 layer, B=128, 12/2 heads, D=128, page 16, P~U[64,1024], T~U[1024,32768], c in {4,8,16}",
        "decode_steps": T_max, "tokens": tokens, "ms_total": ms, "tokens_per_s": tokens / (ms * 1e-3),
        "kv_bytes_read": kv_entries * E, "kv_gbs": kv_entries * E / (ms * 1e-3) / 1e9,
        "pages_high_water": high_water, "pages_high_water_uncompressed": high_water_unc,
        "cache_bytes_high_water": high_water * ps * E, "uncompressed_bytes_high_water": high_water_unc * ps * E,
        "gpu_launches": int(cache.bc_kernel_launches() - n_launch0 + replayed_launches), "host_seconds": host_s,
        "all_pages_returned": True, "graphs": len(graphs),
        "beacon_steps": "paired with the token's attention (one pass over the cache)" if paired else "second attention pass",
        "regular_steps": "bc_append + bc_decode_attn" if (args.no_fused or paired) else "bc_decode_step",
        "note": "between two sequence finishes the batch is fixed and its call pattern repeats every 16 steps: "
                "those steps run as replays of one CUDA graph per epoch, the rest as plain launches"}))


def report_depth(args):
    """The full-depth configuration: 28 layers, batch 256, 12/2 heads, prompt 512, 8192 steps, c = 8,
    page 8.  Per-layer calls in dependency order, whole windows of 8 steps as one CUDA graph, at the
    middle of the generation; footprint against the uncompressed cache; the largest batch one GPU
    holds at c in {1, 4, 8, 16}, computed from the free memory and demonstrated at c = 8."""
    import torch
    from paper_2510_13797_b200 import binding as B
    from paper_2510_13797_b200.workloads import InputStream, make_workload
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = make_workload("depth")
    L, Bn, ps, c, P, T = w.layers, w.batch, w.page_size, w.cs[0], w.prompt_lens[0], w.steps
    E = w.entry_bytes
    cd = lambda a, b_: -(-a // b_)
    free0, total0 = torch.cuda.mem_get_info()

    def pages_per_seq(cc, page):
        return cd(P, page) + cd(cc, page) + cd(cd(T, cc), page) + 1 if cc > 1 else cd(P + T, page) + 1

    def bytes_per_seq(cc):
        page = cc if cc > 1 else 16
        return pages_per_seq(cc, page) * page * E * L

    capacity = {str(cc): int(0.90 * free0 // bytes_per_seq(cc)) for cc in (1, 4, 8, 16)}
    pps = pages_per_seq(c, ps)
    cache = B.Cache(L, w.kv_heads, w.q_heads, w.head_dim, c, ps, max_seqs=Bn, num_pages=Bn * pps,
                    max_pages_per_seq=pps, device=dev)
    slots = torch.arange(Bn, dtype=torch.int32, device=dev)
    cu = torch.arange(0, (Bn + 1) * P, P, dtype=torch.int32, device=dev)
    cache.bc_seq_open(slots, torch.full((Bn,), P, dtype=torch.int32, device=dev))
    stream = InputStream(w, dev)
    ring = 8
    ins = []
    for l in range(L):
        pk, pv = stream.prompt_kv(l)
        cache.bc_prefill(l, slots, cu, Bn * P, pk, pv)
        ins.append((stream.step_chunk(l, 0, ring), stream.beacon_chunk(l, 0, 2)))
        del pk, pv
    out, out_b = cache.new_out(Bn), cache.new_out(Bn)
    paired = not args.no_pair
    state = {"t": 0}

    def step(attend=True):
        t = state["t"]; j = t % ring
        for l in range(L):
            (q, k, v), _ = ins[l]
            if attend and paired and (t + 1) % c == 0:
                # the token fills the window: per layer append, then token and beacon queries in one pass, then compress
                _, (bq, bk, bv) = ins[l]
                m = ((t + 1) // c) % 2
                if not args.no_fused:
                    cache.bc_fill_step(l, slots, q[j], k[j], v[j], bq[m], bk[m], bv[m], out, out_b, w.sm_scale)
                else:
                    cache.bc_append(l, slots, k[j], v[j])
                    cache.bc_decode_attn_pair(l, slots, q[j], out, bq[m], out_b, w.sm_scale, bk[m], bv[m])
                    cache.bc_compress(l, slots, bk[m], bv[m])
            elif attend and not args.no_fused:
                cache.bc_decode_step(l, slots, q[j], k[j], v[j], out, w.sm_scale)
            else:
                cache.bc_append(l, slots, k[j], v[j])
                if attend:
                    cache.bc_decode_attn(l, slots, q[j], out, w.sm_scale)
        state["t"] = t = t + 1
        if t % c == 0 and not (attend and paired):
            m = (t // c) % 2
            for l in range(L):
                _, (bq, bk, bv) = ins[l]
                if attend:
                    cache.bc_decode_attn(l, slots, bq[m], out, w.sm_scale, bk[m], bv[m])
                cache.bc_compress(l, slots, bk[m], bv[m])

    K = max(c, (min(args.steps, 64) // c) * c)
    t_mid = ((T - K) // 2 // c) * c
    while state["t"] < t_mid:
        step(attend=False)
    for _ in range(c):
        step()
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    l0, t_save = cache.bc_kernel_launches(), state["t"]
    with torch.cuda.graph(graph, stream=s, capture_error_mode="thread_local"):
        for _ in range(c):
            step()
    per_graph = cache.bc_kernel_launches() - l0
    state["t"] = t_save
    torch.cuda.current_stream().wait_stream(s)
    graph.replay(); state["t"] += c
    torch.cuda.synchronize()
    t_begin = state["t"]
    e0, e1 = _event_pair(torch)
    e0.record()
    for _ in range(K // c):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    state["t"] += K
    ms = e0.elapsed_time(e1)
    code, slot, call = cache.bc_poll_error()
    assert code == 0, (code, slot, call)
    reg = sum(entries_attended(P, n, c) for n in range(t_begin + 1, t_begin + K + 1))
    bea = 0 if paired else sum(entries_beacon_query(P, n, c) for n in range(t_begin + 1, t_begin + K + 1) if n % c == 0)
    kv = (reg + bea) * E * Bn * L
    end_entries = P + T // c + T % c
    line = {
        "workload": "depth: 28 layers, B=256, 12/2 heads, D=128, P=512, T=8192, c=8, page 8",
        "beacon_steps": "paired with the token's attention (one pass over the cache per layer)" if paired else "second attention pass",
        "regular_steps": "bc_append + bc_decode_attn per layer" if args.no_fused else "bc_decode_step per layer",
        "steps": K, "t_window": [t_begin, t_begin + K], "ms_per_step": ms / K,
        "attention_tokens_per_s": Bn * K / (ms * 1e-3), "layer_tokens_per_s": Bn * K * L / (ms * 1e-3),
        "kv_bytes_per_step": kv / K, "kv_gbs": kv / (ms * 1e-3) / 1e9,
        "pct_of_8tbs": 100 * kv / (ms * 1e-3) / 8e12,
        "gpu_launches": int(per_graph * (K // c)),
        "kv_footprint_end_bytes": end_entries * E * L * Bn, "uncompressed_end_bytes": (P + T) * E * L * Bn,
        "footprint_ratio_end": (P + T) / end_entries,
        "hbm_free_bytes": free0, "hbm_total_bytes": total0,
        "largest_batch_that_fits": capacity,
        "largest_batch_rule": "floor(0.90 * free HBM / (pages per sequence at the end of the run * page bytes * 28 "
                              "layers)), page_size = c (16 for c = 1)",
    }
    # Secondary timing: the same steps with layer = -1, one launch per call for all 28 layers (the layers of a
    # real forward pass depend on one another, so this is the cache traffic alone, without the kernel boundaries).
    Qs, Ks, Vs = (torch.stack([ins[l][0][x] for l in range(L)], dim=1).contiguous() for x in range(3))      # [ring, L, B, H, D]
    BQs, BKs, BVs = (torch.stack([ins[l][1][x] for l in range(L)], dim=1).contiguous() for x in range(3))   # [2, L, B, H, D]
    out_all = torch.empty((L,) + tuple(out.shape), dtype=out.dtype, device=dev)

    def step_all():
        t = state["t"]; j = t % ring
        if (t + 1) % c == 0:
            m = ((t + 1) // c) % 2
            cache.bc_append(-1, slots, Ks[j], Vs[j])
            if paired:
                for l in range(L):
                    cache.bc_decode_attn_pair(l, slots, Qs[j, l], out, BQs[m, l], out_b, w.sm_scale, BKs[m, l], BVs[m, l])
            else:
                cache.bc_decode_attn(-1, slots, Qs[j], out_all, w.sm_scale)
                cache.bc_decode_attn(-1, slots, BQs[m], out_all, w.sm_scale, BKs[m], BVs[m])
            cache.bc_compress(-1, slots, BKs[m], BVs[m])
        else:
            cache.bc_decode_step(-1, slots, Qs[j], Ks[j], Vs[j], out_all, w.sm_scale)
        state["t"] = t + 1

    graph2 = torch.cuda.CUDAGraph()
    l0, t_save = cache.bc_kernel_launches(), state["t"]
    with torch.cuda.graph(graph2, stream=s, capture_error_mode="thread_local"):
        for _ in range(c):
            step_all()
    per_graph2 = cache.bc_kernel_launches() - l0
    state["t"] = t_save
    torch.cuda.current_stream().wait_stream(s)
    graph2.replay(); state["t"] += c
    torch.cuda.synchronize()
    t_begin2 = state["t"]
    e0, e1 = _event_pair(torch)
    e0.record()
    for _ in range(K // c):
        graph2.replay()
    e1.record()
    torch.cuda.synchronize()
    state["t"] += K
    ms2 = e0.elapsed_time(e1)
    code, slot, call = cache.bc_poll_error()
    assert code == 0, (code, slot, call)
    reg2 = sum(entries_attended(P, n, c) for n in range(t_begin2 + 1, t_begin2 + K + 1))
    bea2 = 0 if paired else sum(entries_beacon_query(P, n, c) for n in range(t_begin2 + 1, t_begin2 + K + 1) if n % c == 0)
    kv2 = (reg2 + bea2) * E * Bn * L
    line["all_layers_per_launch"] = {
        "what": "the same steps through layer = -1: a regular step is bc_decode_step(-1) = one bookkeeping kernel and ONE attention "
                "launch whose grid walks the 28 layers; a window fill is bc_append(-1), the per-layer paired attention and bc_compress(-1)",
        "t_window": [t_begin2, t_begin2 + K], "ms_per_step": ms2 / K, "kv_gbs": kv2 / (ms2 * 1e-3) / 1e9,
        "pct_of_8tbs": 100 * kv2 / (ms2 * 1e-3) / 8e12, "gpu_launches": int(per_graph2 * (K // c))}
    # demonstration at c = 8: allocate the pool for that many sequences and decode a window with all of them
    del cache, ins, graph, graph2, Qs, Ks, Vs, BQs, BKs, BVs, out_all
    torch.cuda.empty_cache()
    n_big = capacity["8"]
    big = B.Cache(L, w.kv_heads, w.q_heads, w.head_dim, c, ps, max_seqs=n_big, num_pages=n_big * pps,
                  max_pages_per_seq=pps, device=dev)
    all_slots = torch.arange(n_big, dtype=torch.int32, device=dev)
    big.bc_seq_open(all_slots, torch.full((n_big,), P, dtype=torch.int32, device=dev))
    chunk = 512                                       # sequences per call
    g = torch.Generator(device=dev); g.manual_seed(1)
    rnd = lambda *shape: torch.randn(shape, generator=g, device=dev).to(torch.bfloat16)
    pk, pv = rnd(chunk * P, w.kv_heads, w.head_dim), rnd(chunk * P, w.kv_heads, w.head_dim)
    kq = rnd(chunk, w.q_heads, w.head_dim); kk = rnd(chunk, w.kv_heads, w.head_dim)
    outc = big.new_out(chunk)
    cuc = torch.arange(0, (chunk + 1) * P, P, dtype=torch.int32, device=dev)
    starts = list(range(0, n_big, chunk))
    for l in range(L):
        for a in starts:
            n = min(chunk, n_big - a)
            big.bc_prefill(l, all_slots[a:a + n], cuc[:n + 1], n * P, pk, pv)
    e0, e1 = _event_pair(torch)
    e0.record()
    for t in range(1, c + 1):
        for l in range(L):
            big.bc_append(l, all_slots, rnd(n_big, w.kv_heads, w.head_dim), rnd(n_big, w.kv_heads, w.head_dim))
            for a in starts:
                n = min(chunk, n_big - a)
                big.bc_decode_attn(l, all_slots[a:a + n], kq[:n], outc[:n], w.sm_scale)
        if t == c:
            for l in range(L):
                big.bc_compress(l, all_slots, rnd(n_big, w.kv_heads, w.head_dim), rnd(n_big, w.kv_heads, w.head_dim))
    e1.record()
    torch.cuda.synchronize()
    code, slot, call = big.bc_poll_error()
    st = big.bc_get_state(n_big - 1)
    line["demonstrated"] = {"c": 8, "batch": n_big, "pool_bytes": big.pool_bytes, "steps": c,
                            "ms_per_step": e0.elapsed_time(e1) / c, "device_error": code,
                            "last_slot_state": {k_: st[k_] for k_ in ("prompt_len", "n_beacons", "window_len", "t")}}
    print(json.dumps(line))


def measure_maskform(T, n=8, ratios=RATIOS):
    """The mask-form pass (Section 3.2, Figure 2) on n trajectories of the sweep shape: 32/8 heads,
    D 128, prompt 512, T generated tokens, one beacon per c tokens.  A dense contraction: reported
    in TFLOP/s against the measured bf16 tensor peak.  Useful flops = 4 * D * q_heads * (visible
    keys summed over the token and beacon rows); flops of masked key positions are not counted."""
    import torch
    from paper_2510_13797_b200 import binding as B
    dev = torch.device("cuda", torch.cuda.current_device())
    Hq, Hkv, D, P = 32, 8, 128, 512
    peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
    peak = float(peaks.get("bf16_tflops", 1590.0))
    g = torch.Generator(device=dev); g.manual_seed(0)
    rnd = lambda *shape: torch.randn(shape, generator=g, device=dev).to(torch.bfloat16)
    rows = []
    for c in ratios:
        nb = T // c
        pk, pv = rnd(n * P, Hkv, D), rnd(n * P, Hkv, D)
        tq, tk, tv = rnd(n * T, Hq, D), rnd(n * T, Hkv, D), rnd(n * T, Hkv, D)
        bq, bk, bv = rnd(n * nb, Hq, D), rnd(n * nb, Hkv, D), rnd(n * nb, Hkv, D)
        call = lambda check=False: B.bc_mask_attn_forward([P] * n, [T] * n, c, pk, pv, tq, tk, tv, bq, bk, bv,
                                                          1.0 / math.sqrt(D), check=check)
        call(check=True)
        call()
        torch.cuda.synchronize()
        reps = 3 if T > 4096 else 30                       # short calls: average over more of them
        e0, e1 = _event_pair(torch)
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        keys_tok = sum(P + i // c + i % c + 1 for i in range(T))
        keys_bea = sum(P + m + c for m in range(1, nb + 1))
        flops = 4.0 * D * Hq * (keys_tok + keys_bea) * n
        rows.append({"c": c, "ms": ms, "useful_tflops": flops / (ms * 1e-3) / 1e12,
                     "frac_of_bf16_peak": flops / (ms * 1e-3) / 1e12 / peak, "rows": n * (T + nb)})
        del pk, pv, tq, tk, tv, bq, bk, bv
        torch.cuda.empty_cache()
    return {"workload": f"maskform: {n} trajectories, 32/8 heads, D=128, P={P}, T={T}, c in {list(ratios)}; "
                        "whole calls (host-side tile list and tensor maps included)",
            "roofline": {"bound": "tensor", "unit": "TFLOP/s", "peak": peak, "peak_source": "MEASURED_PEAKS.json bf16_tflops (burst)",
                         "achieved": max(r["useful_tflops"] for r in rows),
                         "frac": max(r["frac_of_bf16_peak"] for r in rows),
                         "min_frac_over_c": min(r["frac_of_bf16_peak"] for r in rows)},
            "rows": rows}


def report_maskform(args):
    import torch
    torch.cuda.set_device(0)
    print(json.dumps(measure_maskform(16384 if args.steps >= 512 else 2048)))


def measure_distill(n_traj):
    """The distillation loss (Eq. 1) at the vocabulary of the 1.5B model the paper trains (151,936)
    with the paper's 100 stored teacher entries per position: n_traj trajectories of 1,000 positions
    (the paper's maximum response length).  One streaming read of the student logits: HBM-bound.
    Algorithmic bytes: rows * vocab * 2 (logits) + rows * 100 * 8 (teacher entries); with the
    gradient, another rows * vocab * 2 written (the second read of a row comes from L2)."""
    import torch
    from paper_2510_13797_b200 import binding as B
    dev = torch.device("cuda", torch.cuda.current_device())
    peak, peak_src = load_peaks()
    T, V, K = 1000, 151936, 100
    rows = n_traj * T
    g = torch.Generator(device=dev); g.manual_seed(0)
    z = torch.empty((rows, V), dtype=torch.bfloat16, device=dev)
    for a in range(0, rows, 2000):                         # drawn in slabs: fp32 randn of the whole matrix would be 9.7 GB
        z[a:a + 2000] = (torch.randn((min(2000, rows - a), V), generator=g, device=dev) * 3).to(torch.bfloat16)
    idx = torch.stack([torch.randperm(V, generator=g, device=dev)[:K] for _ in range(64)]).to(torch.int32)
    idx = idx.repeat(-(-rows // 64), 1)[:rows].contiguous()
    lp = torch.log_softmax(torch.randn((rows, K), generator=g, device=dev) * 2, dim=1).to(torch.float32) + math.log(0.93)
    cu = torch.arange(0, rows + 1, T, dtype=torch.int32, device=dev)
    out = {}
    for with_grad in (False, True):
        for _ in range(2):
            B.bc_distill_loss(cu, z, idx, lp, with_grad=with_grad)
        torch.cuda.synchronize()
        e0, e1 = _event_pair(torch)
        reps = 5
        e0.record()
        for _ in range(reps):
            loss, _, _ = B.bc_distill_loss(cu, z, idx, lp, with_grad=with_grad)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        nbytes = rows * V * 2 * (2 if with_grad else 1) + rows * K * 8
        out["forward_backward" if with_grad else "forward"] = {
            "ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "frac_of_peak": nbytes / (ms * 1e-3) / 1e9 / peak,
            "algorithmic_bytes": nbytes, "positions_per_s": rows / (ms * 1e-3)}
    res = {"workload": f"distill: {n_traj} trajectories x {T} positions, vocab {V}, top-{K} teacher entries, bf16 logits",
           "loss": float(loss), "roofline": {"bound": "hbm", "unit": "GB/s", "peak": peak, "peak_source": peak_src,
                                            "achieved": out["forward"]["gbs"], "frac": out["forward"]["frac_of_peak"]},
           **out}
    del z, idx, lp
    torch.cuda.empty_cache()
    return res


def report_distill(args):
    import torch
    torch.cuda.set_device(0)
    print(json.dumps(measure_distill(16 if args.steps >= 16 else 4)))   # --steps < 16: a 1.2 GB case for profiling


def report_model(args):
    """End-to-end generation with a random-weight decoder of the 1.5B shape around the cache library
    (28 layers, hidden 1536, 12/2 heads, D 128, MLP 8960, vocabulary 151,936; batch 64, prompt 512):
    time to generate N tokens per sequence at ratio c relative to the uncompressed cache -- the
    protocol of the paper's latency table.  The non-attention layers are PyTorch operators."""
    Bn, N, reps = 64, 512 if args.steps >= 512 else 128, 3
    if args.model_ratio is not None:
        # one ratio, in a process of its own (see below): prints its row and nothing else
        import torch
        from bench_model import ToyDecoder
        torch.cuda.set_device(0)
        c = args.model_ratio
        m = ToyDecoder(Bn, c, gen_len=reps * N + 128, device="cuda", paired=not args.no_pair, lib_rope=not args.torch_rope)
        m.capture()
        torch.cuda.synchronize()
        times = []
        for _ in range(reps):                               # best of three: clocks settle during the first
            e0, e1 = _event_pair(torch)
            e0.record()
            m.generate(N)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        st = m.check()
        ms = min(times)
        print(json.dumps({"c": c, "ms": ms, "ms_per_token": ms / N, "tokens_per_s": Bn * N / (ms * 1e-3), "ms_all": times,
                          "cache_entries_end": st["prompt_len"] + st["n_beacons"] + st["window_len"]}))
        return
    # Every ratio runs in a fresh process.  The PyTorch part of a step is some 1100 small kernels in
    # one CUDA graph, and in a process that has already built and dropped a decoder the same graph can
    # replay with about 0.5 us more between consecutive kernels (same kernel times, 12 % more per
    # token): more than the differences between ratios that this protocol is after.
    rows, base = [], None
    for c in (1,) + RATIOS:
        cmd = [sys.executable, os.path.abspath(__file__), "--workload", "model", "--model-ratio", str(c), "--steps", str(args.steps)]
        if args.no_pair:
            cmd.append("--no-pair")
        if args.torch_rope:
            cmd.append("--torch-rope")
        child = subprocess.run(cmd, capture_output=True, text=True)
        if child.returncode != 0:
            sys.stderr.write(child.stderr[-2000:])
            raise SystemExit(f"model workload: the run at c = {c} exited {child.returncode}")
        row = json.loads(child.stdout.strip().splitlines()[-1])
        base = row["ms"] if c == 1 else base
        row["latency_vs_uncompressed"] = row["ms"] / base
        rows.append(row)
    print(json.dumps({"workload": f"model: random-weight decoder of the 1.5B shape, batch {Bn}, prompt 512, {N} generated tokens "
                                  "per sequence, one CUDA graph per token step and per beacon step"
                                  + ("" if args.no_pair else "; the beacon is encoded in the same 2-token pass as the token that fills the window"),
                      "operators_between_the_gemms": "PyTorch operators" if args.torch_rope else
                      "the library's kernels: bc_rope_decode_step / bc_rope_split + bc_fill_step (rotation, append, attention), "
                      "bc_add_rmsnorm (residual add and norm), bc_swiglu, bc_argmax; the GEMMs and the embedding lookup are PyTorch's",
                      "paper_latency_table_qwen_sr": {"2": 1.990, "4": 1.546, "8": 1.593, "16": 1.646, "32": 1.468},
                      "rows": rows}))


def read_stream_peak(dev):
    """GB/s of a read-only pass over 4 GiB with the attention kernel's copy pattern and no arithmetic
    (bc_probe_read_stream): best of five after two warm-up passes."""
    import torch
    from paper_2510_13797_b200 import binding as B
    buf = torch.empty(4 << 30, dtype=torch.uint8, device=dev)
    buf.fill_(1)
    best = 0.0
    for i in range(7):
        e0, e1 = _event_pair(torch)
        e0.record(); B.bc_probe_read_stream(buf); e1.record()
        torch.cuda.synchronize()
        if i >= 2:
            best = max(best, buf.numel() / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    del buf
    torch.cuda.empty_cache()
    return best


def batch_scaling(dev, peak):
    """The attention kernel alone at larger batches (same shape, mid-generation cache): the time per
    launch that does not stream (start-up, merging) is spread over more bytes."""
    import torch
    from paper_2510_13797_b200.workloads import make_workload
    rows = []
    for c in (16, 32):
        for Bn in (128, 256):
            w = make_workload("sweep", c=c, batch=Bn)
            mid = entries_attended(w.prompt_lens[0], w.steps // 2, c)
            w = make_workload("sweep", c=c, batch=Bn, prompt_lens=[mid] * Bn, gen_lens=[256] * Bn)
            r = make_runner(w, dev)
            r.reset_to(c // 2)
            ms, n, nbytes = r.timed_attn_stream(64, 4)
            r.check_error()
            rows.append({"c": c, "batch": Bn, "attn_kernel_us": 1e3 * ms / n, "attn_kernel_gbs": nbytes / (ms * 1e-3) / 1e9,
                         "frac_of_peak": nbytes / (ms * 1e-3) / 1e9 / peak, "pct_of_8tbs": 100 * nbytes / (ms * 1e-3) / 8e12})
            del r
            torch.cuda.empty_cache()
    return rows


# ------------------------------------------------------------------------------ main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--torch-rope", action="store_true",
                    help="--workload model: rotary embedding, QKV split, norms, gated activation and argmax with PyTorch operators instead of the library's kernels")
    ap.add_argument("--no-pair", action="store_true", help="beacon steps as a second attention pass instead of bc_decode_attn_pair")
    ap.add_argument("--pair", action="store_true", help="ragged workload: pair the beacon steps too (off by default there)")
    ap.add_argument("--fused", action="store_true", help="--timeline: regular steps through bc_decode_step")
    ap.add_argument("--no-fused", action="store_true", help="sweep, depth, --profile-case: regular steps as bc_append + bc_decode_attn instead of bc_decode_step")
    ap.add_argument("--ratios", default="")
    ap.add_argument("--skip-uncompressed", action="store_true")
    ap.add_argument("--model-ratio", type=int, default=None, help=argparse.SUPPRESS)   # model workload: one ratio (child process)
    ap.add_argument("--workload", default="sweep", choices=["sweep", "cfg2", "ragged", "depth", "maskform", "distill", "model"],
                    help="sweep (default): the benchmark line; cfg2 / ragged / depth: a report line for that "
                         "benchmark configuration (1 GPU)")
    ap.add_argument("--no-batch-scaling", action="store_true")
    ap.add_argument("--replays", type=int, default=3, help="rewind-and-replay rounds of the timed graph (the first one is the reported time)")
    ap.add_argument("--no-extras", action="store_true", help="skip the short mask-form and distillation runs of the default line")
    ap.add_argument("--timeline", type=int, default=0, metavar="C",
                    help="per-block time stamps of the attention kernel (bc_attn_timeline) on the small case of ratio C")
    ap.add_argument("--timeline-shape", default="sweep", choices=["sweep", "depth"], help="with --timeline: the sweep's head shape and batch, or one layer of the full-depth configuration")
    ap.add_argument("--timeline-raw", action="store_true", help="with --timeline: also print every block's stamps")
    ap.add_argument("--profile-case", type=int, default=0, metavar="C",
                    help="small case for profilers: ratio C with a prompt as long as the mid-generation cache, "
                         "--steps plain decode steps, no fast-forward, no graphs")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.profile_case:
        return run_profile_case(args)
    if args.timeline:
        return run_timeline(args)
    if args.workload != "sweep":
        return {"cfg2": report_cfg2, "ragged": report_ragged, "depth": report_depth, "maskform": report_maskform, "distill": report_distill, "model": report_model}[args.workload](args)

    import torch
    import torch.distributed as dist
    from paper_2510_13797_b200 import sharding
    from paper_2510_13797_b200.workloads import make_workload

    K, W = args.steps, max(args.warmup, 3)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    ratios = tuple(int(x) for x in args.ratios.split(",")) if args.ratios else RATIOS
    peak, peak_src = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    rows, total_ms, total_launches = [], 0.0, 0
    kern_ms = kern_bytes = kern_launches = 0.0
    brack_ms = brack_bytes = step_bytes = 0.0
    e2e_ms = 0.0
    h2d = d2h = 0.0
    sampler = ClockSampler(local)
    sweep = list(ratios) + ([] if args.skip_uncompressed else [1])
    barrier()
    sampler.start()
    for c in sweep:
        w = make_workload("sweep", c=c)
        T = w.steps
        r = make_runner(w, dev, seed_offset=sharding.rank_seed_offset(0, rank), paired=not args.no_pair, fused=not args.no_fused)
        cyc = c if c > 1 else 16
        t_mid = max(0, ((T - K) // 2 // cyc) * cyc)
        # pass A: device-resident inputs, CUDA-graph replays: the headline time
        r.reset_to(max(0, t_mid - W - cyc))
        barrier()
        ms, t_begin, launches = r.timed_graph(K, max(W, t_mid - r.t - cyc), replays=args.replays)
        # pass B: plain launches, every attention kernel bracketed by events: the roofline figures
        Kp = min(K, 256)
        r.reset_to(max(0, t_mid - W))
        b_ms, b_n, b_bytes, plain_ms = r.timed_kernels(Kp, W)
        k_ms, k_n, k_bytes = r.timed_attn_stream(max(Kp, 128), W)   # at least 128 launches: the first one has no launch ahead to start under
        # pass C: host buffers through the C ABI, copies inside the timed region
        r.reset_to(max(0, t_mid - W))
        barrier()
        h_ms = r.timed_host(K, W)
        r.check_error()
        ms, h_ms = sharding.max_over_ranks([ms, h_ms], device=dev)      # the slowest rank counts
        reg, bea = r.kv_bytes(t_begin, K)
        live, unc = r.cache_bytes(t_begin + K // 2)
        end_live, end_unc = r.cache_bytes(T)
        regular, fills = r.graph_steps
        row = {
            "c": c, "page_size": w.page_size, "ms_per_step": ms / K, "tokens_per_s": world * w.batch * K / (ms * 1e-3),
            "graph": f"one CUDA graph of the {K} timed steps ({regular} regular, {fills} window-filling), replayed once under the events",
            "ms_per_step_p50_p99_over_windows": _percentiles(r.window_step_ms),
            "e2e_tokens_per_s": world * w.batch * K / (h_ms * 1e-3),
            "e2e_us_per_step": 1e3 * h_ms / K, "e2e_host_enqueue_us_per_step": 1e3 * r.host_enqueue_ms / K,
            "plain_launch_ms_per_step": plain_ms / Kp,
            "kv_gbs_step": (reg + bea) / (ms * 1e-3) / 1e9,
            "step_frac_of_peak": (reg + bea) / (ms * 1e-3) / 1e9 / peak,
            "step_pct_of_8tbs": 100 * (reg + bea) / (ms * 1e-3) / 8e12,
            "attn_kernel_us": 1e3 * k_ms / k_n, "attn_kernel_gbs": k_bytes / (k_ms * 1e-3) / 1e9,
            "attn_kernel_us_bracketed": 1e3 * b_ms / b_n, "attn_kernel_gbs_bracketed": b_bytes / (b_ms * 1e-3) / 1e9,
            "attn_frac_of_peak_bracketed": b_bytes / (b_ms * 1e-3) / 1e9 / peak,
            "attn_dram_traffic_per_launch": traffic_per_launch(c, k_bytes / k_n),
            "attn_frac_of_peak": k_bytes / (k_ms * 1e-3) / 1e9 / peak,
            "attn_pct_of_8tbs": 100 * k_bytes / (k_ms * 1e-3) / 8e12,
            "kv_bytes_per_step": (reg + bea) / K, "cache_bytes_mid": live, "uncompressed_bytes_mid": unc,
            "cache_bytes_end": end_live, "uncompressed_bytes_end": end_unc,
            "t_window": [t_begin, t_begin + K],
        }
        rows.append(row)
        if c > 1:
            total_ms += ms; total_launches += launches
            kern_ms += k_ms; kern_bytes += k_bytes; kern_launches += k_n
            brack_ms += b_ms; brack_bytes += b_bytes
            step_bytes += reg + bea
            e2e_ms += h_ms
            a, b = r.host_bytes_per_step()
            h2d += a; d2h += b
        del r
        torch.cuda.empty_cache()
    barrier()
    clocks = sampler.stop()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    n_c = sum(1 for c in sweep if c > 1)
    B = 64
    value = world * B * n_c * K / (total_ms * 1e-3)
    achieved = kern_bytes / (kern_ms * 1e-3) / 1e9
    tr = [r["attn_dram_traffic_per_launch"] for r in rows if r["c"] > 1]
    traffic = None if any(x is None for x in tr) else sum(tr) / len(tr)      # equal launch counts per ratio
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "sweep: 1 layer, B=64 per ratio, 32/8 heads, D=128, P=512, T=16384, "
                               "c in {2,4,8,16,32}, page_size=c; one step = one decode step at each ratio, "
                               "timed ratio by ratio around mid-generation",
                   "l2": "inputs larger than L2: every step streams 206 MB (c=32) to 1.2 GB (c=2) of KV, L2 is 126 MB",
                   "launch": "per ratio, the K timed steps are one CUDA graph replayed once under the event pair "
                             "(captured at the timed position, warmed by one replay, caches rewound); sweep[].graph "
                             "gives the steps it holds", "per_gpu_batch": B * n_c,
                   "regular_steps": "bc_append + bc_decode_attn" if args.no_fused else
                                    "bc_decode_step (the append's bookkeeping kernel, then one attention kernel that takes the new entries from the inputs)",
                   "beacon_steps": "second attention pass" if args.no_pair else
                                   ("paired with the token's attention (bc_append, bc_decode_attn_pair: one pass over the cache, bc_compress)"
                                    if args.no_fused else
                                    "bc_fill_step (the append's bookkeeping kernel, one paired attention kernel that takes the token's entry "
                                    "from the inputs and serves the token's and the beacon's rows in one pass over the cache, bc_compress)")},
        "e2e": {"value": world * B * n_c * K / (e2e_ms * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(total_launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "k_attn_pipe", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": kern_bytes / kern_launches,
                     "timing": "achieved / frac: CUDA events around back-to-back launches of the kernel alone at each "
                               "ratio (mid-generation cache): the launch interval, in which a launch begins under the "
                               "tail of the one before.  frac_bracketed: every single launch inside plain decode steps "
                               "bracketed by events (2-3 us of event overhead per launch included).  frac_in_step: the "
                               "algorithmic KV bytes of the timed steps over the whole graph-replayed step time "
                               "(bookkeeping, row writes and launch gaps included).  All three byte-weighted over the "
                               "five ratios; the per-ratio figures are in sweep[] and the minima below",
                     "launches_timed": int(kern_launches),
                     "frac_bracketed": brack_bytes / (brack_ms * 1e-3) / 1e9 / peak,
                     "frac_in_step": step_bytes / (total_ms * 1e-3) / 1e9 / peak,
                     "min_frac_over_c": min(r["attn_frac_of_peak"] for r in rows if r["c"] > 1),
                     "min_frac_bracketed_over_c": min(r["attn_frac_of_peak_bracketed"] for r in rows if r["c"] > 1),
                     "min_frac_in_step": min(r["step_frac_of_peak"] for r in rows if r["c"] > 1),
                     "pct_of_8tbs": 100 * achieved * 1e9 / 8e12,
                     "pct_of_8tbs_per_c": {str(r["c"]): {"kernel_interval": r["attn_pct_of_8tbs"], "in_step": r["step_pct_of_8tbs"]}
                                           for r in rows if r["c"] > 1},
                     "target_bar": "the 70 % bar of the target is read against the nominal 8 TB/s on the kernel's launch "
                                   "interval (pct_of_8tbs_per_c[c].kernel_interval); in_step is the same bytes over the "
                                   "whole step"},
        "sweep": rows,
    }
    if world == 1:
        rs = read_stream_peak(dev)
        line["roofline"]["read_stream_gbs"] = rs
        line["roofline"]["frac_of_read_stream"] = achieved / rs
        line["roofline"]["read_stream_note"] = ("read-only pass with the kernel's own copy pattern and no arithmetic "
                                                "(bc_probe_read_stream): unlike the copy benchmark behind `peak`, a ceiling")
    if not args.no_batch_scaling and world == 1:
        line["batch_scaling"] = batch_scaling(dev, peak)
    if not args.no_extras and world == 1:
        # the two kernels beside the decode path, short cases, so that the same record holds their figures
        line["maskform"] = measure_maskform(2048)
        line["distill"] = measure_distill(4)
    if not args.no_cpu_baseline:
        w = make_workload("sweep", c=16)
        wall, tok, cpu = oracle_sample(w, w.steps // 2, 64, 24)     # about ten seconds of CPU work
        line["cpu_baseline"] = {"value": tok / wall, "unit": "tokens/s", "cores": max(1, round(cpu / wall)),
                                "kind": "oracle",
                                "sample": "64 of 64 sequences, 24 decode steps (one of them fills a window) at c=16, cache at generation step 8192"}
        wall_all, tok_all, procs = oracle_sample_all_cores(16, w.steps // 2, 64, 24)
        line["cpu_baseline"]["cores_all"] = {"value": tok_all / wall_all, "unit": "tokens/s", "cores": procs,
                                             "host_cores": os.cpu_count(),
                                             "sample": "the same sample, the 64 sequences dealt out over one process per host core"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
