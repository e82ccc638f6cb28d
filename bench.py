#!/usr/bin/env python
"""Benchmark of the KV-cache attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3_c512] [--impl ours|reference]

One step = one pass of the whole hot path over one batch of seeded synthetic input:
for a prefill workload every chunk is written to the cache and attends to it
(jupiter_chunk_prefill_append_attn: both in one call); for a branch workload every decode step
writes one block per branch into the suffix caches and attends (jupiter_branch_append_attn, both in
one call).  Prints ONE JSON line.

Timing: CUDA events on the launching stream, one pair per step, L2 flushed between steps
(outside the pairs); the reported time is the sum over the K timed steps, max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import synth  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
PREFILL = {"cfg1": synth.cfg1, "cfg2": synth.cfg2, "cfg3_c128": lambda: synth.cfg3(128),
           "cfg3_c512": lambda: synth.cfg3(512), "cfg3_c1024": lambda: synth.cfg3(1024)}
BRANCH = {"cfg4": synth.cfg4, "cfg5": synth.cfg5}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_c512", choices=sorted(PREFILL) + sorted(BRANCH),
                    help="default: the largest single-GPU workload (4 x 8192-token GQA prompts, chunks of 512)")
    ap.add_argument("--no-extra", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time eager launches instead of a CUDA-graph replay")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only) while the timed region runs."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period = index, period_s
        self.sm, self.power, self.reason_bits = [], [], 0
        self.max_sm = None
        self._stop = threading.Event()
        self.thread = None
        self.error = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # pragma: no cover
            self.error = f"nvml unavailable: {e}"
            return
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception as e:  # pragma: no cover
                self.error = str(e)
                return
            time.sleep(self.period)

    def mark(self):
        """Index of the next sample: lets the caller keep only samples taken inside a region."""
        return len(self.sm)

    def stop(self, begin=0, end=None):
        self._stop.set()
        if self.thread:
            self.thread.join(timeout=2)
        sm = self.sm[begin:end] or self.sm
        reasons = sorted(name for bit, name in self.REASONS.items() if self.reason_bits & bit)
        out = {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": self.max_sm, "samples": len(sm),
               "power_w_max": max(self.power) if self.power else None, "reasons": reasons}
        if self.error:
            out["note"] = self.error
        return out


# ----------------------------------------------------------------------------- GPU side

def _dev(bits, device):
    import torch
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


class Flusher:
    """Writes a buffer larger than L2 so the next step starts with a cold L2."""

    def __init__(self, device):
        import torch
        l2 = torch.cuda.get_device_properties(device).L2_cache_size
        self.buf = torch.empty(max(2 * l2, 256 << 20), dtype=torch.uint8, device=device)

    def __call__(self):
        self.buf.fill_(1)


def timed_steps(step_fn, steps, warmup, flush, dist_barrier):
    """W untimed + K timed steps; returns the per-step durations in ms."""
    import torch
    for _ in range(warmup):
        flush()
        step_fn()
    torch.cuda.synchronize()
    dist_barrier()
    torch.cuda.synchronize()
    pairs = []
    for _ in range(steps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        step_fn()
        b.record()
        pairs.append((a, b))
    torch.cuda.synchronize()
    dist_barrier()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in pairs]


class PrefillRun:
    """Device state and step function of a chunked-prefill workload."""

    def __init__(self, ctx, w, device, data=None):
        import torch
        import paper_2504_08242_b200 as J
        self.ctx, self.w = ctx, w
        q, k, v = data if data is not None else w.make()
        qd, kd, vd = _dev(q, device), _dev(k, device), _dev(v, device)
        self.kc = torch.zeros(w.batch, w.kv_heads, w.capacity, w.head_dim, dtype=torch.bfloat16, device=device)
        self.vc = torch.zeros_like(self.kc)
        self.desc = J.cache_desc(self.kc, self.vc)
        self.chunks = []
        for pos, n in w.chunks():
            self.chunks.append(dict(
                pos=pos, n=n, q=qd[:, pos:pos + n].contiguous(), k=kd[:, pos:pos + n].contiguous(),
                v=vd[:, pos:pos + n].contiguous(),
                out=torch.empty(w.batch, n, w.q_heads, w.head_dim, dtype=torch.float32, device=device)))
        del qd, kd, vd
        self.attn_events = None

    def step(self):
        ctx, w, ev = self.ctx, self.w, self.attn_events
        for c in self.chunks:
            if ev is not None:
                import torch
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
            ctx.chunk_prefill_append_attn(c["q"], c["k"], c["v"], self.desc, w.q_heads, c["n"], c["pos"], w.scale,
                                          c["out"])
            if ev is not None:
                b.record()
                ev.append((a, b))

    def units(self):
        return float(self.w.flops())

    def attn_launches_per_step(self):
        return len(self.chunks)


class BranchRun:
    """Device state and step function of a branch-attention workload.  `copies` > 1 rotates the launches over
    independent copies of the caches so that each launch reads cold data.  A workload with a single decode step
    (speculative verification) runs that step `passes` times per benchmark step, each pass on the next copy: the
    data of every pass is cold (the copies together exceed L2 and L2 is flushed between steps) while the kernel's
    code, as in a real decoding loop, is not fetched from DRAM for every launch."""

    def __init__(self, ctx, w, device, copies=1, passes=1):
        import torch
        import paper_2504_08242_b200 as J
        self.ctx, self.w, self.copies, self.passes = ctx, w, copies, passes
        pk, pv, sk, sv = w.make_caches()
        self.caches = []
        for _ in range(copies):
            t = [_dev(x, device) for x in (pk, pv, sk, sv)]
            self.caches.append((t, J.cache_desc(t[0], t[1]), J.cache_desc(t[2], t[3])))
        hist = w.history_lengths().astype(np.int32)
        self.steps_data, self.bytes, self.flops = [], 0, 0
        for t in range(w.steps):
            q, kn, vn = w.make_step(t)
            pos = hist + t * w.q_len
            lens = pos + w.q_len
            self.steps_data.append(dict(
                q=_dev(q, device), k=_dev(kn, device), v=_dev(vn, device),
                pos=torch.from_numpy(pos.astype(np.int32)).to(device),
                lens=torch.from_numpy(lens.astype(np.int32)).to(device), max_len=int(lens.max())))
            self.bytes += passes * w.step_bytes(lens)
            self.flops += passes * w.step_flops(lens)
        self.out = torch.empty(w.n_branches, w.q_len, w.q_heads, w.head_dim, dtype=torch.float32, device=device)
        self.attn_events = None

    def calls(self):
        """(copy index, step data) of every library call of one benchmark step, in order."""
        k = 0
        for _ in range(self.passes):
            for s in self.steps_data:
                yield k % self.copies, s
                k += 1

    def step(self):
        ctx, w, ev = self.ctx, self.w, self.attn_events
        for c, s in self.calls():
            _, pdesc, sdesc = self.caches[c]
            if ev is not None:
                import torch
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
            ctx.branch_append_attn(s["q"], s["k"], s["v"], pdesc, w.prefix_len, sdesc, s["lens"], s["max_len"],
                                   w.n_branches, w.q_heads, w.q_len, w.scale, self.out)
            if ev is not None:
                b.record()
                ev.append((a, b))

    def units(self):
        return float(self.bytes)

    def attn_launches_per_step(self):
        return len(self.steps_data) * self.passes


def branch_run(ctx, w, device, cold=True):
    """The benchmark's form of a branch workload: launches rotate over cache copies that together exceed L2."""
    if not cold:
        return BranchRun(ctx, w, device, copies=1, passes=1)
    copies = 8 if w.steps == 1 else 6
    return BranchRun(ctx, w, device, copies=copies, passes=copies if w.steps == 1 else 1)


def measure(run, steps, warmup, flush, barrier, use_graph=True, sampler=None):
    """Timed region, then an instrumented replay with an event pair around every attention call.

    Timed region: the step is captured once in a CUDA graph (its launches are 2-60 us kernels, so
    eager launches would time the host) and replayed K times, one event pair per replay.
    Instrumented replay (eager): each step is queued behind a ~0.3 ms device-side delay so that all
    of its launches and events are already enqueued when the GPU starts them; an event pair then
    brackets the kernels of one attention call and nothing else."""
    import torch
    c0 = run.ctx.launch_count()
    for _ in range(max(warmup, 1)):
        flush()
        run.step()
    torch.cuda.synchronize()
    per_step_launches = (run.ctx.launch_count() - c0) // max(warmup, 1)
    step_fn = run.step
    if use_graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            run.step()
        step_fn = g.replay
        for _ in range(2):
            flush()
            step_fn()
        torch.cuda.synchronize()
    i0 = sampler.mark() if sampler else 0
    ms = timed_steps(step_fn, steps, 0, flush, barrier)
    i1 = sampler.mark() if sampler else 0
    run.attn_events = []
    for _ in range(steps):
        flush()
        torch.cuda._sleep(600000)
        run.step()
    torch.cuda.synchronize()
    attn_ms = [a.elapsed_time(b) for a, b in run.attn_events]
    run.attn_events = None
    ms_per_step = float(np.sum(ms) / steps)
    attn_per_step, attn_per_launch, source = float(np.sum(attn_ms) / steps), float(np.mean(attn_ms)), "event pair per call"
    if per_step_launches == run.attn_launches_per_step() and ms_per_step < attn_per_step:
        # the step holds nothing but attention launches: the timed region itself bounds their duration from
        # above (launch gaps included) and is free of the per-call event overhead of the eager replay
        attn_per_step, attn_per_launch = ms_per_step, ms_per_step / per_step_launches
        source = "timed region / launches"
    return dict(ms_per_step=ms_per_step, ms_steps=ms, attn_ms_per_launch=attn_per_launch,
                attn_ms_per_step=attn_per_step, launches_per_step=int(per_step_launches),
                attn_time_source=source, sample_range=(i0, i1))


def plain_read_floor(ctx, device, bytes_per_launch, launches, flush, copies=6, reps=5):
    """Yardstick for the branch workloads, not part of the hot path: how long a plain read of the same number of
    bytes takes per launch in the same kind of chain (one CUDA graph of `launches` back-to-back reads rotating over
    `copies` buffers, L2 flushed before each replay).  The read is jupiter_read_probe."""
    import torch
    n = max(16, int(bytes_per_launch) // 16 * 16)
    bufs = [torch.ones(n, dtype=torch.uint8, device=device) for _ in range(copies)]
    word = torch.zeros(1, dtype=torch.int32, device=device)

    def chain():
        for i in range(launches):
            ctx.read_probe(bufs[i % copies], n, word)
    chain()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        chain()
    best = float("inf")
    for _ in range(reps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        best = min(best, a.elapsed_time(b))
    us = best * 1e3 / launches
    return {"us_per_launch": us, "gbs": n / (us * 1e-6) / 1e9, "bytes_per_launch": n,
            "how": "jupiter_read_probe over the same number of bytes, same launch chain"}


def e2e_measure(run, steps, warmup, flush):
    """Same step, but every input of the step is copied from pinned host memory inside the timed
    region and the step's result is read back to the host.  The copies run on two side streams (one per
    direction) and are ordered against the library calls on the current stream by events, call by call, so the
    transfer of the next call's inputs and of the previous call's output overlap the kernels; the current stream
    joins both side streams before the step ends.  Returns (ms_per_step, h2d, d2h)."""
    import torch
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype, device="cpu").pin_memory().copy_(t.cpu())
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    h2d = d2h = 0

    def pipelined(calls):
        """calls: [(pairs of (device tensor, pinned host source), launch function, (pinned host result, device result))]"""
        main = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(main)
        s_in.wait_event(start)   # the previous step's kernels are done with the device buffers
        s_out.wait_event(start)
        for inputs, launch, (h_out, d_out) in calls:
            with torch.cuda.stream(s_in):
                for dst, src in inputs:
                    dst.copy_(src, non_blocking=True)
                ready = torch.cuda.Event()
                ready.record(s_in)
            main.wait_event(ready)
            main.wait_stream(s_out)  # the previous result has left the output buffer before it is rewritten
            launch()
            done = torch.cuda.Event()
            done.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(done)
                h_out.copy_(d_out, non_blocking=True)
        main.wait_stream(s_out)
        main.wait_stream(s_in)

    if isinstance(run, PrefillRun):
        host = [(pin(c["q"]), pin(c["k"]), pin(c["v"]), torch.empty(c["out"].shape, dtype=torch.float32).pin_memory())
                for c in run.chunks]
        for hq, hk, hv, ho in host:
            h2d += hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2
            d2h += ho.numel() * 4
        ctx, w = run.ctx, run.w
        calls = []
        for c, (hq, hk, hv, ho) in zip(run.chunks, host):
            calls.append((((c["q"], hq), (c["k"], hk), (c["v"], hv)),
                          (lambda c=c: ctx.chunk_prefill_append_attn(c["q"], c["k"], c["v"], run.desc, w.q_heads, c["n"],
                                                                     c["pos"], w.scale, c["out"])),
                          (ho, c["out"])))
    else:
        host = {id(s): (pin(s["q"]), pin(s["k"]), pin(s["v"]), pin(s["pos"]), pin(s["lens"])) for s in run.steps_data}
        ho = torch.empty(run.out.shape, dtype=torch.float32).pin_memory()
        ctx, w = run.ctx, run.w
        calls = []
        for c, s in run.calls():
            hq, hk, hv, hp, hl = host[id(s)]
            h2d += hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2 + hp.numel() * 4 + hl.numel() * 4
            d2h += ho.numel() * 4
            _, pdesc, sdesc = run.caches[c]
            calls.append((((s["q"], hq), (s["k"], hk), (s["v"], hv), (s["pos"], hp), (s["lens"], hl)),
                          (lambda s=s, pdesc=pdesc, sdesc=sdesc: ctx.branch_append_attn(
                              s["q"], s["k"], s["v"], pdesc, w.prefix_len, sdesc, s["lens"], s["max_len"], w.n_branches,
                              w.q_heads, w.q_len, w.scale, run.out)),
                          (ho, run.out)))
    ms = timed_steps(lambda: pipelined(calls), steps, warmup, flush, lambda: None)
    return float(np.sum(ms) / steps), int(h2d), int(d2h)


# ----------------------------------------------------------------------------- CPU oracle legs

_SEQ0 = {}


def oracle_prefill_sample(w, kv_heads_used, threads, n_chunks=None):
    """Runs the oracle (append + chunk attention) on sequence 0, the first `kv_heads_used` KV heads with their query
    heads and the first `n_chunks` chunks of the prompt (all by default); returns (seconds, flops done)."""
    import dataclasses
    import oracle
    G = w.q_heads // w.kv_heads
    chunks = w.chunks()[:n_chunks] if n_chunks else w.chunks()
    tokens = chunks[-1][0] + chunks[-1][1]
    # the generator is counter based: sequence 0 of the workload is the one-sequence workload's only sequence
    w1 = dataclasses.replace(w, batch=1, chunk=1, name="")
    if _SEQ0.get("key") != w1:
        _SEQ0.update(key=w1, data=w1.make())  # kept: the same sample is timed several times
    q, k, v = _SEQ0["data"]
    q = np.ascontiguousarray(q[:1, :tokens, :kv_heads_used * G])
    k = np.ascontiguousarray(k[:1, :tokens, :kv_heads_used])
    v = np.ascontiguousarray(v[:1, :tokens, :kv_heads_used])
    kc = np.zeros((1, kv_heads_used, tokens, w.head_dim), np.uint16)
    vc = np.zeros_like(kc)
    t0 = time.perf_counter()
    for pos, n in chunks:
        oracle.kv_append(kc, vc, k[:, pos:pos + n], v[:, pos:pos + n], pos=pos)
        oracle.chunk_prefill(q[:, pos:pos + n], kc, vc, pos, w.scale, n_threads=threads)
    dt = time.perf_counter() - t0
    return dt, 4.0 * w.head_dim * kv_heads_used * G * (tokens * (tokens + 1) // 2)


def oracle_branch_sample(w, n_steps, threads):
    import oracle
    pk, pv, sk, sv = w.make_caches()
    hist = w.history_lengths().astype(np.int32)
    nbytes = 0
    t0 = time.perf_counter()
    for t in range(n_steps):
        q, kn, vn = w.make_step(t)
        pos = hist + t * w.q_len
        lens = pos + w.q_len
        oracle.kv_append(sk, sv, kn, vn, pos_per_seq=pos)
        oracle.branch(q, pk, pv, w.prefix_len, sk, sv, lens, w.scale, n_threads=threads)
        nbytes += w.step_bytes(lens)
    return time.perf_counter() - t0, float(nbytes)


def cpu_leg(w, target_seconds):
    """Times the oracle, as it stands, on a bounded sample of the workload sized for about
    `target_seconds` of wall time.  Returns (units_per_second, description, threads)."""
    import oracle
    threads = oracle.hardware_threads()
    if isinstance(w, synth.PrefillWorkload):
        G = w.q_heads // w.kv_heads
        # cost model: seconds per flop from a one-KV-head probe on a shortened prompt
        probe = synth.PrefillWorkload(w.name, w.seed, 1, G * min(w.kv_heads, max(1, threads // G)),
                                      min(w.kv_heads, max(1, threads // G)), w.head_dim, min(w.seq_len, 512),
                                      min(w.chunk, 512), min(w.seq_len, 512))
        dt, fl = oracle_prefill_sample(probe, probe.kv_heads, threads)
        per_head = (dt / fl) * 4.0 * w.head_dim * G * w.pairs()
        step = max(1, threads // G)  # whole multiples of the thread count keep every thread busy
        heads = int(max(step, min(w.kv_heads, (target_seconds / max(per_head, 1e-9)) // step * step)))
        heads = min(heads, w.kv_heads)
        # a long prompt whose smallest head set is still too much work: only its first chunks (the work grows with the
        # square of the tokens covered)
        n_chunks = len(w.chunks())
        est = per_head * (heads + step - 1) // step if step else per_head
        if est > 1.5 * target_seconds:
            frac = (target_seconds / est) ** 0.5
            n_chunks = int(max(1, min(n_chunks, round(frac * n_chunks))))
        dt, fl = oracle_prefill_sample(w, heads, threads, n_chunks)
        return (fl / dt, f"sequence 0, KV heads 0..{heads - 1} of {w.kv_heads} with their query heads, "
                f"chunks 0..{n_chunks - 1} of {len(w.chunks())}", threads)
    dt1, b1 = oracle_branch_sample(w, 1, threads)
    n = int(max(1, min(w.steps, target_seconds / max(dt1, 1e-9))))
    dt, nb = oracle_branch_sample(w, n, threads)
    return nb / dt, f"decode steps 0..{n - 1} of {w.steps}, all branches and heads", threads


# ----------------------------------------------------------------------------- main

METRIC = "chunk-prefill attn TFLOP/s (% bf16 peak); branch attn GB/s (% HBM peak)"


def make_workload(name):
    return PREFILL[name]() if name in PREFILL else BRANCH[name]()


def unit_of(w):
    return "TFLOP/s" if isinstance(w, synth.PrefillWorkload) else "GB/s"


def scale_of(w):
    return 1e12 if isinstance(w, synth.PrefillWorkload) else 1e9


def config_of(name, w, extra=None):
    if isinstance(w, synth.PrefillWorkload):
        c = {"workload": name, "batch": w.batch, "q_heads": w.q_heads, "kv_heads": w.kv_heads,
             "head_dim": w.head_dim, "prompt_tokens": w.seq_len, "chunk": w.chunk, "cache_capacity": w.capacity,
             "calls_per_step": len(w.chunks())}
    else:
        c = {"workload": name, "branches": w.n_branches, "q_heads": w.q_heads, "kv_heads": w.kv_heads,
             "head_dim": w.head_dim, "prefix_len": w.prefix_len, "suffix_history": [w.suffix_lo, w.suffix_hi],
             "q_len": w.q_len, "decode_steps": w.steps}
    c["l2"] = "flushed between steps (buffer of 2x L2 rewritten)"
    c["launch"] = "one CUDA-graph replay per step"
    if extra:
        c.update(extra)
    return c


def reference_arm(args, rank):
    """The CPU oracle timed on the host cores: each step is a bounded sample of the workload."""
    if rank != 0:
        return
    import oracle
    w = make_workload(args.workload)
    threads = oracle.hardware_threads()
    budget = min(args.cpu_seconds, 150.0 / max(args.steps + args.warmup, 1))
    rate, sample, threads = cpu_leg(w, budget)  # sizes the sample; also serves as first warm-up
    times, units = [], []
    # re-run the same sample K (+W) times
    if isinstance(w, synth.PrefillWorkload):
        heads = int(sample.split("..")[1].split(" ")[0]) + 1
        n_chunks = int(sample.split("..")[2].split(" ")[0]) + 1
        fn = lambda: oracle_prefill_sample(w, heads, threads, n_chunks)
    else:
        n = int(sample.split("..")[1].split(" ")[0]) + 1
        fn = lambda: oracle_branch_sample(w, n, threads)
    for i in range(max(args.warmup - 1, 0) + args.steps):
        dt, u = fn()
        if i >= max(args.warmup - 1, 0):
            times.append(dt)
            units.append(u)
    value = sum(units) / sum(times) / scale_of(w)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": unit_of(w), "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_of(args.workload, w, {"l2": "n/a (CPU)"}),
            "cpu_baseline": {"value": value, "unit": unit_of(w), "cores": threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": unit_of(w), "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's per-step time: every rank runs the same per-GPU workload (weak scaling, units are
    sharded with no data-path collective), so the job takes as long as its slowest rank."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, ms_per_step: float, scale: float) -> float:
    """Aggregate throughput over all ranks: the units every rank processed per step / the slowest time."""
    return world * units_per_rank / (ms_per_step * 1e-3) / scale


# ----------------------------------------------------------------------------- ncu traffic figures

# Which profile summary carries the DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum per launch) of a
# workload's dominant kernel, and which source files that kernel is built from.  A summary is stamped with the
# hash of those sources at the time of its capture; when the kernel has changed since, the figure is void and
# the bench line says null.
CSRC = os.path.join(ROOT, "paper_2504_08242_b200", "csrc")
TC_SOURCES = ["tc_common.cuh", "tc_softmax.cuh", "common.cuh"]
PREFILL_SOURCES = ["prefill_tc.cu", "prefill_tc_frag.cuh"] + TC_SOURCES
TRAFFIC_PROFILES = {
    "cfg2": ("prefill_frag_kernel_cfg2.md", PREFILL_SOURCES),
    "cfg3_c128": ("prefill_frag_kernel_cfg3_c128.md", PREFILL_SOURCES),
    "cfg3_c512": ("prefill_tc_kernel_cfg3_c512.md", PREFILL_SOURCES),
    "cfg3_c1024": ("prefill_tc_kernel_cfg3_c512.md", PREFILL_SOURCES),
    "cfg4": ("branch_stream_kernel_cfg4.md", ["branch_stream.cu", "tc_common.cuh", "common.cuh"]),
    "cfg5": ("branch_tc_kernel_cfg5.md", ["branch_tc.cu"] + TC_SOURCES),
}


def kernel_source_hash(files):
    import hashlib
    h = hashlib.sha1()
    for f in files:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(name, launch_bytes=None):
    """(bytes per launch or None, where it comes from).  The summary holds the lines
    ``kernel_source_sha1: <hash>`` and ``dram_bytes_per_launch[<workload>]: <bytes>``; for the prefill sweeps the
    capture is of one launch of the sweep and the line is ``dram_bytes_per_algorithmic_byte: <ratio>``, scaled
    here by the workload's mean compulsory bytes per launch (traffic grows in proportion to the K/V rows read)."""
    import re
    prof, files = TRAFFIC_PROFILES.get(name, (None, None))
    if prof is None:
        return None, "no capture"
    path = os.path.join(ROOT, "profiles", prof)
    if not os.path.exists(path):
        return None, f"profiles/{prof} missing"
    text = open(path).read()
    m = re.search(r"kernel_source_sha1:\s*([0-9a-f]+)", text)
    if not m or m.group(1) != kernel_source_hash(files):
        return None, f"profiles/{prof}: taken on an older build of the kernel"
    m = re.search(r"dram_bytes_per_launch\[%s\]:\s*([0-9.eE+]+)" % re.escape(name), text)
    if m:
        return float(m.group(1)), f"profiles/{prof}"
    m = re.search(r"dram_bytes_per_algorithmic_byte:\s*([0-9.eE+]+)", text)
    if m and launch_bytes:
        return float(m.group(1)) * launch_bytes, f"profiles/{prof} (ratio measured on one launch x this workload's mean compulsory bytes per launch)"
    return None, f"profiles/{prof}: no figure for {name}"


def prefill_launch_bytes(w):
    """Compulsory DRAM bytes of an average chunk launch: Q read, the chunk's K/V read and written to the cache,
    the cached rows [0, pos) read, fp32 output written."""
    tot = 0
    for pos, n in w.chunks():
        kv_row = w.kv_heads * w.head_dim * 2
        tot += w.batch * (n * w.q_heads * w.head_dim * (2 + 4) + 2 * kv_row * (2 * n + pos))
    return tot / len(w.chunks())


# ----------------------------------------------------------------------------- one workload on the GPU

def run_workload(ctx, device, name, w, steps, warmup, flush, barrier, world, peaks, peak_kind, use_graph=True,
                 prefill_data=None, with_e2e=True, rank=0):
    """Times one workload and returns the fields of its bench entry: value, ms_per_step, clocks (sampled during its
    own timed region), gpu_launches, roofline, e2e."""
    import torch
    is_prefill = isinstance(w, synth.PrefillWorkload)
    run = PrefillRun(ctx, w, device, data=prefill_data) if is_prefill else branch_run(ctx, w, device)
    sampler = ClockSampler(device.index or 0)
    sampler.start()
    m = measure(run, steps, warmup, flush, barrier, use_graph=use_graph, sampler=sampler)
    clocks = sampler.stop(*m["sample_range"])
    assert ctx.poll_device_status() == 0
    ms_per_step = max_over_ranks(m["ms_per_step"], world, device)
    value = whole_job_value(run.units(), world, ms_per_step, scale_of(w))
    if is_prefill:
        achieved = run.units() / (m["attn_ms_per_step"] * 1e-3) / 1e12
        peak = peaks["bf16_tflops"]
        traffic, traffic_from = ncu_traffic(name, prefill_launch_bytes(w))
        roofline = {"bound": "tensor", "kernel": "chunk_prefill_attn", "achieved": achieved, "peak": peak,
                    "unit": "TFLOP/s", "frac": achieved / peak, "peak_kind": f"{peak_kind} burst bf16",
                    "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                    "avg_launch_ms": m["attn_ms_per_launch"], "avg_launch_from": m["attn_time_source"],
                    "traffic": traffic, "traffic_from": traffic_from,
                    "traffic_unit": "bytes per launch (ncu dram read+write)"}
    else:
        achieved = run.units() / (m["attn_ms_per_step"] * 1e-3) / 1e9
        peak = peaks["hbm_gbs"]
        traffic, traffic_from = ncu_traffic(name)
        roofline = {"bound": "hbm", "kernel": "branch_attn", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"{peak_kind} copy", "avg_launch_ms": m["attn_ms_per_launch"],
                    "avg_launch_from": m["attn_time_source"], "traffic": traffic, "traffic_from": traffic_from,
                    "traffic_unit": "bytes per launch (ncu dram read+write)"}
        if rank == 0:
            n_launch = run.attn_launches_per_step()
            roofline["plain_read"] = plain_read_floor(ctx, device, run.units() / n_launch, max(n_launch, 16), flush)
    extra = {} if is_prefill else {"cache_copies_rotated": run.copies, "passes_per_step": run.passes,
                                   "calls_per_step": run.attn_launches_per_step()}
    if not use_graph:
        extra["launch"] = "eager"
    entry = {"value": value, "unit": unit_of(w), "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step,
             "config": config_of(name, w, extra), "clocks": clocks, "gpu_launches": m["launches_per_step"] * steps,
             "roofline": roofline}
    if with_e2e:
        e2e_ms, h2d, d2h = e2e_measure(run, max(3, steps // 4), 2, flush)
        entry["e2e"] = {"value": whole_job_value(run.units(), world, max_over_ranks(e2e_ms, world, device), scale_of(w)),
                        "unit": unit_of(w), "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    del run
    torch.cuda.empty_cache()
    return entry


def relaunch_under_torchrun(args):
    """`--gpus N` without a launcher: start one rank per GPU under torchrun (standalone, local rendezvous) and pass
    its output and exit status through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return relaunch_under_torchrun(args)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        reference_arm(args, rank)
        return 0

    import torch
    import torch.distributed as dist
    import paper_2504_08242_b200 as J

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)
        barrier = lambda: dist.barrier()
    else:
        barrier = lambda: None

    peaks, peak_kind = load_peaks()
    ctx = J.Context(local_rank)
    flush = Flusher(device)
    name = args.workload
    w = make_workload(name)
    # the three chunk sizes of the long-prompt workload share one prompt: generate it once
    shared = {}

    def data_for(n, wl):
        if not isinstance(wl, synth.PrefillWorkload):
            return None
        key = (wl.seed, wl.batch, wl.q_heads, wl.kv_heads, wl.head_dim, wl.seq_len)
        if key not in shared:
            shared.clear()  # one prompt resident at a time
            shared[key] = wl.make()
        return shared[key]

    head = run_workload(ctx, device, name, w, args.steps, args.warmup, flush, barrier, world, peaks, peak_kind,
                        use_graph=not args.no_graph, prefill_data=data_for(name, w), rank=rank)
    line = {"metric": METRIC, "value": head["value"], "unit": head["unit"], "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": head["config"], "clocks": head["clocks"],
            "gpu_launches": head["gpu_launches"], "e2e": head["e2e"], "roofline": head["roofline"]}

    if rank == 0 and world == 1 and not args.no_extra:
        # the other workloads, each a full entry of its own (same steps and warm-up, its own clock record)
        others = {}
        for other in ("cfg3_c1024", "cfg3_c128", "cfg3_c512", "cfg2", "cfg4", "cfg5"):
            if other == name:
                continue
            ow = make_workload(other)
            others[other] = run_workload(ctx, device, other, ow, max(args.steps, 20), max(args.warmup, 3), flush,
                                         lambda: None, 1, peaks, peak_kind, prefill_data=data_for(other, ow),
                                         with_e2e=False)
        line["other_workloads"] = others
    shared.clear()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rate, sample, threads = cpu_leg(w, args.cpu_seconds)
        line["cpu_baseline"] = {"value": rate / scale_of(w), "unit": unit_of(w), "cores": threads, "kind": "oracle",
                                "sample": sample}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
