#!/usr/bin/env python
"""Benchmark of the per-chunk KV-cache step (append -> evict -> chunk-prefill -> decode steps).

A "step" is one pass of the whole hot path over one one-second chunk of a synthetic stream in
steady state: the chunk's tokens are appended, the cache is evicted/re-indexed, every layer attends
with the chunk's queries, and `decode_steps` single-token decode steps follow (each appends one text
token and attends in every layer).  Layers are called one after another, as a decoder would.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 3] [--impl ours|reference]

Prints one JSON line (rank 0).  `--impl reference` times the CPU checker in oracle/ instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_09608_b200 import streamgen as sg  # noqa: E402


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16_burst=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, torch_device_index: int, period=0.05):
        super().__init__(daemon=True)
        self.period = period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._halt = threading.Event()
        self.h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            for i in range(pynvml.nvmlDeviceGetCount()):
                h = pynvml.nvmlDeviceGetHandleByIndex(i)
                u = pynvml.nvmlDeviceGetUUID(h)
                u = u.decode() if isinstance(u, bytes) else u
                if uuid in u:
                    self.h = h
            if self.h is None:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report that instead of a clock record
            self.err = repr(e)

    NAMES = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
             0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
             0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def run(self):
        if self.h is None:
            return
        while not self._halt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                r = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.NAMES.items():
                    if r & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self._halt.set()
        self.join(timeout=2)
        if self.h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
class StepInputs:
    """Device (and optionally pinned host) inputs of one step, generated from the stream's seed."""

    def __init__(self, wl, stream, chunk, decode, host=False):
        import torch
        L = wl.layers
        gids, types, pos = chunk
        gen = lambda tensor, g, heads: torch.stack(  # noqa: E731
            [sg.rows_bf16_torch(wl.seed, tensor, stream.stream, l, g, heads, wl.head_dim) for l in range(L)])
        self.n = len(gids)
        self.K, self.V, self.Q = gen(sg.TENSOR_K, gids, wl.kv_heads), gen(sg.TENSOR_V, gids, wl.kv_heads), \
            gen(sg.TENSOR_Q, gids, wl.q_heads)
        self.types = torch.from_numpy(types).cuda()
        self.pos = torch.from_numpy(np.ascontiguousarray(pos)).cuda()
        self.out = torch.empty_like(self.Q)
        self.dec = []
        for g1, t1, p1 in decode:
            self.dec.append(dict(K=gen(sg.TENSOR_K, g1, wl.kv_heads), V=gen(sg.TENSOR_V, g1, wl.kv_heads),
                                 Q=gen(sg.TENSOR_Q, g1, wl.q_heads), types=torch.from_numpy(t1).cuda(),
                                 pos=torch.from_numpy(np.ascontiguousarray(p1)).cuda()))
            self.dec[-1]["out"] = torch.empty_like(self.dec[-1]["Q"])
        if host:
            pin = lambda t: t.cpu().pin_memory()  # noqa: E731
            self.h = dict(K=pin(self.K), V=pin(self.V), Q=pin(self.Q), types=pin(self.types), pos=pin(self.pos),
                          out=torch.empty_like(self.Q, device="cpu").pin_memory())
            self.hdec = [dict(K=pin(d["K"]), V=pin(d["V"]), Q=pin(d["Q"]), types=pin(d["types"]), pos=pin(d["pos"]),
                              out=torch.empty_like(d["Q"], device="cpu").pin_memory()) for d in self.dec]

    def h2d_bytes(self):
        tot = 0
        for d in [self.h] + self.hdec:
            tot += sum(d[k].numel() * d[k].element_size() for k in ("K", "V", "Q", "types", "pos"))
        return tot

    def d2h_bytes(self):
        return sum(d["out"].numel() * d["out"].element_size() for d in [self.h] + self.hdec)


def next_step_schedule(stream, wl):
    chunk = stream.next_chunk()
    decode = [stream.next_decode_token() for _ in range(wl.decode_steps)]
    return chunk, decode


def run_step(cache, wl, inp, timers=None):
    """One step through the C ABI, layers in sequence.  timers: dict name -> list of (start,end) events."""
    import torch
    L = wl.layers

    def timed(name, fn):
        if timers is None:
            return fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        timers.setdefault(name, []).append((a, b))

    timed("append", lambda: cache.append(0, inp.K[0], inp.V[0], inp.types, inp.pos))
    timed("evict", lambda: cache.evict())
    timed("prefill", lambda: cache.attend(0, inp.Q[0], inp.pos, inp.out[0]))
    for l in range(1, L):
        timed("append", lambda: cache.append(l, inp.K[l], inp.V[l]))
        timed("prefill", lambda: cache.attend(l, inp.Q[l], inp.pos, inp.out[l]))
    def decode_token(d):   # one generated token: every layer appends its K/V and attends, one launch per layer
        for l in range(L):
            cache.decode_step(l, d["K"][l], d["V"][l], d["types"] if l == 0 else None, d["pos"], d["Q"][l], d["out"][l])

    for d in inp.dec:
        timed("decode_token", lambda: decode_token(d))


def stack_decode_inputs(inps):
    """Per generated token, the streams' one-token inputs side by side: K, V, Q as [layers][streams][heads][d],
    types [streams], pos [streams](x3), the layout of svlm_decode_step_batched."""
    import torch
    toks = []
    for t in range(len(inps[0].dec)):
        d = {k: torch.stack([inp.dec[t][k][:, 0] for inp in inps], dim=1).contiguous() for k in ("K", "V", "Q")}
        d["types"] = torch.cat([inp.dec[t]["types"] for inp in inps]).contiguous()
        d["pos"] = torch.stack([inp.dec[t]["pos"][0] for inp in inps]).contiguous()
        d["out"] = torch.empty_like(d["Q"])
        toks.append(d)
    return toks


def stack_prefill_inputs(inps):
    """The streams' chunk queries one after another, per layer: Q [layers][sum n][q_heads][d], pos [sum n](x3), the
    row counts, and an output buffer of Q's shape (the layout of svlm_attend_batched_varlen)."""
    import torch
    Q = torch.cat([inp.Q for inp in inps], dim=1).contiguous()
    return dict(Q=Q, pos=torch.cat([inp.pos for inp in inps]).contiguous(), n_q=[inp.n for inp in inps], out=torch.empty_like(Q))


def run_step_multi(caches, wl, inps, dec, timers=None, pre=None):
    """One step of several streams that advance in lock step: every stream appends its chunk, ONE batched
    eviction, per layer the streams' K/V appends and ONE chunk-prefill launch for all of them (the chunks differ in
    length), then the generated tokens with one batched decode launch per layer for all streams.
    inps: one StepInputs per stream; dec: stack_decode_inputs; pre: stack_prefill_inputs (outputs land in pre["out"])."""
    import torch
    from paper_2510_09608_b200 import binding
    L = wl.layers

    def timed(name, fn):
        if timers is None:
            return fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        timers.setdefault(name, []).append((a, b))

    for c, inp in zip(caches, inps):
        timed("append", lambda: c.append(0, inp.K[0], inp.V[0], inp.types, inp.pos))
    timed("evict", lambda: binding.evict_batched(caches))
    if pre is None:
        pre = stack_prefill_inputs(inps)
    for l in range(L):
        if l:
            for c, inp in zip(caches, inps):
                timed("append", lambda: c.append(l, inp.K[l], inp.V[l]))
        timed("prefill", lambda: binding.attend_batched_varlen(caches, l, pre["Q"][l], pre["pos"], pre["n_q"], pre["out"][l]))

    def decode_token(d):
        for l in range(L):
            binding.decode_step_batched(caches, l, d["K"][l], d["V"][l], d["types"] if l == 0 else None, d["pos"],
                                        d["Q"][l], d["out"][l])

    for d in dec:
        timed("decode_token", lambda: decode_token(d))


def run_step_host_layered(cache, wl, inp):
    """The step of run_step through the host-buffer entry points, layer by layer as a decoder calls them: every
    call copies its own inputs up from pinned host memory, and the attention calls bring their output down before
    they return."""
    h = inp.h
    cache.append_host(0, h["K"][0], h["V"][0], h["types"], h["pos"])
    cache.evict()
    cache.attend_host(0, h["Q"][0], h["pos"], h["out"][0])
    for l in range(1, wl.layers):
        cache.append_host(l, h["K"][l], h["V"][l], None, None)
        cache.attend_host(l, h["Q"][l], h["pos"], h["out"][l])
    for d in inp.hdec:
        for l in range(wl.layers):
            cache.decode_step_host(l, d["K"][l], d["V"][l], d["types"] if l == 0 else None, d["pos"], d["Q"][l], d["out"][l])


def time_decode_tokens(cache, wl, inp, replays=3):
    """Milliseconds per generated token for the decode part of a step as the step benchmark runs it (one fused
    svlm_decode_step launch per layer, replayed from a CUDA graph): the token launches of `inp` are captured once and
    replayed; an eviction between replays keeps the cache at its steady-state size.  Median of the replays after the
    first (which carries the graph's upload)."""
    import torch

    def tokens():
        for d in inp.dec:
            for l in range(wl.layers):
                cache.decode_step(l, d["K"][l], d["V"][l], d["types"] if l == 0 else None, d["pos"], d["Q"][l], d["out"][l])

    g = torch.cuda.CUDAGraph()
    cur = torch.cuda.current_stream()
    with torch.cuda.graph(g):
        cache.set_stream(torch.cuda.current_stream())
        tokens()
    cache.set_stream(cur)
    ts = []
    for _ in range(replays + 1):
        cache.evict()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) / max(len(inp.dec), 1))
    return statistics.median(ts[1:])


def run_step_host(cache, wl, inp):
    """The same step through the host-buffer entry points (all layers per call): copies included."""
    cache.append_host(-1, inp.h["K"], inp.h["V"], inp.h["types"], inp.h["pos"])
    cache.evict()
    cache.attend_host(-1, inp.h["Q"], inp.h["pos"], inp.h["out"])
    for d in inp.hdec:      # one generated token: all layers' append and attention fused, one call
        cache.decode_step_host(-1, d["K"], d["V"], d["types"], d["pos"], d["Q"], d["out"])


def fill_to_steady_state(cache, wl, stream):
    """Untimed set-up: stream chunks through append+evict (no attention) until the windows are full."""
    import torch
    L = wl.layers
    gen = lambda tensor, g: torch.stack(  # noqa: E731
        [sg.rows_bf16_torch(wl.seed, tensor, stream.stream, l, g, wl.kv_heads, wl.head_dim) for l in range(L)])
    n_text = 0
    chunks = 0
    while n_text < wl.n_sink + wl.text_window + 64 or chunks * wl.vision_per_chunk < wl.vision_window + 1:
        gids, types, pos = stream.next_chunk()
        extra = [stream.next_decode_token() for _ in range(wl.decode_steps)]
        cache.append(-1, gen(sg.TENSOR_K, gids), gen(sg.TENSOR_V, gids), torch.from_numpy(types).cuda(),
                     torch.from_numpy(np.ascontiguousarray(pos)).cuda())
        cache.evict()
        if extra:
            g = np.concatenate([e[0] for e in extra])
            t = np.concatenate([e[1] for e in extra])
            p = np.concatenate([e[2] for e in extra])
            cache.append(-1, gen(sg.TENSOR_K, g), gen(sg.TENSOR_V, g), torch.from_numpy(t).cuda(),
                         torch.from_numpy(np.ascontiguousarray(p)).cuda())
        n_text += int((types == sg.TEXT).sum()) + len(extra)
        chunks += 1
    return chunks


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the attention and eviction kernels come from
# the ncu captures summarised under profiles/: profiles/ncu_dram_traffic.txt lists, per kernel, the bytes per launch on
# the config-3 shape, the source files the kernel is built from and their SHA-256 at the time of the capture.  A kernel
# whose source has changed since reports no traffic (null) until its counters are taken again.
def ncu_dram_traffic():
    import hashlib
    out = {}
    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")
    if not os.path.exists(path):
        return out
    for line in open(path):
        f = line.split()
        if len(f) < 4 or line.startswith("#"):
            continue
        name, nbytes, src, digest = f[0], float(f[1]), f[2], f[3]
        try:      # src: the kernel's files joined by '+', hashed one after another
            now = hashlib.sha256(b"".join(open(os.path.join(ROOT, x), "rb").read() for x in src.split("+"))).hexdigest()
        except OSError:
            now = None
        out[name] = nbytes if now == digest else None
    return out


def max_over_ranks(value: float, world: int, device="cuda") -> float:
    """The slowest rank's figure (replicas run independent streams; the job is as slow as its slowest rank)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, units_per_step: float, ms_per_step: float) -> float:
    """Units per second over all ranks: every rank processes `units_per_step` per step (weak scaling)."""
    return world * units_per_step / (ms_per_step * 1e-3)


def prefill_flops(wl, n_q, lk):
    pairs = n_q * (lk - n_q) + n_q * (n_q + 1) // 2
    return 4 * wl.q_heads * wl.head_dim * pairs


# ------------------------------------------------------------------------------------------------
def oracle_sample(wl, rows=1 << 20, decode=1 << 20, layers=2):
    """Times the CPU checker, as it stands, on a bounded sample of one steady-state step: `layers` layers,
    `rows` query rows of the chunk prefill and `decode` decode steps; the rest is scaled linearly."""
    import oracle
    stream = sg.Stream(wl, 0)
    layers = min(layers, wl.layers)
    ref = oracle.Oracle(layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window,
                        rope_mode=wl.rope_mode, rope_base=wl.rope_base, sections=wl.sections)
    n_text, chunks = 0, 0
    while n_text < wl.n_sink + wl.text_window + 64 or chunks * wl.vision_per_chunk < wl.vision_window + 1:
        gids, types, pos = stream.next_chunk()
        ref.append(None, None, types, pos)
        ref.evict()
        for _ in range(wl.decode_steps):
            g1, t1, p1 = stream.next_decode_token()
            ref.append(None, None, t1, p1)
        n_text += int((types == sg.TEXT).sum()) + wl.decode_steps
        chunks += 1
    gids, types, pos = stream.next_chunk()
    ref.append(None, None, types, pos)
    kept = ref.query()["gids"]
    for l in range(layers):
        ref.set_kv(l, kept, stream.k(l, kept), stream.v(l, kept))
    rows, decode = min(rows, len(gids)), min(decode, wl.decode_steps)
    sel = np.linspace(0, len(gids) - 1, rows).astype(np.int64)
    t0 = time.perf_counter()
    ref.evict()
    t_evict = time.perf_counter() - t0
    t_rows = 0.0
    for l in range(layers):
        Q = stream.q(l, gids)
        t0 = time.perf_counter()
        ref.attend(l, Q, pos, sel)
        t_rows += time.perf_counter() - t0
    t_rows /= layers
    t_dec = 0.0
    for _ in range(decode):
        g1, t1, p1 = stream.next_decode_token()
        ref.append(np.stack([stream.k(l, g1) for l in range(layers)]), np.stack([stream.v(l, g1) for l in range(layers)]), t1, p1)
        for l in range(layers):
            q1 = stream.q(l, g1)
            t0 = time.perf_counter()
            ref.attend(l, q1, p1)
            t_dec += time.perf_counter() - t0
    t_dec /= max(decode * layers, 1)
    # one step = evict (metadata, shared by the layers) + layers x (prefill of all rows + decode steps)
    est = t_evict + wl.layers * (t_rows * len(gids) / rows + wl.decode_steps * t_dec)
    return dict(step_seconds=est, measured_seconds=t_evict + (t_rows + t_dec * decode) * layers, cores=oracle.threads(),
                sample=f"{layers} of {wl.layers} layers, {rows} of {len(gids)} prefill rows, {decode} of {wl.decode_steps} "
                       f"decode steps of one steady-state chunk; scaled linearly to the full step")


def bench_batched_decode(args, wl, base, peaks, rank, world, local):
    """Workload 4: `wl.streams` independent streams at the full retained size; a step is one batched q=1 decode step
    (every stream appends its token and attends: one metadata launch and one attention launch serve all streams); the
    caches are evicted every 16 steps, again with one metadata and one re-rotation launch for all of them.
    Whole cycles of 16 steps + evictions are replayed from a CUDA graph; value = decode tokens/s over all streams."""
    import torch
    from paper_2510_09608_b200 import binding
    cycle = 16
    streams = [sg.Stream(wl, rank * wl.streams + i) for i in range(wl.streams)]
    caches = []
    for st in streams:
        c = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
        c.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
        fill_to_steady_state(c, dataclasses_replace(wl, decode_steps=cycle), st)
        c.evict()
        caches.append(c)

    def make_cycle():
        steps = []
        for _ in range(cycle):
            toks = [st.next_decode_token() for st in streams]
            gen = lambda tensor, heads: torch.stack([sg.rows_bf16_torch(wl.seed, tensor, st.stream, 0, t[0], heads, wl.head_dim)  # noqa: E731
                                                     for st, t in zip(streams, toks)])
            steps.append(dict(K=gen(sg.TENSOR_K, wl.kv_heads), V=gen(sg.TENSOR_V, wl.kv_heads), Q=gen(sg.TENSOR_Q, wl.q_heads),
                              types=torch.zeros(len(streams), dtype=torch.uint8, device="cuda"),
                              pos=torch.from_numpy(np.ascontiguousarray(np.stack([t[2][0] for t in toks]))).cuda()))
            steps[-1]["out"] = torch.empty_like(steps[-1]["Q"])
        return steps

    def run_cycle(steps, timers=None):
        for d in steps:
            if timers is not None:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
            binding.decode_step_batched(caches, 0, d["K"], d["V"], d["types"], d["pos"], d["Q"], d["out"])
            if timers is not None:
                b.record()
                timers.append((a, b))
        binding.evict_batched(caches)

    n_cycles = max(1, (args.warmup + args.steps + cycle - 1) // cycle) + 1
    cycles = [make_cycle() for _ in range(n_cycles)]
    run_cycle(cycles[0])                      # plain once: one-time kernel attributes outside any capture
    torch.cuda.synchronize()
    graphs = []
    cur = torch.cuda.current_stream()
    for cy in cycles[1:]:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for c in caches:
                c.set_stream(torch.cuda.current_stream())
            run_cycle(cy)
        graphs.append(g)
    for c in caches:
        c.set_stream(cur)
    graphs[0].replay()                        # warm-up cycle (>= 3 steps)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    before = binding.launch_count()
    ev0.record()
    for g in graphs[1:] or graphs:
        g.replay()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.finish()
    timed_cycles = len(graphs[1:] or graphs)
    ms_per_step = max_over_ranks(ev0.elapsed_time(ev1), world) / (timed_cycles * cycle)
    launches = (cycle * 2 + 2) * timed_cycles
    timers = []
    run_cycle(make_cycle(), timers)
    torch.cuda.synchronize()
    att_ms = statistics.median(a.elapsed_time(b) for a, b in timers)
    for c in caches:
        assert c.status() == binding.OK
    kv_bytes = wl.retained * 2 * wl.kv_heads * wl.head_dim * 2 * len(caches)
    roof = dict(bound="hbm", kernel="decode step (batched: metadata launch + attention launch)", achieved=kv_bytes / (att_ms * 1e-3) / 1e9, peak=peaks["hbm"], unit="GB/s",
                traffic=None, algorithmic=kv_bytes, avg_ms=att_ms, peak_source=peaks["source"] + " (copy)")
    roof["frac"] = roof["achieved"] / roof["peak"]
    if rank == 0:
        print(json.dumps(dict(base, metric="decode tokens/s, batched q=1 steps with interleaved eviction", unit="tok/s",
                              value=whole_job_value(world, len(caches), ms_per_step), ms_per_step=ms_per_step,
                              config=dict(workload=f"config 4 ({wl.name}): {len(caches)} streams x {wl.layers} layer, {wl.q_heads}/"
                                                   f"{wl.kv_heads} heads, d={wl.head_dim}, retained {wl.retained} tokens per stream, "
                                                   f"evict every {cycle} steps", l2="302 MB of K/V per step, above L2; no flush",
                                          replicas="independent streams per GPU, no collective"),
                              roofline=roof, cpu_baseline=None, e2e=None, gpu_launches=int(launches), clocks=clocks,
                              steps=timed_cycles * cycle)))


def bench_multi_stream(args, wl, base, config, peaks, rank, world, local):
    """Workload 5: `wl.streams` streams of a full attention stack in lock step; a step is one chunk of every stream
    (append, batched eviction, batched chunk prefill, batched decode).  Steps are replayed from CUDA graphs;
    value = frames/s over all streams."""
    import torch
    from paper_2510_09608_b200 import binding
    S = wl.streams
    streams = [sg.Stream(wl, rank * S + i) for i in range(S)]
    caches = []
    fill_chunks = 0
    for st in streams:
        c = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
        c.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
        fill_chunks = fill_to_steady_state(c, wl, st)
        c.evict()
        assert c.status() == binding.OK
        caches.append(c)

    def make_step():
        inps = [StepInputs(wl, st, *next_step_schedule(st, wl)) for st in streams]
        pre = stack_prefill_inputs(inps)
        for inp in inps:          # the per-stream copies of Q and the output are not needed any more
            inp.Q = inp.out = None
        return inps, stack_decode_inputs(inps), pre

    total = args.warmup + args.steps
    steps = [make_step() for _ in range(total)]
    prime = make_step()
    # one plain step on scratch caches: one-time function attributes are set outside any capture
    scratch = []
    for _ in range(S):
        c = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
        c.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
        scratch.append(c)
    run_step_multi(scratch, wl, steps[0][0], steps[0][1], None, steps[0][2])
    torch.cuda.synchronize()
    for c in scratch:
        c.close()

    graphs, launches = [], []
    cur = torch.cuda.current_stream()
    for inps, dec, pre in steps:
        g = torch.cuda.CUDAGraph()
        before = binding.launch_count()
        with torch.cuda.graph(g):
            for c in caches:
                c.set_stream(torch.cuda.current_stream())
            run_step_multi(caches, wl, inps, dec, None, pre)
        launches.append(binding.launch_count() - before)
        graphs.append(g)
    for c in caches:
        c.set_stream(cur)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        graphs[i].replay()
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record()
    for i in range(args.steps):
        graphs[args.warmup + i].replay()
        ev[i + 1].record()
    barrier()
    clocks = sampler.finish()
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    ms_per_step = max_over_ranks(ev[0].elapsed_time(ev[-1]), world) / args.steps
    for c in caches:
        assert c.status() == binding.OK

    # per-kernel durations: one plain pass with events around every call
    timers = {}
    run_step_multi(caches, wl, prime[0], prime[1], timers, prime[2])
    torch.cuda.synchronize()
    kern = {k: [a.elapsed_time(b) for a, b in v] for k, v in timers.items()}
    avg = {k: statistics.mean(v) for k, v in kern.items()}
    tot = {k: sum(v) for k, v in kern.items()}
    n_q = statistics.mean(inp.n for inp in prime[0])
    lk = wl.retained
    flops = sum(prefill_flops(wl, inp.n, lk) for inp in prime[0])          # one prefill launch: all streams, one layer
    kv_bytes_layer = lk * 2 * wl.kv_heads * wl.head_dim * 2 * S          # one batched decode launch: all streams, one layer
    evict_bytes = 2 * (wl.retained - wl.n_sink) * wl.kv_heads * wl.head_dim * 2 * wl.layers * S
    kernels = {
        "prefill": dict(bound="tensor", avg_ms=avg["prefill"], per_step_ms=tot["prefill"],
                        achieved=flops / (avg["prefill"] * 1e-3) / 1e12, unit="TFLOP/s", peak=peaks["bf16_burst"]),
        "decode": dict(bound="hbm", avg_ms=avg["decode_token"] / wl.layers, per_step_ms=tot["decode_token"],
                       achieved=kv_bytes_layer * wl.layers / (avg["decode_token"] * 1e-3) / 1e9, unit="GB/s",
                       peak=peaks["hbm"], note="avg_ms = time of one token step of all streams over all layers / layers"),
        "evict": dict(bound="hbm", avg_ms=avg["evict"], per_step_ms=tot["evict"],
                      achieved=evict_bytes / (avg["evict"] * 1e-3) / 1e9, unit="GB/s", peak=peaks["hbm"]),
        "append": dict(avg_ms=avg["append"], per_step_ms=tot["append"]),
    }
    for k in ("prefill", "decode", "evict"):
        kernels[k]["frac"] = kernels[k]["achieved"] / kernels[k]["peak"]
        # the same rate against the data-sheet figure (dense bf16 2250 TFLOP/s, HBM3e 8000 GB/s), for context
        kernels[k]["frac_of_nominal"] = kernels[k]["achieved"] / (2250.0 if kernels[k]["bound"] == "tensor" else 8000.0)
    dominant = max(("prefill", "decode", "evict"), key=lambda k: kernels[k]["per_step_ms"])
    kd = kernels[dominant]
    roofline = dict(bound="tensor" if dominant == "prefill" else "hbm", kernel=dominant, achieved=kd["achieved"],
                    peak=kd["peak"], unit=kd["unit"], frac=kd["frac"], frac_of_nominal=kd["frac_of_nominal"], traffic=None,
                    algorithmic=(flops if dominant == "prefill" else kv_bytes_layer if dominant == "decode" else evict_bytes),
                    peak_source=peaks["source"] + (" (burst bf16)" if dominant == "prefill" else " (copy)"))
    if rank == 0:
        config = dict(config, replicas="independent streams, no collective",
                      streams=f"{S} streams per GPU in lock step: batched eviction, chunk prefill and decode (one launch per layer for all streams)")
        print(json.dumps(dict(base, value=whole_job_value(world, wl.frames * S, ms_per_step), ms_per_step=ms_per_step,
                              config=config, roofline=roofline, cpu_baseline=None, e2e=None,
                              gpu_launches=int(sum(launches[args.warmup:])), clocks=clocks, kernels=kernels,
                              decode_tok_s=wl.decode_steps * S / (tot["decode_token"] * 1e-3),
                              step_ms=dict(min=min(step_ms), median=statistics.median(step_ms), max=max(step_ms)),
                              state=dict(fill_chunks=fill_chunks, cuda_graph=True))))


def overlap_window(wl, stream_id=0):
    """The tokens a sliding window WITH overlap holds in one second of the stream: what the policy retains once
    the second's chunk has been appended (the chunk included), in stream order.  Returns (gids, types, pos[n,3] or [n]) with positions counted from 0."""
    from paper_2510_09608_b200 import binding
    one = dataclasses_replace(wl, layers=1)
    stream = sg.Stream(one, stream_id)
    cache = binding.Cache(1, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    fill_to_steady_state(cache, one, stream)
    import torch
    gids, types, pos = stream.next_chunk()
    z = torch.zeros(1, len(gids), wl.kv_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda")
    cache.append(-1, z, z, torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda())
    cache.evict()
    q = cache.query()
    cache.close()
    p = q["pos"] if wl.rope_mode else q["pos"][:, 0]
    return q["gids"], q["types"], np.ascontiguousarray(p - p.min()).astype(np.int32)


def bench_overlap(args, wl, base, peaks, rank, world, local):
    """The comparison shape of the paper's efficiency argument (Figure 1(c), Section 3.3): a sliding window WITH
    overlap recomputes the whole window every second instead of reusing the retained KV.  A step drops the cache
    and, layer by layer, appends and chunk-prefills all R window tokens (Lq = Lk) through the same kernels."""
    import torch
    from paper_2510_09608_b200 import binding
    gids, types, pos = overlap_window(wl, rank)
    n = len(gids)
    span = int(pos.max()) + 1
    L = wl.layers
    cap = (n + 127) // 128 * 128
    cache = binding.Cache(L, wl.kv_heads, wl.head_dim, 0, 0, 0, cap)     # nothing is kept from one second to the next
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    gen = lambda tensor, heads: torch.stack(  # noqa: E731
        [sg.rows_bf16_torch(wl.seed, tensor, rank, l, gids, heads, wl.head_dim) for l in range(L)])
    K, V, Q = gen(sg.TENSOR_K, wl.kv_heads), gen(sg.TENSOR_V, wl.kv_heads), gen(sg.TENSOR_Q, wl.q_heads)
    out = torch.empty_like(Q)
    ty = torch.from_numpy(types).cuda()
    total = args.warmup + args.steps + 1
    # the window of second t sits at native positions t*span ..: the stream goes on, the contents are re-drawn
    poss = [torch.from_numpy(np.ascontiguousarray(pos + t * span)).cuda() for t in range(total)]

    def step(t, timers=None):
        def timed(name, fn):
            if timers is None:
                return fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            timers.setdefault(name, []).append((a, b))
        timed("evict", cache.evict)
        for l in range(L):
            timed("append", lambda: cache.append(l, K[l], V[l], ty if l == 0 else None, poss[t] if l == 0 else None))
            timed("prefill", lambda: cache.attend(l, Q[l], poss[t], out[l]))

    step(0)
    torch.cuda.synchronize()
    assert cache.status() == binding.OK
    graphs = []
    cur = torch.cuda.current_stream()
    launches = 0
    for t in range(1, total - 1):
        g = torch.cuda.CUDAGraph()
        before = binding.launch_count()
        with torch.cuda.graph(g):
            cache.set_stream(torch.cuda.current_stream())
            step(t)
        launches = binding.launch_count() - before
        graphs.append(g)
    cache.set_stream(cur)
    for i in range(args.warmup - 1):
        graphs[i].replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for g in graphs[args.warmup - 1:]:
        g.replay()
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.finish()
    ms_per_step = max_over_ranks(ev0.elapsed_time(ev1), world) / args.steps
    timers = {}
    step(total - 1, timers)
    torch.cuda.synchronize()
    assert cache.status() == binding.OK
    avg = {k: statistics.mean(a.elapsed_time(b) for a, b in v) for k, v in timers.items()}
    flops = 4.0 * wl.q_heads * wl.head_dim * (n * (n + 1) / 2)
    roof = dict(bound="tensor", kernel="prefill", achieved=flops / (avg["prefill"] * 1e-3) / 1e12, peak=peaks["bf16_burst"],
                unit="TFLOP/s", traffic=None, algorithmic=flops, avg_ms=avg["prefill"], peak_source=peaks["source"] + " (burst bf16)")
    roof["frac"] = roof["achieved"] / roof["peak"]
    if rank == 0:
        print(json.dumps(dict(base, value=whole_job_value(world, wl.frames, ms_per_step), ms_per_step=ms_per_step,
                              config=dict(workload=f"sliding window with overlap on the config {args.config} shape: all {n} window tokens "
                                                   f"(the retained set, newest chunk included) appended and prefilled again every second, "
                                                   f"{L} layers, causal, Lq = Lk = {n}",
                                          l2="Q and out of a layer (139 MB each) exceed L2; no flush", replicas="independent streams, no collective"),
                              roofline=roof, cpu_baseline=None, e2e=None, gpu_launches=int(launches * args.steps), clocks=clocks,
                              kernels={k: dict(avg_ms=v) for k, v in avg.items()})))


def bench_sweep(args, wl, base, peaks, rank, world, local):
    """Latency over the sink / text-window / vision-window values of the paper's ablations (Section 4.4: sink and
    text window 0..1024 tokens, vision window 0..32 s), one axis at a time around the deployed policy, on the
    config's head shape with `--layers` layers (default 4).  Per point: steady state, three steps of plain calls
    with CUDA events around every call.  One JSON line; `value` is the deployed policy's frames/s by these timings."""
    import torch
    from paper_2510_09608_b200 import binding
    L = args.layers or 4
    per_s = wl.vision_per_chunk          # vision tokens per second of video
    points = [("deployed", wl.n_sink, wl.text_window, wl.vision_window)]
    points += [("sink", v, wl.text_window, wl.vision_window) for v in (0, 64, 256, 1024)]
    points += [("text_window", wl.n_sink, v, wl.vision_window) for v in (0, 64, 256, 1024)]
    points += [("vision_window", wl.n_sink, wl.text_window, sec * per_s) for sec in (0, 1, 4, 8, 32)]
    # the policy switches at the deployed sizes (the paper's Table 4 arms as latency): native positions instead of
    # contiguous ones (eviction then only releases storage: no key is re-rotated), and sinks of any token type
    points += [("policy:native_rope", wl.n_sink, wl.text_window, wl.vision_window),
               ("policy:sink_any_type", wl.n_sink, wl.text_window, wl.vision_window)]
    rows = []
    for axis, S, Tw, Vw in points:
        w = dataclasses_replace(wl, layers=L, n_sink=S, text_window=Tw, vision_window=Vw)
        stream = sg.Stream(w, rank)
        cache = binding.Cache(L, w.kv_heads, w.head_dim, S, Vw, Tw, w.capacity)
        cache.set_rope(w.rope_mode, w.rope_base, w.sections)
        cache.set_policy(sink_any_type=(axis == "policy:sink_any_type"), contiguous=(axis != "policy:native_rope"))
        fill_to_steady_state(cache, w, stream)
        cache.evict()
        timers = {}
        n_q = []
        for i in range(4):
            inp = StepInputs(w, stream, *next_step_schedule(stream, w))
            if i == 0:
                run_step(cache, w, inp)          # warm-up step
                continue
            run_step(cache, w, inp, timers)
            n_q.append(inp.n)
        torch.cuda.synchronize()
        assert cache.status() == binding.OK
        kept = len(cache.query()["gids"])
        cache.close()
        avg = {k: statistics.mean(a.elapsed_time(b) for a, b in v) for k, v in timers.items()}
        tot = {k: sum(a.elapsed_time(b) for a, b in v) / 3 for k, v in timers.items()}
        lk = kept - w.decode_steps                       # keys at the time of the chunk prefill
        nq = int(round(statistics.mean(n_q)))
        flops = prefill_flops(w, nq, lk) if lk >= nq else float("nan")   # the chunk itself is (partly) evicted: no closed form
        kv_bytes = kept * 2 * w.kv_heads * w.head_dim * 2
        moved = max(kept - w.decode_steps - S, 0) if axis != "policy:native_rope" else 0
        ev_bytes = 2 * moved * w.kv_heads * w.head_dim * 2 * L
        step_ms = sum(tot.values())
        rows.append(dict(axis=axis, contiguous=(axis != "policy:native_rope"), sink_any_type=(axis == "policy:sink_any_type"), n_sink=S, text_window=Tw, vision_window_s=Vw // per_s, kept_tokens=kept,
                         step_ms=step_ms, evict_ms=avg["evict"], prefill_ms=avg["prefill"],
                         decode_layer_step_ms=avg["decode_token"] / L,
                         prefill_frac=(flops / (avg["prefill"] * 1e-3) / 1e12 / peaks["bf16_burst"]) if flops == flops else None,
                         decode_frac=kv_bytes * L / (avg["decode_token"] * 1e-3) / 1e9 / peaks["hbm"],
                         evict_frac=ev_bytes / (avg["evict"] * 1e-3) / 1e9 / peaks["hbm"]))
    if rank == 0:
        d = rows[0]
        roof = dict(bound="hbm", kernel="decode", achieved=d["decode_frac"] * peaks["hbm"], peak=peaks["hbm"], unit="GB/s",
                    frac=d["decode_frac"], traffic=None, peak_source=peaks["source"] + " (copy)")
        print(json.dumps(dict(base, value=wl.frames / (d["step_ms"] * 1e-3), ms_per_step=d["step_ms"],
                              config=dict(workload=f"policy sweep on the config {args.config} shape, {L} layers: one axis at a time around "
                                                   f"sinks {wl.n_sink} / text {wl.text_window} / vision {wl.vision_window // per_s} s; plain calls, event-timed",
                                          l2="no flush: the layers' K/V in turn exceed L2 except at the smallest windows (see kept_tokens)",
                                          replicas="independent streams, no collective"),
                              roofline=roof, cpu_baseline=None, e2e=None, gpu_launches=None, clocks=None, sweep=rows)))


def bench_qkv(args, wl, base, peaks, rank, world, local):
    """The step on the input side of the path (svlm_qkv_append): the Q/K/V projection of one layer whose epilogue
    rotates the keys and appends to the cache, timed on the config's head shape with hidden size 3584 for one
    chunk (n ~ 524) and for a long append (n = 4096), graph replay, CUDA events, weights of different layers in turn
    (28 x 33 MB > L2)."""
    import torch
    from paper_2510_09608_b200 import binding
    hidden, L = 3584, args.layers or wl.layers
    n_out = (wl.q_heads + 2 * wl.kv_heads) * wl.head_dim
    g = torch.Generator(device="cuda").manual_seed(wl.seed)
    W = (torch.randn(L, n_out, hidden, generator=g, device="cuda") / hidden ** 0.5).to(torch.bfloat16)
    rows = []
    for n in (wl.vision_per_chunk + wl.text_max // 2, 4096):
        cache = binding.Cache(L, wl.kv_heads, wl.head_dim, 0, 0, 0, (n + 127) // 128 * 128)   # every eviction empties it
        cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
        X = torch.randn(L, n, hidden, generator=g, device="cuda").to(torch.bfloat16)
        Q = torch.empty(n, wl.q_heads, wl.head_dim, dtype=torch.bfloat16, device="cuda")
        ty = torch.ones(n, dtype=torch.uint8, device="cuda")
        def step(it):
            pos = torch.arange(it * n, (it + 1) * n, dtype=torch.int32, device="cuda")
            if wl.rope_mode:
                pos = pos[:, None].repeat(1, 3).contiguous()
            for l in range(L):
                cache.qkv_append(l, X[l], W[l], wl.q_heads, ty if l == 0 else None, pos if l == 0 else None, Q)
            cache.evict()                   # room for the next append

        step(0)                             # plain once: one-time kernel attributes outside any capture
        torch.cuda.synchronize()
        graphs = []
        cur = torch.cuda.current_stream()
        for it in range(1, args.warmup + args.steps + 1):   # replayed from graphs: the host's share of a call is not timed
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr):
                cache.set_stream(torch.cuda.current_stream())
                step(it)
            graphs.append(gr)
        cache.set_stream(cur)
        times = []
        for it, gr in enumerate(graphs):
            a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            gr.replay()
            b2.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times.append(a.elapsed_time(b2) / L)   # per layer; the metadata and eviction launches are inside
        assert cache.status() == binding.OK
        cache.close()
        ms = statistics.median(times)
        flops = 2.0 * n * hidden * n_out
        rows.append(dict(n=n, ms_per_layer=ms, tflops=flops / (ms * 1e-3) / 1e12, frac=flops / (ms * 1e-3) / 1e12 / peaks["bf16_burst"],
                         ctas=(n + 127) // 128 * ((wl.q_heads + 2 * wl.kv_heads + 1) // 2)))
    # decode-time projections (a few tokens): the bandwidth kernel behind svlm_out_proj, weights of the layers in turn
    cache = binding.Cache(1, wl.kv_heads, wl.head_dim, 0, 0, 0, 128)
    small = []
    for n in (1, 16):
        x = torch.randn(n, hidden, generator=g, device="cuda").to(torch.bfloat16)
        y = torch.empty(n, n_out, dtype=torch.bfloat16, device="cuda")
        ts = []
        for it in range(args.warmup + args.steps):
            a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for l in range(L):
                cache.out_proj(x, W[l], y)
            b2.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                ts.append(a.elapsed_time(b2) / L)
        ms = statistics.median(ts)
        wbytes = n_out * hidden * 2
        small.append(dict(n=n, ms_per_layer=ms, gbs=wbytes / (ms * 1e-3) / 1e9, frac_hbm=wbytes / (ms * 1e-3) / 1e9 / peaks["hbm"]))
    cache.close()
    chain = decode_layer_chain(args, wl, peaks, rank, hidden, W, g)
    if rank == 0:
        d = rows[-1]
        roof = dict(bound="tensor", kernel="qkv_append", achieved=d["tflops"], peak=peaks["bf16_burst"], unit="TFLOP/s", frac=d["frac"],
                    traffic=None, algorithmic=2.0 * d["n"] * hidden * n_out, peak_source=peaks["source"] + " (burst bf16)")
        print(json.dumps(dict(base, metric="layers/s of the Q/K/V projection with append epilogue", unit="layers/s",
                              value=1e3 / d["ms_per_layer"], ms_per_step=d["ms_per_layer"],
                              config=dict(workload=f"svlm_qkv_append on the config {args.config} head shape: hidden {hidden} -> "
                                                   f"{wl.q_heads}+{wl.kv_heads}+{wl.kv_heads} heads of {wl.head_dim}, {L} layers in turn",
                                          l2="weights of the layers in turn exceed L2; no flush", replicas="independent streams, no collective"),
                              roofline=roof, cpu_baseline=None, e2e=None, gpu_launches=None, clocks=None, points=rows,
                              decode_projection=small, decode_layer_chain=chain)))


def decode_layer_chain(args, wl, peaks, rank, hidden, W, g):
    """One generated token through the attention half of every layer, as a decoder would call it:
    [q | k | v] = W_qkv x (svlm_out_proj), the fused append + attention (svlm_decode_step), y = W_o a (svlm_out_proj),
    the next layer's x being this layer's y; over the config's steady-state cache, one CUDA graph per token (the
    position advances inside it), CUDA events around the replay.  All three kernels are launched while their
    predecessor may still run and fetch what does not depend on it (weights, retained keys and values) first."""
    import torch
    from paper_2510_09608_b200 import binding
    L = W.shape[0]
    w = dataclasses_replace(wl, layers=L)
    stream = sg.Stream(w, rank)
    cache = binding.Cache(L, w.kv_heads, w.head_dim, w.n_sink, w.vision_window, w.text_window, w.capacity)
    cache.set_rope(w.rope_mode, w.rope_base, w.sections)
    fill_to_steady_state(cache, w, stream)
    cache.evict()
    qd = w.q_heads * w.head_dim
    kd = w.kv_heads * w.head_dim
    Wo = (torch.randn(L, hidden, qd, generator=g, device="cuda") / qd ** 0.5).to(torch.bfloat16)
    x0 = torch.randn(1, hidden, generator=g, device="cuda").to(torch.bfloat16)
    xs = [x0] + [torch.empty(1, hidden, dtype=torch.bfloat16, device="cuda") for _ in range(L)]
    qkv = torch.empty(1, qd + 2 * kd, dtype=torch.bfloat16, device="cuda")
    att = torch.empty(1, w.q_heads, w.head_dim, dtype=torch.bfloat16, device="cuda")
    _, types, pos = stream.next_decode_token()
    ty = torch.from_numpy(types).cuda()
    pos_d = torch.from_numpy(np.ascontiguousarray(pos)).cuda()

    def token():
        for l in range(L):
            cache.out_proj(xs[l], W[l], qkv)
            cache.decode_step(l, qkv[:, qd:qd + kd].view(1, w.kv_heads, w.head_dim), qkv[:, qd + kd:].view(1, w.kv_heads, w.head_dim),
                              ty, pos_d, qkv[:, :qd].view(1, w.q_heads, w.head_dim), att)
            cache.out_proj(att.view(1, qd), Wo[l], xs[l + 1])
        pos_d.add_(1)

    token()                                  # plain once: one-time kernel attributes outside any capture
    torch.cuda.synchronize()
    cur = torch.cuda.current_stream()
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.graph(gr):
        cache.set_stream(torch.cuda.current_stream())
        token()
    cache.set_stream(cur)
    ts = []
    n_tok = max(args.steps, 8)
    for it in range(args.warmup + n_tok):
        a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        gr.replay()
        b2.record()
        torch.cuda.synchronize()
        if it >= args.warmup:
            ts.append(a.elapsed_time(b2))
    assert cache.status() == binding.OK
    q = cache.query()
    cache.close()
    ms = statistics.median(ts)
    # bytes a token must read per layer: both weight matrices and the retained keys and values, once
    per_layer = (qd + 2 * kd) * hidden * 2 + hidden * qd * 2 + w.retained * 2 * kd * 2
    return dict(ms_per_token=ms, us_per_layer=ms * 1e3 / L, tokens_per_s=1e3 / ms, layers=L,
                bytes_per_layer=per_layer, gbs=per_layer * L / (ms * 1e-3) / 1e9,
                frac_hbm=per_layer * L / (ms * 1e-3) / 1e9 / peaks["hbm"], kept_tokens=int(len(q["gids"])),
                note="q/k/v projection + fused append and attention + output projection per layer, graph replay per token")


def bench_drift(args, wl, base, peaks, rank, world, local):
    """The whole stream of the config (3600 one-second chunks = one hour for config 3), every chunk timed: the paper's
    claim is a per-chunk latency that stays flat however long the stream runs (Section 3.3).  Plain calls, one CUDA
    event pair per chunk; key, value and query VALUES are drawn once and reused (they do not influence the time),
    token types and positions follow the stream.  Reports the drift: ratio of the medians of the last and the first
    5 % of the chunks after the windows have filled, and the slope of a straight-line fit."""
    import torch
    from paper_2510_09608_b200 import binding
    L = args.layers or wl.layers
    w = dataclasses_replace(wl, layers=L)
    chunks = args.chunks or w.chunks
    stream = sg.Stream(w, rank)
    cache = binding.Cache(L, w.kv_heads, w.head_dim, w.n_sink, w.vision_window, w.text_window, w.capacity)
    cache.set_rope(w.rope_mode, w.rope_base, w.sections)
    fill = fill_to_steady_state(cache, w, stream)
    cache.evict()
    g = torch.Generator(device="cuda").manual_seed(w.seed)
    nmax = w.max_chunk_tokens
    rnd = lambda *shape: torch.randn(*shape, generator=g, device="cuda").to(torch.bfloat16)  # noqa: E731
    K, V, Q = rnd(L, nmax, w.kv_heads, w.head_dim), rnd(L, nmax, w.kv_heads, w.head_dim), rnd(L, nmax, w.q_heads, w.head_dim)
    out = torch.empty_like(Q)
    k1, v1, q1 = rnd(L, 1, w.kv_heads, w.head_dim), rnd(L, 1, w.kv_heads, w.head_dim), rnd(L, 1, w.q_heads, w.head_dim)
    o1 = torch.empty_like(q1)
    text1 = torch.zeros(1, dtype=torch.uint8, device="cuda")
    sampler = ClockSampler(local)
    sampler.start()
    evs = []
    for i in range(chunks - fill):
        gids, types, pos = stream.next_chunk()
        n = len(gids)
        ty, ps = torch.from_numpy(types).cuda(), torch.from_numpy(np.ascontiguousarray(pos)).cuda()
        dec = [torch.from_numpy(np.ascontiguousarray(stream.next_decode_token()[2])).cuda() for _ in range(w.decode_steps)]
        a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        cache.append(0, K[0, :n], V[0, :n], ty, ps)
        cache.evict()
        cache.attend(0, Q[0, :n], ps, out[0, :n])
        for l in range(1, L):
            cache.append(l, K[l, :n], V[l, :n])
            cache.attend(l, Q[l, :n], ps, out[l, :n])
        for p1 in dec:
            for l in range(L):
                cache.decode_step(l, k1[l], v1[l], text1 if l == 0 else None, p1, q1[l], o1[l])
        b2.record()
        evs.append((a, b2))
        if i % 64 == 63:
            torch.cuda.synchronize()      # keep the host from running far ahead of the device
    torch.cuda.synchronize()
    clocks = sampler.finish()
    assert cache.status() == binding.OK
    meta = cache.query()
    lat = np.array([a.elapsed_time(b2) for a, b2 in evs])
    k5 = max(1, len(lat) // 20)
    first, last = float(np.median(lat[:k5])), float(np.median(lat[-k5:]))
    slope = float(np.polyfit(np.arange(len(lat)), lat, 1)[0]) * 1000.0
    if rank == 0:
        print(json.dumps(dict(base, value=w.frames / (float(np.median(lat)) * 1e-3), ms_per_step=float(np.median(lat)), steps=len(lat),
                              config=dict(workload=f"config {args.config} ({w.name}) run as a whole stream: {chunks} chunks, {L} layers, every chunk "
                                                   f"timed after the windows have filled (chunk {fill}); plain calls, no graph",
                                          l2="working set far exceeds L2; no flush", replicas="independent streams, no collective"),
                              roofline=dict(bound="hbm", kernel="(whole step)", achieved=None, peak=None, unit=None, frac=None, traffic=None),
                              cpu_baseline=None, e2e=None, gpu_launches=None, clocks=clocks,
                              drift=dict(chunks_timed=len(lat), median_ms=float(np.median(lat)), first_5pct_ms=first, last_5pct_ms=last,
                                         ratio_last_to_first=last / first, slope_ms_per_1000_chunks=slope,
                                         max_ms=float(lat.max()), p99_ms=float(np.percentile(lat, 99)),
                                         kept_tokens=int(len(meta["gids"])), max_position=int(meta["pos"].max()),
                                         shift_total=int(meta["shift_total"])))))


TRACE_STATIONS = {0: "kernel entry", 1: "page list in shared memory", 2: "first round's copies issued",
                  3: "previous kernel complete (dependency wait returns)", 4: "rotated query in shared memory",
                  5: "warp 1 has its keys", 14: "warp 1: scores and softmax done", 6: "warp 1 through with its units",
                  7: "all consumer warps through", 8: "CTA's record on its way (tagged stores issued)",
                  12: "combining CTA: its pieces of every split's record in registers",
                  15: "combining CTA: warps' sums exchanged", 11: "combining CTA: output written", 13: "CTA leaves"}


def bench_drift_multi(args, wl, base, peaks, rank, world, local):
    """bench_drift for a workload of several streams in lock step (config 5: 8 streams, 7200 chunks = two hours of
    8 frames/s video each): per chunk every stream appends its tokens, ONE batched eviction, per layer the appends and
    ONE chunk-prefill launch for all streams, then the generated tokens with one batched decode launch per layer;
    every chunk of all streams is timed by its own event pair.  Values are drawn once and reused; token types, counts
    and positions follow each stream."""
    import torch
    from paper_2510_09608_b200 import binding
    L = args.layers or wl.layers
    w = dataclasses_replace(wl, layers=L)
    S = w.streams
    chunks = args.chunks or w.chunks
    streams = [sg.Stream(w, rank * S + i) for i in range(S)]
    caches, fill = [], 0
    for st in streams:
        c = binding.Cache(L, w.kv_heads, w.head_dim, w.n_sink, w.vision_window, w.text_window, w.capacity)
        c.set_rope(w.rope_mode, w.rope_base, w.sections)
        fill = fill_to_steady_state(c, w, st)
        c.evict()
        caches.append(c)
    g = torch.Generator(device="cuda").manual_seed(w.seed)
    nmax = w.max_chunk_tokens
    rnd = lambda *shape: torch.randn(*shape, generator=g, device="cuda").to(torch.bfloat16)  # noqa: E731
    K, V = rnd(L, nmax, w.kv_heads, w.head_dim), rnd(L, nmax, w.kv_heads, w.head_dim)
    Q = rnd(L, S * nmax, w.q_heads, w.head_dim)
    out = torch.empty_like(Q)
    k1, v1, q1 = rnd(L, S, w.kv_heads, w.head_dim), rnd(L, S, w.kv_heads, w.head_dim), rnd(L, S, w.q_heads, w.head_dim)
    o1 = torch.empty_like(q1)
    text1 = torch.zeros(S, dtype=torch.uint8, device="cuda")
    sampler = ClockSampler(local)
    sampler.start()
    evs = []
    for i in range(chunks - fill):
        sched = [st.next_chunk() for st in streams]
        n_q = [len(sc[0]) for sc in sched]
        tys = [torch.from_numpy(sc[1]).cuda() for sc in sched]
        pss = [torch.from_numpy(np.ascontiguousarray(sc[2])).cuda() for sc in sched]
        pos_all = torch.cat(pss).contiguous()
        tot = sum(n_q)
        dec = []
        for _ in range(w.decode_steps):
            toks = [st.next_decode_token() for st in streams]
            dec.append(torch.from_numpy(np.ascontiguousarray(np.stack([t[2][0] for t in toks]))).cuda())
        a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for c, n, ty, ps in zip(caches, n_q, tys, pss):
            c.append(0, K[0, :n], V[0, :n], ty, ps)
        binding.evict_batched(caches)
        for l in range(L):
            if l:
                for c, n in zip(caches, n_q):
                    c.append(l, K[l, :n], V[l, :n])
            binding.attend_batched_varlen(caches, l, Q[l, :tot], pos_all, n_q, out[l, :tot])
        for p1 in dec:
            for l in range(L):
                binding.decode_step_batched(caches, l, k1[l], v1[l], text1 if l == 0 else None, p1, q1[l], o1[l])
        b2.record()
        evs.append((a, b2))
        if i % 32 == 31:
            torch.cuda.synchronize()      # keep the host from running far ahead of the device
    torch.cuda.synchronize()
    clocks = sampler.finish()
    for c in caches:
        assert c.status() == binding.OK
    metas = [c.query() for c in caches]
    lat = np.array([a.elapsed_time(b2) for a, b2 in evs])
    k5 = max(1, len(lat) // 20)
    first, last = float(np.median(lat[:k5])), float(np.median(lat[-k5:]))
    slope = float(np.polyfit(np.arange(len(lat)), lat, 1)[0]) * 1000.0
    if rank == 0:
        med = float(np.median(lat))
        print(json.dumps(dict(base, value=w.frames * S / (med * 1e-3), ms_per_step=med, steps=len(lat),
                              config=dict(workload=f"config {args.config} ({w.name}) run as whole streams: {S} streams in lock step, {chunks} chunks "
                                                   f"each, {L} layers, every chunk (of all streams) timed after the windows have filled "
                                                   f"(chunk {fill}); plain calls, no graph",
                                          l2="working set far exceeds L2; no flush", replicas="independent streams, no collective"),
                              roofline=dict(bound="hbm", kernel="(whole step)", achieved=None, peak=None, unit=None, frac=None, traffic=None),
                              cpu_baseline=None, e2e=None, gpu_launches=None, clocks=clocks,
                              drift=dict(chunks_timed=len(lat), median_ms=med, first_5pct_ms=first, last_5pct_ms=last,
                                         ratio_last_to_first=last / first, slope_ms_per_1000_chunks=slope,
                                         max_ms=float(lat.max()), p99_ms=float(np.percentile(lat, 99)),
                                         kept_tokens=[int(len(m["gids"])) for m in metas],
                                         max_position=int(max(m["pos"].max() for m in metas)),
                                         shift_total=[int(m["shift_total"]) for m in metas]))))


def bench_decode_trace(args, wl, base, peaks, rank, world, local):
    """In-kernel time stamps of the layer-sequential decode chain: the instrumented build of the library
    (paper_2510_09608_b200.build.build_trace) runs generated tokens through svlm_decode_step, one launch per layer,
    replayed from a CUDA graph as in the step benchmark, and every CTA's thread 0 records %globaltimer at the
    stations of the chain.  Prints, per station, the median and the latest CTA's time relative to the moment the
    dependency wait returns, averaged over the traced launches that could read ahead (every layer but a token's first)."""
    import ctypes
    import torch
    from paper_2510_09608_b200 import binding
    lib = binding._lib
    if not hasattr(lib, "svlm_debug_decode_trace_start"):
        raise SystemExit("decode-trace needs the instrumented library: python -m paper_2510_09608_b200.build --trace")
    L = wl.layers
    stream = sg.Stream(wl, rank)
    cache = binding.Cache(L, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    fill_to_steady_state(cache, wl, stream)
    cache.evict()
    n_tok = max(2, 56 // L)
    w1 = dataclasses_replace(wl, decode_steps=n_tok)
    inp = StepInputs(w1, stream, *next_step_schedule(stream, w1))
    run_step(cache, w1, inp)                        # plain once: kernel attributes, warm caches
    torch.cuda.synchronize()
    inp = StepInputs(w1, stream, *next_step_schedule(stream, w1))

    def tokens():
        for d in inp.dec:
            for l in range(L):
                cache.decode_step(l, d["K"][l], d["V"][l], d["types"] if l == 0 else None, d["pos"], d["Q"][l], d["out"][l])

    lib.svlm_debug_decode_trace_start.restype = None
    lib.svlm_debug_decode_trace_start()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        cache.set_stream(torch.cuda.current_stream())
        tokens()
    cache.set_stream(torch.cuda.current_stream())
    a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    g.replay()
    b2.record()
    torch.cuda.synchronize()
    assert cache.status() == binding.OK
    buf = np.zeros((64, 160, 16), np.uint64)
    assert lib.svlm_debug_decode_trace_read(buf.ctypes.data_as(ctypes.c_void_p)) == 0
    t = buf.astype(np.int64)
    rows, periods = [], []
    prev_w = None
    for i in range(min(64, n_tok * L)):
        n = int((t[i, :, 0] > 0).sum())
        if n == 0:
            break
        x = t[i, :n]
        w = float(np.median(x[:, 3]))
        early = bool(np.median(x[:, 0]) < w - 2000)      # entered well before the wait returned: it could read ahead
        if prev_w is not None and early:
            periods.append((w - prev_w) / 1e3)
        prev_w = w
        if early:
            rows.append({k: ((float(np.median(x[:, k][x[:, k] > 0])) - w) / 1e3, (float(x[:, k].max()) - w) / 1e3)
                         for k in TRACE_STATIONS if (x[:, k] > 0).any()})
    table = []
    for k, name in TRACE_STATIONS.items():
        vals = [r[k] for r in rows if k in r]
        if vals:
            table.append(dict(station=name, median_us=round(float(np.mean([v[0] for v in vals])), 2),
                              latest_cta_us=round(float(np.mean([v[1] for v in vals])), 2)))
    table.sort(key=lambda r: r["latest_cta_us"])
    if rank == 0:
        print(json.dumps(dict(base, metric="decode layer-step period (instrumented build)", unit="us", higher_is_better=False,
                              value=float(np.mean(periods)) if periods else None,
                              ms_per_step=a.elapsed_time(b2) / n_tok,
                              config=dict(workload=f"config {args.config} shape, {L} layers: {n_tok} generated tokens, one svlm_decode_step "
                                                   f"launch per layer, graph replay; timer resolution about 0.26 us; the stamps themselves add "
                                                   f"a little to the chain"),
                              roofline=dict(bound="hbm", kernel="decode (instrumented)", achieved=None, peak=None, unit=None, frac=None,
                                            traffic=None),
                              cpu_baseline=None, e2e=None, gpu_launches=n_tok * (L + 1), clocks=None,
                              launches_traced=len(rows), trace=table)))


def dataclasses_replace(obj, **kw):
    import dataclasses
    return dataclasses.replace(obj, **kw)


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="replay nothing: plain calls in the timed region")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (smaller case for profiling)")
    ap.add_argument("--workload", default="step", choices=["step", "overlap", "sweep", "qkv", "drift", "decode-trace"],
                    help="step: the per-chunk KV-cache step (default); overlap: the whole window re-prefilled every second; "
                         "sweep: the step's latency over the paper's sink / window ablation values; qkv: the projection steps; "
                         "drift: the config's whole stream, every chunk timed; decode-trace: in-kernel time stamps of the "
                         "decode chain (needs the instrumented build of the library)")
    ap.add_argument("--chunks", type=int, default=0, help="drift: stream length in chunks (default: the config's)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    wl = sg.workloads()[args.config]
    if args.layers:
        import dataclasses
        wl = dataclasses.replace(wl, layers=args.layers, name=f"{wl.name}, cut to {args.layers} layers")
    frames_per_step = wl.frames
    base = dict(metric="sustainable frames/s of the per-chunk evict+attend step (ms_per_step = per-chunk latency)",
                unit="frames/s", n_gpus=args.gpus, steps=args.steps, warmup=args.warmup, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic")
    kv_mb = wl.retained * 2 * wl.kv_heads * wl.head_dim * 2 * wl.layers / 1e6
    l2_note = (f"working set ({kv_mb:.0f} MB of K/V over all layers) exceeds L2 (126 MB); no flush" if kv_mb > 126 else
               f"working set ({kv_mb:.1f} MB of K/V) stays in L2 (126 MB): bandwidth figures of this configuration are "
               "L2-resident, not HBM")
    config = dict(workload=f"config {args.config} ({wl.name}): {wl.layers} layers, {wl.q_heads}/{wl.kv_heads} heads, "
                           f"d={wl.head_dim}, sinks {wl.n_sink} / vision window {wl.vision_window} / text window "
                           f"{wl.text_window}, chunk = {wl.frames}x{wl.grid_h}x{wl.grid_w} vision + U(0..{wl.text_max}) "
                           f"text tokens, {wl.decode_steps} decode steps per chunk, steady state",
                  layers="sequential calls per layer", l2=l2_note,
                  replicas="one independent stream per GPU, no collective")

    if args.impl == "reference":
        if rank != 0:
            return
        vals = []
        info = None
        for i in range(args.warmup + args.steps):
            info = oracle_sample(wl, decode=2, layers=1)   # one whole layer of prefill rows: the per-call set-up is not scaled up
            if i >= args.warmup:
                vals.append(info["step_seconds"])
        sec = statistics.mean(vals)
        v = frames_per_step / sec
        line = dict(base, impl="reference", value=v, ms_per_step=sec * 1e3, config=config,
                    cpu_baseline=dict(value=v, unit="frames/s", cores=info["cores"], kind="oracle", sample=info["sample"]),
                    e2e=dict(value=v, unit="frames/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0), n_gpus=1)
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist
    if args.workload == "decode-trace":
        import paper_2510_09608_b200 as pkg
        from paper_2510_09608_b200 import build as _build
        pkg.LIB_OVERRIDE = _build.build_trace()       # the instrumented build, before the binding loads a library
    from paper_2510_09608_b200 import binding

    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    if args.workload == "decode-trace":
        bench_decode_trace(args, wl, base, peaks, rank, world, local)
        if world > 1:
            dist.destroy_process_group()
        return
    if args.workload == "drift":
        wd = sg.workloads()[args.config]
        (bench_drift_multi if wd.streams > 1 else bench_drift)(args, wd, base, peaks, rank, world, local)
        if world > 1:
            dist.destroy_process_group()
        return
    if args.workload == "qkv":
        bench_qkv(args, sg.workloads()[args.config], base, peaks, rank, world, local)
        if world > 1:
            dist.destroy_process_group()
        return
    if args.workload == "sweep":
        bench_sweep(args, sg.workloads()[args.config], base, peaks, rank, world, local)
        if world > 1:
            dist.destroy_process_group()
        return
    if args.workload == "overlap":
        bench_overlap(args, wl, base, peaks, rank, world, local)
        if world > 1:
            dist.destroy_process_group()
        return
    if wl.streams > 1 and wl.layers == 1:
        bench_batched_decode(args, wl, base, peaks, rank, world, local)
        if world > 1:
            dist.destroy_process_group()
        return
    if wl.streams > 1:
        bench_multi_stream(args, wl, base, config, peaks, rank, world, local)
        if world > 1:
            dist.destroy_process_group()
        return
    stream = sg.Stream(wl, rank)
    cache = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
    cache.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    fill_chunks = fill_to_steady_state(cache, wl, stream)
    cache.evict()
    assert cache.status() == binding.OK

    total = args.warmup + args.steps
    want_e2e = not args.no_e2e
    inputs = [StepInputs(wl, stream, *next_step_schedule(stream, wl)) for _ in range(total)]
    prime = StepInputs(wl, stream, *next_step_schedule(stream, wl))   # first step of the per-kernel pass
    # one plain step on a scratch cache first: one-time function attributes are set outside any capture
    scratch = binding.Cache(wl.layers, wl.kv_heads, wl.head_dim, wl.n_sink, wl.vision_window, wl.text_window, wl.capacity)
    scratch.set_rope(wl.rope_mode, wl.rope_base, wl.sections)
    run_step(scratch, wl, inputs[0])
    torch.cuda.synchronize()
    scratch.close()

    graphs, launches = [], []
    if not args.no_graph:
        # Capturing only records the launches; the cache's device state is untouched until replay.
        for inp in inputs:
            g = torch.cuda.CUDAGraph()
            before = binding.launch_count()
            with torch.cuda.graph(g):
                cache.set_stream(torch.cuda.current_stream())
                run_step(cache, wl, inp)
            launches.append(binding.launch_count() - before)
            graphs.append(g)
        cache.set_stream(torch.cuda.current_stream())

    def do_step(i):
        if graphs:
            graphs[i].replay()
        else:
            run_step(cache, wl, inputs[i])

    for i in range(args.warmup):
        do_step(i)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    before = binding.launch_count()
    ev[0].record()
    for i in range(args.steps):
        do_step(args.warmup + i)
        ev[i + 1].record()
    barrier()
    clocks = sampler.finish()
    gpu_launches = sum(launches[args.warmup:]) if graphs else binding.launch_count() - before
    step_ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    elapsed_ms = ev[0].elapsed_time(ev[-1])
    assert cache.status() == binding.OK
    kept = len(cache.query()["gids"])

    # ---- per-kernel durations on the same stream (plain calls, CUDA events around each call) -----
    timers = {}
    prof_steps = 3
    lk_list = []
    prof_inputs = [prime] + [StepInputs(wl, stream, *next_step_schedule(stream, wl)) for _ in range(prof_steps - 1)]
    for inp in prof_inputs:
        run_step(cache, wl, inp, timers)
        lk_list.append(inp.n)
    torch.cuda.synchronize()
    kern = {k: [a.elapsed_time(b) for a, b in v] for k, v in timers.items()}
    avg = {k: statistics.mean(v) for k, v in kern.items()}
    tot = {k: sum(v) / prof_steps for k, v in kern.items()}
    n_q = statistics.mean(lk_list)
    lk = wl.retained
    flops = prefill_flops(wl, int(round(n_q)), lk)
    kv_bytes_layer = lk * 2 * wl.kv_heads * wl.head_dim * 2
    moved = wl.retained - wl.n_sink
    evict_bytes = 2 * moved * wl.kv_heads * wl.head_dim * 2 * wl.layers
    # The chunk prefill of all layers back to back inside one event pair: the kernel's duration in the stream,
    # without the host's launch gap that a separately timed call carries (the step itself is replayed from a graph).
    inp_b = StepInputs(wl, stream, stream.next_chunk(), [])
    cache.append(-1, inp_b.K, inp_b.V, inp_b.types, inp_b.pos)
    cache.evict()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record()
    for l in range(wl.layers):
        cache.attend(l, inp_b.Q[l], inp_b.pos, inp_b.out[l])
    eb.record()
    torch.cuda.synchronize()
    prefill_ms = ea.elapsed_time(eb) / wl.layers
    flops_b = prefill_flops(wl, inp_b.n, lk)
    # The decode launches as the step runs them: graph replay of one step's generated tokens (a separately timed
    # plain call would carry the host's launch gaps).
    decode_token_ms = time_decode_tokens(cache, wl, prof_inputs[-1]) if wl.decode_steps else float("nan")
    kernels = {
        "prefill": dict(bound="tensor", avg_ms=prefill_ms, per_step_ms=prefill_ms * wl.layers,
                        achieved=flops_b / (prefill_ms * 1e-3) / 1e12, unit="TFLOP/s", peak=peaks["bf16_burst"],
                        single_call_ms=avg["prefill"], note="avg_ms = the layers' launches back to back / layers"),
        # one launch per layer; the launches of one token overlap (programmatic dependent launch), so the
        # per-launch duration is the token's time over its L launches (the metadata launch is inside it)
        "decode": dict(bound="hbm", avg_ms=decode_token_ms / wl.layers, per_step_ms=decode_token_ms * wl.decode_steps,
                       achieved=kv_bytes_layer * wl.layers / (decode_token_ms * 1e-3) / 1e9, unit="GB/s",
                       peak=peaks["hbm"], plain_call_ms=avg["decode_token"] / wl.layers,
                       note="avg_ms = time of one token's decode over all layers / layers, graph replay of 16 tokens as in "
                            "the step (one launch per layer, the metadata launch inside); plain_call_ms: the same by "
                            "separately timed calls"),
        "evict": dict(bound="hbm", avg_ms=avg["evict"], per_step_ms=tot["evict"],
                      achieved=evict_bytes / (avg["evict"] * 1e-3) / 1e9, unit="GB/s", peak=peaks["hbm"]),
        "append": dict(avg_ms=avg["append"], per_step_ms=tot["append"]),
    }
    for k in ("prefill", "decode", "evict"):
        kernels[k]["frac"] = kernels[k]["achieved"] / kernels[k]["peak"]
        # the same rate against the data-sheet figure (dense bf16 2250 TFLOP/s, HBM3e 8000 GB/s), for context
        kernels[k]["frac_of_nominal"] = kernels[k]["achieved"] / (2250.0 if kernels[k]["bound"] == "tensor" else 8000.0)
    dominant = max(("prefill", "decode", "evict"), key=lambda k: kernels[k]["per_step_ms"])
    kd = kernels[dominant]
    ncu_bytes = ncu_dram_traffic()
    traffic = ncu_bytes.get(dominant)
    if dominant == "evict":
        traffic = ncu_bytes["evict_per_layer"] * wl.layers if ncu_bytes.get("evict_per_layer") is not None else None
    if args.config not in (2, 3):
        traffic = None          # the counters were taken on the config-3 shape
    roofline = dict(bound="tensor" if dominant == "prefill" else "hbm", kernel=dominant, achieved=kd["achieved"],
                    peak=kd["peak"], unit=kd["unit"], frac=kd["frac"], frac_of_nominal=kd["frac_of_nominal"], traffic=traffic,
                    algorithmic=(flops_b if dominant == "prefill" else kv_bytes_layer if dominant == "decode" else evict_bytes),
                    peak_source=peaks["source"] + (" (burst bf16)" if dominant == "prefill" else " (copy)"))

    # ---- extra: one token's decode of ALL layers in one launch (svlm_decode_step with layer -1) -----
    # For callers that hold every layer's inputs at once; the headline above keeps one call per layer.
    all_layers = None
    if wl.layers > 1:
        gen1 = lambda tensor, g, heads: torch.stack(  # noqa: E731
            [sg.rows_bf16_torch(wl.seed, tensor, stream.stream, l, g, heads, wl.head_dim)[0] for l in range(wl.layers)])
        ts = []
        for _ in range(4):
            g1, t1, p1 = stream.next_decode_token()
            K1, V1, Q1 = gen1(sg.TENSOR_K, g1, wl.kv_heads), gen1(sg.TENSOR_V, g1, wl.kv_heads), gen1(sg.TENSOR_Q, g1, wl.q_heads)
            o1 = torch.empty_like(Q1)
            ty1, ps1 = torch.from_numpy(t1).cuda(), torch.from_numpy(np.ascontiguousarray(p1)).cuda()
            a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            cache.decode_step(-1, K1, V1, ty1, ps1, Q1, o1)
            b2.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b2))
        t_all = statistics.median(ts[1:])
        all_layers = dict(ms_per_token=t_all, achieved=kv_bytes_layer * wl.layers / (t_all * 1e-3) / 1e9, unit="GB/s",
                          frac=kv_bytes_layer * wl.layers / (t_all * 1e-3) / 1e9 / peaks["hbm"],
                          note="metadata launch + one attention launch for all layers, CUDA events around the call")
        assert cache.status() == binding.OK

    # ---- end to end through the host-buffer entry points -----------------------------------------
    e2e = None
    e2e_all_layers = None
    if want_e2e:
        hin = [StepInputs(wl, stream, *next_step_schedule(stream, wl), host=True) for _ in range(3)]
        e2e_steps = min(args.steps, 5)

        def timed_host(fn):
            fn(cache, wl, hin[0])
            barrier()
            t0 = time.perf_counter()
            for i in range(e2e_steps):
                fn(cache, wl, hin[1 + i % 2])
            torch.cuda.synchronize()
            return max_over_ranks((time.perf_counter() - t0) / e2e_steps, world)

        lay_s = timed_host(run_step_host_layered)
        all_s = timed_host(run_step_host)
        e2e = dict(value=whole_job_value(world, frames_per_step, lay_s * 1e3), unit="frames/s", ms_per_step=lay_s * 1e3,
                   h2d_bytes_per_step=hin[1].h2d_bytes(), d2h_bytes_per_step=hin[1].d2h_bytes(),
                   api="svlm_cache_append_host / svlm_attend_host / svlm_decode_step_host, one call per layer as in `value` "
                       "(each attention call returns with its output in host memory), pinned host buffers")
        e2e_all_layers = dict(value=whole_job_value(world, frames_per_step, all_s * 1e3), unit="frames/s", ms_per_step=all_s * 1e3,
                              api="the same entry points with all layers per call (layer = -1): the chunk prefill pipelines the "
                                  "layers' copies, a generated token is one launch")

    elapsed_ms = max_over_ranks(elapsed_ms, world)
    ms_per_step = elapsed_ms / args.steps

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        info = oracle_sample(wl, layers=3)
        cpu = dict(value=frames_per_step / info["step_seconds"], unit="frames/s", cores=info["cores"], kind="oracle",
                   sample=info["sample"], est_ms_per_step=info["step_seconds"] * 1e3,
                   measured_seconds=info["measured_seconds"])

    if rank == 0:
        third = max(1, args.steps // 3)
        line = dict(base, value=whole_job_value(world, frames_per_step, ms_per_step), ms_per_step=ms_per_step, config=config,
                    roofline=roofline, cpu_baseline=cpu, e2e=e2e, gpu_launches=int(gpu_launches), clocks=clocks,
                    kernels=kernels, decode_tok_s=1e3 / decode_token_ms,
                    decode_all_layers_one_launch=all_layers, e2e_all_layers_per_call=e2e_all_layers,
                    step_ms=dict(min=min(step_ms), median=statistics.median(step_ms), max=max(step_ms),
                                 first_third=statistics.median(step_ms[:third]),
                                 last_third=statistics.median(step_ms[-third:])),
                    state=dict(fill_chunks=fill_chunks, kept_tokens=kept, cuda_graph=bool(graphs)))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
