#!/usr/bin/env python
"""Benchmark of the chunk-attention hot path on B200.

A step is one pass of the whole path for one new latent chunk of one layer:
RoPE table -> fused RoPE + KV-ring append -> windowed attention, on seeded
synthetic inputs of the 1.3B-class shape (12 heads x 128, 1560 tokens per frame,
3-frame chunk, 18 cached frames + chunk = 32760 keys).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

`--gpus N` with N > 1 starts N ranks by itself (one process per GPU) unless a launcher
already did.  The path shards with no exchange, so the ranks never talk on the data path:
`--parallel replicas` (default) gives every GPU the whole workload (weak scaling),
`--parallel heads` gives every GPU its share of the heads and of the cache (strong scaling).
`--impl reference` times the CPU oracle (numpy, float64) on the host cores instead; it is a
deliberately plain program, reported as a baseline only.

Timing protocol: CUDA events on the launching stream; every step works on the next of several
complete working sets (inputs, q_out, cache, output), more than twice the L2 in total, so that no
kernel finds its inputs or the lines it writes in L2 from an earlier step; a second, seconds-long
leg of back-to-back steps gives the sustained figure under the power cap; SM clock, power and
throttle reasons are sampled through NVML during both legs.
"""

from __future__ import annotations

import argparse
import json
import math
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "windowed-attn TFLOP/s at 1.3B-class shape (whole layer-chunk step: table+append+attention)"
WORKLOAD = "cfg2"
L2_BYTES = 126e6
# dram__bytes_read.sum + dram__bytes_write.sum of one window_attn launch at cfg2 from the ncu
# capture summarised in profiles/window_attn_cfg2_ncu_full.txt, and the range seen over all
# captures of that kernel at that workload (the L2 state at the start of the launch differs)
ATTN_DRAM_TRAFFIC = {"bytes": 401_243_392, "capture": "profiles/window_attn_cfg2_ncu_full.txt",
                     "range_over_captures_mb": [286, 402],
                     "note": "cold L2 (every step on another working set); 286 MB when the cache of the step before is reused"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock, power and throttle reasons of one GPU through NVML, as fast as `period_s`
    allows, with a host time stamp per sample so that a window of the run can be summarised."""

    def __init__(self, index: int, period_s: float = 0.001):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.t, self.mhz, self.power, self.mask = [], [], [], []
        self.max_mhz = None
        self._halt = threading.Event()
        self.ready = threading.Event()     # set after the first sample (NVML start-up can take a while)
        self.error = None
        self.names = {}

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            self.names = {
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
            }
            n, watts = 0, 0.0
            while not self._halt.is_set():
                self.t.append(time.perf_counter())
                self.mhz.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                if n % 4 == 0:                      # a query costs about a millisecond: power less often
                    watts = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                self.power.append(watts)
                self.mask.append(int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)))
                self.ready.set()
                n += 1
                time.sleep(self.period)
        except Exception as exc:  # NVML missing: report it, never fail the benchmark
            self.error = repr(exc)
            self.ready.set()

    def stop(self):
        self._halt.set()
        self.join(timeout=2.0)

    def window(self, t0: float, t1: float):
        """Summary of the samples taken between two host times."""
        idx = [i for i, t in enumerate(self.t[:len(self.mask)]) if t0 <= t <= t1]
        reasons = set()
        for i in idx:
            for bit, name in self.names.items():
                if self.mask[i] & bit:
                    reasons.add(name)
        out = {"sm_mhz": int(np.median([self.mhz[i] for i in idx])) if idx else None,
               "sm_max_mhz": self.max_mhz, "reasons": sorted(reasons), "samples": len(idx),
               "power_w": round(float(np.median([self.power[i] for i in idx])), 1) if idx else None}
        if self.error:
            out["error"] = self.error
        return out


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            return local_rank
    return local_rank


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(wl, heads, rows_per_head, repeats=1):
    """Time the oracle on a bounded sample of the workload: the full append of the measured
    chunk once, then attention for `heads` heads x `rows_per_head` query rows over the
    whole window.  Returns (seconds, attention flops done, description)."""
    import oracle as O
    sh = wl.shape
    s = wl.measured_starts[0]
    ring = O.RingState(1, sh.ring_frames, sh.tokens_per_frame, sh.heads)
    # the history is filled with raw random keys (position-independent content is enough for timing)
    for f in range(s):
        ring.ring_k[0, f % sh.ring_frames] = W.normal_bf16((wl.seed, 900 + f), ring.ring_k.shape[2:])
        ring.ring_v[0, f % sh.ring_frames] = W.normal_bf16((wl.seed, 950 + f), ring.ring_v.shape[2:])
    q, k, v = W.batch_qkv(wl, [s])
    t0 = time.perf_counter()
    for _ in range(repeats):
        cos, sin = O.rope_table(s, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.bands, sh.rope_base)
        q_rot = O.rope_kv_append(ring, [s], q, k, v, cos, sin)
        rows = np.arange(min(rows_per_head, sh.chunk_tokens))
        O.window_attn(ring, [s], wl.window_frames[-1], q_rot, sh.chunk_frames, rows=rows,
                      heads=list(range(heads)))
    dt = (time.perf_counter() - t0) / repeats
    S = wl.keys_attended(wl.window_frames[-1])[0]
    flops = 4.0 * len(rows) * S * sh.head_dim * heads
    desc = (f"{WORKLOAD}: full table+append of the chunk, attention for {heads} of {sh.heads} heads x "
            f"{len(rows)} of {sh.chunk_tokens} query rows over all {S} keys")
    return dt, flops, desc


def reference_sample_size(steps: int, warmup: int):
    """(heads, query rows per head) of one reference step: the largest sample of the table whose
    steps + warmup repetitions stay near two and a half minutes on a few host cores."""
    per_step = 150.0 / max(1, steps + warmup)
    for seconds, heads, rows in ((8.0, 2, 2340), (4.0, 1, 2340), (2.0, 1, 1024)):
        if per_step >= seconds:
            return heads, rows
    return 1, 256


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = W.WORKLOADS[WORKLOAD]
    cores = len(os.sched_getaffinity(0))
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    heads, rows = reference_sample_size(steps, warmup)
    for _ in range(warmup):
        oracle_sample(wl, heads, rows)
    times, flops, desc = [], 0.0, ""
    for _ in range(steps):
        dt, flops, desc = oracle_sample(wl, heads, rows)
        times.append(dt)
    dt = float(np.mean(times))
    val = flops / dt / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def oracle_compare(wl, wf, got_ring_k, got_ring_v, got_out, budget_s=30.0):
    """The CPU baseline leg: the oracle runs the workload's history, the measured chunk and the
    attention from the same host inputs the CUDA arm used for working set 0 (its own table, its
    own cache), is timed, and what it computed is compared with what the GPU produced.
    got_*: uint16 bit arrays copied back from the GPU.  Full comparison when the oracle's
    attention fits the time budget, else a stratified sample of heads and rows."""
    import oracle as O
    sh = wl.shape
    cores = len(os.sched_getaffinity(0))
    starts = list(wl.measured_starts)
    if wl.sink_frames:
        state = O.SinkRingState(sh.batch, wl.sink_frames, sh.ring_frames, sh.tokens_per_frame, sh.heads)
        ring_k, ring_v = state.cache_k, state.cache_v
    else:
        state = O.RingState(sh.batch, sh.ring_frames, sh.tokens_per_frame, sh.heads)
        ring_k, ring_v = state.ring_k, state.ring_v

    def append(st_, q, k, v):
        tabs = [O.rope_table(s_, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.bands, sh.rope_base) for s_ in st_]
        cos, sin = np.stack([t[0] for t in tabs]), np.stack([t[1] for t in tabs])
        if wl.sink_frames:
            return O.rope_kv_append_sink(state, st_, q, k, v, cos, sin)
        return O.rope_kv_append(state, st_, q, k, v, cos, sin)

    for st_ in history_schedule(wl):
        append(st_, *W.batch_qkv(wl, st_))
    q, k, v = W.batch_qkv(wl, starts, tag=0)
    t0 = time.perf_counter()
    q_rot = append(starts, q, k, v)
    t_append = time.perf_counter() - t0
    # sample: everything if the attention fits the budget at ~0.07 TFLOP/s, else a stratified subset
    est = wl.attn_flops(wf) / 0.07e12
    if est <= budget_s:
        rows, heads, mode = None, None, "full"
    else:
        heads = sorted({0, sh.heads // 2, sh.heads - 1})
        per_tile = 8
        while per_tile > 2 and est * len(heads) / sh.heads * per_tile / 128 > budget_s:
            per_tile //= 2
        rows, mode = W.sample_rows(sh.chunk_tokens, per_tile=per_tile), "sampled"
    t0 = time.perf_counter()
    if wl.sink_frames:
        ref = O.window_attn_sink(state, starts, wf, wl.sink_attend, q_rot, sh.chunk_frames, rows=rows, heads=heads)
    else:
        ref = O.window_attn(state, starts, wf, q_rot, sh.chunk_frames, rows=rows, heads=heads)
    t_attn = time.perf_counter() - t0
    n_rows = sh.chunk_tokens if rows is None else len(rows)
    n_heads = sh.heads if heads is None else len(heads)
    flops = sum(4.0 * n_rows * S * sh.head_dim * n_heads for S in wl.keys_attended(wf))
    got = got_out if rows is None else got_out[:, rows]
    if heads is not None:
        got = got[:, :, heads]
    got = O.bf16_bits_to_f32(got).astype(np.float64)
    err = np.abs(got - ref)
    desc = (f"{wl.name}: history + append of the chunk ({t_append:.2f} s), attention for {n_heads} of {sh.heads} "
            f"heads x {n_rows} of {sh.chunk_tokens} query rows x {sh.batch} stream(s) over the whole window")
    return {"value": flops / t_attn / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
            "sample": desc, "seconds": t_attn, "append_seconds": t_append,
            "compared": {"mode": mode, "max_abs": float(err.max()), "mean_abs": float(err.mean()),
                         "rel_l2": float(np.linalg.norm(got - ref) / np.linalg.norm(ref)),
                         "ring_mismatches": int((got_ring_k != ring_k).sum()) + int((got_ring_v != ring_v).sum()),
                         "ring_elements": int(2 * ring_k.size),
                         "note": "the cache is bit-exact wherever the library's own table equals the oracle's "
                                 "(a last-bit difference of a table entry can move a few bf16 results)"}}


def history_schedule(wl):
    """Start frames, per stream, of the appends that come before the measured chunk: streams
    advance together; a stream whose history is shorter repeats its last chunk (an overwrite)."""
    depth = max(len(h) for h in wl.history_starts)
    out = []
    for i in range(depth):
        out.append([h[min(i, len(h) - 1)] if len(h) else wl.measured_starts[b]
                    for b, h in enumerate(wl.history_starts)])
    return out


# --------------------------------------------------------------------------- CUDA arm
def run_ours(args):
    import torch
    import paper_2609_32518_b200 as U
    from paper_2609_32518_b200 import dist as D

    rank, local_rank, world = D.env_ranks()
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if torch.cuda.device_count() <= local_rank:
        raise SystemExit(f"bench.py: rank {rank} has no GPU (visible devices: {torch.cuda.device_count()})")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    D.init("nccl", dev)

    peaks = load_peaks()
    wl_full = W.WORKLOADS[args.workload]
    # --parallel heads: this rank owns a contiguous share of the heads and their cache slices
    my_heads = list(D.shard_heads(wl_full.shape.heads, rank, world)) if args.parallel == "heads" else None
    wl = wl_full if my_heads is None else W.with_heads(wl_full, len(my_heads))
    sh = wl.shape
    abi = U.Shape.make(sh.batch, sh.heads, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.ring_frames)
    s = list(wl.measured_starts)
    wf = args.window if args.window else wl.window_frames[-1]
    sink = wl.sink_frames
    bf = torch.bfloat16
    compare = (not args.no_cpu_baseline) and world == 1 and my_heads is None and not args.rmsnorm

    flops_step = wl.attn_flops(wf)
    distinct = sorted(set(s))
    append_bytes = wl.append_bytes(len(distinct))
    # complete working sets, rotated: more than twice the L2 of append traffic in total, at least 4
    n_sets = max(4, int(math.ceil(2.2 * L2_BYTES / append_bytes)))
    n_sets = min(n_sets, 64)

    ring_shape = (sh.batch, sink + sh.ring_frames, sh.tokens_per_frame, sh.heads, sh.head_dim)
    act_shape = (sh.batch, sh.chunk_tokens, sh.heads, sh.head_dim)
    gen = torch.Generator(device=dev).manual_seed(1000 + wl.seed + rank)
    tab_stride = 0 if len(distinct) == 1 else sh.chunk_tokens * 64
    cos = torch.empty((sh.batch if tab_stride else 1, sh.chunk_tokens, 64), dtype=torch.float32, device=dev)
    sin = torch.empty_like(cos)
    gain_q = 1.0 + 0.1 * torch.randn(sh.heads * sh.head_dim, device=dev, generator=gen)
    gain_k = 1.0 + 0.1 * torch.randn(sh.heads * sh.head_dim, device=dev, generator=gen)

    def build_tables():
        for b, sb in enumerate(s if tab_stride else s[:1]):
            U.rope_table(abi, sb, cos[b], sin[b])

    def append(starts, q, k, v, q_rot, ring_k, ring_v):
        if args.rmsnorm:
            U.rmsnorm_rope_kv_append(abi, sink, starts, q, k, v, gain_q, gain_k, 1e-6, cos, sin, q_rot, ring_k,
                                     ring_v, table_stream_stride=tab_stride)
        elif sink:
            U.rope_kv_append_sink(abi, sink, starts, q, k, v, cos, sin, q_rot, ring_k, ring_v,
                                  table_stream_stride=tab_stride)
        else:
            U.rope_kv_append(abi, starts, q, k, v, cos, sin, q_rot, ring_k, ring_v, table_stream_stride=tab_stride)

    def attend(q_rot, ring_k, ring_v, dst):
        if sink:
            U.window_attn_sink(abi, sink, s, wf, wl.sink_attend, q_rot, ring_k, ring_v, dst)
        else:
            U.window_attn(abi, s, wf, q_rot, ring_k, ring_v, dst)

    def upload(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(bf)

    # ---- working sets ---------------------------------------------------------------------
    # set 0 holds the workload's real history, streamed through the library, so that its result
    # can be compared with the oracle's; the caches of the other sets are random bf16 (content
    # does not change the work)
    sets, host_sets = [], []
    for i in range(n_sets):
        ring_k = torch.empty(ring_shape, dtype=bf, device=dev)
        ring_v = torch.empty_like(ring_k)
        if i == 0 and compare:
            ring_k.view(torch.int16).fill_(0x7FC1)
            ring_v.view(torch.int16).fill_(0x7FC1)
            tmp_q = torch.empty(act_shape, dtype=bf, device=dev)
            for st_ in history_schedule(wl):
                for b, sb in enumerate(st_ if tab_stride else st_[:1]):
                    U.rope_table(abi, sb, cos[b], sin[b])
                hq, hk, hv = W.batch_qkv(wl, st_)
                append(st_, upload(hq), upload(hk), upload(hv), tmp_q, ring_k, ring_v)
            del tmp_q
        else:
            for ring in (ring_k, ring_v):
                for slot in range(ring_shape[1]):
                    ring[:, slot] = torch.randn(ring[:, slot].shape, generator=gen, device=dev).to(bf)
        q, k, v = W.batch_qkv(wl, s, tag=i + 100 * rank)
        if i < 4:
            host_sets.append([torch.from_numpy(x.view(np.int16)).pin_memory() for x in (q, k, v)])
        sets.append({"q": upload(q), "k": upload(k), "v": upload(v), "ring_k": ring_k, "ring_v": ring_v,
                     "q_rot": torch.empty(act_shape, dtype=bf, device=dev),
                     "out": torch.empty(act_shape, dtype=bf, device=dev)})
    set_mb = sum(t.numel() * t.element_size() for t in sets[0].values()) / 1e6
    torch.cuda.synchronize()

    def step(i, ev=None):
        ws = sets[i % n_sets]
        if ev:
            ev[0].record()
        build_tables()
        if ev:
            ev[1].record()
        append(s, ws["q"], ws["k"], ws["v"], ws["q_rot"], ws["ring_k"], ws["ring_v"])
        if ev:
            ev[2].record()
        attend(ws["q_rot"], ws["ring_k"], ws["ring_v"], ws["out"])
        if ev:
            ev[3].record()

    def barrier():
        D.barrier(dev)

    def max_over_ranks(x: float) -> float:
        return D.max_over_ranks(x, dev)

    K, Wm = args.steps, max(args.warmup, 3)
    sampler = ClockSampler(physical_gpu_index(local_rank)) if rank == 0 else None
    if sampler:
        sampler.start()
        sampler.ready.wait(timeout=10.0)   # the short first leg must not be over before NVML is up

    def timed_leg(n_steps):
        """n_steps back-to-back steps with per-kernel events; returns (total ms, per-kernel arrays,
        host time window, launches)."""
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_steps)]
        t_b, t_e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        l0, h0 = U.launch_count(), time.perf_counter()
        t_b.record()
        for i in range(n_steps):
            step(i, evs[i])
        t_e.record()
        barrier()
        h1 = time.perf_counter()
        total = max_over_ranks(t_b.elapsed_time(t_e))
        per = np.array([[e[j].elapsed_time(e[j + 1]) for j in range(3)] for e in evs])   # ms
        return total, per, (h0, h1), U.launch_count() - l0

    # ---- device-resident timing: K steps ------------------------------------------------
    for i in range(Wm):
        step(i)
    total_ms, per, win, launches = timed_leg(K)
    ms_step = total_ms / K
    t_table, t_append, t_attn = (float(x) for x in per.mean(axis=0))
    attn_times = per[:, 2]
    clocks = sampler.window(*win) if sampler else None
    status = U.poll_status()

    # ---- sustained: seconds of back-to-back steps ----------------------------------------
    sustained = None
    if args.sustain_seconds > 0:
        n_long = int(min(max(math.ceil(args.sustain_seconds * 1e3 / ms_step), K), 20000))
        total_l, per_l, win_l, _ = timed_leg(n_long)
        tail = per_l[n_long // 2:]                         # the second half: clocks have settled
        clk_l = sampler.window(win_l[0] + 0.5 * (win_l[1] - win_l[0]), win_l[1]) if sampler else {}
        us = float(tail[:, 2].mean()) * 1e3
        tf = flops_step / (us * 1e-6) / 1e12
        sustained = {"steps": n_long, "seconds": total_l / 1e3, "us": us, "tflops": tf,
                     "frac": tf / peaks["bf16_tflops"], "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"],
                     "ms_per_step": total_l / n_long, "append_us": float(tail[:, 1].mean()) * 1e3,
                     "sm_mhz_median": clk_l.get("sm_mhz"), "power_w": clk_l.get("power_w"),
                     "reasons": clk_l.get("reasons"), "clock_samples": clk_l.get("samples"),
                     "mcycles_per_step": (us * clk_l["sm_mhz"] / 1e6) if clk_l.get("sm_mhz") else None}

    # ---- the same steps on one working set over and over: what the append gains when the lines it
    # writes (and the attention's inputs) are still in L2 from the step before -----------------
    def warm_leg(n=20):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n)]
        for i in range(n):
            step(0, ev[i])
        torch.cuda.synchronize()
        return np.array([[e[j].elapsed_time(e[j + 1]) for j in range(3)] for e in ev[2:]]).mean(axis=0) * 1e3
    warm_us = warm_leg()

    # ---- end to end: pinned host inputs in, result back to the host, every step ---------
    # Copies and kernels run on three streams with two staging buffers, so the upload of step
    # i+1 and the download of step i-1 overlap the kernels of step i.
    cur = torch.cuda.current_stream(dev)
    s_h2d, s_d2h = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    stages = [[torch.empty(act_shape, dtype=bf, device=dev) for _ in range(3)] for _ in range(2)]
    outs2 = [torch.empty(act_shape, dtype=bf, device=dev) for _ in range(2)]
    out_hosts = [torch.empty(act_shape, dtype=torch.int16).pin_memory() for _ in range(2)]
    ev_up = [torch.cuda.Event() for _ in range(2)]
    ev_stage_free = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    ev_down = [torch.cuda.Event() for _ in range(2)]

    def step_e2e(i):
        j = i & 1
        ws = sets[i % n_sets]
        with torch.cuda.stream(s_h2d):
            s_h2d.wait_event(ev_stage_free[j])          # the append of step i-2 has read this buffer
            for d_, h_ in zip(stages[j], host_sets[i % len(host_sets)]):
                d_.view(torch.int16).copy_(h_, non_blocking=True)
            ev_up[j].record(s_h2d)
        cur.wait_event(ev_up[j])
        build_tables()
        append(s, stages[j][0], stages[j][1], stages[j][2], ws["q_rot"], ws["ring_k"], ws["ring_v"])
        ev_stage_free[j].record(cur)
        cur.wait_event(ev_down[j])                      # the download of step i-2 has left this buffer
        attend(ws["q_rot"], ws["ring_k"], ws["ring_v"], outs2[j])
        ev_out[j].record(cur)
        with torch.cuda.stream(s_d2h):
            s_d2h.wait_event(ev_out[j])
            out_hosts[j].copy_(outs2[j].view(torch.int16), non_blocking=True)
            ev_down[j].record(s_d2h)

    def drain_e2e():
        for j in range(2):
            cur.wait_event(ev_down[j])

    for i in range(4):
        step_e2e(i)
    drain_e2e()
    barrier()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for i in range(K):
        step_e2e(i)
    drain_e2e()                                         # the last results are on the host
    t_end.record()
    barrier()
    e2e_ms = max_over_ranks(t_begin.elapsed_time(t_end)) / K
    h2d = 3 * host_sets[0][0].numel() * 2
    d2h = out_hosts[0].numel() * 2

    # ---- what the GPU computed for working set 0, for the comparison with the oracle ------
    got = None
    if compare:
        ws = sets[0]
        hq, hk, hv = W.batch_qkv(wl, s, tag=0)
        build_tables()
        append(s, upload(hq), upload(hk), upload(hv), ws["q_rot"], ws["ring_k"], ws["ring_v"])
        attend(ws["q_rot"], ws["ring_k"], ws["ring_v"], ws["out"])
        torch.cuda.synchronize()
        got = tuple(t.view(torch.int16).cpu().numpy().view(np.uint16) for t in (ws["ring_k"], ws["ring_v"], ws["out"]))
    if sampler:
        sampler.stop()
    D.finalize()
    if rank != 0:
        return

    attn_tflops = flops_step / (t_attn * 1e-3) / 1e12
    total_flops = world * flops_step if my_heads is None else wl_full.attn_flops(wf)
    default_cfg = args.workload == WORKLOAD and not args.window and my_heads is None
    line = {
        "metric": METRIC, "value": total_flops / (ms_step * 1e-3) / 1e12, "unit": "TFLOP/s",
        "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak" if my_heads is None else "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch_per_gpu": sh.batch, "heads_per_gpu": sh.heads, "head_dim": 128,
                   "tokens_per_frame": sh.tokens_per_frame, "chunk_frames": sh.chunk_frames,
                   "queries": sh.chunk_tokens, "keys": wl.keys_attended(wf), "ring_frames": sh.ring_frames,
                   "window_frames": wf, "sink_frames": wl.sink_attend,
                   "parallelism": f"replicas x{world}" if my_heads is None else f"heads split over {world}",
                   "l2": f"every step works on the next of {n_sets} complete working sets (inputs, q_out, cache, "
                         f"output: {set_mb:.0f} MB each, append traffic {n_sets * append_bytes / 1e6:.0f} MB in all; "
                         f"L2 is 126 MB), no flush"},
        "us_per_layer_chunk": ms_step * 1e3,
        "kernels_us": {"rope_table": t_table * 1e3, "rope_kv_append": t_append * 1e3,
                       "window_attn": t_attn * 1e3},
        "window_attn_us_median_min": [float(np.median(attn_times)) * 1e3, float(attn_times.min()) * 1e3],
        "roofline": {"kernel": "window_attn_kernel", "bound": "tensor", "achieved": attn_tflops,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": attn_tflops / peaks["bf16_tflops"],
                     "peak_source": f"{peaks['source']} cuBLAS bf16 burst",
                     "frac_of_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": attn_tflops / 2250.0,
                     "traffic": ATTN_DRAM_TRAFFIC["bytes"] if default_cfg else None,
                     "traffic_source": ATTN_DRAM_TRAFFIC if default_cfg else None,
                     "mcycles_per_launch": (t_attn * 1e3 * clocks["sm_mhz"] / 1e6) if clocks and clocks.get("sm_mhz") else None,
                     "sustained": sustained},
        "append_roofline": {"kernel": "rmsnorm_rope_kv_append_token_kernel" if args.rmsnorm else "rope_kv_append_kernel",
                            "bound": "hbm", "achieved": append_bytes / (t_append * 1e-3) / 1e9,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": append_bytes / (t_append * 1e-3) / 1e9 / peaks["hbm_gbs"],
                            "peak_source": f"{peaks['source']} copy", "bytes": append_bytes,
                            "protocol": "timed inside the step, every step on the next working set (cold inputs, "
                                        "cold outputs); warm_* = the same step repeated on one working set",
                            "warm_us": float(warm_us[1]),
                            "warm_frac": append_bytes / float(warm_us[1]) / 1e3 / peaks["hbm_gbs"],
                            "warm_window_attn_us": float(warm_us[2])},
        "e2e": {"value": total_flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches), "device_status": status, "clocks": clocks,
        "context": "paper end-to-end: 50 FPS on one H100, 77 FPS on GB200 (whole pipeline, not this metric)",
    }
    if got is not None:
        line["cpu_baseline"] = oracle_compare(wl, wf, *got)
    print(json.dumps(line))


def self_launch(args) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks, one per GPU, on this node."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = relaunch_command(args.gpus, port, sys.argv[1:])
    return subprocess.call(cmd)


def relaunch_command(n: int, port: int, argv):
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(W.WORKLOADS),
                    help="configuration to time (default: the 1.3B-class shape the metric is quoted on)")
    ap.add_argument("--rmsnorm", action="store_true",
                    help="use the append with the q/k RMS norm fused in (not the default path)")
    ap.add_argument("--window", type=int, default=0, help="window length in frames (default: the workload's)")
    ap.add_argument("--parallel", choices=["replicas", "heads"], default="replicas",
                    help="what N > 1 GPUs do: each the whole workload, or each its share of the heads")
    ap.add_argument("--sustain-seconds", type=float, default=2.0,
                    help="length of the second, sustained timing leg (0 switches it off)")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(self_launch(args))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
