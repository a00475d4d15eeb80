#!/usr/bin/env python
"""Benchmark of the chunk-attention hot path on B200.

A step is one pass of the whole path for one new latent chunk of one layer:
RoPE table -> fused RoPE + KV-ring append -> windowed attention, on seeded
synthetic inputs of the 1.3B-class shape (12 heads x 128, 1560 tokens per frame,
3-frame chunk, 18 cached frames + chunk = 32760 keys).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun) runs one independent replica per GPU: the path shards by
stream/head with no exchange, so scaling is weak and there is no collective on the
data path.  `--impl reference` times the CPU oracle (numpy, float64) on the host
cores instead; it is a deliberately plain program, reported as a baseline only.
"""

from __future__ import annotations

import argparse
import json
import os
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
# dram__bytes_read.sum + dram__bytes_write.sum of one window_attn launch at this workload,
# from the ncu capture summarised under profiles/ (None until captured)
ATTN_DRAM_TRAFFIC_BYTES = 286_214_400


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
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.power, self.reasons, self.max_mhz = [], [], set(), None
        self._halt = threading.Event()
        self.error = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
            names = {
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
            }
            while not self._halt.is_set():
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
                time.sleep(self.period)
        except Exception as exc:  # NVML missing: report it, never fail the benchmark
            self.error = repr(exc)

    def stop(self):
        self._halt.set()
        self.join(timeout=2.0)
        med = int(np.median(self.samples)) if self.samples else None
        out = {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
               "samples": len(self.samples),
               "power_w": round(float(np.median(self.power)), 1) if self.power else None}
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


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = W.WORKLOADS[WORKLOAD]
    cores = len(os.sched_getaffinity(0))
    oracle_sample(wl, 1, 256)  # warm numpy/BLAS
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample(wl, 1, 1024)
    times, flops, desc = [], 0.0, ""
    for _ in range(max(1, min(args.steps, 3))):
        dt, flops, desc = oracle_sample(wl, 2, 2340)
        times.append(dt)
    dt = float(np.mean(times))
    val = flops / dt / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": len(times), "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- CUDA arm
def run_ours(args):
    import torch
    import paper_2609_32518_b200 as U
    from paper_2609_32518_b200 import dist as D

    rank, local_rank, world = D.env_ranks()
    torch.cuda.set_device(local_rank)
    D.init("nccl", torch.device("cuda", local_rank))

    peaks = load_peaks()
    wl = W.WORKLOADS[args.workload]
    sh = wl.shape
    abi = U.Shape.make(sh.batch, sh.heads, sh.chunk_frames, sh.grid_h, sh.grid_w, sh.ring_frames)
    s = list(wl.measured_starts)
    wf = args.window if args.window else wl.window_frames[-1]
    sink = wl.sink_frames
    dev = torch.device("cuda", local_rank)
    bf = torch.bfloat16

    def dev_bf16(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(bf)

    # cache pre-filled with random bf16 (its content does not change the work; the parity tests
    # stream real histories through the library)
    ring_shape = (sh.batch, sink + sh.ring_frames, sh.tokens_per_frame, sh.heads, sh.head_dim)
    gen = torch.Generator(device=dev).manual_seed(1000 + wl.seed + rank)
    ring_k = torch.empty(ring_shape, dtype=bf, device=dev)
    ring_v = torch.empty_like(ring_k)
    for ring in (ring_k, ring_v):
        for slot in range(ring_shape[1]):
            ring[:, slot] = torch.randn(ring[:, slot].shape, generator=gen, device=dev).to(bf)
    cos = torch.empty((sh.batch, sh.chunk_tokens, 64), dtype=torch.float32, device=dev)
    sin = torch.empty_like(cos)
    tab_stride = 0 if len(set(s)) == 1 else sh.chunk_tokens * 64
    q_rot = torch.empty((sh.batch, sh.chunk_tokens, sh.heads, sh.head_dim), dtype=bf, device=dev)
    out = torch.empty_like(q_rot)
    distinct = sorted(set(s))

    def build_tables():
        for b, sb in enumerate(s if tab_stride else s[:1]):
            U.rope_table(abi, sb, cos[b], sin[b])

    gain_q = 1.0 + 0.1 * torch.randn(sh.heads * sh.head_dim, device=dev, generator=gen)
    gain_k = 1.0 + 0.1 * torch.randn(sh.heads * sh.head_dim, device=dev, generator=gen)

    def append(q, k, v):
        c_, s_ = (cos, sin) if tab_stride else (cos[0], sin[0])
        if tab_stride == 0:
            c_, s_ = c_.contiguous(), s_.contiguous()
        if args.rmsnorm:
            U.rmsnorm_rope_kv_append(abi, sink, s, q, k, v, gain_q, gain_k, 1e-6, c_, s_, q_rot, ring_k, ring_v,
                                     table_stream_stride=tab_stride)
        elif sink:
            U.rope_kv_append_sink(abi, sink, s, q, k, v, c_, s_, q_rot, ring_k, ring_v, table_stream_stride=tab_stride)
        else:
            U.rope_kv_append(abi, s, q, k, v, c_, s_, q_rot, ring_k, ring_v, table_stream_stride=tab_stride)

    def attend(dst=None):
        dst = out if dst is None else dst
        if sink:
            U.window_attn_sink(abi, sink, s, wf, wl.sink_attend, q_rot, ring_k, ring_v, dst)
        else:
            U.window_attn(abi, s, wf, q_rot, ring_k, ring_v, dst)

    # input sets of the measured chunk: rotated over so that the append reads cold data
    n_sets = 4
    host_sets, dev_sets = [], []
    for i in range(n_sets):
        q, k, v = W.batch_qkv(wl, s, tag=i + 10 * rank)
        hp = [torch.from_numpy(x.view(np.int16)).pin_memory() for x in (q, k, v)]
        host_sets.append(hp)
        dev_sets.append([x.to(dev).view(bf) for x in hp])
    stage = [torch.empty_like(t) for t in dev_sets[0]]
    out_host = torch.empty(out.shape, dtype=torch.int16).pin_memory()
    torch.cuda.synchronize()

    def step(i, ev=None):
        q, k, v = dev_sets[i % n_sets]
        if ev:
            ev[0].record()
        build_tables()
        if ev:
            ev[1].record()
        append(q, k, v)
        if ev:
            ev[2].record()
        attend()
        if ev:
            ev[3].record()

    # End to end: the step's q, k, v come from pinned host memory and its result goes back to
    # the host, every step.  Copies and kernels run on three streams with two staging buffers,
    # so the upload of step i+1 and the download of step i-1 overlap the kernels of step i.
    cur = torch.cuda.current_stream(dev)
    s_h2d, s_d2h = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    stages = [stage, [torch.empty_like(t) for t in stage]]
    outs2 = [out, torch.empty_like(out)]
    out_hosts = [out_host, torch.empty(out.shape, dtype=torch.int16).pin_memory()]
    ev_up = [torch.cuda.Event() for _ in range(2)]
    ev_stage_free = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    ev_down = [torch.cuda.Event() for _ in range(2)]

    def step_e2e(i):
        j = i & 1
        hq, hk, hv = host_sets[i % n_sets]
        with torch.cuda.stream(s_h2d):
            s_h2d.wait_event(ev_stage_free[j])          # the append of step i-2 has read this buffer
            for d_, h_ in zip(stages[j], (hq, hk, hv)):
                d_.view(torch.int16).copy_(h_, non_blocking=True)
            ev_up[j].record(s_h2d)
        cur.wait_event(ev_up[j])
        build_tables()
        append(stages[j][0], stages[j][1], stages[j][2])
        ev_stage_free[j].record(cur)
        cur.wait_event(ev_down[j])                      # the download of step i-2 has left this buffer
        attend(outs2[j])
        ev_out[j].record(cur)
        with torch.cuda.stream(s_d2h):
            s_d2h.wait_event(ev_out[j])
            out_hosts[j].copy_(outs2[j].view(torch.int16), non_blocking=True)
            ev_down[j].record(s_d2h)

    def drain_e2e():
        for j in range(2):
            cur.wait_event(ev_down[j])

    def barrier():
        D.barrier(dev)

    def max_over_ranks(x: float) -> float:
        return D.max_over_ranks(x, dev)

    K, Wm = args.steps, max(args.warmup, 3)
    in_mb = sh.batch * sh.chunk_tokens * sh.heads * sh.head_dim * 2 / 1e6
    kv_mb = 2 * sum(wl.keys_attended(wf)) * sh.heads * sh.head_dim * 2 / 1e6
    flush = None if kv_mb > 126 else torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
    flops_step = wl.attn_flops(wf)
    append_bytes = wl.append_bytes(len(distinct))

    # ---- device-resident timing --------------------------------------------------------
    for i in range(Wm):
        step(i)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local_rank)) if rank == 0 else None
    barrier()
    if sampler:
        sampler.start()
    launches0 = U.launch_count()
    t_begin.record()
    for i in range(K):
        if flush is not None:
            flush.fill_(i & 0xFF)   # evict L2 between timed steps (its time is inside the step total,
        step(i, evs[i])             # but outside the per-kernel event pairs)
    t_end.record()
    barrier()
    launches = U.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    total_ms = max_over_ranks(t_begin.elapsed_time(t_end))
    ms_step = total_ms / K
    t_table = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    t_append = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    attn_times = np.array([e[2].elapsed_time(e[3]) for e in evs])
    t_attn = float(attn_times.mean())
    status = U.poll_status()

    # ---- end to end: pinned host inputs in, result back to the host, every step ---------
    for i in range(4):
        step_e2e(i)
    drain_e2e()
    barrier()
    t_begin.record()
    for i in range(K):
        step_e2e(i)
    drain_e2e()                                         # the last results are on the host
    t_end.record()
    barrier()
    e2e_ms = max_over_ranks(t_begin.elapsed_time(t_end)) / K
    h2d = 3 * host_sets[0][0].numel() * 2
    d2h = out_host.numel() * 2

    D.finalize()
    if rank != 0:
        return

    attn_tflops = flops_step / (t_attn * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": world * flops_step / (ms_step * 1e-3) / 1e12, "unit": "TFLOP/s",
        "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch_per_gpu": sh.batch, "heads": sh.heads, "head_dim": 128,
                   "tokens_per_frame": sh.tokens_per_frame, "chunk_frames": sh.chunk_frames,
                   "queries": sh.chunk_tokens, "keys": wl.keys_attended(wf), "ring_frames": sh.ring_frames,
                   "window_frames": wf, "sink_frames": wl.sink_attend, "parallelism": f"replicas x{world}",
                   "l2": f"K/V read per launch {kv_mb:.0f} MB, append inputs rotate over {n_sets} sets "
                         f"({n_sets * 3 * in_mb:.0f} MB); L2 is 126 MB"
                         + ("" if kv_mb > 126 else "; an L2 flush (256 MB write) runs between timed steps")},
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
                     "traffic": ATTN_DRAM_TRAFFIC_BYTES if (args.workload == WORKLOAD and not args.window) else None},
        "append_roofline": {"kernel": "rmsnorm_rope_kv_append_kernel" if args.rmsnorm else "rope_kv_append_kernel", "bound": "hbm",
                            "achieved": append_bytes / (t_append * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                            "unit": "GB/s", "frac": append_bytes / (t_append * 1e-3) / 1e9 / peaks["hbm_gbs"],
                            "peak_source": f"{peaks['source']} copy", "bytes": append_bytes},
        "e2e": {"value": world * flops_step / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches), "device_status": status, "clocks": clocks,
        "context": "paper end-to-end: 50 FPS on one H100, 77 FPS on GB200 (whole pipeline, not this metric)",
    }
    if flush is not None:
        # the flush sits inside the whole-step time: report the step as the sum of its kernels instead
        ms_step = (t_table + t_append + t_attn)
        line["ms_per_step"] = ms_step
        line["us_per_layer_chunk"] = ms_step * 1e3
        line["value"] = world * flops_step / (ms_step * 1e-3) / 1e12
    if not args.no_cpu_baseline and world == 1 and args.workload == WORKLOAD:
        cores = len(os.sched_getaffinity(0))
        oracle_sample(wl, 1, 256)
        dt, fl, desc = oracle_sample(wl, wl.shape.heads, wl.shape.chunk_tokens)
        line["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                                "sample": desc, "seconds": dt}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(W.WORKLOADS),
                    help="configuration to time (default: the 1.3B-class shape the metric is quoted on)")
    ap.add_argument("--rmsnorm", action="store_true",
                    help="use the append with the q/k RMS norm fused in (not the default path)")
    ap.add_argument("--window", type=int, default=0, help="window length in frames (default: the workload's)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
