#!/usr/bin/env python
"""Benchmark of the quantize -> integer aggregate -> reconstruct hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl reference]

One step = one pass of the whole path (agree scale, [select + share scale index,] encode, fused
aggregate+decode) over one batch of synthetic gradients of M workers.  The default workload is
the largest single-GPU configuration, c5.  The metric is gradient
GB/s: bytes of gradient input (M * d * sizeof(element)) per second of the whole step.
The path does not shard: with N GPUs every rank runs an independent replica ("replicas only")
and the value is the sum over ranks; timing is the max over ranks of device-event time.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead (test
infrastructure, executed here only as the reported baseline).
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
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2109_12497_b200 import workloads as wl  # noqa: E402

METRIC = "gradient GB/s through encode+aggregate+decode; % of B200 HBM roofline"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0          # earlier measurement on this machine, used only without MEASURED_PEAKS.json

# DRAM traffic of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum under ncu) in
# bytes per coordinate, from captures of a small case of the same recipe summarised under
# profiles/ (the full workloads are too large to capture); a launch at full size is taken as
# bytes per coordinate * d, since every byte of these kernels belongs to a coordinate.
# Keyed by (workload, kernel); absent = not captured.
NCU_TRAFFIC_BYTES_PER_COORD = {
    ("c5", "select_encode_decode"): 27.64,   # profiles/kernel_select_encode_decode_c5_small_ncu.md: 1381.8 MB for d = 50,000,000
    ("c5", "encode_decode"): 27.39,   # profiles/kernel_encode_decode_c5_small_ncu.md: 1369.4 MB for d = 50,000,000
    ("c5", "encode"): 23.39,      # profiles/kernel_encode_c5_small_ncu.md: 1169.7 MB for d = 50,000,000
    ("c2", "encode"): 38.15,      # profiles/kernel_encode_c2_rng32_ncu.md: 975.7 MB at full size (d = 25,557,032)
}


# ALU-pipe instructions per coordinate and worker of kernels that the ALU pipe, not memory, bounds
# (ncu's per-opcode counts in the same summaries: LOP3, IADD3, PRMT, SHF, ISETP, VIMNMX3, SEL), and the
# pipe's peak: 16 lanes per scheduler (measured: such an instruction occupies its scheduler's pipe for
# 2 cycles), 4 schedulers per SM, 148 SMs, at the SM clock sampled during the run.
NCU_ALU_OPS_PER_COORD_WORKER = {
    ("c5", "select_encode_decode"): 9.99,    # profiles/kernel_select_encode_decode_c5_small_ncu.md
}
ALU_LANES_PER_SM = 64
SM_COUNT = 148


def hbm_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------------
# algorithmic bytes per launch of each kernel (what the method must move)
# ---------------------------------------------------------------------------------------------

def algorithmic_bytes(w: wl.Workload) -> dict:
    e = 4 if w.dtype == wl.F32 else 2
    lev = {"i8": 1.0, "i4x2": 0.5, "i2x4": 0.25, "i6p": 0.75}[w.fmt]
    ib = w.idx_bits / 8.0
    M, d = w.M, w.d
    b = {"agree_scale": e * M * d}
    if w.quantizer == "multi":
        b["select_scale"] = e * M * d + ib * d
        b["encode"] = (e + lev + ib) * M * d          # the shared index counted once per worker
        b["select_encode"] = (e + lev) * M * d + ib * d   # one call: gradients read once, index written once
    else:
        b["encode"] = (e + lev) * M * d
    b["aggregate_decode"] = lev * M * d + ib * d + 4 * d
    b["encode_decode"] = b["encode"] + 4 * d          # one call: the levels are written but not read back
    if w.quantizer == "multi":
        b["select_encode_decode"] = b["select_encode"] + 4 * d      # gradients read once, index, levels, average written
    return b


def step_roofline(w: wl.Workload, ms: float, peak_gbs: float) -> dict:
    """The whole step against the sum of its stages' algorithmic bytes moved at the HBM peak."""
    ab = algorithmic_bytes(w)
    total = sum(ab[k] for k in stages_of(w))
    min_ms = total / peak_gbs / 1e6
    return {"algorithmic_MB": round(total / 1e6, 1), "min_ms_at_peak": round(min_ms, 5), "frac": round(min_ms / ms, 4),
            "ceiling_gradient_GBps": round(w.in_bytes / min_ms / 1e6, 1)}


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict | None:
        if self.proc is None:
            return None
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------

def encoder_decodes(w) -> bool:
    """Whether the step's encoder also aggregates and reconstructs (uq_encode_decode as one kernel:
    int8 levels, 16-bit draws, at most 8 workers; pipeline.Quantizer.fused_decode says the same of its object)."""
    return w.fmt == "i8" and w.M <= 8 and w.rng_bits == 16


def stages_of(w):
    """The calls uq_step makes for this workload (without the integer sums among its outputs)."""
    if w.quantizer == "multi" and encoder_decodes(w):
        return ["agree_scale", "select_encode_decode"]      # the encoder also selects: two calls do the step
    head = ["agree_scale", "select_scale"] if w.quantizer == "multi" else ["agree_scale"]
    return head + (["encode_decode"] if encoder_decodes(w) else ["encode", "aggregate_decode"])


def stage_calls(q, g):
    """{stage: function of the seed} for the separate calls of the step."""
    calls = {"agree_scale": lambda seed: q.agree_scale(g), "aggregate_decode": lambda seed: q.aggregate_decode()}
    calls["encode"] = lambda seed: q.encode(g, seed)
    calls["encode_decode"] = lambda seed: q.encode_decode(g, seed)
    if q.multi:
        calls["select_encode_decode"] = lambda seed: q.select_encode_decode(g, seed)
    if q.multi:
        calls["select_scale"] = lambda seed: q.select_scale(g)
    return calls


def run_stages(q, g, seed, events=None, stages=None):
    """One step; events (if given) is a list of len(stages)+1 CUDA events recorded around the stages.
    Without events the step is the one call a user makes (Quantizer.step)."""
    import torch
    if not events:
        q.step(g, seed)
        return
    st = torch.cuda.current_stream()
    calls = stage_calls(q, g)
    events[0].record(st)
    for k, name in enumerate(stages):
        calls[name](seed)
        events[k + 1].record(st)


def time_device_resident(q, g, w, steps, warmup, barrier):
    """(ms per step, {stage: mean ms}) with inputs resident in HBM, timed with CUDA events.
    The step time comes from a region that holds nothing but the K steps (an event recorded
    between two kernels would keep the second from being scheduled while the first drains, which
    the library's launches otherwise allow); the per-stage times (medians) come from a second pass with
    an event after every stage."""
    import torch
    st = torch.cuda.current_stream()
    stages = stages_of(w)
    for _ in range(warmup):
        run_stages(q, g, w.seed)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(); barrier()
    e0.record(st)
    for k in range(steps):
        run_stages(q, g, w.seed + k)
    e1.record(st)
    torch.cuda.synchronize(); barrier()
    total_ms = e0.elapsed_time(e1)
    # Under continuous load the board reaches its power cap after some 40 ms and every kernel slows by
    # 8-14 % (see time_sustained).  The copy that defines the HBM peak was timed as a burst, so the
    # per-stage pass is kept a burst too: the device idles first, and the pass stays below 40 ms.
    n = max(3, min(steps, 10, int(40.0 / max(total_ms / steps, 1e-3))))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(stages) + 1)] for _ in range(n)]
    time.sleep(BURST_IDLE_S)
    run_stages(q, g, w.seed, [torch.cuda.Event() for _ in range(len(stages) + 1)], stages)      # the separate calls, untimed
    for k in range(n):
        run_stages(q, g, w.seed + k, evs[k], stages)
    torch.cuda.synchronize()
    per_stage = {s: statistics.median(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(n))
                 for i, s in enumerate(stages)}
    return total_ms / steps, per_stage


NOMINAL_HBM_GBS = 8000.0    # the data-sheet figure, reported beside the measured copy rate for context
BURST_IDLE_S = 0.5          # idle time after which the power budget of a burst is available again (measured)


def time_sustained(q, g, w, ms_burst, lead_s=0.6, span_s=0.4):
    """ms per step under continuous load: steps back to back for lead_s seconds untimed, then span_s
    seconds timed.  On a B200 at its 1000 W cap this is 8-14 % above the burst figure."""
    import torch
    st = torch.cuda.current_stream()
    n_lead = max(1, int(lead_s * 1e3 / ms_burst))
    n_span = max(1, int(span_s * 1e3 / ms_burst))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    for k in range(n_lead):
        q.step(g, w.seed + k)
    e0.record(st)
    for k in range(n_span):
        q.step(g, w.seed + k)
    e1.record(st)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n_span, n_lead, n_span


def time_alone(fn, reps, sustained=False, ms_hint=1.0, lead_s=0.6, span_s=0.4):
    """Mean ms of one call of fn(seed) looped alone.  sustained: after lead_s seconds of the same
    calls untimed, over span_s seconds (the rate at the board's power cap); else a burst of reps."""
    import torch
    st = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sustained:
        n_lead = max(1, int(lead_s * 1e3 / ms_hint))
        reps = max(1, int(span_s * 1e3 / ms_hint))
    else:
        n_lead = 2
    torch.cuda.synchronize()
    for k in range(n_lead):
        fn(k)
    e0.record(st)
    for k in range(reps):
        fn(1000 + k)
    e1.record(st)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


COPY_CONTEXT_MAX_BYTES = 1300e6


def time_plain_copy(nbytes, reps=20):
    """Mean ms of a plain device copy that moves nbytes in all (nbytes / 2 read, nbytes / 2
    written; torch's copy_), reps copies back to back between two events (so that no launch latency
    is counted), warm L2.  Context for the short stages: the copy that defines the HBM peak moves
    gigabytes, and a copy of a few hundred megabytes does not get near that rate."""
    import torch
    n = max(16, int(nbytes) // 2)
    a = torch.empty(n, dtype=torch.uint8, device="cuda").fill_(1)
    b = torch.empty_like(a)
    for _ in range(3):
        b.copy_(a)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        b.copy_(a)
    e1.record()
    torch.cuda.synchronize()
    del a, b
    return e0.elapsed_time(e1) / reps


def time_end_to_end(q, g_host, out_host, g_dev, w, steps, warmup, barrier):
    """ms per step with the gradients starting in pinned host memory and the result read back.
    Every step copies its own inputs in and its own result out.  Three streams, ordered by events:
    the inputs of step k+1 arrive (copy stream, into the other of two device buffers) while the
    kernels of step k run (main stream) and the result of step k-1 is read back (a third stream;
    the two directions of the link are independent).  Kernels(k) wait for copy-in(k) and for the
    read-back of result k-1 (the output buffer is reused); copy-in(k+2) waits for kernels(k) (its
    buffer is free again)."""
    import torch
    main = torch.cuda.current_stream()
    copy, back = torch.cuda.Stream(), torch.cuda.Stream()
    bufs = [g_dev, torch.empty_like(g_dev)]
    copied = [torch.cuda.Event() for _ in range(2)]           # inputs of the step using buffer b have arrived
    computed = [torch.cuda.Event() for _ in range(2)]         # kernels of the step using buffer b have finished
    read_back = torch.cuda.Event()                            # the latest result has left the output buffer

    def one(k):
        b = k & 1
        with torch.cuda.stream(copy):
            copy.wait_event(computed[b])                      # the step that used this buffer before is done
            bufs[b].copy_(g_host, non_blocking=True)
            copied[b].record(copy)
        main.wait_event(copied[b])
        main.wait_event(read_back)
        out = q.step(bufs[b], w.seed + k)
        computed[b].record(main)
        with torch.cuda.stream(back):
            back.wait_event(computed[b])
            out_host.copy_(out, non_blocking=True)
            read_back.record(back)

    for ev in computed:
        ev.record(main)
    read_back.record(main)
    for k in range(min(warmup, 3)):
        one(k)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(); barrier()
    e0.record(main)
    copy.wait_event(e0)                                       # no copy of a timed step starts before the clock
    for k in range(steps):
        one(k)
    main.wait_event(read_back)                                # the last read-back is inside the timed region
    e1.record(main)
    torch.cuda.synchronize(); barrier()
    return e0.elapsed_time(e1) / steps


def time_encode_other_mode(q, g, w, reps):
    """Mean ms of the encode kernel alone with the other random-draw width (context: the step
    itself runs in the workload's own mode).  W and idx are those of the last step."""
    keep = q.rng_bits
    q.rng_bits = 32 if keep == 16 else 16
    try:
        return time_alone(lambda k: q.encode(g, w.seed + k), reps)
    finally:
        q.rng_bits = keep


def time_two_kernel_tail(q, g, w, reps):
    """Where the step's encoder also aggregates and reconstructs: mean ms of the encoder alone and of the
    aggregation + reconstruction kernel alone (the two calls the one replaces), each looped by itself."""
    enc = time_alone(lambda k: q.encode(g, w.seed + k), reps)
    time.sleep(BURST_IDLE_S)
    dec = time_alone(lambda k: q.aggregate_decode(), reps)
    return enc, dec


def time_fused_select_encode(q, g, w, reps):
    """Multi-scale: mean ms of selection + encoding as one call (uq_select_encode_multi: one kernel
    for M <= 8; the step runs the two streaming kernels), timed alone."""
    return time_alone(lambda k: q.select_encode(g, w.seed + k), reps)


def time_fused_select_encode_decode(q, g, w, reps):
    """Multi-scale: mean ms of everything behind the scale agreement as one call
    (uq_select_encode_decode_multi), timed alone."""
    return time_alone(lambda k: q.select_encode_decode(g, w.seed + k), reps)


def time_graph_replay(q, g, w, reps, stats=False):
    """ms per step when the step's launches are captured once in a CUDA graph and replayed: the
    figure for a working set so small that launch latency, not memory, sets the time.  stats:
    time every replay by itself and return (mean, median, min) instead of the mean of a burst.
    (A replay repeats the captured seed: a latency figure, not a training loop.)"""
    import torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        q.step(g, w.seed)                       # warm up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        q.step(g, w.seed)
    for _ in range(5):
        graph.replay()
    torch.cuda.synchronize()
    if stats:
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in evs:
            a.record()
            graph.replay()
            b.record()
        torch.cuda.synchronize()
        t = sorted(a.elapsed_time(b) for a, b in evs)
        return statistics.fmean(t), statistics.median(t), t[0]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def time_randk(w, g, K, reps):
    """GlobalRandK step on the workload's gradients: choose + gather K coordinates, the dense
    stages on the K-vector, sparse parameter update.  ms per step as stream launches and as a
    CUDA-graph replay (K is tiny, so launch latency sets the time; the replay repeats one seed
    and is a latency figure only)."""
    import torch
    from paper_2109_12497_b200.pipeline import randk_from_workload
    rq = randk_from_workload(w, K)
    theta = torch.zeros(max(w.d, 1), dtype=torch.float32, device="cuda")

    def step(seed):
        rq.gather(g, seed)
        rq.quantize(seed)
        rq.update(theta, 0.1)

    st = torch.cuda.current_stream()
    for k in range(3):
        step(k)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(st)
    for k in range(reps):
        step(100 + k)
    e1.record(st)
    torch.cuda.synchronize()
    ms_stream = e0.elapsed_time(e1) / reps
    side = torch.cuda.Stream()
    side.wait_stream(st)
    with torch.cuda.stream(side):
        step(7)
    st.wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(7)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return {"K": K, "ms_per_step": round(ms_stream, 5), "cuda_graph_ms_per_step": round(e0.elapsed_time(e1) / reps, 5),
            "kernels_per_step": rq.kernels_per_step(), "status_word": rq.status_bits(),
            "note": "choice + gather, agree-scale, [select], encode, aggregate + reconstruct, sparse update; "
                    "latency-bound (K values per worker)"}


def time_fused_update(q, w, reps):
    """Mean ms of the fused aggregate + reconstruct + SGD-with-momentum kernel alone (the levels
    are those of the last step; it replaces aggregate_decode when the caller wants the update)."""
    import torch
    st = torch.cuda.current_stream()
    theta = torch.zeros(max(w.d, 1), dtype=torch.float32, device="cuda")
    mom = torch.zeros_like(theta)
    for _ in range(2):
        q.aggregate_decode_update(theta, mom, 0.1, 0.9, 5e-4)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(st)
    for _ in range(reps):
        q.aggregate_decode_update(theta, mom, 0.1, 0.9, 5e-4)
    e1.record(st)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def l2_flush_buffer():
    import torch
    return torch.empty(256 << 20, dtype=torch.uint8, device="cuda")


LEVEL_WIRES = {"i8": 127, "i6p": 31, "i4x2": 7, "i2x4": 1}       # wire format -> levels of the smallest scale


def resolve_workload(name, d=None, rng_bits=None, levels=None):
    """The named workload, optionally at a smaller d (same recipe; used for ncu captures, which
    must stay small), with the other random-draw width, or on another level wire format (the
    scale set keeps its ratios and starts at the format's largest level)."""
    w = wl.WORKLOADS[name]
    if levels is not None and levels != w.fmt:
        import dataclasses
        s_new = LEVEL_WIRES[levels]
        w = dataclasses.replace(w, fmt=levels, s=s_new, scales=tuple(s_new * (x // w.scales[0]) for x in w.scales))
    if d is not None and d != w.d:
        import dataclasses
        w = dataclasses.replace(w, d=d, name=f"{name}@{d}")
    if rng_bits is not None:
        import dataclasses
        w = dataclasses.replace(w, rng_bits=rng_bits)
    return w


def bench_workload(w, steps, warmup, barrier, threads, want_e2e, flush_between=False, randk_K=0, sustained=False,
                   device_index=0):
    """Times one workload on the current device.  Returns a dict of raw numbers.  The clocks of
    the device are sampled over everything timed here (res["clocks"])."""
    import torch
    from paper_2109_12497_b200.pipeline import from_workload
    sampler = ClockSampler(device_index)
    sampler.start()
    np_dtype = np.float32 if w.dtype == wl.F32 else np.uint16
    if want_e2e:
        g_host = torch.empty((w.M, w.stride), dtype=torch.float32 if w.dtype == wl.F32 else torch.int16,
                             pin_memory=True)
        wl.generate(w, out=g_host.numpy().view(np_dtype), threads=threads)
    else:
        g_host = torch.from_numpy(wl.generate(w, threads=threads).view(np.float32 if w.dtype == wl.F32 else np.int16))
    if w.dtype == wl.BF16:
        g_host = g_host.view(torch.bfloat16)
    q = from_workload(w)
    g_dev = torch.empty(g_host.shape, dtype=g_host.dtype, device="cuda")
    for m in range(w.M):                       # row by row keeps the staging small for pageable memory
        g_dev[m].copy_(g_host[m])
    torch.cuda.synchronize()

    res = {"workload": w, "q": q, "g_dev": g_dev}
    if flush_between:
        # working set smaller than L2: time each step alone after overwriting L2
        flush = l2_flush_buffer()
        for _ in range(warmup):
            run_stages(q, g_dev, w.seed)
        stages = stages_of(w)
        tot, per = [], {s: [] for s in stages}
        for k in range(steps):
            flush.fill_(k & 0xFF)
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(stages) + 1)]
            if q.one_kernel:                      # the step is one kernel: nothing to time inside it
                evs[0].record()
                q.step(g_dev, w.seed + k)
                evs[-1].record()
            else:
                run_stages(q, g_dev, w.seed + k, evs, stages)
            torch.cuda.synchronize()
            tot.append(evs[0].elapsed_time(evs[-1]))
            for i, s in enumerate(stages):
                if not q.one_kernel:
                    per[s].append(evs[i].elapsed_time(evs[i + 1]))
        res["ms_cold"] = statistics.fmean(tot)
        res["stages_cold_ms"] = {s: statistics.fmean(v) for s, v in per.items() if v}
        del flush
        res["ms_graph"] = time_graph_replay(q, g_dev, w, max(steps, 20))
    res["ms"], res["stages_ms"] = time_device_resident(q, g_dev, w, steps, warmup, barrier)
    time.sleep(BURST_IDLE_S)
    if not q.one_kernel:
        # a plain copy of the same number of bytes beside every stage short enough for its size to matter
        ab = algorithmic_bytes(w)
        res["copy_same_bytes_ms"] = {s: time_plain_copy(ab[s]) for s in res["stages_ms"] if ab[s] <= COPY_CONTEXT_MAX_BYTES}
        time.sleep(BURST_IDLE_S)
    res["encode_other_ms"] = time_encode_other_mode(q, g_dev, w, min(steps, 10))
    if q.fused_decode and not q.one_kernel:
        time.sleep(BURST_IDLE_S)
        res["two_kernel_tail_ms"] = time_two_kernel_tail(q, g_dev, w, min(steps, 10))
        time.sleep(BURST_IDLE_S)
        if q.multi:       # the step's second call also selects: the calls it stands for, each looped alone
            res["alone_ms"] = {}
            for name, fn in (("select_scale", lambda k: q.select_scale(g_dev)),
                             ("encode_decode", lambda k: q.encode_decode(g_dev, w.seed + k))):
                res["alone_ms"][name] = time_alone(fn, min(steps, 10))
                time.sleep(BURST_IDLE_S)
    res["update_ms"] = time_fused_update(q, w, min(steps, 10))
    if q.multi:
        res["fused_select_ms"] = time_fused_select_encode(q, g_dev, w, min(steps, 10))
        if q.fused_decode and not q.one_kernel and "select_encode_decode" not in res["stages_ms"]:
            time.sleep(BURST_IDLE_S)
            res["fused_all_ms"] = time_fused_select_encode_decode(q, g_dev, w, min(steps, 10))
    if randk_K:
        res["randk"] = time_randk(w, g_dev, min(randk_K, w.d), 50)
        if w.quantizer == "single":               # the same choice quantized with a two-scale set (GlobalRandK-MN-TS)
            import dataclasses
            two = dataclasses.replace(w, quantizer="multi", scales=(w.s, w.s * 16), idx_bits=1)
            res["randk_two_scale"] = time_randk(two, g_dev, min(randk_K, w.d), 50)
        res["graph_stats"] = time_graph_replay(q, g_dev, w, max(steps, 20), stats=True)
    res["h2d"], res["d2h"], res["e2e_ms"] = 0, 0, None
    if want_e2e:
        out_host = torch.empty(w.d, dtype=torch.float32, pin_memory=True)
        res["e2e_ms"] = time_end_to_end(q, g_host, out_host, g_dev, w, steps, warmup, barrier)
        res["h2d"] = g_host.numel() * g_host.element_size()
        res["d2h"] = out_host.numel() * 4
    res["clocks"] = sampler.stop()           # the record of the burst figures above
    if sustained:
        # under continuous load: the whole step, then every stage looped alone
        res["sustained"] = time_sustained(q, g_dev, w, res["ms"])
        if not q.one_kernel:
            calls = stage_calls(q, g_dev)
            res["stages_sustained_ms"] = {}
            for name in stages_of(w):
                time.sleep(BURST_IDLE_S)
                res["stages_sustained_ms"][name] = time_alone(calls[name], 0, sustained=True,
                                                              ms_hint=max(res["stages_ms"][name], 1e-3))
        time.sleep(BURST_IDLE_S)
    res["status"] = q.status_bits()
    return res


def sustained_summary(w, timing):
    ms, n_lead, n_span = timing
    return {"ms_per_step": round(ms, 5), "gradient_GBps": round(w.in_bytes / ms / 1e6, 1),
            "steps_before": n_lead, "steps_timed": n_span,
            "note": "steps back to back for 0.6 s untimed, then 0.4 s timed: the rate at the board's power cap"}


def summarize(res, peak_gbs):
    w = res["workload"]
    ab = algorithmic_bytes(w)
    out = {"gradient_GBps": w.in_bytes / res["ms"] / 1e6, "ms_per_step": res["ms"],
           "step_roofline": step_roofline(w, res["ms"], peak_gbs), "kernels": {}}
    if res["q"].one_kernel:
        out["step_form"] = ("one cooperative kernel (uq_step_small): ms_per_step is that kernel; the entries under "
                            "kernels are the separate calls, timed one by one for comparison")
    for s, ms in res["stages_ms"].items():
        gbs = ab[s] / ms / 1e6
        out["kernels"][s] = {"ms": round(ms, 5), "algorithmic_MB": round(ab[s] / 1e6, 2),
                             "GBps": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peak_gbs, 4),
                             "frac_of_nominal_8TBps": round(gbs / NOMINAL_HBM_GBS, 4)}
        if s in res.get("copy_same_bytes_ms", {}):
            cms = res["copy_same_bytes_ms"][s]
            out["kernels"][s]["plain_copy_of_the_same_bytes"] = {
                "ms": round(cms, 5), "frac_of_hbm_peak": round(ab[s] / cms / 1e6 / peak_gbs, 4),
                "note": "torch copy_ moving as many bytes as this stage (half read, half written), copies back to back"}
        if s in res.get("stages_sustained_ms", {}):
            ms_s = res["stages_sustained_ms"][s]
            out["kernels"][s]["ms_sustained"] = round(ms_s, 5)
            out["kernels"][s]["frac_of_hbm_peak_sustained"] = round(ab[s] / ms_s / 1e6 / peak_gbs, 4)
    if res.get("clocks") is not None:
        out["clocks"] = res["clocks"]
    other = 32 if w.rng_bits == 16 else 16
    ms = res["encode_other_ms"]
    out["kernels"][f"encode_rng{other}"] = {
        "ms": round(ms, 5), "algorithmic_MB": round(ab["encode"] / 1e6, 2), "GBps": round(ab["encode"] / ms / 1e6, 1),
        "frac_of_hbm_peak": round(ab["encode"] / ms / 1e6 / peak_gbs, 4), "note": "timed alone, not part of the step"}
    if "two_kernel_tail_ms" in res:
        enc, dec = res["two_kernel_tail_ms"]
        for key, t in (("encode", enc), ("aggregate_decode", dec)):
            out["kernels"][key] = {
                "ms": round(t, 5), "algorithmic_MB": round(ab[key] / 1e6, 2), "GBps": round(ab[key] / t / 1e6, 1),
                "frac_of_hbm_peak": round(ab[key] / t / 1e6 / peak_gbs, 4),
                "note": "timed alone, not part of the step: the step makes the two as one call (encode_decode)"}
        for key, t in res.get("alone_ms", {}).items():
            out["kernels"][key] = {
                "ms": round(t, 5), "algorithmic_MB": round(ab[key] / 1e6, 2), "GBps": round(ab[key] / t / 1e6, 1),
                "frac_of_hbm_peak": round(ab[key] / t / 1e6 / peak_gbs, 4),
                "note": "timed alone, not part of the step: the step makes selection, encoding, aggregation and "
                        "reconstruction as one call (select_encode_decode)"}
        out["kernels"]["encode_decode"]["ms_of_the_two_kernels_it_replaces"] = round(enc + dec, 5)
        if "select_encode_decode" in out["kernels"] and "alone_ms" in res:
            three = res["alone_ms"]["select_scale"] + res["alone_ms"]["encode_decode"]
            out["kernels"]["select_encode_decode"]["ms_of_the_two_kernels_it_replaces"] = round(three, 5)
            out["kernels"]["select_encode_decode"]["gradient_GBps_of_a_step_without_it"] = round(
                w.in_bytes / (res["ms"] - res["stages_ms"]["select_encode_decode"] + three) / 1e6, 1)
            out["kernels"]["select_encode_decode"]["note"] = (
                "selection + encoding + aggregation + reconstruction as one kernel: the gradients are read once and "
                "nothing is read back; bound by instruction issue (ALU pipe), not by memory, so its fraction of the HBM "
                "peak is lower than that of the streaming kernels it replaces (timed alone beside it), and its time shorter")
    if "fused_select_ms" in res:
        ms = res["fused_select_ms"]
        sel = res["stages_ms"].get("select_scale", res.get("alone_ms", {}).get("select_scale", 0.0))
        if "select_encode_decode" in res["stages_ms"]:      # the step already selects inside its second call
            enc_alone, dec_alone = res["two_kernel_tail_ms"]
            two = sel + enc_alone
            step_with = res["ms"] - res["stages_ms"]["select_encode_decode"] + ms + dec_alone
        elif "two_kernel_tail_ms" in res:       # the step's tail is one kernel: compare with selector + encoder alone
            enc_alone, dec_alone = res["two_kernel_tail_ms"]
            two = sel + enc_alone
            step_with = res["ms"] - sel - res["stages_ms"]["encode_decode"] + ms + dec_alone
        else:
            two = sel + res["stages_ms"].get("encode", 0.0)
            step_with = res["ms"] - two + ms
        out["kernels"]["select_encode"] = {
            "ms": round(ms, 5), "algorithmic_MB": round(ab["select_encode"] / 1e6, 2),
            "GBps": round(ab["select_encode"] / ms / 1e6, 1),
            "frac_of_hbm_peak": round(ab["select_encode"] / ms / 1e6 / peak_gbs, 4),
            "ms_of_the_two_kernels_it_replaces": round(two, 5),
            "gradient_GBps_of_a_step_with_it": round(w.in_bytes / step_with / 1e6, 1),
            "note": "selection + encoding as one call (one kernel for M <= 8: the gradients are read once; bound by "
                    "instruction issue, not by memory), timed alone, not part of the step"}
    if "fused_all_ms" in res:
        ms = res["fused_all_ms"]
        nbytes = ab["select_encode"] + 4 * w.d
        two = res["stages_ms"]["select_scale"] + res["stages_ms"]["encode_decode"]
        out["kernels"]["select_encode_decode"] = {
            "ms": round(ms, 5), "algorithmic_MB": round(nbytes / 1e6, 2), "GBps": round(nbytes / ms / 1e6, 1),
            "frac_of_hbm_peak": round(nbytes / ms / 1e6 / peak_gbs, 4),
            "ms_of_the_two_kernels_it_replaces": round(two, 5),
            "gradient_GBps_of_a_step_with_it": round(w.in_bytes / (res["ms"] - two + ms) / 1e6, 1),
            "note": "selection + encoding + aggregation + reconstruction as one call (uq_select_encode_decode_multi: one "
                    "kernel, the gradients are read once and nothing is read back; bound by instruction issue, not by "
                    "memory), timed alone, not part of the step"}
    lev = {"i8": 1.0, "i4x2": 0.5, "i2x4": 0.25, "i6p": 0.75}[w.fmt]
    upd_bytes = lev * w.M * w.d + w.idx_bits / 8.0 * w.d + 16 * w.d      # levels, index, theta and momentum r/w
    ms = res["update_ms"]
    out["kernels"]["aggregate_decode_update"] = {
        "ms": round(ms, 5), "algorithmic_MB": round(upd_bytes / 1e6, 2), "GBps": round(upd_bytes / ms / 1e6, 1),
        "frac_of_hbm_peak": round(upd_bytes / ms / 1e6 / peak_gbs, 4),
        "note": "fused SGD-momentum update, timed alone, not part of the step"}
    if "sustained" in res:
        out["sustained"] = sustained_summary(w, res["sustained"])
    if "ms_cold" in res:
        out["cold_l2"] = {"ms_per_step": res["ms_cold"], "gradient_GBps": w.in_bytes / res["ms_cold"] / 1e6,
                          "kernels_ms": {s: round(v, 5) for s, v in res["stages_cold_ms"].items()}}
        out["cuda_graph_warm_l2"] = {"ms_per_step": res["ms_graph"],
                                     "gradient_GBps": w.in_bytes / res["ms_graph"] / 1e6}
    return out


def cpu_sample(name, max_coords, threads):
    """(workload, n, segment table, gradients) of the oracle's sample: the first n coordinates of the
    workload, n = max_coords rounded down to whole segments where the workload has equal buckets."""
    w = wl.WORKLOADS[name]
    n = min(w.d, max_coords)
    if w.bucket_elems and n < w.d:
        n = max(1, n // w.bucket_elems) * w.bucket_elems           # whole buckets
    seg_full = wl.segment_offsets(w)
    seg = np.unique(np.concatenate([seg_full[seg_full < n], [n]])).astype(np.int64)
    sub = w
    if n < w.d:                                 # same recipe at the window's size
        import dataclasses
        sub = dataclasses.replace(w, d=n, segments="one")
    g = wl.generate(sub, threads=threads)[:, :n]
    return w, n, seg, g


def cpu_pass(w, seg, g, threads):
    """One pass of the whole path through the oracle, as it stands; seconds."""
    from oracle import uq_oracle as o
    o.set_threads(threads)
    norm = o.NORM_L2 if w.norm == wl.NORM_L2 else o.NORM_LINF
    t0 = time.perf_counter()
    W = o.agree_scale(g, seg, norm)
    if w.quantizer == "multi":
        idx = o.select_scale_multi(g, W, w.scales, seg_off=seg)
        lev = o.encode_multi(g, W, w.scales, idx, w.seed, w.rng_bits, seg_off=seg)
        S = o.aggregate(lev)
        o.decode(S, w.M, W, scales=w.scales, idx=idx, seg_off=seg)
    else:
        lev = o.encode_single(g, W, w.s, w.seed, w.rng_bits, seg_off=seg)
        S = o.aggregate(lev)
        o.decode(S, w.M, W, s=w.s, seg_off=seg)
    return time.perf_counter() - t0


def sample_text(w, n, seg):
    if n == w.d:
        return "full workload"
    what = f"{len(seg) - 1} whole buckets" if w.bucket_elems else f"{len(seg) - 1} segments"
    return f"first {n} of {w.d} coordinates ({what}) of all {w.M} workers"


def cpu_baseline(name, threads, max_coords):
    """The oracle on the host cores over a bounded sample of the workload."""
    from oracle import uq_oracle as o
    w, n, seg, g = cpu_sample(name, max_coords, threads)
    dt = cpu_pass(w, seg, g, threads)
    in_bytes = w.M * n * (4 if w.dtype == wl.F32 else 2)
    return {"value": in_bytes / dt / 1e9, "unit": UNIT, "cores": o.get_threads(), "kind": "oracle",
            "sample": sample_text(w, n, seg), "seconds": round(dt, 3)}


def max_over_ranks(values, device):
    """Element-wise max of a list of floats over all ranks (every rank gets the result).
    Replicas do not exchange data; this is the only collective of a multi-GPU run."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_value(world, in_bytes, ms):
    """Gradient GB/s of the whole job: every one of `world` replicas processed in_bytes in ms."""
    return world * in_bytes / ms / 1e6


def bench_distributed(w, steps, warmup, device, threads, kernels=None, return_out=False):
    """The paper's own setting beside the replicas figure: the M workers spread over the processes of
    the job (M / world_size each), the three all-reduces of Algorithm 1 / 2 as real exchanges between
    them (distributed.DistributedQuantizer: NCCL collectives on GPUs, nothing else crosses between them).
    Times the whole step for the gather and the slice form of the last exchange, max over ranks.
    device "cpu" with a stand-in for the C ABI (kernels) runs the same code under gloo in the tests."""
    import torch
    import torch.distributed as dist
    from paper_2109_12497_b200.distributed import DistributedQuantizer
    world, rank = dist.get_world_size(), dist.get_rank()
    if w.M % world:
        return {"skipped": f"{w.M} workers do not divide over {world} processes"}
    on_gpu = str(device).startswith("cuda")
    K = kernels
    if K is None:
        from paper_2109_12497_b200 import binding as K
    M_local = w.M // world
    fmt = {"i8": 0, "i4x2": 1, "i2x4": 2, "i6p": 3}[w.fmt]           # UQ_FMT_* of include/uq.h
    g_np = wl.generate(w, threads=threads, workers=range(rank * M_local, (rank + 1) * M_local))
    t = torch.from_numpy(g_np.view(np.float32 if w.dtype == wl.F32 else np.int16))
    if w.dtype == wl.BF16:
        t = t.view(torch.bfloat16)
    rec = {"processes": world, "workers_per_process": M_local,
           "note": "whole step with the workers spread over the processes: max all-reduce of the scales, [exchange + "
                   "minimum of the packed scale indices,] exchange of the level rows in their wire format, fused sum + "
                   "reconstruction; gradient GB/s counts the gradients of all processes"}
    out_last = None
    for exchange in ("gather", "slices"):
        if exchange == "slices" and w.fmt == "i6p":
            continue                                   # two-plane rows are not cut into slices
        q = DistributedQuantizer(
            M_local, w.d, torch.float32 if w.dtype == wl.F32 else torch.bfloat16, seg_off=wl.segment_offsets(w),
            s=w.s, scales=list(w.scales) if w.quantizer == "multi" else None, fmt=fmt, idx_bits=w.idx_bits,
            norm=K.UQ_NORM_L2 if w.norm == wl.NORM_L2 else K.UQ_NORM_LINF, rng_bits=w.rng_bits, device=device,
            kernels=kernels, exchange=exchange)
        g = torch.zeros((M_local, q.stride), dtype=t.dtype, device=device)
        g[:, : t.shape[1]] = t.to(device)
        for k in range(warmup):
            q.step(g, w.seed + k)
        if on_gpu:
            st = torch.cuda.current_stream()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
        dist.barrier()
        t0 = time.perf_counter()
        if on_gpu:
            e0.record(st)
        for k in range(steps):
            out = q.step(g, w.seed + k)
        if on_gpu:
            e1.record(st)
            torch.cuda.synchronize()
            ms_mine = e0.elapsed_time(e1) / steps
        else:
            ms_mine = (time.perf_counter() - t0) * 1e3 / steps
        dist.barrier()
        (ms,) = max_over_ranks([ms_mine], device)
        rec[exchange] = {"ms_per_step": round(ms, 5), "gradient_GBps": round(w.in_bytes / ms / 1e6, 6),
                         "wire_bytes_received_per_process_and_step": int(q.wire_bytes_per_step()),
                         "status_word": int(q.status.item())}
        if exchange == "gather":
            out_last = out.detach().cpu().numpy().copy()
        del q, g
    return (rec, out_last) if return_out else rec


def other_workloads(rng_bits):
    """The workloads reported beside the headline one: the other four configurations, c2 on the
    2-bit and 6-bit wires, and c3 with its shared index sent in 2, 4 and 8 bits."""
    import dataclasses
    base = {n: resolve_workload(n, None, rng_bits) for n in ("c1", "c2", "c3", "c4", "c5")}
    return [
        ("c1", base["c1"]), ("c2", base["c2"]), ("c3", base["c3"]), ("c4", base["c4"]), ("c5", base["c5"]),
        ("c2_levels_2bit", resolve_workload("c2", None, rng_bits, "i2x4")),      # levels -1, 0, 1
        ("c2_levels_6bit", resolve_workload("c2", None, rng_bits, "i6p")),
        ("c3_idx2", base["c3"]),
        ("c3_idx4", dataclasses.replace(base["c3"], idx_bits=4)),
        ("c3_idx8", dataclasses.replace(base["c3"], idx_bits=8)),
    ]


def wire_bytes_per_coordinate(w):
    """Bytes per coordinate and worker that the method puts on the wire: levels + shared index."""
    return {"i8": 1.0, "i4x2": 0.5, "i2x4": 0.25, "i6p": 0.75}[w.fmt] + w.idx_bits / 8.0


def gpu_main(args):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the quantizer has no CPU path; use --impl reference "
                         "for the oracle baseline)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()

    threads = max(1, min(16, (os.cpu_count() or 8) // max(1, world)))
    peak, peak_kind = hbm_peak()
    name = args.workload
    w = resolve_workload(name, args.d, args.rng_bits, args.levels)

    res = bench_workload(w, args.steps, args.warmup, barrier, threads, want_e2e=not args.no_e2e, sustained=True,
                         flush_between=w.in_bytes < (126 << 20), device_index=local)
    clocks = res["clocks"]
    ms, e2e_ms = max_over_ranks([res["ms"], res["e2e_ms"] or float("nan")], "cuda")
    summ = summarize(res, peak)
    q = res["q"]
    dom = max(res["stages_ms"], key=lambda s: res["stages_ms"][s])
    ab = algorithmic_bytes(w)
    dom_gbs = ab[dom] / res["stages_ms"][dom] / 1e6
    dom_sust = res.get("stages_sustained_ms", {}).get(dom)
    per_coord = NCU_TRAFFIC_BYTES_PER_COORD.get((name, dom))
    alu_ops = NCU_ALU_OPS_PER_COORD_WORKER.get((name, dom))
    line = {
        "metric": METRIC, "value": round(whole_job_value(world, w.in_bytes, ms), 2), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 5),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32" if w.dtype == wl.F32 else "bf16",
        "data": "synthetic",
        "config": {
            "workload": f"{name}: {w.quantizer}-scale, M={w.M}, d={w.d} {w.dtype}, {len(wl.segment_offsets(w)) - 1} "
                        f"segments, s={w.s}, scales={list(w.scales)}, levels {w.fmt}, idx_bits={w.idx_bits}, "
                        f"norm={w.norm}, rng_bits={w.rng_bits}",
            "parallelism": "replicas only" if world > 1 else "single GPU, M workers emulated as resident buffers",
            "l2": (f"inputs {w.in_bytes / 1e6:.0f} MB per step > 126 MB L2, no flush between steps" if w.in_bytes > (126 << 20)
                   else f"inputs {w.in_bytes / 1e6:.0f} MB per step fit in the 126 MB L2: warm-L2 figure"),
            "status_word": res["status"],
        },
        "e2e": None if args.no_e2e else {
            "value": round(whole_job_value(world, w.in_bytes, e2e_ms), 2), "unit": UNIT, "ms_per_step": round(e2e_ms, 4),
            "h2d_bytes_per_step": res["h2d"], "d2h_bytes_per_step": res["d2h"]},
        "gpu_launches": q.kernels_per_step() * args.steps * world,          # all replicas together
        "clocks": clocks,
        "roofline": {
            "bound": "hbm", "kernel": dom, "achieved": round(dom_gbs, 1), "peak": peak, "unit": "GB/s",
            "frac": round(dom_gbs / peak, 4), "peak_kind": f"of {peak_kind}",
            "frac_sustained": None if dom_sust is None else round(ab[dom] / dom_sust / 1e6 / peak, 4),
            "frac_of_nominal_8TBps": round(dom_gbs / NOMINAL_HBM_GBS, 4),
            "algorithmic_bytes_per_launch": int(ab[dom]),
            "avg_launch_ms": round(res["stages_ms"][dom], 5),
            "avg_launch_ms_sustained": None if dom_sust is None else round(dom_sust, 5),
            "traffic": None if per_coord is None else int(per_coord * w.d),
            "traffic_note": None if per_coord is None else
                            f"{per_coord} B per coordinate under ncu at a smaller d of the same recipe, times d",
        },
        "step_roofline": step_roofline(w, ms, peak),
        "kernels": summ["kernels"],
        "sustained": sustained_summary(w, res["sustained"]),
    }
    if alu_ops is not None:
        # this kernel is bound by the ALU pipe and instruction issue, not by memory: the same launch
        # against that pipe, beside the fraction of the HBM peak that the metric asks for
        mhz = (clocks or {}).get("sm_mhz") or 1965.0
        alu_peak = SM_COUNT * ALU_LANES_PER_SM * mhz * 1e6
        alu_rate = alu_ops * w.M * w.d / (res["stages_ms"][dom] * 1e-3)
        line["roofline"]["limiter"] = ("ALU pipe and instruction issue, not memory (ncu on a smaller case: ALU pipe 70 %, "
                                       "DRAM 49 % busy); the streaming kernels whose work it does are timed alone under "
                                       "kernels: select_scale, encode, aggregate_decode")
        line["roofline"]["alu"] = {"achieved": round(alu_rate / 1e12, 2), "peak": round(alu_peak / 1e12, 2),
                                   "unit": "T ALU-pipe thread instructions/s", "frac": round(alu_rate / alu_peak, 4),
                                   "ops_per_coordinate_and_worker": alu_ops}
    if "cold_l2" in summ:
        line["cold_l2"], line["cuda_graph_warm_l2"] = summ["cold_l2"], summ["cuda_graph_warm_l2"]
    if rank == 0 and world == 1:
        # the other workloads (parity-test cases; reported for context, a few steps each)
        if not args.no_extra and args.d is None:
            extra = {}
            for other, wo in other_workloads(args.rng_bits):
                if other == name:
                    continue
                del res, q
                torch.cuda.empty_cache()
                small = wo.in_bytes < (126 << 20)
                res = bench_workload(wo, max(3, min(args.steps, 10)), 3, lambda: None, threads,
                                     want_e2e=False, flush_between=small, sustained=True,
                                     randk_K=10_000 if other == "c2" else 0, device_index=local)
                q = res["q"]
                extra[other] = summarize(res, peak)
                extra[other]["status_word"] = res["status"]
                extra[other]["rng_bits"] = wo.rng_bits
                extra[other]["wire_bytes_per_coordinate_and_worker"] = wire_bytes_per_coordinate(wo)
                if "randk" in res:
                    extra[other]["global_randk"] = res["randk"]
                if "randk_two_scale" in res:
                    extra[other]["global_randk_two_scale"] = res["randk_two_scale"]
                if "graph_stats" in res:
                    mean, med, lo = res["graph_stats"]
                    extra[other]["cuda_graph_replay"] = {
                        "ms_per_step_mean": round(mean, 5), "ms_per_step_median": round(med, 5), "ms_per_step_min": round(lo, 5),
                        "gradient_GBps_median": round(wo.in_bytes / med / 1e6, 1),
                        "note": "the whole step captured once and replayed, each replay timed by itself"}
            line["other_workloads"] = extra
        if not args.no_cpu:
            cores = max(1, os.cpu_count() or 1)
            line["cpu_baseline"] = cpu_baseline(name, cores, args.cpu_coords)
            one = cpu_baseline(name, 1, max(1, args.cpu_coords // 16))      # one thread, a sixteenth of the sample
            line["cpu_baseline"]["single_thread"] = {"value": one["value"], "unit": UNIT, "sample": one["sample"],
                                                     "seconds": one["seconds"]}
    if world > 1:
        # the workers of the same workload spread over the processes, with real exchanges (every rank takes part)
        del res, q
        torch.cuda.empty_cache()
        try:
            line["distributed"] = bench_distributed(w, args.steps, args.warmup, "cuda", threads)
        except Exception as e:           # the replicas figure above stands by itself
            line["distributed"] = {"error": f"{type(e).__name__}: {e}"[:300]}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# reference arm: the CPU oracle
# ---------------------------------------------------------------------------------------------

def reference_main(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import uq_oracle as o
    threads = max(1, os.cpu_count() or 1)
    w, n, seg, g = cpu_sample(args.workload, args.ref_coords, threads)      # the inputs are made once, outside the steps
    secs = []
    for k in range(args.warmup + args.steps):
        dt = cpu_pass(w, seg, g, threads)
        if k >= args.warmup:
            secs.append(dt)
    sec = statistics.fmean(secs)
    in_bytes = w.M * n * (4 if w.dtype == wl.F32 else 2)
    value = in_bytes / sec / 1e9
    sample = sample_text(w, n, seg)
    line = {
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(sec * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if w.dtype == wl.F32 else "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: CPU oracle on the {sample}; a step = one pass of the whole path over that sample"},
        "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": o.get_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--no-extra", action="store_true", help="skip the context workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end timing")
    ap.add_argument("--d", type=int, default=None, help="run the workload's recipe at this smaller d (profiling)")
    ap.add_argument("--rng-bits", type=int, default=None, choices=[16, 32], help="override the draw width")
    ap.add_argument("--levels", default=None, choices=sorted(LEVEL_WIRES), help="override the level wire format")
    ap.add_argument("--cpu-coords", type=int, default=2 * 13_107_200,
                    help="coordinates of the workload the CPU baseline covers (c5: two whole 25 MiB buckets)")
    ap.add_argument("--ref-coords", type=int, default=13_107_200,
                    help="coordinates per step of the reference (oracle) arm (c5: one whole bucket)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        reference_main(args)
    else:
        gpu_main(args)


if __name__ == "__main__":
    main()
