#!/usr/bin/env python
"""Benchmark of the MXFP4 weight-only linear path on B200.

Workload (BASELINE.json config "7B-Llama-shaped decode layer set", M=1): one *step* is one
draft-token pass over the linear projections of ``--layers`` (default 32) distinct 7B decoder
layers -- q/k/v/o 4096x4096, gate/up 11008x4096, down 4096x11008 -- i.e. 224 independent layer
problems per step, streaming 3.44 GB of MXFP4 weights (far larger than the 126 MB L2, so every
step reads HBM).  They run through mxq_linear_batch, ``--layers-per-call`` (default 8) layer
sets = 56 layers per launch, the step's independent calls issued round-robin on ``--streams``
(default 2) CUDA streams with a workspace each; the same step on one stream, with four and with one
layer set per launch and as 224 separate mxq_linear calls is timed beside it (``extra.routes``).  Weights are synthetic (Student-t, seeded), direct-cast on the device by
mxq_quantize before timing; the offline cast and the greedy-accept step are timed separately and
reported under "extra".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead (the only other
place this file may execute anything under oracle/ is the cpu_baseline leg).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_13565_b200 import replicas, synth  # noqa: E402

METRIC = "mxq_linear_hbm_gbs"
UNIT = "GB/s"
HBM_DATASHEET_GBS = 8000.0


# DRAM bytes (read + write) over algorithmic bytes of one launch, from the committed profiler summaries:
#   mxq_linear_batch, eight 7B layer sets at M=1 (profiles/mxq_linear_batch_m1_8x7B_layer_sets_full.md):
#     866.23 MB read + 5.45 MB written against 862.02 MB algorithmic (mean of the two captured launches)
#   one mxq_linear call, 11008x4096 at M=1 (profiles/mxq_linear_fp4_m1_11008x4096_full.md): 24.034816 MB / 23.957504 MB
DRAM_OVER_ALGORITHMIC_BATCH = (866.232704 + 5.452672) / 862.023680
DRAM_OVER_ALGORITHMIC = 24.034816 / 23.957504


def algorithmic_bytes(m: int, n: int, k: int, y_bytes: int = 4) -> int:
    """4.25 bits per weight + activations + outputs (the byte count the metric is defined on)."""
    return n * k // 2 + n * k // 32 + 2 * m * k + y_bytes * m * n


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


# ---------------------------------------------------------------------------------------------
# clocks: NVML polling thread (read-only) running during the timed region
# ---------------------------------------------------------------------------------------------
class ClockMonitor:
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
        0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
        0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, device_index: int):
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            self._nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = int(vis.split(",")[device_index]) if vis and vis.split(",")[device_index].isdigit() else device_index
                self._h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self._h is not None:
            self._stop.clear()
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self):
        bits = self.reason_bits & ~0x1  # idle between samples is not a throttle
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": [name for bit, name in self.REASONS.items() if bits & bit],
            "samples": len(self.samples),
        }


# ---------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------
def build_layers(mxq, n_layers: int, shapes, device):
    """Direct-cast `n_layers` seeded layer sets on the device; returns [(name, n, k, codes, scales)]."""
    out = []
    for layer in range(n_layers):
        for i, (name, n, k) in enumerate(shapes):
            w = synth.weight(3, layer * len(shapes) + i, n, k, device=device)
            codes, scales = mxq.mxq_quantize(w)
            out.append((name, n, k, codes, scales))
            del w
    torch.cuda.synchronize()
    return out


class LinearPass:
    """One pass over a list of quantised matrices at M token rows, replayed from a CUDA graph."""

    def __init__(self, mxq, mats, m: int, device, seed: int, use_graph: bool = True, per_call: int = 0, streams: int = 1):
        """per_call = 0: one mxq_linear call per matrix; > 0: mxq_linear_batch, that many matrices per call.
        streams > 1 (batch route): the calls, which are independent of one another, are issued round-robin on that many
        streams, each with a workspace of its own, between a fork and a join on the timing stream: a call then does not
        wait for the call before it to drain."""
        self.mxq, self.mats, self.m = mxq, mats, m
        ks = sorted({k for _, _, k, _, _ in mats})
        self.x = {k: synth.normal_bf16((m, k), 1.0, seed + k, device) for k in ks}
        self.y = [torch.empty((m, n), dtype=torch.float32, device=device) for _, n, _, _, _ in mats]
        self.bytes = sum(algorithmic_bytes(m, n, k) for _, n, k, _, _ in mats)
        self.batches = None
        if per_call > 0:
            self.batches = [mxq.LinearBatch([dict(x=self.x[k], codes=c, scales=s, out=y)
                                             for (_, n, k, c, s), y in zip(mats[i:i + per_call], self.y[i:i + per_call])])
                            for i in range(0, len(mats), per_call)]
            self.calls = mxq.IndependentBatches(self.batches, streams)
            self.nstreams = max(1, len(self.calls.streams))
            self.ws = self.calls.workspaces[0]
            self.launches = len(self.batches)
            self.info = self.batches[0].info()
        else:
            ws_bytes = max([mxq.mxq_linear_workspace_bytes(m, n, k) for _, n, k, _, _ in mats] + [16])
            self.nstreams = max(1, min(streams, len(mats)))
            self.wss = [mxq.new_workspace(ws_bytes, device) for _ in range(self.nstreams)]
            self.ws = self.wss[0]
            self.side = [torch.cuda.Stream(device=device) for _ in range(self.nstreams)] if self.nstreams > 1 else []
            self.launches = len(mats)
        self.graph = None
        self.stream = torch.cuda.Stream(device=device)
        self.stream.wait_stream(torch.cuda.current_stream(device))   # the inputs were produced on the current stream
        if use_graph:
            with torch.cuda.stream(self.stream):
                self.enqueue()          # first call outside capture (lazy module loading)
                self.stream.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=self.stream):
                    self.enqueue()
                self.graph = g

    def enqueue(self):
        if self.batches is not None:
            self.calls.run(self.stream)
            return
        if not self.side:
            for (_, n, k, codes, scales), y in zip(self.mats, self.y):
                self.mxq.mxq_linear(self.x[k], codes, scales, out=y, workspace=self.ws)
            return
        # the independent calls round-robin on several streams, a workspace each, between a fork and a join
        fork = torch.cuda.Event()
        fork.record(self.stream)
        for s_ in self.side:
            s_.wait_event(fork)
        for i, ((_, n, k, codes, scales), y) in enumerate(zip(self.mats, self.y)):
            self.mxq.mxq_linear(self.x[k], codes, scales, out=y, workspace=self.wss[i % self.nstreams], stream=self.side[i % self.nstreams])
        for s_ in self.side:
            join = torch.cuda.Event()
            join.record(s_)
            self.stream.wait_event(join)

    def step(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.enqueue()

    def time(self, steps: int, warmup: int, monitor: ClockMonitor = None):
        """seconds for `steps` passes, CUDA events on the launching stream, sync on both sides."""
        with torch.cuda.stream(self.stream):
            for _ in range(warmup):
                self.step()
            self.stream.synchronize()
            replicas.barrier()
            torch.cuda.synchronize()
            if monitor:
                monitor.start()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            for _ in range(steps):
                self.step()
            e1.record(self.stream)
            self.stream.synchronize()
            torch.cuda.synchronize()
            if monitor:
                monitor.stop()
            replicas.barrier()
        return e0.elapsed_time(e1) * 1e-3


def time_e2e(mxq, mats, m: int, steps: int, warmup: int, device):
    """Same pass through mxq_linear_host: activations come from pinned host memory and results go
    back to pinned host memory inside the timed region (weights stay resident)."""
    ks = sorted({k for _, _, k, _, _ in mats})
    xh = {k: synth.normal_bf16((m, k), 1.0, 77 + k).pin_memory() for k in ks}
    xs = {k: torch.empty((m, k), dtype=torch.bfloat16, device=device) for k in ks}
    yh = [torch.empty((m, n), dtype=torch.float32).pin_memory() for _, n, _, _, _ in mats]
    ys = [torch.empty((m, n), dtype=torch.float32, device=device) for _, n, _, _, _ in mats]
    ws = mxq.new_workspace(max([mxq.mxq_linear_workspace_bytes(m, n, k) for _, n, k, _, _ in mats] + [16]), device)
    stream = torch.cuda.Stream(device=device)
    stream.wait_stream(torch.cuda.current_stream(device))
    h2d = sum(2 * m * k for _, _, k, _, _ in mats)
    d2h = sum(4 * m * n for _, n, _, _, _ in mats)

    def one():
        for (_, n, k, codes, scales), yh_i, ys_i in zip(mats, yh, ys):
            mxq.mxq_linear_host(xh[k], codes, scales, yh_i, xs[k], ys_i, workspace=ws, stream=stream)

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            one()
        stream.synchronize()
        replicas.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record(stream)
        for _ in range(steps):
            one()
        e1.record(stream)
        stream.synchronize()
        wall = time.perf_counter() - t0
        replicas.barrier()
    return max(e0.elapsed_time(e1) * 1e-3, 0.0), wall, h2d, d2h


def time_e2e_batch(mxq, mats, m: int, per_call: int, steps: int, warmup: int, device, streams: int = 1):
    """The same pass through mxq_linear_batch with the activations and the results in pinned HOST memory: the kernel
    reads every layer's X across the bus itself and stores Y straight into host memory, inside the timed region.
    Every layer of a call has a host buffer of its own (the library shares the rewriting of X only between layers
    that pass the same pointer), so each layer's activations cross the bus, as with one call per layer."""
    xh = [synth.normal_bf16((m, k), 1.0, 77 + i).pin_memory() for i, (_, _, k, _, _) in enumerate(mats[:per_call])]
    yh = [torch.empty((m, n), dtype=torch.float32).pin_memory() for _, n, _, _, _ in mats]
    batches = []
    for i in range(0, len(mats), per_call):
        lays = []
        for j, ((_, n, k, c, s_), y) in enumerate(zip(mats[i:i + per_call], yh[i:i + per_call])):
            assert xh[j].shape[1] == k   # every call holds the same sequence of shapes
            lays.append(dict(x=xh[j], codes=c, scales=s_, out=y))
        batches.append(mxq.LinearBatch(lays))
    calls = mxq.IndependentBatches(batches, streams)
    stream = torch.cuda.Stream(device=device)
    stream.wait_stream(torch.cuda.current_stream(device))
    h2d = sum(2 * m * k for _, _, k, _, _ in mats)
    d2h = sum(4 * m * n for _, n, _, _, _ in mats)

    def one():
        calls.run(stream)

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            one()
        stream.synchronize()
        replicas.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record(stream)
        for _ in range(steps):
            one()
        e1.record(stream)
        stream.synchronize()
        wall = time.perf_counter() - t0
        replicas.barrier()
    return max(e0.elapsed_time(e1) * 1e-3, 0.0), wall, h2d, d2h


def time_fn(fn, iters: int, warmup: int = 3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / iters


def time_graph(fn, iters: int, warmup: int = 3):
    """Device time per replay of a CUDA graph of fn() (no host launch overhead between the kernels)."""
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())   # the inputs were produced on the current stream
    with torch.cuda.stream(st):
        fn()
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            fn()
        for _ in range(warmup):
            g.replay()
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(iters):
            g.replay()
        e1.record(st)
        st.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / iters


def round_robin(calls, nstreams: int):
    """fn() that issues the independent `calls` (each takes the stream to run on) round-robin on `nstreams` streams between a
    fork from and a join to the current stream: a call then starts in the SMs the other stream's call leaves, without
    waiting for it to drain."""
    side = [torch.cuda.Stream() for _ in range(nstreams)]

    def fn():
        cur = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(cur)
        for s_ in side:
            s_.wait_event(fork)
        for i, call in enumerate(calls):
            call(side[i % nstreams])
        for s_ in side:
            join = torch.cuda.Event()
            join.record(s_)
            cur.wait_event(join)
    return fn


def cpu_baseline_leg(m: int, budget_s: float = 15.0):
    """The oracle, as it stands, on one 7B layer set (host cores of this machine)."""
    import numpy as np

    import oracle
    mats = []
    for i, (name, n, k) in enumerate(synth.LAYERS_7B):
        rng = np.random.default_rng(i)
        mats.append((n, k, rng.integers(0, 256, (n, k // 2), dtype=np.uint8),
                     rng.integers(110, 126, (n, k // 32), dtype=np.uint8),
                     synth.bits_of(synth.normal_bf16((m, k), 1.0, 5 + i))))
    nbytes = sum(algorithmic_bytes(m, n, k) for n, k, *_ in mats)
    reps, t_total = 0, 0.0
    while t_total < budget_s and reps < 50:
        t0 = time.perf_counter()
        for n, k, codes, scales, x in mats:
            oracle.linear(x, codes, scales)
        t_total += time.perf_counter() - t0
        reps += 1
    out = {"value": nbytes * reps / t_total / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
           "sample": "%d pass(es) over one 7B layer set (7 matrices, 202M weights) at M=%d, FP64" % (reps, m),
           "us_per_layer_set": t_total / reps * 1e6}
    # beside it, each once: the same layer set at eight token rows and on one thread, and the cast of one 4096 x 4096 matrix
    cores = oracle.threads()
    try:
        x8 = {k: synth.bits_of(synth.normal_bf16((8, k), 1.0, 9)) for k in (4096, 11008)}
        t0 = time.perf_counter()
        for n, k, codes, scales, _ in mats:
            oracle.linear(x8[k], codes, scales)
        out["m8_us_per_layer_set"] = (time.perf_counter() - t0) * 1e6
        oracle.set_threads(1)
        t0 = time.perf_counter()
        n, k, codes, scales, x = mats[0]
        oracle.linear(x, codes, scales)
        out["one_thread_us_4096x4096_m%d" % m] = (time.perf_counter() - t0) * 1e6
        w = synth.bits_of(synth.normal_bf16((4096, 4096), 0.02, 3))
        t0 = time.perf_counter()
        oracle.quantize(w)
        out["one_thread_quantize_us_4096x4096"] = (time.perf_counter() - t0) * 1e6
        oracle.set_threads(cores)
        t0 = time.perf_counter()
        oracle.quantize(w)
        out["quantize_us_4096x4096"] = (time.perf_counter() - t0) * 1e6
    finally:
        oracle.set_threads(cores)
    return out


def run_ours(args):
    rank, local_rank, world = replicas.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    replicas.init("nccl")
    import paper_2503_13565_b200 as mxq
    mxq.binding.lib()  # fail loudly now if the extension is missing

    shapes = synth.LAYERS_7B
    mats = build_layers(mxq, args.layers, shapes, device)
    m = args.m
    monitor = ClockMonitor(local_rank)

    per_call = len(shapes) * max(1, min(args.layers_per_call, args.layers))   # layers (matrices) per mxq_linear_batch call
    if args.route == "separate" or m > 8:
        per_call = 0
    streams = max(1, args.streams) if per_call else 1
    main = LinearPass(mxq, mats, m, device, seed=31, use_graph=not args.no_graph, per_call=per_call, streams=streams)
    secs = main.time(args.steps, args.warmup, monitor)
    secs_max = replicas.max_over_ranks(secs, device)
    bytes_step = main.bytes
    value = replicas.sum_over_ranks(bytes_step * args.steps, device) / secs_max / 1e9
    ms_per_step = secs_max / args.steps * 1e3
    per_launch_s = secs / (args.steps * main.launches)
    achieved = bytes_step / main.launches / per_launch_s / 1e9
    peaks, peak_kind = measured_peaks()
    route_text = ("mxq_linear_batch, %d layer set(s) = %d layers per launch%s" %
                  (per_call // len(shapes), per_call, ", the independent calls issued round-robin on %d streams" % main.nstreams if main.nstreams > 1 else "")) \
        if per_call else "one mxq_linear call per layer"

    # end to end with host buffers
    e2e_steps = max(3, min(args.steps, 50))
    if per_call:
        e2e_dev, e2e_wall, h2d, d2h = time_e2e_batch(mxq, mats, m, per_call, e2e_steps, 3, device, streams)
    else:
        e2e_dev, e2e_wall, h2d, d2h = time_e2e(mxq, mats, m, e2e_steps, 3, device)
    e2e_secs = replicas.max_over_ranks(max(e2e_dev, e2e_wall), device)
    e2e_value = replicas.sum_over_ranks(bytes_step * e2e_steps, device) / e2e_secs / 1e9

    extra = {}
    if rank == 0 and not args.quick:
        # the same step through the other routes: one launch per layer set, and one mxq_linear call per layer
        routes = {}
        n7 = len(shapes)
        st_r = max(3, min(args.steps, 40))
        nper = max(1, min(args.layers_per_call, args.layers))
        head = "batch_%d_layer_sets_per_call%s" % (nper, "_%d_streams" % streams if streams > 1 else "")
        todo = [(head, per_call, streams)]
        for name, pc, ns in (("batch_%d_layer_sets_per_call" % nper, per_call, 1), ("batch_4_layer_sets_per_call_%d_streams" % streams, 4 * n7, streams),
                             ("batch_4_layer_sets_per_call", 4 * n7, 1), ("batch_1_layer_set_per_call_%d_streams" % streams, n7, streams),
                             ("batch_1_layer_set_per_call", n7, 1), ("separate_calls_%d_streams" % streams, 0, streams), ("separate_calls", 0, 1)):
            if (pc, ns) != (per_call, streams) and pc <= n7 * args.layers and name not in [t_[0] for t_ in todo] and (ns == 1 or streams > 1):
                todo.append((name, pc, ns))
        for name, pc, ns in todo:
            if (pc, ns) == (per_call, streams):
                routes[name] = {"us_per_layer_set": ms_per_step * 1e3 / args.layers, "gbs": value, "launches_per_step": main.launches,
                                "frac_of_peak": value / peaks["hbm_gbs"], "headline": True}
                continue
            if m > 8 and pc:
                continue
            pr = LinearPass(mxq, mats, m, device, seed=31, use_graph=not args.no_graph, per_call=pc, streams=ns)
            sr = pr.time(st_r, 3)
            routes[name] = {"us_per_layer_set": sr / st_r / args.layers * 1e6, "gbs": pr.bytes * st_r / sr / 1e9,
                            "launches_per_step": pr.launches, "frac_of_peak": pr.bytes * st_r / sr / 1e9 / peaks["hbm_gbs"]}
            del pr
        extra["routes"] = routes
        # the verify-side pass (M=8) over the same layers, through the same route and as separate calls
        st8 = max(3, args.steps // 2)
        p8 = LinearPass(mxq, mats, 8, device, seed=32, use_graph=not args.no_graph, per_call=per_call, streams=streams)
        s8 = p8.time(st8, 3)
        extra["m8"] = {"gbs": p8.bytes * st8 / s8 / 1e9, "us_per_layer_set": s8 / st8 / args.layers * 1e6,
                       "route": "batch" if per_call else "separate", "launches_per_step": p8.launches}
        del p8
        p8 = LinearPass(mxq, mats, 8, device, seed=32, use_graph=not args.no_graph)
        s8 = p8.time(st8, 3)
        extra["m8"]["separate_calls_us_per_layer_set"] = s8 / st8 / args.layers * 1e6
        del p8
        # and the token counts between (verifying 1..7 speculated tokens)
        mrows = {}
        for mm in (2, 3, 4, 5, 6):
            if not per_call:
                break
            pm = LinearPass(mxq, mats, mm, device, seed=35, use_graph=not args.no_graph, per_call=per_call, streams=streams)
            sm_ = pm.time(5, 3)
            mrows["m%d" % mm] = {"us_per_layer_set": sm_ / 5 / args.layers * 1e6, "gbs": pm.bytes * 5 / sm_ / 1e9}
            del pm
        extra["m8"]["other_token_counts"] = mrows
        # per-shape, one matrix at a time, rotating over the layers (each pass > L2)
        per_shape = {}
        for name, n, k in [("4096x4096", 4096, 4096), ("11008x4096", 11008, 4096), ("4096x11008", 4096, 11008)]:
            sel = [t for t in mats if (t[1], t[2]) == (n, k)]
            for mm in (1, 8):
                p = LinearPass(mxq, sel, mm, device, seed=33, use_graph=not args.no_graph)
                s = p.time(20, 3)
                per_shape["%s_m%d" % (name, mm)] = {"us_per_call": s / 20 / len(sel) * 1e6,
                                                    "gbs": p.bytes * 20 / s / 1e9}
        extra["per_shape"] = per_shape
        # vocabulary projections (one launch streams 70 / 279 MB): where launch latency no longer hides the kernel;
        # and the token-count curves of the 13B layer shapes and of the paper's own 8192 x 8192 micro-benchmark shape
        def m_curve(n, k, ms, iters=10):
            copies = max(2, int(300e6 // (n * k * 0.53125)) + 1)   # rotated, together larger than L2
            gen = torch.Generator(device=device).manual_seed(n + k)
            sel = [("w", n, k,
                    torch.randint(0, 256, (n, k // 2), dtype=torch.uint8, device=device, generator=gen),
                    torch.randint(110, 126, (n, k // 32), dtype=torch.uint8, device=device, generator=gen)) for _ in range(copies)]
            out = {}
            for mm in ms:
                p = LinearPass(mxq, sel, mm, device, seed=34, use_graph=not args.no_graph)
                s = p.time(iters, 3)
                out["%dx%d_m%d" % (n, k, mm)] = {"us_per_call": s / iters / len(sel) * 1e6, "gbs": p.bytes * iters / s / 1e9,
                                                 "frac_of_peak": p.bytes * iters / s / 1e9 / peaks["hbm_gbs"],
                                                 "kernel": mxq.mxq_linear_plan_info(mm, n, k)["kernel"]}
            return out
        vocab = {}
        for n in (32000, 128256):
            vocab.update(m_curve(n, 4096, (1, 2, 4, 8, 16)))
        curves = {}
        for n, k in ((5120, 5120), (13824, 5120), (5120, 13824), (8192, 8192)):
            curves.update(m_curve(n, k, (1, 2, 4, 8, 16) if (n, k) != (8192, 8192) else (1, 2, 4, 8)))
        extra["m_curves"] = curves
        extra["vocab_projection"] = vocab
        # vocabulary projection + greedy verification: one fused launch against mxq_linear followed by mxq_greedy_accept
        fused = {}
        for v_, r_ in ((32000, 1), (32000, 9), (128256, 1), (128256, 9)):
            copies = 3 if v_ == 32000 else 2
            gen = torch.Generator(device=device).manual_seed(v_ + r_)
            mats_ = [(torch.randint(0, 256, (v_, 2048), dtype=torch.uint8, device=device, generator=gen),
                      torch.randint(110, 126, (v_, 128), dtype=torch.uint8, device=device, generator=gen)) for _ in range(copies)]
            x_ = synth.normal_bf16((r_, 4096), 1.0, 5, device)
            t_ = r_ - 1
            draft_ = torch.zeros(max(t_, 1), dtype=torch.int32, device=device)
            wsf = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(r_, v_, 4096), device)
            wsl = mxq.new_workspace(max(mxq.mxq_linear_workspace_bytes(r_, v_, 4096), 16), device)
            wsa = mxq.new_workspace(mxq.mxq_accept_workspace_bytes(1, r_, v_), device)
            lg_ = torch.empty((1, r_, v_), dtype=torch.float32, device=device)

            def fused_pass():
                for c_, s_ in mats_:
                    mxq.mxq_lm_head_accept(x_, c_, s_, draft_[:t_] if t_ else None, workspace=wsf)

            draft2d = draft_[:max(t_, 1)].view(1, -1)   # (R = 1: a one-token draft stands in; the work is the same)

            def unfused_pass():
                for c_, s_ in mats_:
                    mxq.mxq_linear(x_, c_, s_, out=lg_[0], workspace=wsl)
                    mxq.mxq_greedy_accept(lg_, draft2d, workspace=wsa)
            tf = time_graph(fused_pass, 10) / copies
            tu = time_graph(unfused_pass, 10) / copies
            fused["%dx4096_r%d" % (v_, r_)] = {"fused_us": tf * 1e6, "linear_then_accept_us": tu * 1e6}
            del mats_
        extra["lm_head_accept"] = fused
        # the paper's comparison point: the same layer set with unquantised BF16 weights (16 bits per weight against 4.25)
        bf = {}
        shapes7 = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
        for mm in (1, 8):
            nl = 3   # 3 x 404 MB of BF16 weights: larger than L2
            wl = [[synth.normal_bf16((n_, k_), 0.02, 100 + 10 * li + j, device) for j, (n_, k_) in enumerate(shapes7)] for li in range(nl)]
            xk = {k_: synth.normal_bf16((mm, k_), 1.0, 7, device) for k_ in (4096, 11008)}
            ys_ = {n_: torch.empty((mm, n_), dtype=torch.float32, device=device) for n_ in (4096, 11008)}

            def bf_pass():
                for lay in wl:
                    for w_ in lay:
                        mxq.mxq_linear_bf16(xk[w_.shape[1]], w_, out=ys_[w_.shape[0]])
            tb = time_graph(bf_pass, 10) / nl
            nbytes = sum(n_ * k_ * 2 + 2 * mm * k_ + 4 * mm * n_ for n_, k_ in shapes7)
            bf["7B_layer_set_m%d" % mm] = {"us_per_layer_set": tb * 1e6, "gbs": nbytes / tb / 1e9, "bytes": nbytes}
            del wl
        bf["status"] = mxq.mxq_linear_device_status()
        extra["bf16_weights"] = bf
        # The same 7B layer as four calls with fused epilogues (Sec. III-D-2: operators fused into the linear layers):
        # q/k/v as one 12288 x 4096 matrix, o + residual, gate/up interleaved by rows with SiLU(gate)*up, down + residual.
        # BF16 in and out; o -> gate/up -> down is a true dependent chain (each call's output is the next one's input).
        fl = {}
        nlay = 8   # 8 x 107.5 MB of weights: larger than L2
        lay4 = []
        for li in range(nlay):
            mats4 = []
            for j, (n_, k_) in enumerate([(12288, 4096), (4096, 4096), (22016, 4096), (4096, 11008)]):
                w_ = synth.weight(3, 500 + 4 * li + j, n_, k_, device=device)
                mats4.append(mxq.mxq_quantize(w_))
                del w_
            lay4.append(mats4)
        for mm in (1, 8):
            h0 = synth.normal_bf16((mm, 4096), 1.0, 11, device)
            att = synth.normal_bf16((mm, 4096), 1.0, 12, device)
            qkv = torch.empty((mm, 12288), dtype=torch.bfloat16, device=device)
            h1 = torch.empty((mm, 4096), dtype=torch.bfloat16, device=device)
            act = torch.empty((mm, 11008), dtype=torch.bfloat16, device=device)
            h2 = torch.empty((mm, 4096), dtype=torch.bfloat16, device=device)
            wsf = torch.empty(max(mxq.mxq_linear_fused_workspace_bytes(mm, 22016, 4096),
                                  mxq.mxq_linear_fused_workspace_bytes(mm, 4096, 11008),
                                  mxq.mxq_linear_workspace_bytes(mm, 12288, 4096), 16), dtype=torch.uint8, device=device)

            def fused_pass():
                for (wqkv, wo, wgu, wd) in lay4:
                    mxq.mxq_linear(h0, wqkv[0], wqkv[1], out=qkv, workspace=wsf)
                    mxq.mxq_linear_residual(att, wo[0], wo[1], h0, out=h1, workspace=wsf)
                    mxq.mxq_linear_swiglu(h1, wgu[0], wgu[1], out=act, workspace=wsf)
                    mxq.mxq_linear_residual(act, wd[0], wd[1], h1, out=h2, workspace=wsf)
            tf_ = time_graph(fused_pass, 10) / nlay
            wbytes = sum(n_ * k_ * 17 // 32 for n_, k_ in [(12288, 4096), (4096, 4096), (22016, 4096), (4096, 11008)])
            fl["m%d" % mm] = {"us_per_layer": tf_ * 1e6, "gbs": wbytes / tf_ / 1e9, "calls": 4, "weight_bytes": wbytes}
            # what was timed is the chain it claims to be: issued without any synchronisation it leaves bit for bit what it
            # leaves with a device synchronisation after every call (a kernel that read its input early would not)
            fused_pass()
            torch.cuda.synchronize()
            free_running = [t_.clone() for t_ in (qkv, h1, act, h2)]
            for (wqkv, wo, wgu, wd) in lay4:
                mxq.mxq_linear(h0, wqkv[0], wqkv[1], out=qkv, workspace=wsf)
                torch.cuda.synchronize()
                mxq.mxq_linear_residual(att, wo[0], wo[1], h0, out=h1, workspace=wsf)
                torch.cuda.synchronize()
                mxq.mxq_linear_swiglu(h1, wgu[0], wgu[1], out=act, workspace=wsf)
                torch.cuda.synchronize()
                mxq.mxq_linear_residual(act, wd[0], wd[1], h1, out=h2, workspace=wsf)
                torch.cuda.synchronize()
            fl["m%d" % mm]["free_running_equals_synchronised"] = all(torch.equal(a_, b_) for a_, b_ in zip(free_running, (qkv, h1, act, h2)))
            # the same layer, dependences included, as ONE mxq_linear_batch call of three groups:
            # {q/k/v, o + residual} | {gate/up with SiLU(gate) * up} | {down + residual}
            one = [mxq.LinearBatch([dict(x=h0, codes=wqkv[0], scales=wqkv[1], out=qkv),
                                    dict(x=att, codes=wo[0], scales=wo[1], out=h1, epilogue="residual", residual=h0),
                                    dict(x=h1, codes=wgu[0], scales=wgu[1], out=act, epilogue="swiglu", depends=True),
                                    dict(x=act, codes=wd[0], scales=wd[1], out=h2, epilogue="residual", residual=h1, depends=True)])
                   for (wqkv, wo, wgu, wd) in lay4]
            ws1 = mxq.new_workspace(one[0].workspace_bytes(), device)

            def one_call_pass():
                for b_ in one:
                    b_.run(ws1)
            t1_ = time_graph(one_call_pass, 10) / nlay
            fl["m%d" % mm]["one_call_three_groups_us_per_layer"] = t1_ * 1e6
            fl["m%d" % mm]["one_call_three_groups_gbs"] = wbytes / t1_ / 1e9
        fl["status"] = mxq.mxq_linear_device_status()
        extra["fused_layer"] = fl
        del lay4
        # Speculative decoding with the quantised draft (Sec. III-B): a 4-layer slice of the 7B stack plus a 32000-row
        # vocabulary projection, target in BF16, draft = its MXFP4 cast; acceptance is simulated (random weights accept
        # nothing), the kernels and the control flow are real.  Measured tokens per second against Eq. 1 fed with the measured S.
        import random as _random
        from paper_2503_13565_b200 import specdec
        nl_, n_draft = 4, 8
        tw = [[synth.normal_bf16((n_, k_), 0.02, 300 + 10 * li + j, device) for j, (n_, k_) in enumerate(shapes7)] for li in range(nl_)]
        th = synth.normal_bf16((32000, 4096), 0.02, 399, device)
        dq = [[mxq.mxq_quantize(w_) for w_ in lay] for lay in tw]
        dh = mxq.mxq_quantize(th)
        xs_ = {(r_, k_): synth.normal_bf16((r_, k_), 1.0, 9, device) for r_ in (1, n_draft + 1) for k_ in (4096, 11008)}
        yo_ = {(r_, n_): torch.empty((r_, n_), dtype=torch.float32, device=device) for r_ in (1, n_draft + 1) for n_ in (4096, 11008)}
        lg_ = {r_: torch.empty((1, r_, 32000), dtype=torch.float32, device=device) for r_ in (1, n_draft + 1)}
        dr_ = torch.zeros((1, n_draft), dtype=torch.int32, device=device)
        wsa_ = mxq.new_workspace(mxq.mxq_accept_workspace_bytes(1, n_draft + 1, 32000), device)
        wsf_ = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(1, 32000, 4096), device)

        def target_step(r_):
            for lay in tw:
                for w_ in lay:
                    mxq.mxq_linear_bf16(xs_[(r_, w_.shape[1])], w_, out=yo_[(r_, w_.shape[0])])
            mxq.mxq_linear_bf16(xs_[(r_, 4096)], th, out=lg_[r_][0])
            mxq.mxq_greedy_accept(lg_[r_], dr_[:, :max(r_ - 1, 1)], workspace=wsa_)

        def draft_step_separate():   # one mxq_linear call per layer
            for lay in dq:
                for (c_, s_) in lay:
                    mxq.mxq_linear(xs_[(1, c_.shape[1] * 2)], c_, s_, out=yo_[(1, c_.shape[0])], workspace=self_ws)
            mxq.mxq_lm_head_accept(xs_[(1, 4096)], dh[0], dh[1], None, workspace=wsf_)

        # the draft's 28 layers in one mxq_linear_batch launch (here, as in the timed step above, the layers' inputs are
        # fixed buffers: a real decoder's layers depend on one another, which bounds what a call may hold)
        d_batch = mxq.LinearBatch([dict(x=xs_[(1, c_.shape[1] * 2)], codes=c_, scales=s_,
                                        out=torch.empty((1, c_.shape[0]), dtype=torch.float32, device=device)) for lay in dq for (c_, s_) in lay])
        d_ws = mxq.new_workspace(d_batch.workspace_bytes(), device)

        def draft_step():
            d_batch.run(d_ws)
            mxq.mxq_lm_head_accept(xs_[(1, 4096)], dh[0], dh[1], None, workspace=wsf_)
        self_ws = mxq.new_workspace(16, device)
        st_ = torch.cuda.Stream()
        st_.wait_stream(torch.cuda.current_stream())
        graphs = {}
        with torch.cuda.stream(st_):
            for name_, fn_ in (("t1", lambda: target_step(1)), ("tv", lambda: target_step(n_draft + 1)), ("d", draft_step),
                               ("ds", draft_step_separate)):
                fn_()
                st_.synchronize()
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_, stream=st_):
                    fn_()
                graphs[name_] = g_

            def timed(launch, reps):
                for _ in range(2):
                    launch()
                st_.synchronize()
                e0_, e1_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0_.record(st_)
                for _ in range(reps):
                    launch()
                e1_.record(st_)
                st_.synchronize()
                return e0_.elapsed_time(e1_) * 1e-3 / reps
            t_t1 = timed(graphs["t1"].replay, 20)
            t_tv = timed(graphs["tv"].replay, 20)
            t_d = timed(graphs["d"].replay, 20)
            t_ds = timed(graphs["ds"].replay, 20)
            sd = {"layers": nl_, "draft_tokens_per_round": n_draft, "target_step_us": t_t1 * 1e6, "target_verify_us": t_tv * 1e6,
                  "draft_step_us": t_d * 1e6, "S": t_t1 / t_d, "draft_route": "mxq_linear_batch (28 layers in one launch) + mxq_lm_head_accept",
                  "draft_step_one_call_per_layer_us": t_ds * 1e6, "S_one_call_per_layer": t_t1 / t_ds, "runs": {}}
            for p_ in (0.7, 0.9):
                rng_ = _random.Random(1)
                steps_ = []
                tally = specdec.simulate(2, [n_draft], lambda lvl, k_: specdec.leading_successes(rng_, p_, k_), tokens=400,
                                         on_step=lambda lvl, rows: steps_.append("d" if lvl == 1 else "tv"))

                def run_all():
                    for nm in steps_:
                        graphs[nm].replay()
                t_all = timed(run_all, 3)
                produced = tally.accepted[0] + tally.steps[0]
                alpha_ = tally.accepted[0] / tally.proposed[0]
                sd["runs"]["p=%.1f" % p_] = {"alpha": alpha_, "tokens": produced, "us_per_token": t_all / produced * 1e6,
                                             "speedup_measured": produced * t_t1 / t_all,
                                             "speedup_eq1": specdec.eq1_speedup(alpha_, n_draft, t_t1 / t_d)}
            # Two levels (Sec. III-C): a tiny draft (2 layers of the 68M-like shapes, MXFP4) drafts for the MXFP4 model, which
            # verifies with 9 rows and in turn drafts for the BF16 target.
            n_tiny = 4
            tiny_shapes = [(768, 768)] * 4 + [(3072, 768)] * 2 + [(768, 3072)]
            tq = [[mxq.mxq_quantize(synth.normal_bf16((n_, k_), 0.02, 500 + 10 * li + j, device)) for j, (n_, k_) in enumerate(tiny_shapes)]
                  for li in range(2)]
            tqh = mxq.mxq_quantize(synth.normal_bf16((32000, 768), 0.02, 599, device))
            xt_ = {k_: synth.normal_bf16((1, k_), 1.0, 11, device) for k_ in (768, 3072)}
            yt_ = {n_: torch.empty((1, n_), dtype=torch.float32, device=device) for n_ in (768, 3072)}
            wsf_t = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(1, 32000, 768), device)
            rv = n_tiny + 1
            xv_ = {k_: synth.normal_bf16((rv, k_), 1.0, 12, device) for k_ in (4096, 11008)}
            yv_ = {n_: torch.empty((rv, n_), dtype=torch.float32, device=device) for n_ in (4096, 11008)}
            wsv = mxq.new_workspace(max(mxq.mxq_linear_workspace_bytes(rv, n_, k_) for n_, k_ in shapes7), device)
            wsfv = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(rv, 32000, 4096), device)
            drv = torch.zeros(n_tiny, dtype=torch.int32, device=device)

            t_batch = mxq.LinearBatch([dict(x=xt_[c_.shape[1] * 2], codes=c_, scales=s_,
                                            out=torch.empty((1, c_.shape[0]), dtype=torch.float32, device=device)) for lay in tq for (c_, s_) in lay])
            t_ws = mxq.new_workspace(t_batch.workspace_bytes(), device)
            v_batch = mxq.LinearBatch([dict(x=xv_[c_.shape[1] * 2], codes=c_, scales=s_,
                                            out=torch.empty((rv, c_.shape[0]), dtype=torch.float32, device=device)) for lay in dq for (c_, s_) in lay])
            v_ws = mxq.new_workspace(v_batch.workspace_bytes(), device)

            def tiny_step():
                t_batch.run(t_ws)
                mxq.mxq_lm_head_accept(xt_[768], tqh[0], tqh[1], None, workspace=wsf_t)

            def draft_verify():   # the MXFP4 model checks the tiny draft's n_tiny tokens in one pass of n_tiny + 1 rows
                v_batch.run(v_ws)
                mxq.mxq_lm_head_accept(xv_[4096], dh[0], dh[1], drv, workspace=wsfv)
            for name_, fn_ in (("y", tiny_step), ("dv", draft_verify)):
                fn_()
                st_.synchronize()
                g_ = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_, stream=st_):
                    fn_()
                graphs[name_] = g_
            t_y = timed(graphs["y"].replay, 20)
            t_dv = timed(graphs["dv"].replay, 20)
            p_lv = [0.9, 0.6]
            rng_ = _random.Random(2)
            steps_ = []
            tally = specdec.simulate(3, [n_draft, n_tiny], lambda lvl, k_: specdec.leading_successes(rng_, p_lv[lvl], k_), tokens=400,
                                     on_step=lambda lvl, rows: steps_.append({0: "tv", 1: "dv", 2: "y"}[lvl]))

            def run_all2():
                for nm in steps_:
                    graphs[nm].replay()
            t_all = timed(run_all2, 3)
            produced = tally.accepted[0] + tally.steps[0]
            alphas = [tally.accepted[i] / tally.proposed[i] for i in range(2)]
            sd["two_level"] = {"tiny_step_us": t_y * 1e6, "draft_verify_us": t_dv * 1e6, "tiny_tokens_per_round": n_tiny,
                               "p": p_lv, "alpha": alphas, "tokens": produced, "us_per_token": t_all / produced * 1e6,
                               "speedup_measured": produced * t_t1 / t_all,
                               "speedup_nested_eq1": specdec.multilevel_speedup([t_t1, t_d, t_y], [n_draft, n_tiny], alphas)}
        extra["specdec"] = sd
        del tw, th, dq, dh
        # direct cast throughput (2 B read + 0.53125 B written per weight)
        w = synth.student_t_bf16((11008, 4096), 0.02, 1, device=device)
        ws_ = [w.clone() for _ in range(4)]   # 360 MB rotated: larger than L2
        codes = torch.empty((11008, 2048), dtype=torch.uint8, device=device)
        scales = torch.empty((11008, 128), dtype=torch.uint8, device=device)

        def q():   # one replay = the four matrices once
            for w_ in ws_:
                mxq.mxq_quantize(w_, codes, scales)
        tq = time_graph(q, 10) / 4
        extra["quantize"] = {"gbs": 11008 * 4096 * 2.53125 / tq / 1e9, "us_per_call": tq * 1e6, "shape": "11008x4096",
                             "frac_of_peak": 11008 * 4096 * 2.53125 / tq / 1e9 / peaks["hbm_gbs"]}
        # the same casts, which are independent of one another, round-robin on two streams (outputs of their own)
        outs2 = [(torch.empty_like(codes), torch.empty_like(scales)) for _ in ws_]
        tq2 = time_graph(round_robin([(lambda st_, w_=w_, o_=o_: mxq.mxq_quantize(w_, o_[0], o_[1], stream=st_)) for w_, o_ in zip(ws_, outs2)], 2), 10) / 4
        extra["quantize"]["two_streams"] = {"gbs": 11008 * 4096 * 2.53125 / tq2 / 1e9, "us_per_call": tq2 * 1e6,
                                            "frac_of_peak": 11008 * 4096 * 2.53125 / tq2 / 1e9 / peaks["hbm_gbs"]}
        del w, ws_, outs2
        # config 5: the direct cast of all 40 layers of a 13B-shaped model (12.69 G weights, 25.4 GB of BF16 in, 6.7 GB
        # out), every matrix resident, one replayed graph of the 280 casts
        try:
            shapes13 = [(n_, k_) for _, n_, k_ in synth.LAYERS_13B]
            w13 = [synth.weight(5, 100 + li * len(shapes13) + j, n_, k_, device=device) for li in range(40) for j, (n_, k_) in enumerate(shapes13)]
            c13 = [torch.empty((w_.shape[0], w_.shape[1] // 2), dtype=torch.uint8, device=device) for w_ in w13]
            s13 = [torch.empty((w_.shape[0], w_.shape[1] // 32), dtype=torch.uint8, device=device) for w_ in w13]

            def q13():
                for w_, c_, s_ in zip(w13, c13, s13):
                    mxq.mxq_quantize(w_, c_, s_)
            t13 = time_graph(q13, 3)
            weights13 = sum(w_.numel() for w_ in w13)
            extra["quantize_13b"] = {"ms_per_sweep": t13 * 1e3, "weights": weights13, "gbs": weights13 * 2.53125 / t13 / 1e9,
                                     "frac_of_peak": weights13 * 2.53125 / t13 / 1e9 / peaks["hbm_gbs"], "matrices": len(w13)}
            t13b = time_graph(round_robin([(lambda st_, w_=w_, c_=c_, s_=s_: mxq.mxq_quantize(w_, c_, s_, stream=st_))
                                           for w_, c_, s_ in zip(w13, c13, s13)], 2), 3)
            extra["quantize_13b"]["two_streams"] = {"ms_per_sweep": t13b * 1e3, "gbs": weights13 * 2.53125 / t13b / 1e9,
                                                    "frac_of_peak": weights13 * 2.53125 / t13b / 1e9 / peaks["hbm_gbs"]}
            del w13, c13, s13
        except torch.OutOfMemoryError as e:   # (a GPU with less memory than the 32 GB this leg holds)
            extra["quantize_13b"] = {"skipped": str(e)[:80]}
        # greedy accept: 250 sequences x 17 rows x 32000 logits (FP32), one call
        lg, draft, _, _ = synth.accept_trials(250, 16, 17, 32000, seed=1, device=device)
        ws2 = mxq.new_workspace(mxq.mxq_accept_workspace_bytes(250, 17, 32000), device)
        ta = time_graph(lambda: mxq.mxq_greedy_accept(lg, draft, workspace=ws2), 20)
        extra["greedy_accept"] = {"gbs": lg.numel() * 4 / ta / 1e9, "us_per_call": ta * 1e6, "shape": "250x17x32000 f32"}
        # two such batches, independent of each other, on two streams (logits, workspace and outputs of their own)
        lg_b, draft_b, _, _ = synth.accept_trials(250, 16, 17, 32000, seed=2, device=device)
        ws2b = mxq.new_workspace(mxq.mxq_accept_workspace_bytes(250, 17, 32000), device)
        outs_a = [tuple(torch.empty(250, dtype=torch.int32, device=device) for _ in range(2)) for _ in range(2)]
        ta2 = time_graph(round_robin([lambda st_: mxq.mxq_greedy_accept(lg, draft, workspace=ws2, stream=st_, out=outs_a[0]),
                                      lambda st_: mxq.mxq_greedy_accept(lg_b, draft_b, workspace=ws2b, stream=st_, out=outs_a[1])], 2), 20) / 2
        extra["greedy_accept"]["two_streams"] = {"gbs": lg.numel() * 4 / ta2 / 1e9, "us_per_call": ta2 * 1e6}
        del lg_b, draft_b
        del lg

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline_leg(m)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": "7B decode layer set (q,k,v,o 4096x4096; gate,up 11008x4096; down 4096x11008), "
                               "M=%d, %d distinct layer sets (%d independent layers) per step, run as: %s"
                               % (m, args.layers, len(mats), route_text),
                   "M": m, "layers": args.layers, "route": route_text, "calls_per_step": main.launches, "streams": streams, "bytes_per_step": bytes_step,
                   "y_dtype": "f32", "l2": "inputs larger than L2 (%.2f GB of weights per step)" % (bytes_step / 1e9),
                   "cuda_graph": not args.no_graph, "multi_gpu": "replicas only"},
        "us_per_layer_set": ms_per_step * 1e3 / args.layers,
        "pct_of_8000": 100.0 * value / world / HBM_DATASHEET_GBS,
        "clocks": monitor.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps},
        "gpu_launches": main.launches * args.steps,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "traffic": (DRAM_OVER_ALGORITHMIC_BATCH if per_call else DRAM_OVER_ALGORITHMIC) * bytes_step / main.launches,
                     "traffic_kind": ("dram read+write bytes of a profiler capture of one mxq_linear_batch launch of eight 7B layer sets "
                                      "(871.7 MB against 862.0 MB algorithmic), scaled to this launch's bytes") if per_call else
                                     ("dram read+write bytes of one profiler capture of the 11008x4096 launch "
                                      "(24.03 MB against 23.96 MB algorithmic), scaled to the average launch"),
                     "peak_kind": "of " + peak_kind,
                     "kernel": ("linear_batch_kernel" if per_call else "linear_fp4_kernel") + " M=%d" % m,
                     "bytes_per_launch": bytes_step / main.launches},
        "cpu_baseline": cpu,
        "extra": extra,
    }
    if rank == 0:
        print(json.dumps(line))
    replicas.shutdown()


# ---------------------------------------------------------------------------------------------
# reference arm: the oracle on the host cores
# ---------------------------------------------------------------------------------------------
def run_case(args):
    """One mxq_linear shape, launched `steps` times on a few distinct weight matrices (together larger than L2):
    the small case that profiler captures run on.  Prints one JSON line with the device time per call."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    import paper_2503_13565_b200 as mxq
    mxq.binding.lib()
    device = torch.device("cuda", 0)
    case = args.case.lower()
    if case.split(":")[0] in ("quantize", "accept", "bf16", "swiglu", "residual"):
        return run_case_other(mxq, case, args.steps, device)
    if case.split(":")[0] == "batch":
        return run_case_batch(mxq, case, args.steps, device)
    n, k, m = (int(v) for v in case.split("x"))
    nbytes = algorithmic_bytes(m, n, k)
    copies = max(2, min(8, int(200e6 // nbytes) + 1))
    gen = torch.Generator(device=device).manual_seed(7)
    mats = [(torch.randint(0, 256, (n, k // 2), dtype=torch.uint8, device=device, generator=gen),
             torch.randint(110, 126, (n, k // 32), dtype=torch.uint8, device=device, generator=gen)) for _ in range(copies)]
    x = synth.normal_bf16((m, k), 1.0, 3, device)
    y = torch.empty((m, n), dtype=torch.float32, device=device)
    for c, s in mats[:1]:
        mxq.mxq_linear(x, c, s, out=y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        c, s = mats[i % copies]
        mxq.mxq_linear(x, c, s, out=y)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / args.steps
    print(json.dumps({"case": args.case, "kernel": mxq.mxq_linear_plan_info(m, n, k)["kernel"], "launches": args.steps,
                      "us_per_call": us, "gbs": nbytes / us / 1e3, "bytes_per_call": nbytes,
                      "device_status": mxq.mxq_linear_device_status()}))


def run_case_batch(mxq, case: str, steps: int, device):
    """--case batch:LxM : mxq_linear_batch calls of L 7B layer sets (7 L layers per launch) at M token rows, launched
    `steps` times over distinct weights (together larger than L2): the small case profiler captures of the persistent
    kernel run on."""
    lsets, m = (int(v) for v in case.split(":")[1].split("x"))
    copies = max(2, 300 // (108 * lsets) + 1)
    gen = torch.Generator(device=device).manual_seed(7)
    x = {k: synth.normal_bf16((m, k), 1.0, 3 + k, device) for k in (4096, 11008)}
    batches, nbytes = [], 0
    for _ in range(copies):
        lays = []
        for _ in range(lsets):
            for _, n, k in synth.LAYERS_7B:
                lays.append(dict(x=x[k], codes=torch.randint(0, 256, (n, k // 2), dtype=torch.uint8, device=device, generator=gen),
                                 scales=torch.randint(110, 126, (n, k // 32), dtype=torch.uint8, device=device, generator=gen),
                                 out=torch.empty((m, n), dtype=torch.float32, device=device)))
        batches.append(mxq.LinearBatch(lays))
        nbytes = sum(algorithmic_bytes(m, d["codes"].shape[0], d["x"].shape[1]) for d in lays)
    ws = mxq.new_workspace(batches[0].workspace_bytes(), device)
    batches[0].run(ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        batches[i % copies].run(ws)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / steps

    def all_copies():
        for b in batches:
            b.run(ws)
    graph_us = time_graph(all_copies, 10) / copies * 1e6
    print(json.dumps({"case": case, "launches": steps, "us_per_call_from_python": us, "us_per_call": graph_us,
                      "gbs": nbytes / graph_us / 1e3, "bytes_per_call": nbytes, "layout": batches[0].info(),
                      "device_status": mxq.mxq_linear_device_status()}))


def run_case_other(mxq, case: str, steps: int, device):
    """--case quantize:NxK (direct cast of `steps` distinct BF16 matrices, rotated), accept:BxRxV (greedy accept of FP32
    logits, T = R - 1), bf16:NxKxM (the unquantised comparison layer), swiglu:FxKxM (gate / up rows interleaved, 2F x K
    weights, SiLU(gate) * up in the epilogue) or residual:NxKxM (residual add in the epilogue): the small cases profiler
    captures of those kernels run on."""
    op, dims = case.split(":")
    dims = [int(v) for v in dims.split("x")]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if op == "quantize":
        n, k = dims
        copies = max(2, min(8, int(400e6 // (n * k * 2)) + 1))
        ws_ = [synth.student_t_bf16((n, k), 0.02, 1 + i, device=device) for i in range(copies)]
        codes = torch.empty((n, k // 2), dtype=torch.uint8, device=device)
        scales = torch.empty((n, k // 32), dtype=torch.uint8, device=device)
        mxq.mxq_quantize(ws_[0], codes, scales)
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            mxq.mxq_quantize(ws_[i % copies], codes, scales)
        e1.record()
        nbytes = n * k * 2.53125

        def all_copies():
            for w_ in ws_:
                mxq.mxq_quantize(w_, codes, scales)
        graph_us = time_graph(all_copies, 10) / copies * 1e6
    elif op in ("swiglu", "residual"):
        n, k, m = dims
        rows = 2 * n if op == "swiglu" else n
        nbytes = algorithmic_bytes(m, rows, k, 2) - (2 * m * n if op == "swiglu" else -2 * m * n)   # BF16 out (half as many for gate / up), + the residual
        copies = max(2, min(8, int(200e6 // nbytes) + 1))
        gen = torch.Generator(device=device).manual_seed(7)
        mats = [(torch.randint(0, 256, (rows, k // 2), dtype=torch.uint8, device=device, generator=gen),
                 torch.randint(110, 126, (rows, k // 32), dtype=torch.uint8, device=device, generator=gen)) for _ in range(copies)]
        x = synth.normal_bf16((m, k), 1.0, 3, device)
        res = synth.normal_bf16((m, n), 1.0, 4, device)
        y = torch.empty((m, n), dtype=torch.bfloat16, device=device)
        ws = torch.empty(max(16, mxq.mxq_linear_fused_workspace_bytes(m, rows, k)), dtype=torch.uint8, device=device)

        def call(c, s_):
            if op == "swiglu":
                mxq.mxq_linear_swiglu(x, c, s_, out=y, workspace=ws)
            else:
                mxq.mxq_linear_residual(x, c, s_, res, out=y, workspace=ws)
        call(*mats[0])
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            call(*mats[i % copies])
        e1.record()

        def all_copies():
            for c, s_ in mats:
                call(c, s_)
        graph_us = time_graph(all_copies, 10) / copies * 1e6
    elif op == "bf16":
        n, k, m = dims
        copies = max(2, min(8, int(400e6 // (n * k * 2)) + 1))
        ws_ = [synth.normal_bf16((n, k), 0.02, 1 + i, device=device) for i in range(copies)]
        x = synth.normal_bf16((m, k), 1.0, 3, device)
        y = torch.empty((m, n), dtype=torch.float32, device=device)
        mxq.mxq_linear_bf16(x, ws_[0], out=y)
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            mxq.mxq_linear_bf16(x, ws_[i % copies], out=y)
        e1.record()
        nbytes = n * k * 2 + 2 * m * k + 4 * m * n

        def all_copies():
            for w_ in ws_:
                mxq.mxq_linear_bf16(x, w_, out=y)
        graph_us = time_graph(all_copies, 10) / copies * 1e6
    else:
        b, r, v = dims
        lg, draft, _, _ = synth.accept_trials(b, r - 1, r, v, seed=1, device=device)
        ws = mxq.new_workspace(mxq.mxq_accept_workspace_bytes(b, r, v), device)
        mxq.mxq_greedy_accept(lg, draft, workspace=ws)
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            mxq.mxq_greedy_accept(lg, draft, workspace=ws)
        e1.record()
        nbytes = lg.numel() * 4
        graph_us = time_graph(lambda: mxq.mxq_greedy_accept(lg, draft, workspace=ws), 10) * 1e6
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / steps
    print(json.dumps({"case": case, "launches": steps, "us_per_call_from_python": us, "us_per_call": graph_us,
                      "gbs": nbytes / graph_us / 1e3, "bytes_per_call": nbytes,
                      "note": "us_per_call: replayed CUDA graph; from_python adds the host launch overhead"}))


def run_reference(args):
    rank, _, world = replicas.env_world()
    if rank != 0:
        return
    import numpy as np

    import oracle
    m = args.m
    frac = 8  # every 8th row of each matrix: a bounded sample of the layer set
    mats = []
    for i, (name, n, k) in enumerate(synth.LAYERS_7B):
        rng = np.random.default_rng(i)
        rows = np.arange(0, n, frac, dtype=np.int64)
        mats.append((n, k, rows, rng.integers(0, 256, (n, k // 2), dtype=np.uint8),
                     rng.integers(110, 126, (n, k // 32), dtype=np.uint8),
                     synth.bits_of(synth.normal_bf16((m, k), 1.0, 5 + i))))
    nbytes = sum(algorithmic_bytes(m, len(rows), k) for n, k, rows, *_ in mats)

    def one():
        for n, k, rows, codes, scales, x in mats:
            oracle.linear(x, codes, scales, rows=rows)

    for _ in range(args.warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one()
    secs = time.perf_counter() - t0
    value = nbytes * args.steps / secs / 1e9
    sample = "every %dth output row of one 7B layer set per step (%.1fM weights), M=%d, FP64" % (
        frac, sum(len(r) * k for _, k, r, *_ in mats) / 1e6, m)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "7B decode layer set, M=%d (CPU oracle, bounded sample)" % m, "M": m, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--layers", type=int, default=32, help="distinct 7B layer sets per step")
    ap.add_argument("--m", type=int, default=1, help="token rows (1 = draft step)")
    ap.add_argument("--route", choices=["batch", "separate"], default="batch",
                    help="batch: mxq_linear_batch, --layers-per-call layer sets per launch; separate: one mxq_linear call per layer")
    ap.add_argument("--streams", type=int, default=2,
                    help="batch route: the step's independent mxq_linear_batch calls are issued round-robin on this many streams (a workspace each)")
    ap.add_argument("--layers-per-call", type=int, default=8, help="layer sets (7 layers each) per mxq_linear_batch call, 1..9")
    ap.add_argument("--no-graph", action="store_true", help="launch from Python instead of replaying a CUDA graph")
    ap.add_argument("--quick", action="store_true", help="skip the extra measurements")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--case", default=None, metavar="NxKxM",
                    help="instead of the benchmark: launch this one mxq_linear shape --steps times (profiler captures)")
    args = ap.parse_args()
    if args.case:
        run_case(args)
        return
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
