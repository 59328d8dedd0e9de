#!/usr/bin/env python
"""Benchmark of the HLQ LUT-GEMM hot path on B200.

A "step" is one pass of the whole hot path (table build, weight stream, look-up/accumulate,
per-plane scales, offset term, K-split reduce) over one batch of synthetic input: by default the
twelve M = 1 decode linears of the LLaMA-3.1-8B shapes at q in {2,3,4}, G = 128.  One JSON line is
printed by rank 0:

  value       achieved GB/s = algorithmic bytes of the step (bit-planes + fp16 scales + fp16 offsets +
              X + Y, summed over the calls) / device time, inputs resident in HBM.  M = 1 workloads run
              the step through the chained decode entry (elutq_chain_run: the list of calls in one
              persistent launch); the same step as separate elutq_lut_gemm calls replayed
              from a CUDA graph is timed beside it (`secondary`).  The working set of a step exceeds
              the L2 capacity
  e2e         the same metric with host buffers, host<->device transfers inside the timed region: M = 1
              workloads through elutq_chain_run_host (all X in one pinned host arena, fetched by a small kernel;
              Y stored into a pinned host arena), the others through elutq_lut_gemm_host per call
  roofline    achieved / measured HBM copy bandwidth for the decode kernel
  cpu_baseline  the fp64 oracle timed on the host cores on a bounded sample of the same workload
  secondary   short same-run measurements of the other configurations (70B decode, one 2-bit GEMV
              isolated / L2-hot, small-batch sweep, prefill, 32-layer stack), each with its own roofline
              fraction; their inputs are drawn on the device (same shapes and distributions)

`--impl reference` times the oracle alone (the only reference there is: the paper ships no code).
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

import workloads  # noqa: E402
from workloads import synth  # noqa: E402

METRIC = "HLQ LUT-GEMM achieved HBM GB/s at M=1, 8B shapes (us/call alongside)"
UNIT = "GB/s"
FALLBACK_TENSOR_TFLOPS = 1400.0
FALLBACK_HBM_GBS = 6650.0


def _calls(name: str):
    if name.startswith("custom:"):
        # custom:q:N:K[:M],q:N:K[:M],...  (G = 128) - used for profiler captures of single shapes
        out = []
        for i, spec in enumerate(name[len("custom:"):].split(",")):
            f = [int(x) for x in spec.split(":")]
            out.append(workloads.shapes.Call(f"custom{i}", f[3] if len(f) > 3 else 1, f[1], f[2], f[0]))
        return out
    return {
        "cfg0": workloads.config0,
        "cfg1": workloads.config1_calls,
        "cfg2": workloads.config2_calls,
        "cfg3": workloads.config3_calls,
        "cfg4_prefill": workloads.config4_prefill_calls,
        "cfg4_stack": workloads.config4_stack_calls,
    }[name]()


WORKLOAD_NAMES = {
    "cfg0": "config 0: single 2-bit GEMV M=1 N=K=4096 G=128",
    "cfg1": "config 1: LLaMA-3.1-8B decode linears (qkv, o, gate_up, down) at M=1, q in {2,3,4}, G=128",
    "cfg2": "config 2: small-batch sweep on the 8B shapes, q in {2,3}, M in {1..32}, outlier activations",
    "cfg3": "config 3: LLaMA-3.1-70B decode linears at M=1, q in {2,3}, G=128",
    "cfg4_prefill": "config 4a: prefill-sized GEMM on the 8B shapes, q=2, M in {128,512,2048}",
    "cfg4_stack": "config 4b: 32-layer LLaMA-3.1-8B linear stack at M=1, q=2",
}


def _bytes_of(calls) -> int:
    return sum(workloads.algorithmic_bytes(c.M, c.N, c.K, c.q, c.G) for c in calls)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier pool measurement, MEASURED_PEAKS.json absent)"


def _tensor_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json bf16_tflops_sustained, cuBLAS)"
    except Exception:
        return FALLBACK_TENSOR_TFLOPS, "fallback (earlier pool measurement, sustained, MEASURED_PEAKS.json absent)"


def _traffic_note():
    """Per-launch DRAM traffic of the decode kernel from the committed ncu summary, if present."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as f:
            return json.load(f)
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int, period_ms: int = 20):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", str(period_ms), "-i", str(device_index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def wait_first(self, timeout_s: float = 5.0) -> None:
        """Returns when the first sample has arrived (nvidia-smi can take a second to start), or after the timeout."""
        t_end = time.time() + timeout_s
        while self.proc is not None and not self.rows and time.time() < t_end and self.proc.poll() is None:
            time.sleep(0.01)

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        inside = [r for (t, r) in self.rows if t0 <= t <= t1 + 0.05] or [r for (_, r) in self.rows]
        sm, smax, reasons = [], [], set()
        for r in inside:
            p = [x.strip() for x in r.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0]))
                smax.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# reference arm: the oracle on the host cores
# ---------------------------------------------------------------------------------------------

def _oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return len(os.sched_getaffinity(0))


def _oracle_sample(calls, rows_per_layer: int, seed: int):
    """Row-sampled sub-problems of the calls: (X, planes, scales, offsets, G, bytes)."""
    out = []
    for c in calls:
        n = min(c.N, rows_per_layer)
        rows = np.arange(n)
        Gn = c.K // c.G
        out.append((synth.activations(seed, c.tag + "/x", c.M, c.K, outliers=c.outliers),
                    synth.bit_planes(seed, c.tag, c.q, c.N, c.K, rows=rows),
                    synth.scales(seed, c.tag, c.N, Gn, c.q, rows=rows),
                    synth.offsets(seed, c.tag, c.N, Gn, rows=rows),
                    c.G, workloads.algorithmic_bytes(c.M, n, c.K, c.q, c.G)))
    return out


def _time_oracle(sample, steps: int, warmup: int):
    from oracle import hlq
    for _ in range(warmup):
        for (X, p, s, z, G, _) in sample[:1]:
            hlq.matmul(X, p, s, z, G)
    t0 = time.perf_counter()
    for _ in range(steps):
        for (X, p, s, z, G, _) in sample:
            hlq.matmul(X, p, s, z, G)
    dt = (time.perf_counter() - t0) / steps
    nbytes = sum(b for *_, b in sample)
    return nbytes / dt / 1e9, dt


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    calls = _calls(args.workload)
    # size the per-step sample so that steps + warmup passes of the oracle end within about two minutes
    probe_rows = 16
    _, probe_dt = _time_oracle(_oracle_sample(calls, probe_rows, seed=0), 1, 0)
    budget_s = 100.0 / (args.steps + 1)
    rows = int(max(8, min(1024, probe_rows * budget_s / max(probe_dt, 1e-6))))
    rows -= rows % 8
    sample = _oracle_sample(calls, rows, seed=0)
    gbs, dt = _time_oracle(sample, args.steps, min(args.warmup, 1))
    cores = _oracle_threads()
    desc = f"first {rows} output rows of each of the {len(calls)} layers per step (fp64 numpy oracle)"
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAMES[args.workload], "sample": desc},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------

def max_over_ranks(values_ms, device="cuda"):
    """Element-wise maximum of per-rank timings over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values_ms), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_value(step_bytes: int, world: int, ms_per_step: float) -> float:
    """Whole-job GB/s: every rank processes its own batch of step_bytes in the (max-over-ranks) step time."""
    return world * step_bytes / (ms_per_step * 1e-3) / 1e9


MIN_TIMED_SECONDS = 0.2      # the timed region replays the step until it lasts at least this long


def _device_layer(torch, elutq, c, gen):
    """Packed layer with inputs drawn on the device (timing-only: same shapes and distributions as the recipe)."""
    Gn = c.K // c.G
    planes = torch.randint(0, 2, (c.q, c.N, c.K), dtype=torch.uint8, device="cuda", generator=gen)
    scales = (torch.randn((c.N, Gn, c.q), device="cuda", generator=gen) * 0.02).abs().to(torch.float16)
    offsets = (torch.randn((c.N, Gn), device="cuda", generator=gen) * 0.01).to(torch.float16)
    packed = elutq.elutq_pack(planes, scales, offsets, c.q, c.G, c.N, c.K)
    torch.cuda.synchronize()
    return packed


class _Runner:
    """One step of a call list, replayed over rotating copies of its buffers: as one chain (M = 1 lists) or as a
    CUDA graph of separate C-ABI calls."""

    def __init__(self, torch, elutq, sets, mode, stream, flags=0):
        self.torch, self.elutq, self.sets, self.mode, self.stream = torch, elutq, sets, mode, stream
        self.copies = len(sets)
        self.n = len(sets[0])
        self.plans, self.graphs = [], []
        with torch.cuda.stream(stream):
            if mode == "chain":
                for st in sets:
                    self.plans.append(elutq.elutq_chain_plan(
                        [(l["X"], l["packed"], l["Y"], l["call"].N, l["call"].K) for l in st], stream=stream))
                self.one(0)
                stream.synchronize()
                c0 = elutq.elutq_launch_count()
                self.one(0)
                self.launches_per_step = int(elutq.elutq_launch_count() - c0)
            else:
                self._eager(0, flags)          # allocates the library's scratch before capture
                stream.synchronize()
                c0 = elutq.elutq_launch_count()
                self._eager(0, flags)
                self.launches_per_step = int(elutq.elutq_launch_count() - c0)
                stream.synchronize()
                for r in range(self.copies):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        self._eager(r, flags)
                    self.graphs.append(g)
            stream.synchronize()

    def _eager(self, r, flags):
        for l in self.sets[r]:
            c = l["call"]
            if flags:
                self.elutq.elutq_lut_gemm_ws(l["X"], l["packed"], l["Y"], c.M, c.N, c.K, flags, l["ws"], stream=self.stream)
            else:
                self.elutq.elutq_lut_gemm(l["X"], l["packed"], l["Y"], c.M, c.N, c.K, stream=self.stream)

    def one(self, i):
        r = i % self.copies
        if self.mode == "chain":
            self.elutq.elutq_chain_run(self.plans[r], self.n, stream=self.stream)
        else:
            self.graphs[r].replay()

    def timed(self, steps, warmup, barrier=None):
        """Device time (ms) of exactly steps * reps steps; reps makes the region last MIN_TIMED_SECONDS."""
        torch = self.torch
        with torch.cuda.stream(self.stream):
            for i in range(warmup):
                self.one(i)
            self.stream.synchronize()
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            probe = max(3, min(steps, 20))
            p0.record(self.stream)
            for i in range(probe):
                self.one(i)
            p1.record(self.stream)
            self.stream.synchronize()
            per = max(p0.elapsed_time(p1) / probe, 1e-4)
            reps = max(1, int(-(-MIN_TIMED_SECONDS * 1e3 // (per * steps))))
            if barrier:
                barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.time()
            e0.record(self.stream)
            for i in range(steps * reps):
                self.one(i)
            e1.record(self.stream)
            if barrier:
                barrier()
            self.stream.synchronize()
            t1 = time.time()
            return e0.elapsed_time(e1), reps, t0, t1

    def status(self):
        if self.mode == "chain":
            return max(self.elutq.elutq_chain_status(p, stream=self.stream) for p in self.plans)
        return self.elutq.elutq_device_status(self.stream)

    def close(self):
        for p in self.plans:
            self.elutq.elutq_chain_forget(p)
        self.plans, self.graphs = [], []


def _make_sets(torch, elutq, layers, l2_bytes, flags=0, max_copies=8):
    """Rotating copies of the packed layers (and X / Y) so that >= 3x L2 is touched between two uses of a copy."""
    working_set = sum(l["packed"].numel() for l in layers)
    copies = max(1, min(max_copies, -(-3 * l2_bytes // max(working_set, 1))))
    if copies * working_set > (24 << 30):
        copies = 1
    sets = [layers]
    for _ in range(1, copies):
        dup = []
        for l in layers:
            c = l["call"]
            d = dict(l)
            d["packed"] = l["packed"].clone()
            elutq.elutq_describe(d["packed"], c.N, c.K)
            d["X"] = l["X"].clone()
            d["Y"] = torch.empty_like(l["Y"])
            if flags:
                d["ws"] = torch.empty_like(l["ws"])
                elutq.elutq_workspace_init(d["ws"])
            dup.append(d)
        sets.append(dup)
    torch.cuda.synchronize()
    return sets, copies, working_set


def _secondary(torch, elutq, name, stream, l2_bytes, hbm_peak, tensor_peak, device_index):
    """Short same-run measurement of another configuration; inputs drawn on the device."""
    calls = _calls(name)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234)
    cache = {}
    layers = []
    for c in calls:
        key = (c.q, c.G, c.N, c.K) if name != "cfg4_stack" else (c.name,)
        if key not in cache:
            cache[key] = _device_layer(torch, elutq, c, gen)
        X = torch.randn((c.M, c.K), device="cuda", generator=gen).to(torch.float16)
        layers.append(dict(call=c, packed=cache[key], X=X, Y=torch.empty((c.M, c.N), dtype=torch.float16, device="cuda")))
    step_bytes = _bytes_of(calls)
    all_m1 = all(c.M == 1 for c in calls)
    tensor = all(c.M >= 9 and c.G == 128 for c in calls)           # (every call a tensor-core contraction at any N)
    # distinct blobs are shared between the calls of a step here, so rotate whole copies only while they are small
    distinct = sum(t.numel() for t in cache.values())
    out = {"workload": WORKLOAD_NAMES[name], "calls_per_step": len(calls), "algorithmic_bytes_per_step": step_bytes,
           "data": "synthetic, drawn on the device (timing only)"}
    results = {}
    for mode in (("chain", "graph") if all_m1 else ("graph",)):
        sets = [layers]
        copies = 1
        if distinct < 3 * l2_bytes:
            copies = max(1, min(8, -(-3 * l2_bytes // max(distinct, 1))))
            sets = [layers]
            for _ in range(1, copies):
                dup_cache = {k: v.clone() for k, v in cache.items()}
                dup = []
                for l in layers:
                    c = l["call"]
                    key = (c.q, c.G, c.N, c.K) if name != "cfg4_stack" else (c.name,)
                    elutq.elutq_describe(dup_cache[key], c.N, c.K)
                    dup.append(dict(call=c, packed=dup_cache[key], X=l["X"].clone(), Y=torch.empty_like(l["Y"])))
                sets.append(dup)
        runner = _Runner(torch, elutq, sets, mode, stream)
        sampler = ClockSampler(device_index)
        sampler.wait_first()
        ms, reps, t0, t1 = runner.timed(10, 5)
        clocks = sampler.stop(t0, t1)
        ms_step = ms / (10 * reps)
        r = {"ms_per_step": ms_step, "us_per_call_mean": ms_step * 1e3 / len(calls), "launches_per_step": runner.launches_per_step,
             "device_status": runner.status(), "clocks": clocks,
             "l2": f"{copies} rotating copies of the distinct layers ({copies * distinct / l2_bytes:.1f}x L2)"}
        if tensor:
            tf = sum(2.0 * c.M * c.N * c.K for c in calls) / (ms_step * 1e-3) / 1e12
            r.update({"bound": "tensor", "achieved": tf, "unit": "TFLOP/s", "peak": tensor_peak, "frac": tf / tensor_peak})
        else:
            gbs = step_bytes / (ms_step * 1e-3) / 1e9
            r.update({"bound": "hbm", "achieved": gbs, "unit": "GB/s", "peak": hbm_peak, "frac": gbs / hbm_peak})
        results["chain (elutq_chain_run)" if mode == "chain" else "separate calls (CUDA graph)"] = r
        runner.close()
        del runner, sets
    out["runs"] = results
    if name == "cfg0":
        # one 2-bit GEMV, isolated (one launch between two synchronisations) and L2-hot (the same blob again and again):
        # labelled figures, not HBM-roofline figures
        l = layers[0]
        c = l["call"]
        with torch.cuda.stream(stream):
            ts = []
            for _ in range(60):
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                stream.synchronize()
                a0.record(stream)
                elutq.elutq_lut_gemm(l["X"], l["packed"], l["Y"], c.M, c.N, c.K, stream=stream)
                a1.record(stream)
                stream.synchronize()
                ts.append(a0.elapsed_time(a1) * 1e3)
            ts = sorted(ts[10:])
            hot = _Runner(torch, elutq, [layers], "graph", stream)
            ms, reps, _, _ = hot.timed(50, 10)
            out["isolated_call_us_median"] = ts[len(ts) // 2]
            out["l2_hot_us_per_call"] = ms * 1e3 / (50 * reps)
            out["isolated_note"] = "one elutq_lut_gemm between two stream synchronisations (launch latency included); " \
                                   "L2-hot: the same 5 MB blob replayed back to back from a graph; neither is an HBM figure"
            hot.close()
    for t in cache.values():
        elutq.elutq_forget(t)
    del layers, cache
    torch.cuda.empty_cache()
    return out


def run_cuda(args) -> None:
    import torch
    import torch.distributed as dist

    import paper_2510_19482_b200 as elutq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")

    calls = _calls(args.workload)
    seed = rank           # every rank works on its own, independently drawn batch (weak scaling, no exchange)

    # ---- build the workload: pack each layer once (offline step), keep X / Y per call --------------
    layers = []
    for c in calls:
        lay = workloads.hlq_layer(seed, c.tag, c.q, c.G, c.N, c.K)
        planes = torch.from_numpy(lay.planes).cuda()
        scales = torch.from_numpy(lay.scales.view(np.int16)).cuda().view(torch.float16)
        offsets = torch.from_numpy(lay.offsets.view(np.int16)).cuda().view(torch.float16)
        packed = elutq.elutq_pack(planes, scales, offsets, c.q, c.G, c.N, c.K)
        torch.cuda.synchronize()
        del planes, scales, offsets, lay
        Xh = torch.from_numpy(synth.activations(seed, c.tag + "/x", c.M, c.K, outliers=c.outliers).view(np.int16)) \
            .view(torch.float16).pin_memory()
        Yh = torch.empty((c.M, c.N), dtype=torch.float16).pin_memory()
        layers.append(dict(call=c, packed=packed, X=Xh.cuda(), Y=torch.empty((c.M, c.N), dtype=torch.float16, device="cuda"),
                           Xh=Xh, Yh=Yh))
    step_bytes = _bytes_of(calls)

    if args.flags:
        # variant runs go through the caller-workspace entry point, one workspace per call
        for l in layers:
            c = l["call"]
            l["ws"] = torch.empty(elutq.elutq_workspace_bytes(c.M, c.N, c.K), dtype=torch.uint8, device="cuda")
            elutq.elutq_workspace_init(l["ws"])
        torch.cuda.synchronize()

    # HBM-cold protocol: consecutive steps rotate over distinct copies of the packed layers (and of X / Y) so
    # that the bytes touched between two uses of the same copy are at least 3x the L2 capacity
    l2_bytes = int(getattr(torch.cuda.get_device_properties(local_rank), "L2_cache_size", 126 << 20))
    layer_sets, copies, working_set = _make_sets(torch, elutq, layers, l2_bytes, args.flags)

    stream = torch.cuda.Stream()
    use_chain = all(c.M == 1 for c in calls) and not args.flags and not args.no_chain and not args.no_graph
    peak, peak_src = _peaks()
    tpeak, tsrc = _tensor_peak()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.no_graph:
        # plain stream of C-ABI calls (no graph, no chain): a debugging mode
        class _Eager(_Runner):
            def __init__(self):
                self.torch, self.elutq, self.sets, self.mode, self.stream = torch, elutq, layer_sets, "eager", stream
                self.copies, self.n, self.plans, self.graphs = copies, len(layers), [], []
                with torch.cuda.stream(stream):
                    c0 = elutq.elutq_launch_count()
                    self._eager(0, args.flags)
                    stream.synchronize()
                    self.launches_per_step = int(elutq.elutq_launch_count() - c0)

            def one(self, i):
                self._eager(i % self.copies, args.flags)
        main = _Eager()
    else:
        main = _Runner(torch, elutq, layer_sets, "chain" if use_chain else "graph", stream, args.flags)

    # ---- device-resident timing -------------------------------------------------------------
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.wait_first()
    ms, reps, t_wall0, t_wall1 = main.timed(args.steps, args.warmup, barrier)
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    launches = main.launches_per_step * args.steps * reps
    main_status = main.status()

    # ---- spread of single steps (separate pass; the headline above is the timed region) --------------
    with torch.cuda.stream(stream):
        spread_n = max(3, min(args.steps, 200))
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(spread_n + 1)]
        evs[0].record(stream)
        for i in range(spread_n):
            main.one(i)
            evs[i + 1].record(stream)
        stream.synchronize()
        singles = sorted(evs[i].elapsed_time(evs[i + 1]) for i in range(spread_n))
        ms_median, ms_min = singles[len(singles) // 2], singles[0]

    # ---- the same step as separate calls (when the headline is the chain) ------------------------------
    separate = None
    graph_runner = main if (not use_chain and not args.no_graph) else None
    if use_chain:
        graph_runner = _Runner(torch, elutq, layer_sets, "graph", stream)
        sms, sreps, _, _ = graph_runner.timed(min(args.steps, 200), min(args.warmup, 20))
        sms_step = sms / (min(args.steps, 200) * sreps)
        sg = step_bytes / (sms_step * 1e-3) / 1e9
        separate = {"ms_per_step": sms_step, "us_per_call_mean": sms_step * 1e3 / len(calls), "achieved": sg, "unit": "GB/s",
                    "frac": sg / peak, "launches_per_step": graph_runner.launches_per_step,
                    "launch": "the same step as separate elutq_lut_gemm calls, CUDA graph, programmatic dependent launch"}

    # ---- end to end through the host entry point ---------------------------------------------
    # (a CUDA graph of the public host-buffer calls, whose copy nodes read the pinned inputs and write the pinned
    #  outputs on every replay)
    host_chain = None
    if use_chain:
        # The chained step with host buffers: every call's X in one pinned host arena and every Y in another; a step
        # is one copy in and the chain's launches (elutq_chain_run_host), which write Y into the host arena.
        x_off, y_off = [0], [0]
        for l in layers:
            c = l["call"]
            x_off.append(x_off[-1] + (c.K + 127) // 128 * 128)
            y_off.append(y_off[-1] + (c.N + 127) // 128 * 128)
        xh_arena = torch.zeros(x_off[-1], dtype=torch.float16).pin_memory()
        yh_arena = torch.zeros(y_off[-1], dtype=torch.float16).pin_memory()
        for i, l in enumerate(layers):
            xh_arena[x_off[i]:x_off[i] + l["call"].K] = l["Xh"].reshape(-1)
        xd_arena = torch.zeros(x_off[-1], dtype=torch.float16, device="cuda")
        # the calls' Y point into the pinned host arena: the reduction's stores cross the bus during the launch
        plan_h = elutq.elutq_chain_plan([(xd_arena[x_off[i]:], l["packed"], yh_arena[y_off[i]:], l["call"].N, l["call"].K)
                                         for i, l in enumerate(layers)])
        host_chain = {"plan": plan_h, "h2d": xh_arena.numel() * 2, "d2h": sum(2 * l["call"].N for l in layers)}

    def step_host():
        if host_chain is not None:
            elutq.elutq_chain_run_host(host_chain["plan"], len(layers), xd_arena, xh_arena, stream=stream)
            return
        for l in layers:
            c = l["call"]
            elutq.elutq_lut_gemm_host(l["Xh"], l["packed"], l["Yh"], c.M, c.N, c.K, stream=stream)

    e2e_steps = max(1, min(args.steps, 200))
    with torch.cuda.stream(stream):
        step_host()
        stream.synchronize()
        host_graph = None
        if not args.no_graph and host_chain is None:
            host_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(host_graph, stream=stream):
                step_host()

        def run_host():
            if host_graph is not None:
                host_graph.replay()
            else:
                step_host()

        for _ in range(min(args.warmup, 20)):
            run_host()
        barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(e2e_steps):
            run_host()
        h1.record(stream)
        barrier()
        ms_host = h0.elapsed_time(h1)
        host_chain_bytes, e2e_how = None, "elutq_lut_gemm_host per call (pinned host X in, Y out), CUDA graph"
        if host_chain is not None:
            host_chain_bytes = (host_chain["h2d"], host_chain["d2h"])
            e2e_how = ("elutq_chain_run_host: a fetch kernel reads the pinned host arena of all X across the bus, then the chain's launch, "
                       "whose calls have their Y in a pinned host arena (the reduction stores straight into host memory), per step")
            e2e_status = elutq.elutq_chain_status(host_chain["plan"], stream=stream)
            if e2e_status:
                e2e_how += f"; DEVICE STATUS {e2e_status:#x}"
            elutq.elutq_chain_forget(host_chain["plan"])

        # ---- per-call times: marginal device time of one extra call inside the graph-replayed step -------
        # (the extra call reads its own copy of the packed layer, so it is HBM-cold like the others and
        #  does not warm the L2 for the step's own call)
        per_call = []
        if rank == 0 and not args.no_per_call and graph_runner is not None:
            reps_pc = max(20, min(args.steps, 300))
            graph = graph_runner.graphs[0]

            def time_graph(g):
                for _ in range(3):
                    g.replay()
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a0.record(stream)
                for _ in range(reps_pc):
                    g.replay()
                a1.record(stream)
                stream.synchronize()
                return a0.elapsed_time(a1) * 1e3 / reps_pc

            seen = {}
            for l in layers:
                c = l["call"]
                key = (c.name.split(".")[-1], c.q, c.M, c.N, c.K)
                if key in seen:
                    continue
                seen[key] = True
                clone = l["packed"].clone()
                elutq.elutq_describe(clone, c.N, c.K)
                Y2 = torch.empty_like(l["Y"])
                g2 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g2, stream=stream):
                    elutq.elutq_lut_gemm(l["X"], clone, Y2, c.M, c.N, c.K, stream=stream)
                    graph_runner._eager(0, 0)
                t_base = time_graph(graph)
                us = max(time_graph(g2) - t_base, 0.0)
                b = workloads.algorithmic_bytes(c.M, c.N, c.K, c.q, c.G)
                per_call.append({"name": key[0], "q": c.q, "M": c.M, "N": c.N, "K": c.K, "us": round(us, 3),
                                 "GBps": round(b / max(us, 1e-3) / 1e3, 1),
                                 "frac_of_hbm_peak": round(b / max(us, 1e-3) / 1e3 / peak, 3),
                                 "tflop_eq": round(2.0 * c.M * c.N * c.K / max(us, 1e-3) / 1e6, 3),
                                 "how": "marginal time of one extra separate call inside the graph-replayed step"})
                if c.M == 1:
                    # the same shape inside the chained entry: chains of n copies of the layer against chains of one, per
                    # extra call; the launches rotate over enough distinct blobs (more than twice the L2) that every
                    # call streams from HBM
                    n_in = 9
                    n_plans = max(2, -(-(2 * l2_bytes + (64 << 20)) // (n_in * l["packed"].numel())))
                    clones = [l["packed"].clone() for _ in range(n_plans * n_in)]
                    for cl in clones:
                        elutq.elutq_describe(cl, c.N, c.K)
                    Ys = [torch.empty_like(l["Y"]) for _ in range(n_in)]
                    plans_n = [elutq.elutq_chain_plan([(l["X"], clones[s_ * n_in + i], Ys[i], c.N, c.K) for i in range(n_in)])
                               for s_ in range(n_plans)]
                    plans_1 = [elutq.elutq_chain_plan([(l["X"], clones[s_ * n_in], Ys[0], c.N, c.K)]) for s_ in range(n_plans)]

                    def time_chain(plans, n):
                        for i_ in range(3):
                            elutq.elutq_chain_run(plans[i_ % len(plans)], n, stream=stream)
                        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a0.record(stream)
                        for i_ in range(reps_pc):
                            elutq.elutq_chain_run(plans[i_ % len(plans)], n, stream=stream)
                        a1.record(stream)
                        stream.synchronize()
                        return a0.elapsed_time(a1) * 1e3 / reps_pc

                    us_c = max(time_chain(plans_n, n_in) - time_chain(plans_1, 1), 0.0) / (n_in - 1)
                    per_call[-1].update({"us_in_chain": round(us_c, 3),
                                         "frac_of_hbm_peak_in_chain": round(b / max(us_c, 1e-3) / 1e3 / peak, 3),
                                         "how_in_chain": f"(chain of 9 copies of the layer - chain of 1) / 8, elutq_chain_run, "
                                                         f"launches rotating over {n_plans} sets of distinct blobs"})
                    st_ = [elutq.elutq_chain_status(pl) for pl in plans_n + plans_1]
                    if any(st_):
                        per_call[-1]["in_chain_device_status"] = [x_ for x_ in st_ if x_]
                    for pl in plans_n + plans_1:
                        elutq.elutq_chain_forget(pl)
                    for cl in clones:
                        elutq.elutq_forget(cl)
                    del clones, Ys, plans_n, plans_1
                elutq.elutq_forget(clone)
                del g2, clone, Y2

    # ---- the other configurations, measured briefly in the same run -----------------------------------
    secondary = []
    if rank == 0 and args.workload == "cfg1" and not args.no_secondary and not args.flags:
        main.close()
        if graph_runner is not None and graph_runner is not main:
            graph_runner.close()
        del main, graph_runner, layer_sets, host_graph
        for l in layers:
            elutq.elutq_forget(l["packed"])
        layers_meta = [l["call"] for l in layers]
        del layers
        torch.cuda.empty_cache()
        for name in ("cfg3", "cfg0", "cfg2", "cfg4_prefill", "cfg4_stack"):
            try:
                secondary.append(_secondary(torch, elutq, name, stream, l2_bytes, peak, tpeak, local_rank))
            except Exception as ex:      # a failed side measurement must not lose the headline
                secondary.append({"workload": WORKLOAD_NAMES[name], "error": repr(ex)})

    # ---- reduce over ranks ---------------------------------------------------------------------
    ms, ms_host = max_over_ranks([ms, ms_host])
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms / (args.steps * reps)
    value = aggregate_value(step_bytes, world, ms_per_step)
    e2e_value = aggregate_value(step_bytes, world, ms_host / e2e_steps)
    per_gpu = step_bytes / (ms_per_step * 1e-3) / 1e9
    traffic = _traffic_note() if args.workload == "cfg1" and not args.flags else None
    roofline = {"bound": "hbm", "achieved": per_gpu, "peak": peak, "unit": "GB/s", "frac": per_gpu / peak,
                "peak_source": peak_src,
                "traffic": traffic.get("dram_bytes_per_step") if traffic else None,
                "traffic_note": traffic.get("note") if traffic else None}
    tensor_path = all(c.M >= 9 and c.G == 128 for c in calls) and not (args.flags & 0x3F0)   # ELUTQ_TENSOR_MIN_M
    if tensor_path:
        # every call of the step is a dense contraction on the tensor cores: report FLOP/s against the measured
        # GEMM peak (the sustained figure, since the kernels are timed inside a long step)
        tf = sum(2.0 * c.M * c.N * c.K for c in calls) / (ms_per_step * 1e-3) / 1e12
        roofline = {"bound": "tensor", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak,
                    "peak_source": tsrc, "traffic": None,
                    "traffic_note": "fp16 operands, fp32 accumulation; fp16 and bf16 share one tensor-core rate"}

    # ---- CPU baseline: the oracle on a bounded sample of the same workload -------------------------
    cpu = None
    if not args.no_cpu_baseline:
        cpu = _cpu_baseline(calls)

    if use_chain:
        launch_desc = ("chained decode entry: elutq_chain_run, the list of calls in persistent launches "
                       f"({main_launches_per_step(launches, args.steps * reps)} per step), calls ordered as if run one after another")
    elif args.no_graph:
        launch_desc = "stream of C-ABI calls"
    else:
        launch_desc = "CUDA graph of C-ABI calls, programmatic dependent launch"
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_NAMES[args.workload], "calls_per_step": len(calls),
                   "us_per_call_mean": ms_per_step * 1e3 / len(calls),
                   "algorithmic_bytes_per_step": step_bytes, "packed_working_set_bytes": working_set,
                   "timed_region": f"{args.steps} steps x {reps} replays = {args.steps * reps} steps in {ms:.1f} ms",
                   "ms_per_step_median": ms_median, "ms_per_step_min": ms_min,
                   "l2": (f"no flush: consecutive steps rotate over {copies} distinct copies of the packed layers, "
                          f"{copies * working_set / l2_bytes:.1f}x the {l2_bytes >> 20} MiB L2 between two uses of a copy")
                         if copies * working_set >= 3 * l2_bytes
                         else "working set below 3x L2 (partly L2-hot number, not an HBM figure)",
                   "launch": launch_desc, "device_status": main_status,
                   "parallelism": "replicas only (independent batch per rank, no collective)"},
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": host_chain_bytes[0] if host_chain_bytes else sum(2 * c.M * c.K for c in calls),
                "d2h_bytes_per_step": host_chain_bytes[1] if host_chain_bytes else sum(2 * c.M * c.N for c in calls),
                "how": e2e_how},
        "gpu_launches": launches,
        "clocks": clocks,
        "cpu_baseline": cpu,
        "separate_calls": separate,
        "per_call": per_call,
        "secondary": secondary,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main_launches_per_step(launches: int, steps: int) -> int:
    return launches // max(steps, 1)


def _cpu_baseline(calls):
    """The oracle as it stands on a bounded sample: all cores, one thread, and one M = 32 call."""
    # a short probe sizes the sample for about 12 s of CPU work (bounded below and above)
    probe_rows = 256
    _, probe_dt = _time_oracle(_oracle_sample(calls, probe_rows, seed=0), 1, 0)
    rows = int(max(256, min(12288, probe_rows * 12.0 / max(probe_dt, 1e-3))))   # generation time bounds it too
    sample = _oracle_sample(calls, rows, seed=0)
    gbs, dt = _time_oracle(sample, 1, 0)
    cpu = {"value": gbs, "unit": UNIT, "cores": _oracle_threads(), "kind": "oracle",
           "sample": f"first {rows} output rows (or all, where a layer has fewer) of each of the {len(calls)} layers, "
                     f"one pass ({dt:.1f} s)"}
    try:
        from threadpoolctl import threadpool_limits
        small = _oracle_sample(calls, max(64, rows // 8), seed=0)
        with threadpool_limits(limits=1):
            g1, d1 = _time_oracle(small, 1, 0)
        cpu["single_thread"] = {"value": g1, "unit": UNIT, "cores": 1,
                                "sample": f"first {max(64, rows // 8)} output rows of each layer, one pass ({d1:.1f} s)"}
    except Exception as ex:
        cpu["single_thread"] = {"error": repr(ex)}
    try:
        c = workloads.shapes.Call("o", 32, 4096, 4096, 2)
        m32 = _oracle_sample([c], 2048, seed=0)
        g32, d32 = _time_oracle(m32, 1, 0)
        cpu["m32"] = {"value": g32, "unit": UNIT, "cores": _oracle_threads(), "tflop_eq": 2.0 * 32 * 2048 * 4096 / d32 / 1e12,
                      "sample": f"M = 32, first 2048 rows of the 4096 x 4096 2-bit layer, one pass ({d32:.1f} s)"}
    except Exception as ex:
        cpu["m32"] = {"error": repr(ex)}
    return cpu


def run_fit(args) -> None:
    """Offline step before the path: elutq_hlq_fit (Algorithm 1) on one dense fp16 layer, `fit:q:G:N:K`."""
    import torch

    import paper_2510_19482_b200 as elutq

    q, G, N, K = [int(x) for x in args.workload.split(":")[1:5]]
    t_max = 10
    W = torch.from_numpy(synth.dense_weights(0, "bench-fit", N, K).view(np.int16)).cuda().view(torch.float16)
    for _ in range(args.warmup):
        out = elutq.elutq_hlq_fit(W, q, G, t_max)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        out = elutq.elutq_hlq_fit(W, q, G, t_max)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import fit as ofit
        rows = max(1, min(N, (1 << 21) // K))
        Wh = synth.dense_weights(0, "bench-fit", N, K)[:rows]
        t0 = time.time()
        ofit.fit(Wh, q, G, t_max)
        dt = time.time() - t0
        cpu = {"value": rows * K / dt / 1e9, "unit": "Gweight/s", "cores": _oracle_threads(), "kind": "oracle",
               "sample": f"first {rows} rows ({dt:.1f} s)"}
    del out
    # fp64 pipe work per group and round: selection (1 + 2 * 2^q per weight), error-free right-hand sides are
    # integer; the (q+1)^3/3-ish solve is repeated by every lane.  Peak: 64 fp64 lanes per clock per SM.
    sel = G * (1 + 2 * (1 << q))
    solve = 32 * sum((q + 1 - c - 1) * (2 * (q + 1 - c - 1) + 3) for c in range(q + 1))
    ops = (N * K // G) * t_max * (sel + solve)
    peak = 148 * 64 * 1.965e9
    line = {"metric": "HLQ Algorithm-1 fit throughput", "value": N * K / (ms * 1e-3) / 1e9, "unit": "Gweight/s",
            "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"Algorithm 1 on a dense fp16 layer N={N} K={K}, q={q}, G={G}, T_max={t_max}"},
            "roofline": {"bound": "alu", "achieved": ops / (ms * 1e-3) / 1e12, "peak": peak / 1e12, "unit": "T fp64 lane-op/s",
                         "frac": ops / (ms * 1e-3) / peak,
                         "peak_source": "148 SMs x 64 fp64 lanes per clock x 1965 MHz (nominal unit count and clock)",
                         "traffic": None},
            "gpu_launches": args.steps, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg1",
                    help="one of %s, custom:q:N:K[:M],... (G = 128), or fit:q:G:N:K (the offline parameter fit)"
                         % ", ".join(sorted(WORKLOAD_NAMES)))
    ap.add_argument("--flags", type=lambda v: int(v, 0), default=0,
                    help="ELUTQ_FLAG_* bits for every call (kernel-variant comparisons; 0 = the default path)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-call", action="store_true")
    ap.add_argument("--no-chain", action="store_true", help="time M = 1 steps as separate calls only")
    ap.add_argument("--no-secondary", action="store_true", help="skip the short measurements of the other configurations")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="the timed region replays the K steps until it lasts this long (0: exactly K steps; profiler captures)")
    args = ap.parse_args()
    if args.workload.startswith("fit:"):
        args.steps = args.steps or 5
        args.warmup = max(args.warmup or 3, 3)
        run_fit(args)
        return
    if args.workload not in WORKLOAD_NAMES:
        if not args.workload.startswith("custom:"):
            ap.error("unknown workload")
        WORKLOAD_NAMES[args.workload] = "custom shapes " + args.workload[len("custom:"):]
    if args.steps is None:
        args.steps = 2000 if args.impl == "cuda" else 10
    if args.warmup is None:
        args.warmup = 200 if args.impl == "cuda" else 3
    if args.warmup < 3:
        args.warmup = 3
    globals()["MIN_TIMED_SECONDS"] = max(0.0, args.min_seconds)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
