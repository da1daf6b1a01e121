#!/usr/bin/env python
"""Benchmark of the conv-merging hot path on B200.

One step = one pass of the whole path over one batch of synthetic input: merge the run of
convolutions (dc_merge_chain: BN fold, composition, skip fold, repack) and run the merged
convolution forward over the batch (dc_conv_forward).  Headline workload: the MobileNetV2-1.0
inverted-residual block at 56x56, batch 64, bf16 (1x1 24->144, dw3x3, 1x1 144->24, skip folded ->
one 3x3 conv 24->24).  The default run also measures the stride-2 merge (cfg2), the cross-block
merge (cfg3) and the full depth-compressed MobileNetV2-1.0 (cfg4: with every valid span of a seeded
pattern merged, and cut by Algorithm 1 over the latency table measured on the spot) and reports them
under `per_config` of the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|cfg1|cfg2|cfg3|cfg4|vgg] [--impl reference]

Prints one JSON line (rank 0).  `value` = images/s with inputs resident in HBM; `e2e` = the same
through the host-buffer entry point with the copies inside the timed region; `roofline` = the
merged-conv kernel alone against the measured and the nominal HBM (or tensor) peak; `cpu_baseline`
= the fp64 oracle on the host cores (a baseline, not a target).  Kernel-only figures are the median
of at least 20 CUDA-graph replays after 3 warm-up replays, whatever --steps says.
"""
from __future__ import annotations

import argparse
import ctypes
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

WORKLOADS = {"cfg1": 1, "cfg2": 2, "cfg3": 3, "cfg4": 4}
METRIC = "merged-conv fwd TFLOP/s & images/s on 1 B200 vs roofline; merge latency us"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}      # the datasheet figures the target is stated against
L2_BYTES = 126 * 1024 * 1024
KERNEL_REPLAYS, KERNEL_WARMUPS = 24, 3


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"])}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def profiled_traffic(kernel, workload):
    """DRAM bytes per launch of `kernel` on `workload` from profiles/dram_traffic.md (written from an
    ncu capture by paper_2301_12187_b200/ncu_summary.py), or None when there is no capture or the
    kernel's source has changed since it was taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    try:
        lines = open(path).read().splitlines()
    except OSError:
        return None
    for line in lines:
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if len(cells) < 5 or cells[0] != kernel or cells[1] != workload:
            continue
        src = os.path.join(ROOT, "paper_2301_12187_b200", "csrc", cells[3])
        try:
            digest = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
        except OSError:
            return None
        return int(cells[2]) if digest == cells[4] else None
    return None


def conv_facts(shape_in, g):
    """Algorithmic flops and bytes of one conv launch: read x once, write y once, read W' once."""
    n, h, w, c = shape_in
    ho = (h + 2 * g.pad - g.k) // g.stride + 1
    wo = (w + 2 * g.pad - g.k) // g.stride + 1
    flops = 2.0 * n * ho * wo * g.c_out * g.c_in * g.k * g.k
    bytes_ = 2.0 * n * h * w * c + 2.0 * n * ho * wo * g.c_out + 2.0 * g.c_out * g.c_in * g.k * g.k + 4.0 * g.c_out
    return flops, bytes_, (n, ho, wo, g.c_out)


def roofline_entry(flops, abytes, seconds, peaks, peak_src):
    """Roofline of one kernel launch: bound by the slower of bytes / HBM peak and flops / tensor peak;
    the fraction against the measured peaks and, beside it, against the nominal 8 TB/s / 2.25 PFLOP/s."""
    t_hbm, t_tc = abytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_tc:
        r = {"bound": "hbm", "achieved": abytes / seconds / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        r = {"bound": "tensor", "achieved": flops / seconds / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    r["frac"] = r["achieved"] / r["peak"]
    nom = max(abytes / (NOMINAL_PEAKS["hbm_gbs"] * 1e9), flops / (NOMINAL_PEAKS["bf16_tflops"] * 1e12))
    r.update({"peak_source": peak_src, "frac_of_nominal": nom / seconds,
              "nominal": "slower of 8 TB/s HBM and 2.25 PFLOP/s dense bf16", "roofline_us": max(t_hbm, t_tc) * 1e6,
              "algorithmic_bytes": abytes, "flops": flops, "tflops": flops / seconds / 1e12})
    return r


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the load runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def count_since(self, t):
        return sum(1 for ts, _ in self.rows if ts >= t)

    def stop(self, t_begin, t_end):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ts, line in self.rows:
            if ts < t_begin or ts > t_end:
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def count_kernel_nodes(graph) -> int:
    """Kernel nodes of a captured CUDA graph (cudaGraphGetNodes / cudaGraphNodeGetType)."""
    rt = None
    for name in ("libcudart.so.12", "libcudart.so"):
        try:
            rt = ctypes.CDLL(name)
            break
        except OSError:
            continue
    if rt is None:
        return -1
    h = ctypes.c_void_p(graph.raw_cuda_graph())
    n = ctypes.c_size_t(0)
    if rt.cudaGraphGetNodes(h, None, ctypes.byref(n)) != 0:
        return -1
    nodes = (ctypes.c_void_p * n.value)()
    rt.cudaGraphGetNodes(h, nodes, ctypes.byref(n))
    kernels = 0
    for i in range(n.value):
        t = ctypes.c_int(-1)
        rt.cudaGraphNodeGetType(ctypes.c_void_p(nodes[i]), ctypes.byref(t))
        kernels += 1 if t.value == 0 else 0
    return kernels


def replay_stats(graph, stream, per_replay, replays=KERNEL_REPLAYS, warmups=KERNEL_WARMUPS):
    """Median / min / max time (us) of one unit of work: the graph holds `per_replay` units and is
    replayed `replays` times, each replay timed by its own pair of CUDA events on `stream`."""
    import torch
    for _ in range(warmups):
        graph.replay()
    stream.synchronize()
    ts = []
    for _ in range(replays):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        stream.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e3 / per_replay)
    return {"median": float(np.median(ts)), "min": float(min(ts)), "max": float(max(ts)), "replays": replays,
            "launches_per_replay": per_replay}


# --------------------------------------------------------------------------------------------- ours


class ChainBench:
    """One merge workload (cfg1..cfg3) resident on the device: rotating (x, y) pool, graphs of the
    step, of the conv forward alone and of the merge alone."""
    MERGES_PER_GRAPH = 10            # a one-merge graph would time the graph launch, not the merge

    def __init__(self, name, seed, stream, case=None):
        import torch
        from paper_2301_12187_b200 import dc, inputs as I
        self.torch, self.dc, self.name, self.stream = torch, dc, name, stream
        case = self.case = case if case is not None else I.chain_case(WORKLOADS[name], seed=seed)
        n, h, w, c = case.x_shape
        self.layers = [dc.DeviceLayer(s) for s in case.layers]
        g, merge_ws_bytes = dc.merge_query(self.layers, case.residuals)
        self.g = g
        self.flops, self.abytes, self.yshape = conv_facts(case.x_shape, g)
        self.wm = torch.empty((g.c_out, g.c_in, g.k, g.k), dtype=torch.float32, device="cuda")
        self.bm = torch.empty((g.c_out,), dtype=torch.float32, device="cuda")
        self.merge_ws = torch.empty(merge_ws_bytes, dtype=torch.uint8, device="cuda")
        self.packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
        self.conv_ws = torch.zeros(dc.conv_workspace_bytes(), dtype=torch.uint8, device="cuda")
        # rotating pool of (x, y) pairs: more than 2.5x L2 in total, so no step finds its input in L2
        self.pair_bytes = 2 * (n * h * w * c + int(np.prod(self.yshape)))
        self.slots = max(4, int(np.ceil(2.5 * L2_BYTES / self.pair_bytes)))
        self.x_host = torch.from_numpy(case.x()).to(torch.bfloat16)
        self.xs = [self.x_host.to("cuda").clone() for _ in range(self.slots)]
        self.ys = [torch.empty(self.yshape, dtype=torch.bfloat16, device="cuda") for _ in range(self.slots)]
        self.kernel = dc.conv_kernel_name(n, h, w, g, dc.BF16)
        with torch.cuda.stream(stream):
            for i in range(min(self.slots, 3)):
                self.step(i)
            stream.synchronize()
            self.graphs = []         # one step per slot (the remainder of a timed run that is no whole round)
            self.launches_per_step = -1
            for i in range(self.slots):
                gr = torch.cuda.CUDAGraph(keep_graph=(i == 0))
                with torch.cuda.graph(gr, stream=stream):
                    self.step(i)
                if i == 0:
                    self.launches_per_step = count_kernel_nodes(gr)
                    gr.instantiate()
                self.graphs.append(gr)
            self.g_conv = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.g_conv, stream=stream):
                for i in range(self.slots):
                    self.conv(i)
            self.g_merge = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.g_merge, stream=stream):
                for _ in range(self.MERGES_PER_GRAPH):
                    self.merge()
            # a whole round of steps (every slot once): the gap between two graph launches is paid once
            # per round, not once per step
            self.g_round = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.g_round, stream=stream):
                for i in range(self.slots):
                    self.step(i)

    def merge(self):
        self.dc.merge_chain(self.layers, self.case.residuals, self.wm, self.bm, self.packed, self.dc.BF16, self.merge_ws)

    def conv(self, i):
        self.dc.conv_forward(self.xs[i], self.g, self.packed, self.bm, self.dc.ACT_IDENTITY, None, self.ys[i], self.conv_ws)

    def step(self, i):
        self.merge()
        self.conv(i)

    def run_steps(self, k):
        for _ in range(k // self.slots):
            self.g_round.replay()
        for i in range(k % self.slots):
            self.graphs[i].replay()

    def kernel_figures(self, peaks, peak_src):
        """Conv forward alone (L2-cold by rotation), merge alone, whole step: medians over graph replays."""
        with self.torch.cuda.stream(self.stream):
            conv = replay_stats(self.g_conv, self.stream, self.slots)
            merge = replay_stats(self.g_merge, self.stream, self.MERGES_PER_GRAPH)
            step = replay_stats(self.g_round, self.stream, self.slots)
        if self.dc.workspace_status(self.conv_ws, self.stream) != self.dc.OK:
            raise RuntimeError("device-side wait timed out during the benchmark (%s)" % self.name)
        n = self.case.x_shape[0]
        roof = roofline_entry(self.flops, self.abytes, conv["median"] * 1e-6, peaks, peak_src)
        roof.update({"kernel": self.kernel, "us_per_launch": conv["median"], "us_min": conv["min"], "us_max": conv["max"],
                     "replays": conv["replays"], "launches_per_replay": conv["launches_per_replay"],
                     "traffic": profiled_traffic(self.kernel, self.name),
                     "images_per_s_kernel_only": n / (conv["median"] * 1e-6)})
        return {"conv_forward_us": conv, "merge_latency_us": merge, "step_us": step, "roofline": roof}

    def e2e(self, world, barrier, steps, n_slots=3):
        """End to end through the host-buffer entry point: every step copies its input (and the run's
        parameters, one pinned block) from pinned host memory, merges, runs the forward and copies the
        output back.  Steps rotate over three streams, each with its own workspace and pinned buffers,
        so the copies of one step overlap the work of its neighbours; a slot is reused only after its
        previous step has finished."""
        torch, dc, case = self.torch, self.dc, self.case
        n, h, w, c = case.x_shape
        arr, keep = dc.host_layer_array(case.layers, pinned=True)
        ws_bytes = dc.chain_host_workspace_bytes(arr, len(case.layers), case.residuals, n, h, w, dc.BF16)
        e_ws = [torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda") for _ in range(n_slots)]
        e_x = [self.x_host.clone().pin_memory() for _ in range(n_slots)]
        e_y = [torch.empty(self.yshape, dtype=torch.bfloat16).pin_memory() for _ in range(n_slots)]
        e_st = [torch.cuda.Stream() for _ in range(n_slots)]

        def run(k):
            for i in range(k):
                s = i % n_slots
                e_st[s].synchronize()            # the slot's previous step is done, its output consumed
                dc.chain_forward_host_async(arr, len(case.layers), case.residuals, e_x[s], dc.ACT_IDENTITY, e_y[s],
                                            e_ws[s], e_st[s])
            for s in range(n_slots):
                e_st[s].synchronize()

        stream = self.stream
        with torch.cuda.stream(stream):
            run(2 * n_slots)
            barrier()
            h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            h0.record(stream)
            for s in range(n_slots):
                e_st[s].wait_event(h0)
            run(steps)
            for s in range(n_slots):
                stream.wait_stream(e_st[s])
            h1.record(stream)
            barrier()
        ms = h0.elapsed_time(h1) / steps
        for s in range(n_slots):
            if dc.workspace_status(e_ws[s], e_st[s]) != dc.OK:
                raise RuntimeError("device-side wait timed out during the end-to-end run (%s)" % self.name)
        param_bytes = sum(int(s.weight.size) * 4 + 4 * int(s.c_out) * 4 for s in case.layers)
        return ms, {"h2d_bytes_per_step": int(2 * n * h * w * c + param_bytes), "d2h_bytes_per_step": int(2 * np.prod(self.yshape)),
                    "steps": steps, "api": "dc_chain_forward_host_async (pinned host buffers, one parameter block, %d streams in flight)" % n_slots}

    def config(self):
        g = self.g
        return {"workload": self.case.name, "batch_per_gpu": self.case.x_shape[0], "input_nhwc": list(self.case.x_shape),
                "merged_conv": {"c_in": g.c_in, "c_out": g.c_out, "k": g.k, "stride": g.stride, "pad": g.pad},
                "step": "dc_merge_chain + dc_conv_forward; CUDA graphs of %d consecutive steps (one per input slot)" % self.slots,
                "l2": "inputs rotate over %d (x, y) pairs = %.0f MB > L2" % (self.slots, self.slots * self.pair_bytes / 1e6),
                "parallelism": "batch-sharded replicas, no collective"}

    def free(self):
        self.xs = self.ys = self.graphs = self.g_conv = self.g_round = self.g_merge = None
        self.torch.cuda.empty_cache()


def measure_network(args, peaks, peak_src):
    """cfg4: the whole depth-compressed MobileNetV2-1.0 forward at batch 128.  The roofline of the plan
    is the sum over its launch groups of max(bytes / HBM peak, flops / tensor peak), each group reading
    its input, writing its output and reading its weights once (an unmerged block: input and output
    only, its 6x wider maps counted as avoidable)."""
    import torch
    from paper_2301_12187_b200 import dc, inputs as I
    from paper_2301_12187_b200.network import CompressedNetwork, HostRunner
    net = I.mobilenet_v2(seed=0, batch=128)
    acts, plan = I.plan_spans(net, seed=0)
    plan_name = "every valid span merged"
    if args.plan == "latency":
        # the same kept activations, cut by Algorithm 1 over the latency table measured on this GPU
        from paper_2301_12187_b200 import latency as LT
        T, _ = LT.measure_latency_table(net, unit_us=0.1, reps=10, max_span=9)
        plan, _, _ = LT.latency_optimal_plan(net, acts, T)
        plan_name = "latency-optimal pattern (Algorithm 1 over the measured table)"
    cn = CompressedNetwork(net, acts, plan)
    x_np = I.make_input(0, net.x_shape, bf16=True)
    x = torch.from_numpy(x_np).to("cuda", dtype=torch.bfloat16)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        cn.merge()
        stream.synchronize()
        g_merge = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_merge, stream=stream):
            cn.merge()
    g_fwd = cn.capture(x, keep_graph=True)
    n_launch = count_kernel_nodes_of(g_fwd)
    g_step = cn.capture_step(x)
    with torch.cuda.stream(stream):
        fwd = replay_stats(g_fwd, stream, 1)
        merge = replay_stats(g_merge, stream, 1)
        step = replay_stats(g_step, stream, 1)
        # one launch group at a time: a graph of three launches of the group on the maps the forward left
        groups = []
        cur = x
        for i, op in enumerate(cn.ops):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=stream):
                for _ in range(3):
                    cn.launch(i, cur, x)
            groups.append(replay_stats(gr, stream, 3, replays=10, warmups=2))
            cur = op.y
    if cn.status() != dc.OK:
        raise RuntimeError("device-side wait timed out during the network benchmark")
    roof_s, roof_nom_s, flops_all, table = 0.0, 0.0, 0.0, []
    for op, st in zip(cn.ops, groups):
        n, h, w, c = op.in_shape
        _, ho, wo, co = op.out_shape
        specs = [net.layers[i] for i in op.layers]
        if op.kind == "conv":
            g = op.geom
            f = 2.0 * n * ho * wo * g.c_out * g.c_in * g.k * g.k
            b = 2.0 * (n * h * w * c + n * ho * wo * co + g.c_out * g.c_in * g.k * g.k) + (2.0 * n * ho * wo * co if op.add_from >= -1 else 0)
            kern = dc.conv_kernel_name(n, h, w, g, dc.BF16)
        elif op.kind == "dw":
            g = op.geom
            f = 2.0 * n * ho * wo * co * g.k * g.k
            b = 2.0 * (n * h * w * c + n * ho * wo * co)
            kern = "k_dwconv"
        else:
            f = sum(2.0 * n * (ho * wo if s.role != "expand" else h * w) * s.c_out * (s.c_in // s.groups) * s.k * s.k for s in specs)
            b = 2.0 * (n * h * w * c + n * ho * wo * co)
            kern = "block (3 launches)"
        t = max(b / (peaks["hbm_gbs"] * 1e9), f / (peaks["bf16_tflops"] * 1e12))
        roof_s += t
        roof_nom_s += max(b / (NOMINAL_PEAKS["hbm_gbs"] * 1e9), f / (NOMINAL_PEAKS["bf16_tflops"] * 1e12))
        flops_all += f
        table.append({"layers": "+".join(s.name for s in specs), "kind": op.kind + ("/merged" if op.merged else ""),
                      "kernel": kern, "in": list(op.in_shape), "out": list(op.out_shape), "us": round(st["median"], 2),
                      "roofline_us": round(t * 1e6, 2), "frac": round(t * 1e6 / st["median"], 3)})
    fwd_s = fwd["median"] * 1e-6
    # end to end from pinned host buffers
    runner = HostRunner(cn)
    x_pin = torch.from_numpy(x_np).to(torch.bfloat16).pin_memory()
    y_pin = [torch.empty(cn.out_shape, dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    for i in range(4):
        runner.submit(x_pin, y_pin[i & 1])
    runner.synchronize()
    e2e_steps = 20
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(runner.compute_stream)
    runner.copy_stream.wait_event(e0)
    for i in range(e2e_steps):
        runner.submit(x_pin, y_pin[i & 1])
    runner.join()                                # the last step's copy back is inside the timed region
    e1.record(runner.compute_stream)
    runner.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    if cn.status() != dc.OK:
        raise RuntimeError("device-side wait timed out during the network end-to-end run")
    roof = {"bound": "hbm", "achieved": roof_s / fwd_s, "peak": 1.0, "unit": "fraction of the summed per-group roofline time",
            "frac": roof_s / fwd_s, "traffic": None, "roofline_ms": roof_s * 1e3, "peak_source": peak_src,
            "frac_of_nominal": roof_nom_s / fwd_s,
            "tflops": flops_all / fwd_s / 1e12, "kernel": "%d launch groups" % len(cn.ops)}
    return {
        "config": {"workload": "cfg4_mbv2_full_batch128", "launch_groups": len(cn.ops), "kernel_launches": n_launch,
                   "merged_spans": sum(1 for op in cn.ops if op.merged), "plan_seed": 0, "plan": plan_name,
                   "step": "all dc_merge_chain calls + forward in one graph (a launch group waits for the merge of its own span only)",
                   "l2": "activation maps (0.1-0.6 GB each) exceed L2"},
        "value": 128 / (step["median"] * 1e-6), "unit": "images/s",
        "ms_per_step": step["median"] * 1e-3,
        "step_ms": {k: (v * 1e-3 if k in ("median", "min", "max") else v) for k, v in step.items()},
        "forward_ms": {k: (v * 1e-3 if k in ("median", "min", "max") else v) for k, v in fwd.items()},
        "forward_images_per_s": 128 / fwd_s, "merge_latency_us": merge, "roofline": roof, "groups": table,
        "e2e": {"value": 128 / (e2e_ms * 1e-3), "unit": "images/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(x_pin.numel() * 2), "d2h_bytes_per_step": int(y_pin[0].numel() * 2), "steps": e2e_steps,
                "api": "network.HostRunner (pinned host buffers; the input copy of a step runs under the previous forward, the copy back under the next)"},
    }, net, cn


def count_kernel_nodes_of(graph):
    try:
        return count_kernel_nodes(graph)
    except Exception:
        return -1


# --------------------------------------------------------------------------------------------- oracle


def oracle_step(case, O, images):
    """One pass of the path by the oracle: merge by the formula, then the sequential chain on `images`."""
    x = case.x(images).transpose(0, 3, 1, 2)
    t0 = time.time()
    O.merge_formula(case.layers, case.residuals)
    O.chain_forward_reordered(x, case.layers, case.residuals)
    return time.time() - t0


def cpu_baseline(case, seconds_cap):
    """The oracle as it stands on a bounded sample: as many images of the batch as fit half the cap in one
    step, and, when the whole batch takes less, whole steps until about `seconds_cap` seconds are spent."""
    from oracle import dc_oracle as O
    n = case.x_shape[0]
    t1 = oracle_step(case, O, 1)
    images = int(max(1, min(n, (seconds_cap / 2) / max(t1, 1e-3))))
    dt = oracle_step(case, O, images)
    steps, total = 1, dt
    while images == n and total + dt <= seconds_cap and steps < 64:
        total += oracle_step(case, O, images)
        steps += 1
    return {"value": images * steps / total, "unit": "images/s", "cores": O.num_threads(), "kind": "oracle",
            "sample": "fp64 merge by the formula + unmerged sequential chain on %d of %d images, %d step%s"
                      % (images, n, steps, "" if steps == 1 else "s"),
            "seconds": total}


def cpu_baseline_network(net, cn, images=16):
    """The oracle's sequential network (every launch group's layers in fp64) on the first `images`
    images; images/s extrapolated from that sample."""
    from oracle import dc_oracle as O
    from paper_2301_12187_b200 import inputs as I
    x = I.make_input(0, (images,) + tuple(net.x_shape[1:]), bf16=True).transpose(0, 3, 1, 2).astype(np.float64)
    t0 = time.time()
    cur, outs = x, []
    for op in cn.ops:
        specs = [net.layers[i] for i in op.layers]
        if op.kind == "block":
            y = cur
            for s in specs:
                Wf, bf = O.fold_bn(s)
                y = O.conv_direct(y, Wf, bf, s.k, s.stride, s.pad, s.groups)
                if s.act == "relu6":
                    y = O.relu6(y)
            if net.blocks[specs[0].block]["residual"]:
                y = y + cur
        else:
            po = cn.plan_ops[op.plan_index[0]]
            if len(specs) > 1:
                O.merge_formula(specs, po.residuals)
            y = O.chain_forward_reordered(cur, specs, po.residuals)
            if op.add_from == -1:
                y = y + x
            elif op.add_from >= 0:
                y = y + outs[op.add_from]
            if po.act == "relu6":
                y = O.relu6(y)
        outs.append(y)
        cur = y
    dt = time.time() - t0
    return {"value": images / dt, "unit": "images/s", "cores": O.num_threads(), "kind": "oracle",
            "sample": "fp64 merges by the formula + sequential network on %d of 128 images, 1 step (images/s extrapolated)" % images,
            "seconds": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import dc_oracle as O
    from paper_2301_12187_b200 import inputs as I
    name = "cfg1" if args.workload in ("all", "cfg4") else args.workload
    case = I.chain_case(WORKLOADS[name])
    n = case.x_shape[0]
    t1 = oracle_step(case, O, 1)
    budget = 120.0 / max(1, args.steps + args.warmup)
    images = int(max(1, min(n, budget / max(t1, 1e-3))))
    for _ in range(args.warmup):
        oracle_step(case, O, images)
    t0 = time.time()
    for _ in range(args.steps):
        oracle_step(case, O, images)
    dt = (time.time() - t0) / args.steps
    val = images / dt
    sample = "fp64 oracle: merge by the formula + unmerged sequential chain on %d of %d images per step" % (images, n)
    print(json.dumps({
        "impl": "reference", "metric": METRIC,
        "value": val, "unit": "images/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": case.name, "batch_per_gpu": n, "input_nhwc": list(case.x_shape)},
        "cpu_baseline": {"value": val, "unit": "images/s", "cores": O.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def chain_entry(cb, figs, e2e_ms, e2e_info, world, cpu):
    """per_config entry of one merge workload."""
    from paper_2301_12187_b200 import replicas as R
    n = cb.case.x_shape[0]
    out = {"config": cb.config(), "value": R.job_throughput(n, world, figs["step_us"]["median"] * 1e-6), "unit": "images/s",
           "ms_per_step": figs["step_us"]["median"] * 1e-3, "step_us": figs["step_us"],
           "conv_forward_us": figs["conv_forward_us"], "merge_latency_us": figs["merge_latency_us"],
           "launches_per_step": cb.launches_per_step, "roofline": figs["roofline"],
           "e2e": dict({"value": R.job_throughput(n, world, e2e_ms * 1e-3), "unit": "images/s", "ms_per_step": e2e_ms}, **e2e_info)}
    if cpu is not None:
        out["cpu_baseline"] = cpu
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2301_12187_b200 import dc, replicas as R

    rank, world, local = R.env_rank_world()
    torch.cuda.set_device(local)
    R.init_group("nccl", world, torch.device("cuda", local))
    dc.lib()
    peaks, peak_src = load_peaks()
    want_cpu = world == 1 and not args.no_cpu_baseline

    if args.workload == "cfg4":
        entry, net, cn = measure_network(args, peaks, peak_src)
        if want_cpu:
            entry["cpu_baseline"] = cpu_baseline_network(net, cn)
        if rank == 0:
            line = {"metric": METRIC, "n_gpus": world, "steps": entry["forward_ms"]["replays"], "warmup": KERNEL_WARMUPS,
                    "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                    "gpu_launches": entry["config"]["kernel_launches"] * entry["forward_ms"]["replays"]}
            line.update(entry)
            print(json.dumps(line))
        if world > 1:
            dist.destroy_process_group()
        return

    if args.workload == "vgg":
        # VGG-style runs (two dense 3x3 layers of 64..512 channels -> one 5x5 layer): merge latency and the merged
        # layer's forward by the same protocol (graph replays, L2-cold by rotation), kernel figures only
        from paper_2301_12187_b200 import inputs as I
        stream = torch.cuda.Stream()
        per = {}
        for c in sorted(I.VGG_MAPS):
            cb = ChainBench("vgg_c%d" % c, R.replica_seed(0, rank), stream, case=I.vgg_case(c, seed=R.replica_seed(0, rank)))
            f = cb.kernel_figures(peaks, peak_src)
            f["config"] = cb.config()
            per[cb.name] = f
            cb.free()
        if rank == 0:
            head = per["vgg_c512"]
            print(json.dumps({"metric": METRIC, "value": head["roofline"]["images_per_s_kernel_only"] * world, "unit": "images/s",
                              "n_gpus": world, "steps": head["conv_forward_us"]["replays"], "warmup": KERNEL_WARMUPS,
                              "ms_per_step": head["step_us"]["median"] * 1e-3, "higher_is_better": True, "scaling": "weak",
                              "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": head["config"],
                              "roofline": head["roofline"], "per_config": per}))
        if world > 1:
            dist.destroy_process_group()
        return

    headline = "cfg1" if args.workload == "all" else args.workload
    stream = torch.cuda.Stream()
    hb = ChainBench(headline, R.replica_seed(0, rank), stream)

    def barrier():
        stream.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    with torch.cuda.stream(stream):
        hb.run_steps(args.warmup)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_begin = time.time()
        e0.record(stream)
        hb.run_steps(args.steps)
        e1.record(stream)
        barrier()
        t_end = time.time()
        ms_total = e0.elapsed_time(e1)
        # keep the same load running (untimed) until the clock sampler has a few samples
        if rank == 0 and sampler.proc is not None:
            deadline = time.time() + 2.0
            while sampler.count_since(t_begin) < 4 and time.time() < deadline:
                hb.run_steps(200)
                stream.synchronize()
            t_end = time.time()
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    figs = hb.kernel_figures(peaks, peak_src)
    e2e_ms, e2e_info = hb.e2e(world, barrier, max(9, min(args.steps, 60)), args.e2e_streams)
    times = torch.tensor([ms_total, e2e_ms], dtype=torch.float64, device="cuda")
    R.max_over_ranks(times, world)
    ms_total, e2e_ms = float(times[0]), float(times[1])
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    n = hb.case.x_shape[0]
    ms_step = ms_total / args.steps
    out = {
        "metric": METRIC,
        "value": R.job_throughput(n, world, ms_step * 1e-3), "unit": "images/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": hb.config(),
        "merge_latency_us": figs["merge_latency_us"]["median"], "conv_forward_us": figs["conv_forward_us"]["median"],
        "gpu_launches": (hb.launches_per_step if hb.launches_per_step > 0 else 3) * args.steps,
        "launches_per_step": hb.launches_per_step,
        "roofline": figs["roofline"],
        "e2e": dict({"value": R.job_throughput(n, world, e2e_ms * 1e-3), "unit": "images/s", "ms_per_step": e2e_ms}, **e2e_info),
        "clocks": clocks,
    }
    cpu = cpu_baseline(hb.case, seconds_cap=10.0) if want_cpu else None
    if cpu is not None:
        out["cpu_baseline"] = cpu
    if args.workload == "all" and world == 1:
        per = {headline: chain_entry(hb, figs, e2e_ms, e2e_info, world, cpu)}
        hb.free()
        for name in ("cfg2", "cfg3"):
            cb = ChainBench(name, R.replica_seed(0, rank), stream)
            f = cb.kernel_figures(peaks, peak_src)
            ms, info = cb.e2e(world, barrier, 30, args.e2e_streams)
            per[name] = chain_entry(cb, f, ms, info, world, cpu_baseline(cb.case, seconds_cap=8.0) if want_cpu else None)
            cb.free()
        entry, net, cn = measure_network(args, peaks, peak_src)
        if want_cpu:
            entry["cpu_baseline"] = cpu_baseline_network(net, cn)
        per["cfg4"] = entry
        # the same network cut by Algorithm 1 over the latency table measured here (the paper's own way to pick
        # the merge pattern; the plan above merges every valid span of a fixed seeded pattern instead)
        del cn, net
        import copy
        args_lat = copy.copy(args)
        args_lat.plan = "latency"
        per["cfg4_latency_plan"] = measure_network(args_lat, peaks, peak_src)[0]
        out["per_config"] = per
    print(json.dumps(out))


def relaunch_with_ranks(args):
    """--gpus N without a launcher: start N ranks of this script on this node (one per GPU)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--workload", default="all", choices=["all", "vgg"] + sorted(WORKLOADS),
                    help="all: cfg1 as the headline line plus cfg1..cfg4 (cfg4 under both plans) under per_config (one GPU); cfgN: that workload alone")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-streams", type=int, default=3, help="steps in flight in the end-to-end measurement of the chain workloads")
    ap.add_argument("--plan", default="spans", choices=["spans", "latency"],
                    help="cfg4: merge every valid span, or cut by Algorithm 1 over the measured latency table")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        if args.steps == 20000:
            args.steps, args.warmup = 5, 3
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        relaunch_with_ranks(args)
    run_ours(args)


if __name__ == "__main__":
    main()
