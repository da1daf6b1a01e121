#!/usr/bin/env python
"""Benchmark of the conv-merging hot path on B200.

One step = one pass of the whole path over one batch of synthetic input: merge the run of
convolutions (dc_merge_chain: BN fold, composition, skip fold, repack) and run the merged
convolution forward over the batch (dc_conv_forward).  Default workload: the MobileNetV2-1.0
inverted-residual block at 56x56, batch 64, bf16 (1x1 24->144, dw3x3, 1x1 144->24, skip folded ->
one 3x3 conv 24->24).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1|cfg2|cfg3] [--impl reference]

Prints one JSON line (rank 0).  `value` = images/s with inputs resident in HBM; `e2e` = the same
through the host-buffer entry point with the copies inside the timed region; `roofline` = the
merged-conv kernel alone against the measured HBM (or tensor) peak; `cpu_baseline` = the fp64
oracle on the host cores (a baseline, not a target).
"""
from __future__ import annotations

import argparse
import ctypes
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
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
L2_BYTES = 126 * 1024 * 1024


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"])}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def workload_facts(case, g):
    """Algorithmic flops and bytes of one merged-conv launch: read x once, write y once, read W'."""
    n, h, w, c = case.x_shape
    ho = (h + 2 * g.pad - g.k) // g.stride + 1
    wo = (w + 2 * g.pad - g.k) // g.stride + 1
    flops = 2.0 * n * ho * wo * g.c_out * g.c_in * g.k * g.k
    bytes_ = 2.0 * n * h * w * c + 2.0 * n * ho * wo * g.c_out + 2.0 * g.c_out * g.c_in * g.k * g.k + 4.0 * g.c_out
    return flops, bytes_, (n, ho, wo, g.c_out)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the load runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index
        self.t0 = None

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
    import torch  # noqa: F401
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


# --------------------------------------------------------------------------------------------- ours


def run_network(args):
    """cfg4: the whole depth-compressed MobileNetV2-1.0 forward at batch 128 (reported beside the
    headline workload; the per-layer roofline is the sum over launch groups of
    max(bytes / HBM peak, flops / tensor peak) with each group reading its input, writing its
    output and reading its weights once)."""
    import torch
    from paper_2301_12187_b200 import dc, inputs as I
    from paper_2301_12187_b200.network import CompressedNetwork
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
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
    x = torch.from_numpy(I.make_input(0, net.x_shape, bf16=True)).to("cuda", dtype=torch.bfloat16)
    stream = torch.cuda.Stream()
    peaks, peak_src = load_peaks()
    with torch.cuda.stream(stream):
        cn.merge()
        stream.synchronize()
        g_merge = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_merge, stream=stream):
            cn.merge()
    g_fwd = cn.capture(x)
    with torch.cuda.stream(stream):
        for _ in range(max(3, args.warmup // 50)):
            g_merge.replay(); g_fwd.replay()
        stream.synchronize()
        steps = max(3, min(args.steps, 50))
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        e[0].record(stream)
        for _ in range(steps):
            g_merge.replay(); g_fwd.replay()
        e[1].record(stream)
        for _ in range(steps):
            g_fwd.replay()
        e[2].record(stream)
        for _ in range(steps):
            g_merge.replay()
        e[3].record(stream)
        stream.synchronize()
    assert cn.status() == dc.OK
    ms_step, ms_fwd, ms_merge = (e[i].elapsed_time(e[i + 1]) / steps for i in range(3))
    roof_s, flops = 0.0, 0.0
    per_group = []
    for op in cn.ops:
        n, h, w, c = op.in_shape
        _, ho, wo, co = op.out_shape
        specs = [net.layers[i] for i in op.layers]
        if op.kind == "conv":
            g = op.geom
            f = 2.0 * n * ho * wo * g.c_out * g.c_in * g.k * g.k
            b = 2.0 * (n * h * w * c + n * ho * wo * co + g.c_out * g.c_in * g.k * g.k) + (2.0 * n * ho * wo * co if op.add_from >= -1 else 0)
        elif op.kind == "dw":
            g = op.geom
            f = 2.0 * n * ho * wo * co * g.k * g.k
            b = 2.0 * (n * h * w * c + n * ho * wo * co)
        else:
            f = sum(2.0 * n * (ho * wo if s.role != "expand" else h * w) * s.c_out * (s.c_in // s.groups) * s.k * s.k for s in specs)
            b = 2.0 * (n * h * w * c + n * ho * wo * co)
        t = max(b / (peaks["hbm_gbs"] * 1e9), f / (peaks["bf16_tflops"] * 1e12))
        roof_s += t
        flops += f
        per_group.append(t)
    print(json.dumps({
        "metric": "merged-conv fwd TFLOP/s & images/s on 1 B200 vs roofline; merge latency us",
        "value": 128 / (ms_step * 1e-3), "unit": "images/s", "n_gpus": 1, "steps": steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "cfg4_mbv2_full_batch128", "launch_groups": len(cn.ops),
                   "merged_spans": sum(1 for op in cn.ops if op.merged), "plan_seed": 0, "plan": plan_name,
                   "step": "all dc_merge_chain calls + forward graph", "l2": "activation maps (0.1-0.6 GB each) exceed L2"},
        "forward_ms": ms_fwd, "forward_images_per_s": 128 / (ms_fwd * 1e-3), "merge_latency_us": ms_merge * 1e3,
        "roofline": {"bound": "hbm", "achieved": roof_s / (ms_fwd * 1e-3), "peak": 1.0, "unit": "fraction of summed per-group roofline time",
                     "frac": roof_s / (ms_fwd * 1e-3), "traffic": None, "roofline_ms": roof_s * 1e3,
                     "tflops": flops / (ms_fwd * 1e-3) / 1e12, "peak_source": peak_src},
    }))


def run_ours(args):
    if args.workload == "cfg4":
        return run_network(args)
    import torch
    import torch.distributed as dist
    from paper_2301_12187_b200 import dc, inputs as I, replicas as R

    rank, world, local = R.env_rank_world()
    torch.cuda.set_device(local)
    R.init_group("nccl", world, torch.device("cuda", local))
    dc.lib()

    case = I.chain_case(WORKLOADS[args.workload], seed=R.replica_seed(0, rank))
    n, h, w, c = case.x_shape
    layers = [dc.DeviceLayer(s) for s in case.layers]
    g, merge_ws_bytes = dc.merge_query(layers, case.residuals)
    flops, abytes, yshape = workload_facts(case, g)
    wm = torch.empty((g.c_out, g.c_in, g.k, g.k), dtype=torch.float32, device="cuda")
    bm = torch.empty((g.c_out,), dtype=torch.float32, device="cuda")
    merge_ws = torch.empty(merge_ws_bytes, dtype=torch.uint8, device="cuda")
    packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
    conv_ws = torch.zeros(dc.conv_workspace_bytes(), dtype=torch.uint8, device="cuda")

    # rotating pool of (x, y) pairs: more than 2x L2 in total, so no step finds its input in L2
    pair_bytes = 2 * (n * h * w * c + int(np.prod(yshape)))
    slots = max(4, int(np.ceil(2.5 * L2_BYTES / pair_bytes)))
    x_host = torch.from_numpy(case.x()).to(torch.bfloat16)
    xs = [x_host.to("cuda").clone() for _ in range(slots)]
    ys = [torch.empty(yshape, dtype=torch.bfloat16, device="cuda") for _ in range(slots)]

    def step(i):
        dc.merge_chain(layers, case.residuals, wm, bm, packed, dc.BF16, merge_ws)
        dc.conv_forward(xs[i], g, packed, bm, dc.ACT_IDENTITY, None, ys[i], conv_ws)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(min(slots, 3)):
            step(i)
        stream.synchronize()
        # one graph per slot (merge + conv); one graph with only the conv launches over all slots;
        # one with only the merge
        graphs = []
        for i in range(slots):
            gr = torch.cuda.CUDAGraph(keep_graph=(i == 0))
            with torch.cuda.graph(gr, stream=stream):
                step(i)
            if i == 0:
                launches_per_step = count_kernel_nodes(gr)
                gr.instantiate()
            graphs.append(gr)
        g_conv = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_conv, stream=stream):
            for i in range(slots):
                dc.conv_forward(xs[i], g, packed, bm, dc.ACT_IDENTITY, None, ys[i], conv_ws)
        MERGES_PER_GRAPH = 10            # a one-merge graph would time the graph launch, not the merge
        g_merge = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_merge, stream=stream):
            for _ in range(MERGES_PER_GRAPH):
                dc.merge_chain(layers, case.residuals, wm, bm, packed, dc.BF16, merge_ws)
        # one graph with a whole round of steps (every slot once): the timed loop replays rounds,
        # so that the gap between two graph launches is paid once per round, not once per step
        g_round = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_round, stream=stream):
            for i in range(slots):
                step(i)

        def barrier():
            stream.synchronize()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()

        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        def run_steps(k):
            for _ in range(k // slots):
                g_round.replay()
            for i in range(k % slots):
                graphs[i].replay()

        run_steps(args.warmup)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_begin = time.time()
        e0.record(stream)
        run_steps(args.steps)
        e1.record(stream)
        barrier()
        t_end = time.time()
        ms_total = e0.elapsed_time(e1)
        # kernel-level timing, same stream, CUDA events: merged conv alone (L2-cold by rotation), merge alone
        reps = max(3, min(200, args.steps // slots + 1))
        for _ in range(3):
            g_conv.replay()
        stream.synchronize()
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        k0.record(stream)
        for _ in range(reps):
            g_conv.replay()
        k1.record(stream)
        stream.synchronize()
        conv_us = k0.elapsed_time(k1) * 1e3 / (reps * slots)
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            g_merge.replay()
        m0.record(stream)
        for _ in range(50):
            g_merge.replay()
        m1.record(stream)
        stream.synchronize()
        merge_us = m0.elapsed_time(m1) * 1e3 / (50 * MERGES_PER_GRAPH)
        # keep the same load running (untimed) until the clock sampler has a few samples
        if rank == 0 and sampler.proc is not None:
            deadline = time.time() + 2.0
            while sampler.count_since(t_begin) < 4 and time.time() < deadline:
                run_steps(200)
                stream.synchronize()
            t_end_clk = time.time()
        else:
            t_end_clk = t_end
        status = dc.workspace_status(conv_ws, stream)
        if status != dc.OK:
            raise RuntimeError("device-side wait timed out during the benchmark")

        # End to end through the host-buffer entry point: every step copies its input from pinned host
        # memory, merges, runs the forward and copies the output back.  Steps rotate over three
        # streams, each with its own workspace and pinned buffers, so the copies of one step overlap
        # the work of its neighbours; a slot is reused only after its previous step has finished.
        arr, keep = dc.host_layer_array(case.layers, pinned=True)
        ws_bytes = dc.chain_host_workspace_bytes(arr, len(case.layers), case.residuals, n, h, w, dc.BF16)
        n_slots = 3
        e_ws = [torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda") for _ in range(n_slots)]
        e_x = [x_host.clone().pin_memory() for _ in range(n_slots)]
        e_y = [torch.empty(yshape, dtype=torch.bfloat16).pin_memory() for _ in range(n_slots)]
        e_st = [torch.cuda.Stream() for _ in range(n_slots)]
        e2e_steps = max(3 * n_slots, min(args.steps, 60))

        def e2e_run(steps):
            for i in range(steps):
                k = i % n_slots
                e_st[k].synchronize()            # the slot's previous step is done, its output consumed
                dc.chain_forward_host_async(arr, len(case.layers), case.residuals, e_x[k], dc.ACT_IDENTITY, e_y[k],
                                            e_ws[k], e_st[k])
            for k in range(n_slots):
                e_st[k].synchronize()

        e2e_run(2 * n_slots)
        barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for k in range(n_slots):
            e_st[k].wait_event(h0)
        e2e_run(e2e_steps)
        for k in range(n_slots):
            stream.wait_stream(e_st[k])
        h1.record(stream)
        barrier()
        e2e_ms = h0.elapsed_time(h1) / e2e_steps
        for k in range(n_slots):
            if dc.workspace_status(e_ws[k], e_st[k]) != dc.OK:
                raise RuntimeError("device-side wait timed out during the end-to-end run")

    times = torch.tensor([ms_total, e2e_ms], dtype=torch.float64, device="cuda")
    R.max_over_ranks(times, world)
    ms_total, e2e_ms = float(times[0]), float(times[1])
    clocks = sampler.stop(t_begin, t_end_clk) if rank == 0 else None
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return

    peaks, peak_src = load_peaks()
    t_hbm = abytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    conv_s = conv_us * 1e-6
    if t_hbm >= t_tc:
        roof = {"bound": "hbm", "achieved": abytes / conv_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": flops / conv_s / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = PROFILED_TRAFFIC.get(args.workload)
    roof.update({"kernel": dc.conv_kernel_name(n, h, w, g, dc.BF16), "us_per_launch": conv_us, "peak_source": peak_src,
                 "algorithmic_bytes": abytes, "flops": flops, "tflops": flops / conv_s / 1e12,
                 "images_per_s_kernel_only": n / conv_s})

    ms_step = ms_total / args.steps
    param_bytes = sum(int(s.weight.size) * 4 + 4 * int(s.c_out) * 4 for s in case.layers)
    out = {
        "metric": "merged-conv fwd TFLOP/s & images/s on 1 B200 vs roofline; merge latency us",
        "value": R.job_throughput(n, world, ms_step * 1e-3), "unit": "images/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": case.name, "batch_per_gpu": n, "input_nhwc": list(case.x_shape),
                   "merged_conv": {"c_in": g.c_in, "c_out": g.c_out, "k": g.k, "stride": g.stride, "pad": g.pad},
                   "step": "dc_merge_chain + dc_conv_forward; CUDA graphs of %d consecutive steps (one per input slot)" % slots,
                   "l2": "inputs rotate over %d (x, y) pairs = %.0f MB > L2" % (slots, slots * pair_bytes / 1e6),
                   "parallelism": "batch-sharded replicas, no collective"},
        "merge_latency_us": merge_us, "conv_forward_us": conv_us,
        "gpu_launches": (launches_per_step if launches_per_step > 0 else 10) * args.steps,
        "launches_per_step": launches_per_step,
        "roofline": roof,
        "e2e": {"value": R.job_throughput(n, world, e2e_ms * 1e-3), "unit": "images/s",
                "h2d_bytes_per_step": int(2 * n * h * w * c + param_bytes),
                "d2h_bytes_per_step": int(2 * np.prod(yshape)), "ms_per_step": e2e_ms,
                "api": "dc_chain_forward_host_async (pinned host buffers, 3 streams in flight)"},
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(case, seconds_cap=30.0)
    print(json.dumps(out))


# ncu dram__bytes_read.sum + dram__bytes_write.sum per launch of the conv forward kernel (profiles/);
# None until captured, and again once the kernel has changed since
PROFILED_TRAFFIC = {"cfg1": 9743104, "cfg2": None, "cfg3": None}   # cfg1: profiles/k_conv_tc_pairrows_cfg1.md


# --------------------------------------------------------------------------------------------- oracle


def oracle_step(case, O, images):
    """One pass of the path by the oracle: merge by the formula, then the sequential chain on `images`."""
    x = case.x(images).transpose(0, 3, 1, 2)
    t0 = time.time()
    O.merge_formula(case.layers, case.residuals)
    O.chain_forward_reordered(x, case.layers, case.residuals)
    return time.time() - t0


def cpu_baseline(case, seconds_cap=30.0):
    from oracle import dc_oracle as O
    n = case.x_shape[0]
    t1 = oracle_step(case, O, 1)
    images = int(max(1, min(n, (seconds_cap / 2) / max(t1, 1e-3))))
    dt = oracle_step(case, O, images)
    return {"value": images / dt, "unit": "images/s", "cores": O.num_threads(), "kind": "oracle",
            "sample": "fp64 merge by the formula + unmerged sequential chain on %d of %d images, 1 step" % (images, n),
            "seconds": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import dc_oracle as O
    from paper_2301_12187_b200 import inputs as I
    case = I.chain_case(WORKLOADS[args.workload])
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
        "impl": "reference", "metric": "merged-conv fwd TFLOP/s & images/s on 1 B200 vs roofline; merge latency us",
        "value": val, "unit": "images/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": case.name, "batch_per_gpu": n, "input_nhwc": list(case.x_shape)},
        "cpu_baseline": {"value": val, "unit": "images/s", "cores": O.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--workload", default="cfg1", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--plan", default="spans", choices=["spans", "latency"],
                    help="cfg4 only: merge every valid span, or cut by Algorithm 1 over the measured latency table")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        if args.steps == 20000:
            args.steps, args.warmup = 5, 3
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
