"""Latency table T[i][j] of a network on this GPU and the latency-optimal merge pattern.

T[i][j] (Sec. 4.1) is the measured forward time of the one convolution that layers i+1..j merge
into when the activations between them are identities: the span is merged with dc_merge_chain and
its dc_conv_forward (dc_dwconv_forward for a lone depthwise layer) is timed with CUDA events.
Spans that cannot be merged carry dc.DP_INF.  Algorithm 1 (dc_dp_optimal_latency) then gives, for
every span, the pattern that merges only where merging is faster.

Host logic only: which spans are valid, buffers, timing loops.  All arithmetic runs in the library.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

from . import dc


def _out_extent(h, k, s, p):
    return (h + 2 * p - k) // s + 1


def span_residuals(net, i: int, j: int, max_k: int = 7) -> Optional[List[Tuple[int, int]]]:
    """Skip groups (relative to the span) if layers i..j-1 (0-based; boundaries i and j) may be
    merged into one convolution, else None.  Rules: a skip block lies wholly inside the span (it is
    folded as an identity kernel, App. E.1), does not touch it, or contains the whole span (the
    block's addition then stays an explicit step after its last layer); no layer with k > 1 after a
    stride-2 layer of the span (App. B.2); merged kernel size at most max_k (a limit of this
    harness, not of the method)."""
    L = net.layers
    if j - i == 1:
        return []
    res = []
    for blk in net.blocks:
        if not blk["residual"]:
            continue
        f, l = blk["first"], blk["last"]
        inside = i <= f and l < j
        disjoint = l < i or f >= j
        within = f <= i and j - 1 <= l
        if inside:
            res.append((f - i, l - i))
        elif not disjoint and not within:
            return None
    k, s, seen_s2 = 1, 1, False
    for a in range(i, j):
        if seen_s2 and L[a].k > 1:
            return None
        k += (L[a].k - 1) * s
        s *= L[a].stride
        seen_s2 = seen_s2 or L[a].stride > 1
    if k > max_k:
        return None
    return res


def boundary_shapes(net):
    """NHWC shape of the feature map at every boundary 0..L."""
    n, h, w, c = net.x_shape
    shapes = [(n, h, w, c)]
    for lay in net.layers:
        h, w = _out_extent(h, lay.k, lay.stride, lay.pad), _out_extent(w, lay.k, lay.stride, lay.pad)
        shapes.append((n, h, w, lay.c_out))
    return shapes


def measure_latency_table(net, unit_us: float = 1.0, reps: int = 10, max_span: int = 9, max_k: int = 7,
                          cold: bool = False):
    """Returns (T, us): T[i][j] = ceil(latency / unit_us) as Python ints (dc.DP_INF where the span
    is not mergeable or longer than max_span layers), us[i][j] the measured microseconds (None where
    not measured).  bf16, this process's current CUDA device.  Warm (default): each span's forward is
    captured `reps` times in one CUDA graph and the graph's time divided by reps, so inputs of small
    maps stay in L2 -- the state a layer finds inside a running network, whose input the previous
    layer has just written.  cold=True: every launch is timed on its own after a buffer larger than L2
    has been overwritten, and the median of `reps` launches is taken (inputs come from HBM; a CUDA
    event pair around one launch adds ~2 us to every entry alike)."""
    import math
    import torch

    nL = len(net.layers)
    shapes = boundary_shapes(net)
    devs = [dc.DeviceLayer(s) for s in net.layers]
    T = [[0] * (nL + 1) for _ in range(nL + 1)]
    us = [[None] * (nL + 1) for _ in range(nL + 1)]
    conv_ws = torch.zeros(dc.conv_workspace_bytes(), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if cold else None
    for i in range(nL):
        x = torch.zeros(shapes[i], dtype=torch.bfloat16, device="cuda")
        for j in range(i + 1, nL + 1):
            T[i][j] = dc.DP_INF
            if j - i > max_span:
                continue
            res = span_residuals(net, i, j, max_k)
            if res is None:
                continue
            layers = devs[i:j]
            try:
                g, ws_bytes = dc.merge_query(layers, res)
            except dc.DcError:
                continue
            y = torch.empty(shapes[j], dtype=torch.bfloat16, device="cuda")
            lone_dw = j - i == 1 and net.layers[i].groups != 1
            with torch.cuda.stream(stream):
                if lone_dw:
                    lay = net.layers[i]
                    wf = torch.empty_like(devs[i].weight)
                    bf = torch.empty(lay.c_out, device="cuda")
                    dc.fold_bn(devs[i], wf, bf)
                    gd = dc.geom(lay.c_in, lay.c_out, lay.groups, lay.k, lay.stride, lay.pad)
                    packed = torch.empty(dc.packed_bytes(gd, dc.F32), dtype=torch.uint8, device="cuda")
                    dc.pack_weights(wf, gd, dc.F32, packed)

                    def run():
                        dc.dwconv_forward(x, lay.k, lay.stride, lay.pad, packed, bf, dc.ACT_IDENTITY, y)
                else:
                    wm = torch.empty((g.c_out, g.c_in, g.k, g.k), dtype=torch.float32, device="cuda")
                    bm = torch.empty((g.c_out,), dtype=torch.float32, device="cuda")
                    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
                    packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
                    dc.merge_chain(layers, res, wm, bm, packed, dc.BF16, ws)

                    def run():
                        dc.conv_forward(x, g, packed, bm, dc.ACT_IDENTITY, None, y, conv_ws)
                run()
                stream.synchronize()
                if cold:
                    times = []
                    for _ in range(reps):
                        flush.zero_()
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record(stream)
                        run()
                        e1.record(stream)
                        stream.synchronize()
                        times.append(e0.elapsed_time(e1) * 1e3)
                    t_us = sorted(times)[len(times) // 2]
                else:
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=stream):
                        for _ in range(reps):
                            run()
                    graph.replay()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    graph.replay()
                    e1.record(stream)
                    stream.synchronize()
                    t_us = e0.elapsed_time(e1) * 1e3 / reps
            if dc.workspace_status(conv_ws) != dc.OK:
                raise RuntimeError("device-side wait timed out while timing span (%d, %d)" % (i, j))
            us[i][j] = t_us
            T[i][j] = max(1, int(math.ceil(t_us / unit_us)))
    return T, us


def optimal_pattern(T, L: int):
    """Algorithm 1 on a measured table: (T_opt[0][L], S_opt[0][L], T_opt, split)."""
    t_opt, split = dc.dp_optimal_latency(T, L)
    return t_opt[0][L], dc.dp_pattern(split, L, 0, L), t_opt, split


def latency_optimal_plan(net, acts, T):
    """Merge pattern for a network whose kept activations are fixed (`acts[l]` is None where layer
    l's activation is an identity): spans that would swallow a kept activation become unmergeable,
    Algorithm 1 picks the fastest pattern among the rest, and the pieces become plan ops.  Returns
    (ops, boundaries, T_opt[0][L])."""
    from . import inputs as I
    L = len(net.layers)
    Tm = [row[:] for row in T]
    for i in range(L + 1):
        for j in range(i + 2, L + 1):
            if any(acts[a] is not None for a in range(i, j - 1)):
                Tm[i][j] = dc.DP_INF
    total, S, _, _ = optimal_pattern(Tm, L)
    bounds = [0] + S + [L]
    ops = I.plan_from_boundaries(net, acts, bounds, lambda a, c: span_residuals(net, a, c))
    return ops, bounds, total
