"""Sequencing of a depth-compressed network: a span plan becomes a list of C-ABI calls on one
stream (merged spans through dc_merge_chain + dc_conv_forward, untouched layers through
dc_conv_forward / dc_dwconv_forward / dc_block_forward), optionally captured in a CUDA graph.

Host logic only: shapes, buffers and the order of calls.  All arithmetic runs in the library.
The total latency of the result is the sum over its merged layers (the paper's decomposition of
T(network) in Sec. 4.1).
"""
from __future__ import annotations

from typing import List, Optional

from . import dc


def _out_extent(h, k, s, p):
    return (h + 2 * p - k) // s + 1


class _Op:
    def __init__(self):
        self.kind = ""            # 'conv' | 'dw' | 'block'
        self.plan_index = []      # indices into the plan's ops this launch group covers
        self.layers = []          # network layer indices
        self.geom = None
        self.packed = None
        self.bias = None
        self.act = dc.ACT_IDENTITY
        self.add_from = -2
        self.block = None
        self.keep = []
        self.in_shape = None
        self.out_shape = None
        self.y = None
        self.merged = False
        self.merge_job = -1       # index into the network's merge jobs (merged spans only)


class CompressedNetwork:
    """Device-resident compressed network built from `inputs.Network` and `inputs.plan_spans`."""

    def __init__(self, net, acts, plan_ops, batch: Optional[int] = None, use_block_calls: bool = True):
        import torch
        self.torch = torch
        self.net = net
        self.acts = acts
        self.plan_ops = plan_ops
        n, h, w, c = net.x_shape
        self.batch = batch or n
        self.in_shape = (self.batch, h, w, c)
        self.layers = [dc.DeviceLayer(s) for s in net.layers]
        self.conv_ws = torch.zeros(dc.conv_workspace_bytes(), dtype=torch.uint8, device="cuda")
        self.ops: List[_Op] = []
        self._merge_jobs = []
        self._build(use_block_calls)
        self.graph = None

    # ------------------------------------------------------------------ construction
    def _act(self, name):
        return dc.ACT_RELU6 if name == "relu6" else dc.ACT_IDENTITY

    def _build(self, use_block_calls):
        torch = self.torch
        L = self.net.layers
        plan = self.plan_ops
        produced = {}                      # plan op index -> launch group index
        shape = self.in_shape
        i = 0
        while i < len(plan):
            po = plan[i]
            op = _Op()
            op.in_shape = shape
            n, h, w, c = shape
            blk3 = None
            if use_block_calls and len(po.layers) == 1 and i + 1 < len(plan):
                blk3 = self._vanilla_block_at(i)
            if blk3 is not None:
                cnt, blk = blk3
                first = L[plan[i].layers[0]]
                dwl = L[plan[i + cnt - 2].layers[0]]
                prj = L[plan[i + cnt - 1].layers[0]]
                op.kind = "block"
                op.plan_index = list(range(i, i + cnt))
                op.layers = [plan[j].layers[0] for j in op.plan_index]
                parts = [self._fold_pack(li) for li in op.layers]
                has_exp = cnt == 3
                pe = parts[0] if has_exp else (None, None)
                pd, pp = parts[-2], parts[-1]
                ho, wo = _out_extent(h, dwl.k, dwl.stride, dwl.pad), _out_extent(w, dwl.k, dwl.stride, dwl.pad)
                op.block = dc.Block(first.c_in, dwl.c_in, prj.c_out, int(has_exp), dwl.k, dwl.stride, dwl.pad,
                                    int(blk["residual"]), dc.ACT_RELU6, dc.ACT_RELU6,
                                    pe[0].data_ptr() if has_exp else None, pe[1].data_ptr() if has_exp else None,
                                    pd[0].data_ptr(), pd[1].data_ptr(), pp[0].data_ptr(), pp[1].data_ptr())
                op.keep = parts
                op.out_shape = (n, ho, wo, prj.c_out)
                op.ws = torch.zeros(dc.block_workspace_bytes(n, h, w, op.block, dc.BF16), dtype=torch.uint8,
                                    device="cuda")
                i += cnt
            else:
                op.plan_index = [i]
                op.layers = list(po.layers)
                op.act = self._act(po.act)
                op.add_from = po.add_from
                if len(po.layers) == 1:
                    lay = L[po.layers[0]]
                    op.geom = dc.geom(lay.c_in, lay.c_out, lay.groups, lay.k, lay.stride, lay.pad)
                    op.packed, op.bias = self._fold_pack(po.layers[0])
                    op.kind = "dw" if lay.groups != 1 else "conv"
                else:
                    devs = [self.layers[j] for j in po.layers]
                    g, ws_bytes = dc.merge_query(devs, po.residuals)
                    op.geom = g
                    op.merged = True
                    op.kind = "conv"
                    wm = torch.empty((g.c_out, g.c_in, g.k, g.k), dtype=torch.float32, device="cuda")
                    op.bias = torch.empty((g.c_out,), dtype=torch.float32, device="cuda")
                    op.packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
                    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
                    op.merge_job = len(self._merge_jobs)
                    self._merge_jobs.append((devs, list(po.residuals), wm, op.bias, op.packed, ws))
                    op.keep = [wm, ws]
                g = op.geom
                op.out_shape = (n, _out_extent(h, g.k, g.stride, g.pad), _out_extent(w, g.k, g.stride, g.pad), g.c_out)
                i += 1
            op.y = torch.empty(op.out_shape, dtype=torch.bfloat16, device="cuda")
            for pi in op.plan_index:
                produced[pi] = len(self.ops)
            self.ops.append(op)
            shape = op.out_shape
        # explicit skip additions: plan op index -> launch group index (or -1 for the network input)
        for op in self.ops:
            if op.add_from >= 0:
                op.add_from = produced[op.add_from]
        self.out_shape = shape

    def _vanilla_block_at(self, i):
        """(count, block) when plan ops i.. are the untouched layers of one inverted-residual block."""
        L = self.net.layers
        plan = self.plan_ops
        first = L[plan[i].layers[0]]
        blk = self.net.blocks[first.block]
        if first.role not in ("expand", "dw") or plan[i].layers[0] != blk["first"]:
            return None
        cnt = blk["last"] - blk["first"] + 1
        if cnt not in (2, 3) or i + cnt > len(plan):
            return None
        for j in range(cnt):
            po = plan[i + j]
            if len(po.layers) != 1 or po.layers[0] != blk["first"] + j:
                return None
            if j < cnt - 1 and po.act != "relu6":
                return None
        last = plan[i + cnt - 1]
        if last.act is not None:
            return None
        if blk["residual"] and last.add_from != (i - 1 if i > 0 else -1):
            return None
        return cnt, blk

    def _fold_pack(self, li):
        """BN-folded, packed weights and bias of one untouched layer (launched immediately)."""
        torch = self.torch
        lay = self.layers[li]
        s = lay.spec
        wf = torch.empty_like(lay.weight)
        bf = torch.empty((s.c_out,), dtype=torch.float32, device="cuda")
        dc.fold_bn(lay, wf, bf)
        g = dc.geom(s.c_in, s.c_out, s.groups, s.k, s.stride, s.pad)
        packed = torch.empty(dc.packed_bytes(g, dc.BF16), dtype=torch.uint8, device="cuda")
        dc.pack_weights(wf, g, dc.BF16, packed)
        return packed, bf

    # ------------------------------------------------------------------ the two halves of the path
    def merge(self, n_streams: int = 10):
        """Merge every span of two or more layers (dc_merge_chain).  The runs are independent of each
        other (own layers, own outputs, own workspace) and each is a short chain of small dependent
        launches, so they are spread over `n_streams` side streams forked from and joined back into the
        current stream (largest runs first); the work is ordered like any other work on the current
        stream and can be captured in a CUDA graph."""
        torch = self.torch
        jobs = self._merge_jobs
        if n_streams <= 1 or len(jobs) <= 1:
            for devs, res, wm, bm, packed, ws in jobs:
                dc.merge_chain(devs, res, wm, bm, packed, dc.BF16, ws)
            return len(jobs)
        if not hasattr(self, "_merge_streams") or len(self._merge_streams) < n_streams:
            self._merge_streams = [torch.cuda.Stream() for _ in range(n_streams)]
        cur = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(cur)
        order = sorted(range(len(jobs)), key=lambda i: -jobs[i][2].numel())
        used = []
        for n, i in enumerate(order):
            st = self._merge_streams[n % n_streams]
            if n < n_streams:
                st.wait_event(fork)
                used.append(st)
            devs, res, wm, bm, packed, ws = jobs[i]
            dc.merge_chain(devs, res, wm, bm, packed, dc.BF16, ws, stream=st)
        for st in used:
            done = torch.cuda.Event()
            done.record(st)
            cur.wait_event(done)
        return len(jobs)

    def step(self, x, n_streams: int = 10):
        """The whole path once: every merge, then the forward, as one piece of work on the current stream.
        The merges run on side streams in the order the forward needs them, and a launch group waits only
        for the merge of its own span.  (Measured on cfg4: 1.13 ms, the same as the merges followed by the
        forward, 0.24 + 0.88 ms: the forward's persistent kernels fill every SM, so the merges' small
        launches get their turn between them either way; high-priority merge streams did not change it.)"""
        torch = self.torch
        jobs = self._merge_jobs
        if not hasattr(self, "_merge_streams") or len(self._merge_streams) < n_streams:
            self._merge_streams = [torch.cuda.Stream() for _ in range(n_streams)]
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        done = []
        for j, (devs, res, wm, bm, packed, ws) in enumerate(jobs):
            st = self._merge_streams[j % n_streams]
            if j < n_streams:
                st.wait_event(fork)
            dc.merge_chain(devs, res, wm, bm, packed, dc.BF16, ws, stream=st)
            ev = torch.cuda.Event()
            ev.record(st)
            done.append(ev)
        cur = x
        for i, op in enumerate(self.ops):
            if op.merge_job >= 0:
                main.wait_event(done[op.merge_job])
            cur = self.launch(i, cur, x)
        return cur

    def capture_step(self, x):
        """Capture step(x) into a CUDA graph; replay with .replay()."""
        torch = self.torch
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            self.step(x)
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                self.step(x)
        torch.cuda.current_stream().wait_stream(stream)
        return graph

    def launch(self, i, cur, x):
        """Launch group i on `cur` (the previous group's map); x is the network input (skip source -1)."""
        op = self.ops[i]
        if op.kind == "block":
            dc.block_forward(cur, op.block, op.y, op.ws)
        elif op.kind == "dw":
            g = op.geom
            dc.dwconv_forward(cur, g.k, g.stride, g.pad, op.packed, op.bias, op.act, op.y)
        else:
            res = None
            if op.add_from == -1:
                res = x
            elif op.add_from >= 0:
                res = self.ops[op.add_from].y
            dc.conv_forward(cur, op.geom, op.packed, op.bias, op.act, res, op.y, self.conv_ws)
        return op.y

    def forward(self, x):
        """Run the compressed network on x (NHWC bf16, batch == self.batch); returns the last map."""
        cur = x
        for i in range(len(self.ops)):
            cur = self.launch(i, cur, x)
        return cur

    def capture(self, x, keep_graph: bool = False):
        """Capture forward(x) into a CUDA graph on a side stream; replay with .replay().  keep_graph
        keeps the captured graph inspectable (node counts) beside its executable form."""
        torch = self.torch
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(stream):
            self.forward(x)
            stream.synchronize()
            self.graph = torch.cuda.CUDAGraph(keep_graph=keep_graph)
            with torch.cuda.graph(self.graph, stream=stream):
                self.forward(x)
            if keep_graph:
                self.graph.instantiate()
        torch.cuda.current_stream().wait_stream(stream)
        return self.graph

    def status(self):
        """DC_OK unless a bounded device-side wait ran out in any launch so far."""
        st = dc.workspace_status(self.conv_ws)
        for op in self.ops:
            if op.kind == "block":
                st = max(st, dc.workspace_status(op.ws))
        return st


class HostRunner:
    """The captured network fed from pinned host buffers: a step copies its input to the device, replays
    the forward graph and copies the last map back.  Two device input buffers and a copy stream let
    the input copy of step i+1 run under the forward of step i; the last map is copied to one of two
    device staging buffers behind the forward (a few microseconds) and goes to the host from there on a
    third stream, under the next forward.  The forwards themselves are serial (they share the
    intermediate maps)."""

    def __init__(self, cn: CompressedNetwork):
        torch = cn.torch
        self.cn, self.torch = cn, torch
        self.copy_stream, self.compute_stream, self.out_stream = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        self.x = [torch.zeros(cn.in_shape, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        self.y = [torch.zeros(cn.out_shape, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        self.graphs = [cn.capture(x) for x in self.x]
        self.in_ready = [torch.cuda.Event() for _ in range(2)]
        self.in_free = [torch.cuda.Event() for _ in range(2)]
        self.out_ready = [torch.cuda.Event() for _ in range(2)]
        self.out_free = [torch.cuda.Event() for _ in range(2)]
        self.count = 0

    def submit(self, x_host, y_host):
        """Queue one step; y_host is valid once synchronize() has returned."""
        torch = self.torch
        b = self.count & 1
        with torch.cuda.stream(self.copy_stream):
            if self.count >= 2:
                self.copy_stream.wait_event(self.in_free[b])
            self.x[b].copy_(x_host, non_blocking=True)
            self.in_ready[b].record(self.copy_stream)
        with torch.cuda.stream(self.compute_stream):
            self.compute_stream.wait_event(self.in_ready[b])
            self.graphs[b].replay()
            self.in_free[b].record(self.compute_stream)
            if self.count >= 2:
                self.compute_stream.wait_event(self.out_free[b])
            self.y[b].copy_(self.cn.ops[-1].y, non_blocking=True)
            self.out_ready[b].record(self.compute_stream)
        with torch.cuda.stream(self.out_stream):
            self.out_stream.wait_event(self.out_ready[b])
            y_host.copy_(self.y[b], non_blocking=True)
            self.out_free[b].record(self.out_stream)
        self.count += 1

    def join(self):
        """Make compute_stream wait for the copies queued so far (so that an event recorded on it afterwards
        marks the end of every queued step)."""
        self.compute_stream.wait_stream(self.copy_stream)
        self.compute_stream.wait_stream(self.out_stream)

    def synchronize(self):
        self.copy_stream.synchronize()
        self.compute_stream.synchronize()
        self.out_stream.synchronize()
