"""Full depth-compressed MobileNetV2-1.0 forward (batch 128, 224x224, bf16) against the oracle.

Per launch group: the GPU output of images 0, 63 and 127 against the oracle applied to the GPU's
own previous output (isolates each layer, 2e-2 each; 3 x 2e-2 for an unmerged block, which rounds
two intermediate maps), with the element-wise bound of parity_util beside the norm.  End to end:
the first 8 images against the oracle's sequential network.  Every output map is pre-filled with NaN
and sits between sentinel bands."""
import numpy as np
import pytest

from oracle import dc_oracle as O
from paper_2301_12187_b200 import inputs as I
from parity_util import Guarded, assert_close, rel_l2

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 2e-2


def nchw(t):
    return t.float().cpu().numpy().astype(np.float64).transpose(0, 3, 1, 2)


def oracle_group(net, cn, op, x_prev, skip):
    """What one launch group computes, by the oracle, from the map x_prev (NCHW fp64)."""
    specs = [net.layers[i] for i in op.layers]
    if op.kind == "block":
        cur = x_prev
        for s in specs:
            Wf, bf = O.fold_bn(s)
            cur = O.conv_direct(cur, Wf, bf, s.k, s.stride, s.pad, s.groups)
            if s.act == "relu6":
                cur = O.relu6(cur)
        if net.blocks[specs[0].block]["residual"]:
            cur = cur + x_prev
        return cur
    po = cn.plan_ops[op.plan_index[0]]
    cur = O.chain_forward_reordered(x_prev, specs, po.residuals)
    if skip is not None:
        cur = cur + skip
    return O.relu6(cur) if po.act == "relu6" else cur


@pytest.fixture(scope="module")
def run():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_12187_b200 import dc
    from paper_2301_12187_b200.network import CompressedNetwork
    net = I.mobilenet_v2(seed=0, batch=128)
    acts, plan = I.plan_spans(net, seed=0)
    cn = CompressedNetwork(net, acts, plan)
    # every launch group writes into a guarded, NaN-filled map
    guards = []
    for op in cn.ops:
        gy = Guarded(torch, tuple(op.out_shape), torch.bfloat16, fill=float("nan"))
        op.y = gy.t
        guards.append(gy)
    n_merged = cn.merge()
    x_np = I.make_input(0, net.x_shape, bf16=True)
    x = torch.from_numpy(x_np).to("cuda", dtype=torch.bfloat16)
    y = cn.forward(x)
    torch.cuda.synchronize()
    assert cn.status() == dc.OK
    for op, gy in zip(cn.ops, guards):
        gy.check("output of " + "+".join(net.layers[i].name for i in op.layers))
        assert not torch.isnan(op.y.float()).any(), [net.layers[i].name for i in op.layers]
    return dict(dc=dc, net=net, cn=cn, x=x, x_np=x_np, y=y, n_merged=n_merged)


def test_plan_covers_the_network_and_uses_every_kind_of_call(run):
    cn = run["cn"]
    kinds = {op.kind for op in cn.ops}
    assert kinds >= {"conv", "dw"}
    assert run["n_merged"] >= 8 and any(op.merged for op in cn.ops)
    assert sorted(i for op in cn.ops for i in op.layers) == list(range(52))
    assert tuple(run["y"].shape) == (128, 7, 7, 1280)
    assert not torch.isnan(run["y"].float()).any()


def test_each_launch_group_matches_the_oracle_on_sampled_images(run):
    net, cn, x = run["net"], run["cn"], run["x"]
    sel = [0, 63, 127]
    prev = x
    worst = 0.0
    for op in cn.ops:
        skip = None
        if op.kind != "block" and op.add_from == -1:
            skip = nchw(x[sel])
        elif op.kind != "block" and op.add_from >= 0:
            skip = nchw(cn.ops[op.add_from].y[sel])
        ref = oracle_group(net, cn, op, nchw(prev[sel]), skip)
        k = 3.0 if op.kind == "block" else 1.0
        err, _, _ = assert_close(nchw(op.y[sel]), ref, k * TOL, scale=k,
                                 what="+".join(net.layers[i].name for i in op.layers))
        worst = max(worst, err)
        prev = op.y
    print("worst per-group rel-L2: %.3e" % worst)


def test_end_to_end_against_the_sequential_network(run):
    """First 8 images through all launch groups by the oracle (fp64 throughout) against the GPU's
    last map.  bf16 rounding of ~40 consecutive maps accumulates: the norm over the 8 images is held
    to 2e-2 and reported per image; element-wise, an error may reach 8 x the single-layer bound (the
    rel-L2 here is ~8 x a single layer's 2.5e-3) but no more."""
    net, cn, x = run["net"], run["cn"], run["x"]
    N = 8
    cur = nchw(x[:N])
    outs = []
    for op in cn.ops:
        skip = None
        if op.kind != "block" and op.add_from == -1:
            skip = nchw(x[:N])
        elif op.kind != "block" and op.add_from >= 0:
            skip = outs[op.add_from]
        cur = oracle_group(net, cn, op, cur, skip)
        outs.append(cur)
    got = nchw(run["y"][:N])
    per_image = [rel_l2(got[i], cur[i]) for i in range(N)]
    print("end-to-end rel-L2 after %d launch groups, per image: %s" % (len(cn.ops), " ".join("%.2e" % e for e in per_image)))
    err, worst, max_abs = assert_close(got, cur, TOL, scale=8.0, what="end to end, 8 images")
    print("end-to-end rel-L2 over 8 images %.3e; worst element at %.2f of 8 x the single-layer bound" % (err, worst))
    assert max(per_image) <= TOL


def test_graph_replay_reproduces_the_eager_result(run):
    cn, x = run["cn"], run["x"]
    ref = run["y"].clone()
    g = cn.capture(x)
    cn.ops[-1].y.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(cn.ops[-1].y, ref)
    assert cn.status() == run["dc"].OK


def test_step_graph_merges_and_runs_with_per_span_dependencies(run):
    """The whole path as one graph: the merged weights are wiped before every replay, so a launch group
    that ran before the merge of its span had finished would read zeros."""
    cn, x = run["cn"], run["x"]
    ref = run["y"].clone()
    g = cn.capture_step(x)
    for _ in range(3):
        for op in cn.ops:
            if op.merged:
                op.packed.zero_()
                op.bias.zero_()
        cn.ops[-1].y.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(cn.ops[-1].y, ref)
    assert cn.status() == run["dc"].OK


def test_host_runner_returns_every_steps_own_result(run):
    """Steps fed from pinned host buffers with the copies running under neighbouring forwards: each step's
    output is the forward of its own input (two inputs alternate, five steps in flight)."""
    from paper_2301_12187_b200.network import HostRunner
    cn, x = run["cn"], run["x"]
    x2 = torch.flip(x, dims=[0]).contiguous()
    ref = [cn.forward(x).clone(), cn.forward(x2).clone()]
    torch.cuda.synchronize()
    assert not torch.equal(ref[0], ref[1])
    runner = HostRunner(cn)
    xs = [x.cpu().pin_memory(), x2.cpu().pin_memory()]
    ys = [torch.zeros(cn.out_shape, dtype=torch.bfloat16).pin_memory() for _ in range(5)]
    for i in range(5):
        runner.submit(xs[i & 1], ys[i])
    runner.synchronize()
    for i in range(5):
        assert torch.equal(ys[i], ref[i & 1].cpu()), "step %d" % i
    assert cn.status() == run["dc"].OK
