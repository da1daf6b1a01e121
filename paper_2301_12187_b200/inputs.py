"""Seeded synthetic inputs: tensors, layer chains, the MobileNetV2-1.0 table and its span plan.

This module only *describes and generates data*.  It contains none of the
method's arithmetic (no BN folding, no kernel composition, no convolution) and
imports neither the CUDA binding nor the CPU oracle, so both sides can read
identical buffers from it.

Generator: counter-based.  Element `i` of tensor `tensor_id` under `seed` is a
function of (seed, tensor_id, i) alone: splitmix64 finaliser -> 53-bit uniform
-> Box-Muller for normals.  Layouts: feature maps NHWC float32; kernels
[c_out][c_in/groups][k][k] float32 (the paper's theta_l with out/in swapped,
Sec. 3).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)


def _mix(z):
    """splitmix64 output function on a uint64 array (wrapping arithmetic)."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


def _stream(seed: int, tensor_id: int, start: int, count: int):
    """uint64 words start..start+count-1 of the stream (seed, tensor_id)."""
    with np.errstate(over="ignore"):
        base = _mix(np.uint64(seed) * _GOLD + np.uint64(0x1234567))
        base = _mix(base + np.uint64(tensor_id) * np.uint64(0xD1B54A32D192ED03))
        idx = np.arange(start, start + count, dtype=np.uint64)
        return _mix(base + (idx + np.uint64(1)) * _GOLD)


def uniform01(seed: int, tensor_id: int, count: int, start: int = 0):
    """count doubles in [0, 1)."""
    w = _stream(seed, tensor_id, start, count)
    return (w >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def uniform(seed, tensor_id, shape, lo, hi):
    n = int(np.prod(shape))
    return (lo + (hi - lo) * uniform01(seed, tensor_id, n)).astype(np.float32).reshape(shape)


def normal(seed, tensor_id, shape, std=1.0):
    """N(0, std^2) by Box-Muller on the uniforms (2i, 2i+1)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)
    step = 1 << 22
    for s in range(0, n, step):
        m = min(step, n - s)
        u = uniform01(seed, tensor_id, 2 * m, start=2 * s)
        r = np.sqrt(-2.0 * np.log(1.0 - u[0::2]))
        out[s:s + m] = (std * r * np.cos(2.0 * np.pi * u[1::2])).astype(np.float32)
    return out.reshape(shape)


def round_bf16(a):
    """float32 array rounded to the nearest bfloat16 (ties to even), returned as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


# --------------------------------------------------------------------------- layers


@dataclass
class LayerSpec:
    """One convolution followed by batch-norm (and, in a network, an activation)."""
    c_in: int
    c_out: int
    groups: int
    k: int
    stride: int
    pad: int
    weight: np.ndarray
    bias: Optional[np.ndarray]
    bn: Optional[Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]]
    eps: float = 1e-5
    act: Optional[str] = None          # activation after the layer ('relu6' or None)
    name: str = ""
    block: int = -1                    # index of the network block the layer belongs to
    role: str = ""


_KIND_W, _KIND_G, _KIND_B, _KIND_M, _KIND_V, _KIND_BIAS = range(6)
_X_TENSOR_ID = 1 << 20


def make_layer(seed, index, c_in, c_out, k, stride, pad, depthwise=False, act=None, name="",
               block=-1, role="", with_bn=True, with_bias=False) -> LayerSpec:
    """Weights N(0, 1/fan_in) (variance), fan_in = (c_in/groups) k^2; BN gamma, var ~ U[0.5,1.5),
    beta, running mean ~ N(0, 0.1^2); no conv bias unless asked for (then N(0, 0.1^2))."""
    groups = c_in if depthwise else 1
    if depthwise:
        assert c_in == c_out
    cg = c_in // groups
    fan_in = cg * k * k
    tid = 16 * index
    w = normal(seed, tid + _KIND_W, (c_out, cg, k, k), std=fan_in ** -0.5)
    bn = None
    if with_bn:
        bn = (uniform(seed, tid + _KIND_G, (c_out,), 0.5, 1.5),
              normal(seed, tid + _KIND_B, (c_out,), std=0.1),
              normal(seed, tid + _KIND_M, (c_out,), std=0.1),
              uniform(seed, tid + _KIND_V, (c_out,), 0.5, 1.5))
    bias = normal(seed, tid + _KIND_BIAS, (c_out,), std=0.1) if with_bias else None
    return LayerSpec(c_in, c_out, groups, k, stride, pad, w, bias, bn, 1e-5, act, name, block, role)


def make_input(seed, shape_nhwc, bf16=False):
    x = normal(seed, _X_TENSOR_ID, shape_nhwc, std=1.0)
    return round_bf16(x) if bf16 else x


@dataclass
class ChainCase:
    """A run of convolutions with identity activations in between, plus its input shape."""
    name: str
    dtype: str                                     # 'f32' or 'bf16'
    layers: List[LayerSpec]
    residuals: List[Tuple[int, int]]
    x_shape: Tuple[int, int, int, int]             # N, H, W, C (NHWC)
    seed: int = 0
    final_act: Optional[str] = None

    def x(self, n: Optional[int] = None):
        """Input NHWC float32 (bf16-rounded for bf16 cases); first n images if given."""
        shp = self.x_shape if n is None else (n,) + tuple(self.x_shape[1:])
        return make_input(self.seed, shp, bf16=(self.dtype == "bf16"))


def inverted_residual(seed, index0, c_in, c_out, t, stride, block=-1, acts=("relu6", "relu6")):
    """expand 1x1 (c_in -> t c_in), depthwise 3x3 (stride, pad 1), project 1x1 (-> c_out)."""
    hid = c_in * t
    L = []
    if t != 1:
        L.append(make_layer(seed, index0 + len(L), c_in, hid, 1, 1, 0, act=acts[0],
                            name="b%d.expand" % block, block=block, role="expand"))
    L.append(make_layer(seed, index0 + len(L), hid, hid, 3, stride, 1, depthwise=True, act=acts[1],
                        name="b%d.dw" % block, block=block, role="dw"))
    L.append(make_layer(seed, index0 + len(L), hid, c_out, 1, 1, 0, act=None,
                        name="b%d.project" % block, block=block, role="project"))
    return L


def chain_case(idx: int, seed: int = 0, batch: Optional[int] = None) -> ChainCase:
    """The four single-span workloads (all inner activations already identities).

    0: tiny fp32   1x1 16->96, dw3x3 96 s1 p1, 1x1 96->24;  x 2x16x16x16
    1: bf16 block  24->144->24 at 56x56, skip folded;         x 64x56x56x24
    2: bf16 s2     24->144 (dw stride 2) ->32;                x 128x56x56x24
    3: bf16 cross  two blocks 32->192->32 at 28x28, both skips folded; x 128x28x28x32
    """
    none2 = (None, None)
    if idx == 0:
        L = inverted_residual(seed, 0, 16, 24, 6, 1, block=0, acts=none2)
        return ChainCase("cfg0_tiny_fp32", "f32", L, [], (batch or 2, 16, 16, 16), seed)
    if idx == 1:
        L = inverted_residual(seed, 0, 24, 24, 6, 1, block=0, acts=none2)
        return ChainCase("cfg1_mbv2_block56", "bf16", L, [(0, 2)], (batch or 64, 56, 56, 24), seed)
    if idx == 2:
        L = inverted_residual(seed, 0, 24, 32, 6, 2, block=0, acts=none2)
        return ChainCase("cfg2_stride2", "bf16", L, [], (batch or 128, 56, 56, 24), seed)
    if idx == 3:
        L = inverted_residual(seed, 0, 32, 32, 6, 1, block=0, acts=none2)
        L += inverted_residual(seed, 3, 32, 32, 6, 1, block=1, acts=none2)
        return ChainCase("cfg3_cross_block", "bf16", L, [(0, 2), (3, 5)],
                         (batch or 128, 28, 28, 32), seed)
    raise ValueError("chain_case index must be 0..3")


VGG_MAPS = {64: 224, 128: 112, 256: 56, 512: 28}       # channel width -> feature-map side of that VGG stage


def vgg_case(c: int, seed: int = 0, batch: int = 32) -> ChainCase:
    """Two dense 3x3 layers c -> c -> c (stride 1, padding 1, BN each) with an identity in between, on the
    feature map of the VGG stage of that width: the run that merges into one 5x5 layer."""
    L = [make_layer(seed, 0, c, c, 3, 1, 1, act=None, name="conv_a"),
         make_layer(seed, 1, c, c, 3, 1, 1, act=None, name="conv_b")]
    hw = VGG_MAPS[c]
    return ChainCase("vgg_c%d" % c, "bf16", L, [], (batch, hw, hw, c), seed)


# --------------------------------------------------------------------------- MobileNetV2-1.0


MBV2_SETTING = ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2),
                (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1))


@dataclass
class Network:
    layers: List[LayerSpec]
    blocks: List[dict]                 # {'first','last','residual'} per block (stem and head included)
    x_shape: Tuple[int, int, int, int]
    seed: int


def mobilenet_v2(seed: int = 0, batch: int = 128, res: int = 224) -> Network:
    """Stem 3x3 s2 3->32, the 17 inverted-residual blocks of MBV2_SETTING, head 1x1 320->1280.
    ReLU6 after stem, every expand, every depthwise and the head; identity after every project."""
    layers: List[LayerSpec] = []
    blocks: List[dict] = []
    layers.append(make_layer(seed, 0, 3, 32, 3, 2, 1, act="relu6", name="stem", block=0, role="stem"))
    blocks.append(dict(first=0, last=0, residual=False))
    c = 32
    b = 1
    for t, co, n, s in MBV2_SETTING:
        for j in range(n):
            stride = s if j == 0 else 1
            first = len(layers)
            layers += inverted_residual(seed, first, c, co, t, stride, block=b)
            blocks.append(dict(first=first, last=len(layers) - 1,
                               residual=(stride == 1 and c == co)))
            c = co
            b += 1
    layers.append(make_layer(seed, len(layers), c, 1280, 1, 1, 0, act="relu6", name="head",
                             block=b, role="head"))
    blocks.append(dict(first=len(layers) - 1, last=len(layers) - 1, residual=False))
    return Network(layers, blocks, (batch, res, res, 3), seed)


@dataclass
class PlanOp:
    """One launch group of the compressed network.

    layers      indices (consecutive) of the network layers the op covers
    residuals   skip additions folded into the op, as (first, last) relative to `layers`
    act         activation after the op
    add_from    -2: nothing added; -1: add the network input; j >= 0: add the output of op j
                (a skip addition that stays explicit)
    """
    layers: List[int]
    residuals: List[Tuple[int, int]] = field(default_factory=list)
    act: Optional[str] = None
    add_from: int = -2


def plan_spans(net: Network, seed: int = 0, n_remove: int = 17, max_k3: int = 3):
    """Choose which ReLU6 become identities and cut the network into spans.

    Returns (acts, ops): acts[l] is the activation after layer l in the
    compressed network; ops is the list of PlanOp.
      1. the ReLU6 positions other than the head's are ordered by a seeded hash;
         the first n_remove become identities;
      2. a span ends at every remaining ReLU6;
      3. inside a linear run a span also ends (a) at the entry and exit of a
         skip block that still holds a ReLU6 (its addition stays explicit),
         (b) before a layer with k > 1 when the span already holds a stride-2
         layer (App. B.2), (c) before the (max_k3+1)-th 3x3 layer; a skip block
         with no ReLU6 left is never split: the cut moves to its entry.
    """
    L = net.layers
    nL = len(L)
    cand = [i for i in range(nL - 1) if L[i].act == "relu6"]
    keys = _stream(seed, (1 << 21) + 7, 0, len(cand))
    order = [cand[j] for j in np.argsort(keys, kind="stable")]
    removed = set(order[:n_remove])
    acts = [None if (i in removed) else L[i].act for i in range(nL)]

    # atoms: a whole skip block with no activation left inside, or a single layer
    atoms = []                         # (layer indices, is_folded_skip, forced_cut_before, forced_cut_after)
    for blk in net.blocks:
        idx = list(range(blk["first"], blk["last"] + 1))
        inner_linear = all(acts[i] is None for i in idx[:-1])
        if blk["residual"] and inner_linear:
            atoms.append((idx, True, False, False))
        elif blk["residual"]:
            for j, i in enumerate(idx):
                atoms.append(([i], False, j == 0, j == len(idx) - 1))
        else:
            for i in idx:
                atoms.append(([i], False, False, False))

    spans = []                         # (layer indices, folded skips relative)
    cur, cur_res, has_s2, n_k3 = [], [], False, 0
    prev_forced_after = False

    def close():
        nonlocal cur, cur_res, has_s2, n_k3
        if cur:
            spans.append((cur, cur_res))
        cur, cur_res, has_s2, n_k3 = [], [], False, 0

    for idx, folded, cut_before, cut_after in atoms:
        a_k3 = sum(1 for i in idx if L[i].k > 1)
        a_s2 = any(L[i].stride > 1 for i in idx)
        join = bool(cur) and acts[cur[-1]] is None and not cut_before and not prev_forced_after
        if join and has_s2 and a_k3 > 0:
            join = False
        if join and n_k3 + a_k3 > max_k3:
            join = False
        if not join:
            close()
        if folded:
            cur_res.append((len(cur), len(cur) + len(idx) - 1))
        cur += idx
        has_s2 = has_s2 or a_s2
        n_k3 += a_k3
        prev_forced_after = cut_after
    close()

    return acts, ops_from_spans(net, acts, spans)


def ops_from_spans(net: Network, acts, spans) -> List[PlanOp]:
    """PlanOps for a list of spans (consecutive layer indices, folded skip groups relative to the
    span), with the skip additions that stay explicit wired to the op that produced the block
    input."""
    L = net.layers
    ops: List[PlanOp] = []
    produced_by = {}                   # layer index -> op index whose output is that layer's output
    for idx, res in spans:
        op = PlanOp(layers=idx, residuals=res, act=acts[idx[-1]])
        blk = net.blocks[L[idx[-1]].block]
        explicit = blk["residual"] and not any(
            (idx[0] + f == blk["first"] and idx[0] + l == blk["last"]) for f, l in res)
        if explicit and idx[-1] == blk["last"]:
            op.add_from = produced_by.get(blk["first"] - 1, -1)
        ops.append(op)
        produced_by[idx[-1]] = len(ops) - 1
    return ops


def removed_activations(net: Network, seed: int = 0, n_remove: int = 17):
    """acts[l] after the seeded choice of plan_spans: the first n_remove ReLU6 positions (head
    excluded) in the order of a seeded hash become identities."""
    L = net.layers
    cand = [i for i in range(len(L) - 1) if L[i].act == "relu6"]
    keys = _stream(seed, (1 << 21) + 7, 0, len(cand))
    order = [cand[j] for j in np.argsort(keys, kind="stable")]
    removed = set(order[:n_remove])
    return [None if (i in removed) else L[i].act for i in range(len(L))]


def plan_from_boundaries(net: Network, acts, boundaries, span_residuals) -> List[PlanOp]:
    """PlanOps for the pieces (b_0, b_1], (b_1, b_2], ... of `boundaries` (0 = b_0 < ... < b_n = L):
    the merge pattern S of Sec. 4 with the kept activations `acts`.  span_residuals(i, j) gives the
    folded skip groups of a piece (or None if the piece cannot be merged: an error here)."""
    spans = []
    for a, c in zip(boundaries[:-1], boundaries[1:]):
        res = span_residuals(a, c)
        if res is None or any(acts[i] is not None for i in range(a, c - 1)):
            raise ValueError("piece (%d, %d] cannot be merged" % (a, c))
        spans.append((list(range(a, c)), list(res)))
    return ops_from_spans(net, acts, spans)


def random_dp_tables(rng, L, inf, unmergeable=0.2, neg_inf=0.0):
    """Seeded latency / importance tables for the selector's dynamic programmes: T[i][j] small
    positive integers growing with the span (`inf` for a share of the spans longer than one layer),
    I[i][j] = 0 for single layers and negative for longer blocks (-infinity for a share of them).
    `rng` is a random.Random."""
    T = [[0] * (L + 1) for _ in range(L + 1)]
    I = [[0.0] * (L + 1) for _ in range(L + 1)]
    for i in range(L + 1):
        for j in range(i + 1, L + 1):
            T[i][j] = rng.randint(1, 9) + (j - i - 1) * rng.randint(0, 3)
            if j - i > 1 and rng.random() < unmergeable:
                T[i][j] = inf
            I[i][j] = 0.0 if j - i == 1 else -rng.random() * (j - i)
            if j - i > 1 and rng.random() < neg_inf:
                I[i][j] = float("-inf")
    return T, I


def random_dp_tables_ext(rng, L, inf, unmergeable=0.2, p_identity=0.4):
    """Tables for the extended selector (App. B): T as random_dp_tables; I[i][j][a][b] the importance
    of block (i, j] with end indicators (a, b) (single layers near 0, longer blocks more negative, a
    kept non-linearity at an end slightly better); sigma_id[p] for p = 0..L says whether the original
    activation at boundary p is an identity (each inner boundary with probability p_identity; the
    network input counts as one, the last activation does not)."""
    T, _ = random_dp_tables(rng, L, inf, unmergeable, 0.0)
    I = [[[[0.0, 0.0], [0.0, 0.0]] for _ in range(L + 1)] for _ in range(L + 1)]
    for i in range(L + 1):
        for j in range(i + 1, L + 1):
            base = -rng.random() * (j - i - 0.5)
            for a in range(2):
                for b in range(2):
                    I[i][j][a][b] = base + 0.3 * rng.random() * (a + b) - 0.1 * rng.random()
    sigma_id = [True] + [rng.random() < p_identity for _ in range(L - 1)] + [False]
    return T, I, sigma_id
